"""Writes tests/golden/full_width_step.json: the ORACLE's hashes of one replayed step at the benchmark's full width.

    python tests/golden/make_full_width_step.py

The case is one decoder layer of the 1B shape (d_model 2048, 16 heads, FFN 8192, sequence 2048, micro-batch 4, Hadamard
block 128) with the vocabulary cut to 8192 so that the oracle finishes in minutes.  Only `oracle/` and `synth/` are
imported: no value in the file ever comes from the CUDA path.  The file is keyed by a hash of the oracle's and the input
generator's sources; the GPU test recomputes the step with the oracle when that key no longer matches.
"""
import hashlib
import json
import os
import sys
import time

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

CASE = dict(n_layers=1, d_model=2048, n_heads=16, ffn=8192, vocab=8192, seq=2048, micro_batch=4, mesh=(1, 1, 1),
            hadamard_block=128, z_weight=0.0, lr=3e-4, betas=(0.9, 0.95), eps=1e-8, wd=0.1, clip=1.0, step=1)
SEED = 0
OUT = os.path.join(HERE, "full_width_step.json")


def source_key():
    """SHA-256 over the sources that define the expected values (oracle + input generator)."""
    h = hashlib.sha256()
    for rel in ("oracle/prim.h", "oracle/oracle.c", "oracle/__init__.py", "oracle/step.py", "synth/__init__.py"):
        h.update(rel.encode())
        h.update(open(os.path.join(ROOT, rel), "rb").read())
    return h.hexdigest()


def compute():
    import synth
    from oracle import step as ostep
    params = synth.model_params(CASE, seed=SEED)
    tokens = synth.model_tokens(CASE, 1, seed=SEED)
    out = ostep.run_step(dict(CASE), params, tokens)
    return {"hashes": out["hashes"], "losses": [float(x) for x in out["losses"]], "grad_norm": float(out["grad_norm"]),
            "coef": float(out["coef"])}


if __name__ == "__main__":
    import oracle
    oracle.build()
    t0 = time.time()
    res = compute()
    res.update(key=source_key(), case={k: (list(v) if isinstance(v, tuple) else v) for k, v in CASE.items()}, seed=SEED,
               oracle_seconds=round(time.time() - t0, 1), cores=os.cpu_count())
    with open(OUT, "w") as f:
        json.dump(res, f, indent=1, sort_keys=True)
        f.write("\n")
    print("wrote", OUT, "in", res["oracle_seconds"], "s")
