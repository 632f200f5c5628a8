// Ordered full-precision contractions for the LM head (Sec. 3.2: the head stays out of quantisation).
//
// Every output is ONE f32 accumulator that starts at +0 (or at the value already in the output) and
// receives its terms in ascending order of the contraction index, each term an exact bf16 x bf16 product
// added with a separate rounding.  That fixes the order, so these GEMMs run on the FP32 ALUs:
// 128x256 output tile per CTA, 8x16 register tile per consumer thread, 16-deep slabs staged through a three-slot
// shared-memory ring as f32 by dedicated producer warps (k_ogemm_ws in ogemm_core.cuh), packed two-lane FP32
// instructions.  Because the product of two
// bf16 values is exact in binary32, "multiply, then add" and a fused multiply-add round the same exact sum
// once and give the same bits, unless the product is subnormal (the unfused product is then flushed to zero,
// the fused one is not).  Each slab is therefore checked for factors below 2^-63 while it is staged; clean
// slabs use the fused instruction, the others the two-instruction sequence.
#include "ogemm_core.cuh"

using namespace det;

// The two gradient contractions of the LM head are independent; the input-gradient grid (512 blocks on 148 SMs at
// the benchmark shape) ends in a partial wave, so the weight-gradient kernel runs beside it on an auxiliary stream
// and fills the idle SMs (aux_fork / aux_join keep plain stream order for the caller).
static OgemmArgs plain_args(const void* A, const void* B, void* out, int I, int J, int C, int lda, int ldb, int ldo, int init) {
  OgemmArgs p = {};
  p.A = A; p.B = B; p.out = out; p.I = I; p.J = J; p.C = C; p.lda = lda; p.ldb = ldb; p.ldo = ldo; p.init = init; p.H = 1;
  return p;
}

extern "C" int det_lmhead_fwd(const det_bf16* H, const det_bf16* W, int M, int V, int K, float* logits, void* stream) {
  if (!H || !W || !logits || M <= 0 || V <= 0 || K <= 0) return DET_ERR_ARG;
  if (K % 16 || V % 4) return DET_ERR_SHAPE;
  if (!aligned16(H) || !aligned16(W) || !aligned16(logits)) return DET_ERR_ALIGN;
  int rc = ogemm_ws_launch<CONTIG, CONTIG, false, false>(plain_args(H, W, logits, M, V, K, K, K, V, 0), (cudaStream_t)stream);
  if (rc != DET_OK) return rc;
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_lmhead_bwd(const float* dlogits, const det_bf16* H, const det_bf16* W, int M, int V, int K, det_bf16* dH,
                              float* dW, int first_chunk, void* stream) {
  if (!dlogits || !H || !W || !dH || !dW || M <= 0 || V <= 0 || K <= 0) return DET_ERR_ARG;
  if (K % 16 || V % 16 || M % 8) return DET_ERR_SHAPE;
  if (!aligned16(dlogits) || !aligned16(H) || !aligned16(W) || !aligned16(dH) || !aligned16(dW)) return DET_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  AuxScope aux(st);   // the auxiliary streams start where the caller's stream stands now; joined on every way out
  // dH[m,k] = sum over v ascending of bf16(dlogits[m,v]) * W[v,k]
  int rc = ogemm_ws_launch<CONTIG, STRIDED, true, true>(plain_args(dlogits, W, dH, M, K, V, V, K, K, 0), st);
  if (rc != DET_OK) return rc;
  // dW[v,k] (+)= sum over m ascending of bf16(dlogits[m,v]) * H[m,k], beside the first kernel
  rc = ogemm_ws_launch<STRIDED, STRIDED, true, false>(plain_args(dlogits, H, dW, V, K, M, V, K, K, first_chunk ? 0 : 1),
                                                      aux.aux(0));
  if (rc != DET_OK) return rc;
  if (!aux.join()) return DET_ERR_CUDA;
  DET_CHECK_LAUNCH();
  return DET_OK;
}
