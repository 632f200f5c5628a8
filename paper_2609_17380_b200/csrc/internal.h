// Host-side helpers shared between the translation units of libdet.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace det {
// every kernel launch of the library passes its grid through DET_L, which counts it
int note_launch();
#define DET_L(grid) (det::note_launch(), (grid))
// floats of scratch the multi-level tree sum needs for n elements
size_t sum_ws_floats(size_t n);
// out[0] = det_sum(x[0..n)) (squares: of x^2); launches on st, scratch in ws (sum_ws_floats(n) floats)
int sum_launch(const float* x, size_t n, int squares, float* out, float* ws, cudaStream_t st);

// Epilogue descriptions.  All data-dependent scalars are read from device memory.
enum { EPI_RAW = 0, EPI_FWD = 1, EPI_DX = 2, EPI_DW = 3 };
struct EpiParams {
  void* out;              // RAW: int32 [I,J]; FWD: bf16 [I,J]; DX: bf16 [I,J]; DW: f32 [I,J]
  const float* s_x;       // FWD, DX, DW: activation step (device scalar)
  const float* s_w;       // FWD: per column j; DW: per row i
  const uint32_t* amax1;  // DX: float bits of absmax(A); DW: float bits of absmax(G)
  const uint32_t* amax2;  // DW: int absmax(Z) (NULL: scale 1)
  const float* s_u;       // DX: step of the rotated weights
  const uint16_t* ref;    // DX: X bf16 [I,J]; DW: W bf16 [I,J] (range masks)
  float rot;              // 2^-7 with rotation, 1 without
  float* ds_partial;      // DX: [I, J/128] partial sums of dXhat * phi
};

// Independent kernels of one call may run side by side so that the partial last wave of one grid is filled by blocks of
// another.  aux_fork makes up to two auxiliary streams of the current device start where `st` stands now; aux_join makes
// `st` wait for them, so the caller still sees plain stream order.  Returns NULL / false when the streams cannot be
// had (the caller then launches everything on `st`).
struct AuxStreams {
  cudaStream_t s[2];
  cudaEvent_t fork, join[2];
  bool ok;
};
AuxStreams* aux_fork(cudaStream_t st);
bool aux_join(cudaStream_t st, AuxStreams* a);
// Joins the auxiliary streams on every way out of a call that forked them (error returns included), so that the
// caller's stream never keeps an unjoined fork.
struct AuxScope {
  cudaStream_t st;
  AuxStreams* a;
  AuxScope(cudaStream_t s) : st(s), a(aux_fork(s)) {}
  ~AuxScope() { if (a) aux_join(st, a); }
  cudaStream_t aux(int i) const { return a ? a->s[i] : st; }
  bool join() { AuxStreams* t = a; a = nullptr; return aux_join(st, t); }
};

// Kernel attributes and the SM count belong to a device, not to the process: DevOnce remembers per device whether a
// kernel's opt-in for large dynamic shared memory has been made there.  Both helpers act on the CURRENT device.
constexpr int MAX_DEVICES = 64;
struct DevOnce { bool done[MAX_DEVICES]; };
int dev_ensure_smem(DevOnce& once, const void* fn, size_t bytes);  // DET_OK or DET_ERR_CUDA
int dev_sm_count();                                                 // SMs of the current device (0 on error)

// C[i,j] = sum_k A[i,k] B[j,k] on the tensor cores with the chosen epilogue; host-side checks included
// force_one_cta != 0 keeps the one-CTA kernel even where the two-CTA tiles would apply (the results are identical)
int igemm_launch(int epi, const int8_t* A, const int8_t* B, int I, int J, int K, const EpiParams& ep, int* status,
                 cudaStream_t st, int force_one_cta = 0);

// Sliced (arithmetic version 2) contractions: out = round(I 2^(Ea + Eb - 280)) from the int8 slices of both operands,
// Z problems per launch (lmhead_v2.cu).
enum { SL_F32 = 0, SL_BF16 = 1, SL_BF16_ROWSCALE = 2 };
struct SlArgs {
  const int32_t* Ea;       // [Z*I] row exponents of A (bit 30: non-finite row)
  const int32_t* Eb;       // [Z*J]
  void* out;               // f32 or bf16, element (z, i, j) at (z / hdiv) * o_b + (z % hdiv) * o_h + i * ldo + j
  const float* rowscale;   // [Z*I], SL_BF16_ROWSCALE only
  int I, J, K, Z, hdiv;
  long long o_b, o_h;
  int ldo;
  int causal_tiles;        // only tiles with j0 <= i0
  int krange;              // 0 all steps, 1 steps <= the row tile's, 2 steps >= the row tile's
  int epi;
};
int sliced_gemm_launch(const int8_t* Ah, const int8_t* Al, const int8_t* Bh, const int8_t* Bl, const SlArgs& p, int* status,
                       cudaStream_t st);
}  // namespace det
