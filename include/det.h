/* det.h -- C-ABI of libdet: the replayed, bit-exact training-step arithmetic on B200 (sm_100a).
 *
 * The sequence of calls below is the normative statement of one training step of the paper's auditable
 * regime (Sec. 2.2 "forward pass, gradient calculation, weight updates"; Sec. 6, Algorithm 1 for the
 * gradient reduction).  Every tensor that crosses a call boundary is rounded to its declared type.
 *
 * Conventions for every call
 *  - returns DET_OK (0) or a negative det_status; errors that the host can see (bad shape, misaligned
 *    pointer, workspace too small) return before anything is launched;
 *  - every tensor pointer is a DEVICE pointer owned by the caller, row-major and contiguous unless a
 *    leading dimension is given; the library allocates no device memory, frees nothing and keeps no pointer after
 *    it returns.  Scratch comes from the caller's `ws` buffer of `ws_bytes` bytes (256-byte aligned),
 *    sized by the matching det_*_ws_bytes() query;
 *  - work is asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream), except
 *    det_tensor_hash which synchronises that stream (det_tensor_hash_async does not).  det_linear_bwd, det_attn_bwd
 *    and det_lmhead_bwd run independent kernels of the call side by side on two auxiliary streams per device that
 *    the library creates on first use: they start where `stream` stands when the call is made and `stream` waits
 *    for them on every way out of the call (error returns included), so the caller still sees plain stream order.
 *    What the library keeps between calls is per DEVICE and set up under a lock on first use there: those two streams,
 *    the one-time opt-in of each kernel for large shared memory, the SM count, and the address of det_sum_static's
 *    scratch.  None of it outlives a cudaDeviceReset (do not call the library again after one).  No mode or option
 *    is process-wide.  Calls for one device may come from several host threads, except that two calls of the three
 *    functions above on one device at the same time would share the auxiliary streams: give those one thread per device;
 *  - data-dependent scalars (LSQ steps, norms, losses) are device scalars so that no call forces a sync;
 *  - device-detected conditions (bad target index, a bounded wait that expired, a non-finite norm) are
 *    OR-ed into *status_dev (device int, may be NULL) as DET_DEV_* bits; kernels never trap;
 *  - floating point: IEEE binary32, round-to-nearest-even, multiply and add never fused, subnormal
 *    inputs and results flushed to zero (Sec. 2.1).  Sums run in the fixed pairwise tree "det_sum":
 *    level by level, adjacent elements paired, an odd last element carried up unchanged, so the tree
 *    shape depends only on the length, never on the launch configuration.
 *  - bf16 tensors are passed as uint16_t bit patterns;
 *  - operands are expected to be finite.  The LSQ linears, norms, losses and reductions propagate an infinity or a NaN
 *    exactly as the definition does (max/min ignore a NaN operand; NaN payloads are unspecified); the attention calls
 *    multiply masked pairs in with weight +0, so a non-finite q, k, v or dout entry can turn more elements of its block
 *    into NaN than the definition names.  Every finite element is still exact.
 */
#ifndef DET_H
#define DET_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t det_bf16;

typedef enum {
  DET_OK = 0,
  DET_ERR_ARG = -1,       /* NULL pointer, negative size, inconsistent arguments */
  DET_ERR_SHAPE = -2,     /* dimension not supported by the kernels (see each call) */
  DET_ERR_ALIGN = -3,     /* pointer or leading dimension not 16-byte aligned */
  DET_ERR_WORKSPACE = -4, /* ws_bytes too small */
  DET_ERR_RANGE = -5,     /* contraction length >= 2^17 could overflow the int32 accumulator */
  DET_ERR_CUDA = -6       /* launch or runtime error (no synchronisation beyond the stream query) */
} det_status;

/* bits OR-ed into *status_dev by kernels */
#define DET_DEV_TARGET 1    /* cross-entropy target outside [0, V) */
#define DET_DEV_TIMEOUT 2   /* a bounded in-kernel wait expired; outputs of that launch are undefined */
#define DET_DEV_NONFINITE 4 /* non-finite gradient norm */

typedef enum { DET_F32 = 0, DET_BF16 = 1 } det_dtype;

/* library / device information: returns the number of SMs of the current device (or a negative status) */
int det_device_sm_count(void);
/* number of kernels this library has launched in this process so far (host-side atomic counter) */
unsigned long long det_launch_count(void);

/* ---- order-fixed sums (Sec. 2.1 "Reduction order") ----------------------------------------------- */
/* out[0] = det_sum_i x[i]^2 (squares == 1) or det_sum_i x[i] (squares == 0).  n >= 0. */
size_t det_sum_ws_bytes(size_t n);
int det_sum(const float* x, size_t n, int squares, float* out, void* ws, size_t ws_bytes, void* stream);

/* det_sum for callers that cannot allocate.  The paper has no counterpart for this entry point; it exists for users
 * of this library who may not call cudaMalloc: code running inside a host application that owns all device memory
 * and passes in only input and output buffers, or a loop that must not block on the allocator's device-wide
 * synchronisation.  Same result as det_sum, bit for bit, but the scratch is a fixed 256 KiB array inside the library
 * image (held by every GPU that loads the library until the process exits), so the call allocates and frees nothing.
 *  - n may be at most DET_SUM_STATIC_MAX_N (also returned by det_sum_static_max_n()); larger n returns DET_ERR_SHAPE
 *    and launches nothing.
 *  - The first call on each device looks up the array's device address (one cudaGetSymbolAddress with that device
 *    current); make that first call before starting any stream capture.
 *  - All calls on a device share the one array and it keeps what the last call left there.  Nothing in it needs to
 *    start at zero.  Two calls that overlap on the GPU (different streams, no ordering between them) race on it and
 *    give undefined results: order them. */
#define DET_SUM_STATIC_MAX_N (1u << 29)
size_t det_sum_static_max_n(void);
int det_sum_static(const float* x, size_t n, int squares, float* out, void* stream);

/* Global gradient norm and clip coefficient (Sec. 3.2 "Optimizer": clip to global l2 norm 1.0).
 * g_ptrs / n_elems are HOST arrays of ntensors device pointers / lengths in canonical parameter order.
 * per-tensor det_sum(g^2), then det_sum over the per-tensor sums, norm = sqrt(total),
 * coef = min(1, max_norm / (norm + 1e-6)); max_norm <= 0 gives coef = 1.  norm_out, coef_out: device. */
size_t det_grad_norm_ws_bytes(const size_t* n_elems, int ntensors);
int det_grad_norm(const float* const* g_ptrs, const size_t* n_elems, int ntensors, float max_norm, float* norm_out,
                  float* coef_out, void* ws, size_t ws_bytes, void* stream, int* status_dev);
/* g[i] *= *coef_dev, in place */
int det_scale_inplace(float* g, size_t n, const float* coef_dev, void* stream);

/* ---- LSQ int8 linear (Sec. 3.1 "int8 quantization-aware training"; Sec. 3.2 "int8 computation";
 *      Sec. 4.4 "Quantizer Step-Size Drift": weight steps re-pinned every optimizer step) ------------- */
/* s_w[n] = max(2 * mean_k|W[n,k]| / sqrt(127), 2^-40); per_tensor != 0 fills all N entries with the
 * whole-tensor value.  W bf16 [N,K]; K % 8 == 0. */
size_t det_lsq_weight_scale_ws_bytes(int N, int K);
int det_lsq_weight_scale(const det_bf16* W, int N, int K, int per_tensor, float* s_w, void* ws, size_t ws_bytes,
                         void* stream);
/* s_x[0] = max(2 * mean|x| / sqrt(127), 2^-40) over n elements (LSQ initialisation of the activation step) */
size_t det_lsq_act_scale_init_ws_bytes(size_t n);
int det_lsq_act_scale_init(const det_bf16* X, size_t n, float* s_x, void* ws, size_t ws_bytes, void* stream);
/* Once per optimizer step per linear: qW[n,k] = rne(clamp(W[n,k] * (1/s_w[n]), -128, 127)) (int8 [N,K]) and,
 * for the backward, qWt_bwd int8 [K,N] = quantised (hadamard_block == 128: block-128 Walsh-Hadamard rotated
 * along n, per-tensor absmax step s_u[0]; hadamard_block == 0: plain transpose, s_u[0] = 1) copy.
 * N % 128 == 0, K % 128 == 0.  qWt_bwd / s_u may be NULL to skip the backward copy. */
size_t det_lsq_quantize_weight_ws_bytes(int N, int K);
int det_lsq_quantize_weight(const det_bf16* W, const float* s_w, int N, int K, int hadamard_block, int8_t* qW,
                            int8_t* qWt_bwd, float* s_u, void* ws, size_t ws_bytes, void* stream);

/* Forward: qX = rne(clamp(X * (1/s_x), -128, 127)) (saved to qX_save, int8 [M,K], required),
 * acc = qX . qW^T in int32 on the tensor cores (exact), Y[m,n] = bf16(float(acc) * (s_x * s_w[n])).
 * X bf16 [M,K], qW int8 [N,K], Y bf16 [M,N].  M % 128 == 0, N % 128 == 0, K % 128 == 0, K < 2^17. */
int det_linear_fwd(const det_bf16* X, const int8_t* qW, const float* s_x, const float* s_w, int M, int N, int K,
                   det_bf16* Y, int8_t* qX_save, void* stream, int* status_dev);
/* The activation quantiser fused into the kernel that produces the activation (Sec. 3.2 "int8 computation": the
 * linears consume int8 activations).  In a step the step size s_x of a linear is known before its input is produced,
 * so the producer can write the int8 codes beside its bf16 output and the linear takes them ready-made:
 *   det_rmsnorm_fwd_q / det_swiglu_fwd_q / det_attn_fwd_q  =  the plain call, plus q = rne(clamp(y * (1/s_q), -128, 127))
 *   of the bf16 values y it stores (s_q: device scalar; q: int8, same shape and leading dimension as y, 8-byte
 *   aligned, 4-byte for the attention); det_linear_fwd_q = det_linear_fwd without its quantiser pass (qX given).
 * Every output has exactly the bits of the unfused sequence det_<producer>, det_linear_fwd. */
int det_linear_fwd_q(const int8_t* qX, const int8_t* qW, const float* s_x, const float* s_w, int M, int N, int K,
                     det_bf16* Y, void* stream, int* status_dev);
/* Backward (straight-through estimator; both gradient GEMMs in int8 after a block-`hadamard_block`
 * Walsh-Hadamard rotation along the contraction dimension, 0 = no rotation):
 *   dX bf16 [M,K]  = mask_x ? 2^-7 s_a s_u (A_q . U_q) : 0,   A = rotate_n(dY * s_w[n]) quantised per tensor
 *   dW f32  [N,K]  = mask_w ? 2^-7 s_g s_z s_x (G_q^T . Z_q) : 0 (overwritten), G = rotate_m(dY), Z = rotate_m(qX)
 *   ds_x f32 [1]   = LSQ step gradient: det_sum over (m,k) of dXhat * phi, times 1/sqrt(M K 127)
 * mask_x: -128 <= X/s_x <= 127; mask_w likewise per channel.  Same shape limits as the forward, M < 2^17. */
size_t det_linear_bwd_ws_bytes(int M, int N, int K);
int det_linear_bwd(const det_bf16* dY, const det_bf16* X, const int8_t* qX, const det_bf16* W, const int8_t* qWt_bwd,
                   const float* s_x, const float* s_w, const float* s_u, int M, int N, int K, int hadamard_block,
                   det_bf16* dX, float* dW, float* ds_x, void* ws, size_t ws_bytes, void* stream, int* status_dev);
/* ---- RMSNorm (Sec. 3.1 "RMSNorm", FP32 internals) -------------------------------------------------
 * y = (x * rstd) * gamma, rstd = 1 / sqrt(det_sum(x^2) * (1/D) + eps); gamma NULL = gain-free.
 * io: dtype of x, y, gamma, dy, dx (DET_F32 or DET_BF16); rstd f32 [rows]; D % 8 == 0, D <= 8192. */
int det_rmsnorm_fwd(int io, const void* x, const void* gamma, int rows, int D, float eps, void* y, float* rstd,
                    void* stream);
/* bf16 in and out, D <= 2048; also writes the next linear's int8 input (see det_linear_fwd_q) */
int det_rmsnorm_fwd_q(const det_bf16* x, const det_bf16* gamma, int rows, int D, float eps, det_bf16* y, float* rstd,
                      const float* s_q, int8_t* qy, void* stream);
/* dx = rstd * (w - xhat * c), w = dy*gamma, xhat = x*rstd, c = det_sum(w*xhat) * (1/D);
 * dgamma[j] = det_sum over rows of dy[r,j] * xhat[r,j] (f32 [D], may be NULL). */
size_t det_rmsnorm_bwd_ws_bytes(int rows, int D);
int det_rmsnorm_bwd(int io, const void* dy, const void* x, const void* gamma, const float* rstd, int rows, int D,
                    void* dx, float* dgamma, void* ws, size_t ws_bytes, void* stream);

/* ---- per-head operations of the attention block (Sec. 3.1 "QK-norm", "RoPE") --------------------------
 * Rows of 128 values (one head of one token) inside wider token rows: element (t, h, i) of x sits at
 * x[t*ld + h*128 + i]; ld, ld_y, ... are row strides in elements (multiples of 4, >= nh*128); pointers 8-byte
 * aligned; in-place use (y == x) is allowed.  All device pointers; stream-ordered.
 * det_headnorm_fwd: gain-free RMS normalisation of every head: y = bf16(x * rstd),
 *   rstd[t*nh + h] = 1 / sqrt(det_sum(x^2) * 2^-7 + eps)  (the paper normalises queries and keys before RoPE).
 * det_headnorm_bwd: dx = bf16(rstd * (dy - xhat * c)), xhat = x * rstd, c = det_sum(dy * xhat) * 2^-7. */
int det_headnorm_fwd(const det_bf16* x, int ld, int T, int nh, float eps, det_bf16* y, int ld_y, float* rstd,
                     void* stream);
int det_headnorm_bwd(const det_bf16* dy, int ld_dy, const det_bf16* x, int ld, const float* rstd, int T, int nh,
                     det_bf16* dx, int ld_dx, void* stream);
/* Rotary embedding with caller-supplied tables cos_tab, sin_tab f32 [S, 64] (inputs of the step; the paper uses
 * theta = 5e5): the position of token t is t mod S; pairs are (i, i+64):
 *   y_i = bf16(x_i c_i - x_{i+64} s_i),  y_{i+64} = bf16(x_{i+64} c_i + x_i s_i),  every product rounded on its own.
 * inverse != 0 rotates by the opposite angle, which is the backward pass of the rotation. */
int det_rope(const det_bf16* x, int ld, int T, int nh, int S, const float* cos_tab, const float* sin_tab, int inverse,
             det_bf16* y, int ld_y, void* stream);

/* ---- cross-entropy with optional z-loss (Sec. 3.1 "Z-loss"; loss in FP32) ---------------------------
 * per row: m = max z, S = det_sum exp(z - m), lse = m + log S, loss_row = lse - z[target];
 * loss_mean[0] = det_sum(loss_row)/rows (+ z_weight * z_mean), z_mean[0] = det_sum(lse^2)/rows.
 * A target outside [0,V) sets DET_DEV_TARGET and its row contributes zero.  V % 4 == 0. */
size_t det_xent_ws_bytes(int rows, int V);
int det_xent_fwd(const float* logits, const int32_t* target, int rows, int V, float z_weight, float* loss_row,
                 float* lse, float* loss_mean, float* z_mean, void* ws, size_t ws_bytes, void* stream, int* status_dev);
/* in place: logits[r,j] <- (p - [j == target] (+ 2 z_weight lse p)) * scale, p = exp(z - lse) */
int det_xent_bwd(float* logits_inout, const int32_t* target, const float* lse, int rows, int V, float z_weight,
                 float scale, void* stream);

/* ---- causal attention, head_dim 128 (Sec. 3.2: QK^T and softmax in higher precision; BF16 flash
 *      backward that recomputes the weights; Sec. 3.1: grouped queries, sliding windows) -------------------
 * q, k, v: bf16, row (b*S + i) of head h starts at element ld*(b*S+i) + h*128.  H query heads share Hkv
 * key/value heads (H % Hkv == 0; query head h reads key/value head h / (H/Hkv); Hkv == H is multi-head
 * attention).  window == 0: row i sees the keys j <= i; window = W > 0 (multiple of 128): the keys j in (i - W, i].
 * Online softmax over KV tiles of 128 keys in ascending order (a row visits the tiles that hold one of its keys);
 * dot products are sequential over the 128 dimensions; tile row sums are adjacent trees over the 128 slots; P is
 * rounded to bf16 before P.V.  lse f32 [B,H,S].  S % 64 == 0. */
int det_attn_fwd(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int Hkv, int S,
                 int window, det_bf16* out, int ld_out, float* lse, void* stream);
/* det_attn_fwd that also writes the output projection's int8 input qout [B*S, ld_out] (see det_linear_fwd_q) */
int det_attn_fwd_q(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int Hkv, int S,
                   int window, det_bf16* out, int ld_out, float* lse, const float* s_q, int8_t* qout, void* stream);
/* The same forward with the P.V product of every block of 128 keys on the int8 tensor cores (Sec. 3.2: "int8 P.V
 * per block"; the scales are this library's reading): per (batch, key/value head, block) s_v = absmax(V block)/127,
 * q_v = rne(clamp(v * (127/absmax))); per row and block q_p = rne(p * 127) with p = exp(s - m) in [0,1];
 * u = float(sum_j q_p q_v) * (s_v/127); logits, statistics, row sums and o = o*alpha + u as in det_attn_fwd, so lse is
 * identical to det_attn_fwd's and det_attn_bwd applies unchanged.  status_dev (device int, may be NULL) receives
 * DET_DEV_TIMEOUT if the bounded wait for the tensor-core product expires; the output is then undefined. */
int det_attn_fwd_int8pv(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int Hkv, int S,
                        int window, det_bf16* out, int ld_out, float* lse, void* stream, int* status_dev);
/* dq (H heads), dk, dv (Hkv heads) with leading dimension ld_d; every contraction is one sequential ascending sum
 * from +0; the gradient of a shared key/value head runs over its query heads in ascending order and, within a
 * head, over the queries in ascending order.  ws (16-byte aligned, det_attn_bwd_ws_bytes) holds bf16(P) and
 * bf16(dS), [B*H, S, S] each, Delta [B*H, S], and for Hkv < H the f32 accumulators carried between query heads. */
size_t det_attn_bwd_ws_bytes(int B, int H, int Hkv, int S);
int det_attn_bwd(const det_bf16* dout, const det_bf16* q, const det_bf16* k, const det_bf16* v, const det_bf16* out,
                 const float* lse, int ld, int ld_out, int B, int H, int Hkv, int S, int window, det_bf16* dq,
                 det_bf16* dk, det_bf16* dv, int ld_d, void* ws, size_t ws_bytes, void* stream);
/* The same backward with the query gradient accumulated over the key blocks in 64-bit fixed point (Sec. 3.2: "accumulates
 * the query gradient in 64-bit fixed point for bitwise reproducibility"; scale and rounding are this library's
 * reading): per block of 128 keys the ordered f32 sum u over the block's keys from +0; its contribution is
 * rne(u * 2^48) as a signed 64-bit integer (saturated at the ends of the range, NaN -> 0); integer additions wrap, so
 * the order of the blocks cannot matter; dq = bf16(f32(acc) * 2^-48) with the conversion rounding to nearest even.
 * dk and dv as in det_attn_bwd; the 64-bit accumulators live in registers, so the workspace has det_attn_bwd's size. */
size_t det_attn_bwd_fixq_ws_bytes(int B, int H, int Hkv, int S);
int det_attn_bwd_fixq(const det_bf16* dout, const det_bf16* q, const det_bf16* k, const det_bf16* v, const det_bf16* out,
                      const float* lse, int ld, int ld_out, int B, int H, int Hkv, int S, int window, det_bf16* dq,
                      det_bf16* dk, det_bf16* dv, int ld_d, void* ws, size_t ws_bytes, void* stream);

/* ---- elementwise glue (Sec. 3.1: SwiGLU with fused gate/up projection, pre-norm residuals, embedding) */
/* gu bf16 [rows, 2F] (gate | up), h bf16 [rows, F] = silu(gate) * up;  F % 8 == 0 */
int det_swiglu_fwd(const det_bf16* gu, int rows, int F, det_bf16* h, void* stream);
/* det_swiglu_fwd that also writes the down projection's int8 input qh [rows, F] (see det_linear_fwd_q) */
int det_swiglu_fwd_q(const det_bf16* gu, int rows, int F, det_bf16* h, const float* s_q, int8_t* qh, void* stream);
int det_swiglu_bwd(const det_bf16* dh, const det_bf16* gu, int rows, int F, det_bf16* dgu, void* stream);
/* y = bf16(a + b); y may alias a or b; n % 8 == 0 */
int det_residual_add(const det_bf16* a, const det_bf16* b, size_t n, det_bf16* y, void* stream);
int det_embed_fwd(const int32_t* tok, int T, const det_bf16* E, int V, int D, det_bf16* y, void* stream);
/* dE f32 [V,D] is overwritten: rows of unused tokens are zero; a row used several times is the sequential
 * sum of its positions' gradients in ascending position, from +0.  D % 4 == 0. */
int det_embed_bwd(const int32_t* tok, int T, const det_bf16* dy, int V, int D, float* dE, void* stream);

/* ---- LM head in full precision (Sec. 3.2: excluded from quantisation) -------------------------------
 * logits[m,n] = sequential-k f32 sum from +0 of the exact products H[m,k] W[n,k].  K % 16 == 0. */
int det_lmhead_fwd(const det_bf16* H, const det_bf16* W, int M, int V, int K, float* logits, void* stream);
/* dlogits is rounded to bf16 first.  dH bf16 [M,K]: sum over the vocabulary ascending.  dW f32 [V,K]: sum over
 * tokens ascending, continuing from the value already in dW unless first_chunk != 0.  V % 16 == 0, M % 8 == 0. */
int det_lmhead_bwd(const float* dlogits, const det_bf16* H, const det_bf16* W, int M, int V, int K, det_bf16* dH,
                   float* dW, int first_chunk, void* stream);

/* Arithmetic version 2 of the forward contraction (optional mode; version 1 above stays the default and the benchmark's
 * arithmetic).  Built from the paper's two integer devices (Sec. 3.2: int8 products accumulated exactly in int32; a wide
 * exact integer total "for bitwise reproducibility"): the result does not depend on the order of the terms at all.
 *   per row x of H and of W:  E = largest biased bf16 exponent of the row (0 for an all-zero row; subnormals count as 0);
 *     T_k = ((128 + fraction_k) << 6) >> (E - E_k) with the sign of x_k: x_k is replaced by T_k 2^(E - 140) (values within
 *     2^-6 of the row's largest are exact, smaller ones truncated toward zero); T_k = 128 hi_k + lo_k, two signed int8 slices
 *   logits[m,n] = binary32 nearest-even rounding of I 2^(E(H_m) + E(W_n) - 280),  I = sum_k Ta_k Tb_k
 *     = 2^14 sum(ha hb) + 2^7 (sum(ha lb) + sum(la hb)) + sum(la lb), the four sums exact in int32 on the tensor cores;
 *     ONE rounding; a result below 2^-126 after it is a signed zero; a row with an infinity or a NaN gives NaN.
 * M % 128 == 0, V % 128 == 0, K % 128 == 0, contraction length < 2^16 (the accumulator of the two cross products holds
 * 2 K 127^2).  ws: det_lmhead_fwd_v2_ws_bytes (the int8 slices and row exponents). */
size_t det_lmhead_fwd_v2_ws_bytes(int M, int V, int K);
int det_lmhead_fwd_v2(const det_bf16* H, const det_bf16* W, int M, int V, int K, float* logits, void* ws, size_t ws_bytes,
                      void* stream, int* status_dev);
/* The two gradient contractions in version 2: the same contraction on transposed operands, the shared exponent always taken
 * over the contracted index.  g = bf16(dlogits) (rounded once, as in version 1);
 *   dH[m,k] bf16 = bf16(contraction over the vocabulary of row m of g with column k of W),
 *   dW[v,k] f32  = contraction over the tokens of column v of g with column k of H (overwritten; a micro-batch is one call).
 * Same shape limits; M, V < 2^16.  ws: det_lmhead_bwd_v2_ws_bytes (about 4 M V + 2 K (M + V) bytes). */
size_t det_lmhead_bwd_v2_ws_bytes(int M, int V, int K);
int det_lmhead_bwd_v2(const float* dlogits, const det_bf16* H, const det_bf16* W, int M, int V, int K, det_bf16* dH, float* dW,
                      void* ws, size_t ws_bytes, void* stream, int* status_dev);

/* Causal attention in arithmetic version 2 (optional mode; head dimension 128, one key/value head per query head, no
 * window): the two contractions of the forward pass become the order-free contraction of det_lmhead_fwd_v2 (Sec. 3.2:
 * exact integer products and a wide exact total "for bitwise reproducibility"), the softmax keeps the binary32
 * arithmetic of det_attn_fwd.  With no order to respect there are no key tiles and no rescaling:
 *   s_ij = fmul(C(q_i, k_j), 1/sqrt(128) in binary32), C over the 128 dimensions with the exponents of the two rows;
 *   m_i = max_j s_ij, p_ij = det_exp(s_ij - m_i), l_i = det_sum(p_i0 .. p_ii), lse_i = m_i + det_log(l_i);
 *   u_ic = C(bf16(p_i.), v_.c) over the keys 0 .. i, the exponent of a row of weights over its keys and the exponent of a
 *   column of v over ALL keys of its sequence; out_ic = bf16(fmul(u_ic, fdiv(1, l_i))).
 * q, k, v, out, lse laid out as for det_attn_fwd.  S % 128 == 0, S <= 8192, ld % 8 == 0.  ws: det_attn_fwd_v2_ws_bytes
 * (slices, exponents, the f32 logits [B*H, S, S] and the sliced weights: about 6 B H S^2 bytes).  status_dev (device
 * int, may be NULL) receives DET_DEV_TIMEOUT if a bounded wait of the tensor-core kernels expires. */
size_t det_attn_fwd_v2_ws_bytes(int B, int H, int S);
int det_attn_fwd_v2(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int S, det_bf16* out,
                    int ld_out, float* lse, void* ws, size_t ws_bytes, void* stream, int* status_dev);

/* ---- gradient accumulation = single-device replay of the data-parallel reduction
 *      (Sec. 6, Algorithm 1; Appendix A, Algorithm 2 "TreeFold"; A.3 reciprocal-multiply averages) -------
 * The state is a caller-owned POD; bufs holds det_grad_accum_nbufs(dp_replicate) * n floats on the device. */
typedef struct {
  int accum, dp_shard, dp_replicate, pushes, nstack;
  int level[34];
  int slot[34];
  unsigned long long free_mask;
  size_t n;
  float* bufs;
  int inner_slot, gr_slot;
} det_accum;
int det_grad_accum_nbufs(int dp_replicate);
int det_grad_accum_init(det_accum* st, int accum, int dp_shard, int dp_replicate, size_t n, float* bufs);
/* micro-batch gradients in mesh order: rank r = replica * dp_shard + shard, then k = 0..accum-1 */
int det_grad_accum_push(det_accum* st, const float* g_microbatch, void* stream);
/* DET_ERR_ARG unless exactly accum * dp_shard * dp_replicate pushes were made */
int det_grad_accum_result(det_accum* st, float* g_out, void* stream);

/* ---- AdamW (Sec. 3.2 "Optimizer", "Optimizer-state precision": FP32 moments, one BF16 rounding) ------- */
typedef struct {
  double lr, beta1, beta2, eps, weight_decay; /* weight_decay = 0 for embedding, norms and LSQ steps */
  int step;                                   /* t >= 1 */
} det_adamw_desc;
/* p: bf16 (pdtype DET_BF16) or f32 (DET_F32) parameters, updated in place; g, m, v f32 */
int det_adamw_step(const det_adamw_desc* h, int pdtype, void* p, const float* g, float* m, float* v, size_t n,
                   void* stream);

/* ---- tensor hash (Appendix B: per-step state hash, here on the device) --------------------------------
 * Level 1: SHA-256 of every 4 KiB chunk of the raw bytes (last chunk may be shorter).  While more than 128
 * digests remain, the concatenated digests are hashed again in 4 KiB blocks (128 digests each).  root = SHA-256(remaining digests
 * || u64le(nbytes)), finished on the host; every level below it runs on the device.  p device, 16-byte aligned;
 * ws device, 16-byte aligned, det_tensor_hash_ws_bytes(nbytes) bytes; out32_host receives 32 bytes.
 * Synchronises `stream`. */
size_t det_tensor_hash_ws_bytes(size_t nbytes);
int det_tensor_hash(const void* p, size_t nbytes, uint8_t* out32_host, void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif
