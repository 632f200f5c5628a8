/* det_test.h -- test hooks of libdet.  Not part of the product boundary (include/det.h): these calls exist so that
 * tests can reach pieces that no product call exposes on their own.  Same conventions as det.h (device pointers,
 * stream-ordered, status codes). */
#ifndef DET_TEST_H
#define DET_TEST_H
#include "det.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Elementwise evaluation of one primitive of Sec. 2.1 ("Reproducible Operations") on device arrays: op 0 add, 1 sub,
 * 2 mul, 3 div, 4 sqrt(a), 5 det_exp(a), 6 det_log(a), 7 max, 8 bf16 round trip of a, 9 unfused a*b+b, 10 the form of
 * det_exp the softmax kernels use for arguments a <= 0 or NaN (same bits as op 5 there).  b may be NULL for unary ops.  Lets a test compare the device arithmetic with the CPU statement of the same rule. */
int det_test_prim(int op, const float* a, const float* b, float* out, size_t n, void* stream);

/* The GEMM core of the LSQ linears alone (Sec. 3.2 "int8 computation"): exact int8 x int8 -> int32 contraction
 * C[i,j] = sum_k A[i,k] B[j,k] on tcgen05.  I % 128 == 0, J % 128 == 0, K % 128 == 0, K < 2^17.  force_one_cta != 0
 * keeps the one-CTA kernel where the two-CTA 256 x 256 tiles (cta_group::2) would otherwise be chosen (both output
 * dimensions multiples of 256); integer accumulation is exact, so both give the same result. */
int det_test_igemm_tn(const int8_t* A, const int8_t* B, int I, int J, int K, int32_t* C, int force_one_cta, void* stream,
                      int* status_dev);

/* The bounded wait used by every kernel that waits on an mbarrier (TMA loads, tensor-core commits): one warp waits on a
 * barrier that nothing completes; after limit_cycles SM clocks (at most 4e9) the wait gives up, ORs DET_DEV_TIMEOUT into
 * *status_dev (device int) and the kernel returns, leaving the context usable.  No counterpart in the paper: it exists
 * so that the time-out path can be exercised without making a real kernel hang. */
int det_test_wait_timeout(int* status_dev, long long limit_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif
