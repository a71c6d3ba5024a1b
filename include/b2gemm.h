/*
 * b2gemm -- real GEMM for NVIDIA B200 (sm_100a) computed as a register-blocked sequence of
 * rank-1 outer-product updates over staged panels of A and B, plus a complex entry built
 * from four real-kernel calls.
 *
 * Source of the operation.  The paper's micro-kernel (Section 2.1, "The micro-kernel") is
 *     C += A B = sum_{p<kc} a_p b_p^T          (C is mr x nr, A is mr x kc, B is kc x nr)
 * wrapped in the GotoBLAS/BLIS loop nest (Section 2, Figure 1).  The paper stops at
 * C += A B; scaling by alpha and beta, transposition, leading dimensions and edge sizes
 * follow the level-3 BLAS statement of GEMM:
 *     C := alpha * op(A) * op(B) + beta * C,   op(X) = X or X^T,
 * with column-major storage, X(r, c) = X[r + c * ldx].
 *
 * Conventions shared by every entry point unless its comment says otherwise
 *   - A, B, C (and any workspace) are DEVICE pointers owned by the caller.  No call allocates
 *     or frees device or host memory.  What the library does hold, from the moment it is loaded
 *     (or from the first call that needs it) until the process exits, is: the scratch array of
 *     b2_zgemm4m_static (B2_ZGEMM4M_STATIC_BYTES of device memory on every GPU that loads the
 *     library), two device status words (b2_device_status), per-device caches of symbol
 *     addresses, shared-memory attributes and the SM count, per host thread the last sixteen
 *     kernel choices of the selector (a pure function of the problem's shape), and, for the
 *     host-buffer forms, two helper streams and a few events per device.  None of it carries
 *     results from one call to the next.
 *   - Threads: the per-device caches are filled on first use through atomic slots and one-time
 *     initialisers, so host threads may make their first calls concurrently.  Calls that share
 *     an output or a workspace must be ordered by the caller.
 *   - Scalars are passed by value from the host.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t cast to void*; NULL = the legacy
 *     default stream) and the call returns without synchronising.
 *   - trans in {N,n,T,t,C,c}; for real data C means T.
 *   - m, n, k >= 0;  lda >= max(1, transa==N ? m : k);  ldb >= max(1, transb==N ? k : n);
 *     ldc >= max(1, m).
 *   - Return value: 0 on success; -i when the i-th argument is illegal, counted as in the
 *     reference BLAS: transa 1, transb 2, m 3, n 4, k 5, alpha 6, A 7, lda 8, B 9, ldb 10,
 *     beta 11, C 12, ldc 13 (nothing is launched); a positive b2_status for run-time failures.
 *   - Quick returns: m==0 or n==0 does nothing.  alpha==0 or k==0 computes C := beta*C and
 *     never reads A or B.  beta==0 writes C without reading it (NaN/Inf in the old C do
 *     not propagate).  alpha==0 and beta==1 does nothing.
 *   - Rows r >= m of a column of C, and rows of A/B beyond the operand's row count (the
 *     padding ld - rows), are never written and their contents never influence a result.
 *   - A and B must not overlap C.
 *   - Arithmetic: IEEE round-to-nearest, fused multiply-add, denormals kept; fp32 entries
 *     use FP32 FMA only (no TF32).  The order of the k-summation is unspecified.
 */
#ifndef B2GEMM_H_
#define B2GEMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  B2_OK = 0,
  B2_ERR_TIMEOUT = 1001,   /* a bounded device-side wait gave up */
  B2_ERR_LAUNCH = 1002,    /* the CUDA runtime refused a launch or a copy */
  B2_ERR_WORKSPACE = 1003, /* workspace pointer null, misaligned or too small */
  B2_ERR_VARIANT = 1004,   /* unknown or inapplicable kernel variant */
  B2_ERR_STATIC_LIMIT = 1005 /* problem needs more scratch than the built-in array of b2_zgemm4m_static holds */
} b2_status;

/* Kernel variants (micro-kernel x tile).  B2_VARIANT_AUTO lets the analytic selector choose. */
#define B2_VARIANT_AUTO (-1)

/*
 * Double-precision GEMM, C := alpha*op(A)*op(B) + beta*C  (micro-kernel sum of Section 2.1;
 * BLAS semantics as stated at the top of this file).  All pointers are device pointers.
 */
int b2_dgemm(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha, const double* A,
             int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
             void* cuda_stream);

/* Single-precision GEMM, same definition; FP32 FMA arithmetic only. */
int b2_sgemm(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
             int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
             void* cuda_stream);

/*
 * The same two operations with an explicit kernel variant, 0 <= variant < b2_variant_count(dtype),
 * or B2_VARIANT_AUTO.  Used by tests and benchmarks to exercise every micro-kernel; a variant
 * that cannot serve the given shape/alignment returns B2_ERR_VARIANT and launches nothing
 * (the TMA-staged variants need 16-byte aligned columns of A and B; the fp32 one, "ffma2_tma",
 * reads each operand in the layout it has in memory and also declines transa = T with transb = N,
 * where neither operand has its C index contiguous).
 * An explicit variant is launched with one CTA per tile; variant + 256*s (s = 2 or 4) asks for
 * the k-loop of every tile to be split over a thread-block cluster of s CTAs, whose partial
 * sums are added in rank order through distributed shared memory (Section 2's kc loop, cut in
 * s pieces; same error bound, bit-exact on integer-valued data, the same bits on every run).
 * Variants that cannot split (the TMA-staged and scalar-FMA ones) return B2_ERR_VARIANT.
 */
int b2_dgemm_variant(int variant, char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha,
                     const double* A, int64_t lda, const double* B, int64_t ldb, double beta, double* C,
                     int64_t ldc, void* cuda_stream);
int b2_sgemm_variant(int variant, char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha,
                     const float* A, int64_t lda, const float* B, int64_t ldb, float beta, float* C,
                     int64_t ldc, void* cuda_stream);

/*
 * Device-side status.  Kernels that wait on hardware barriers (the TMA-staged variants) bound
 * every wait; when a bound is hit they record B2_ERR_TIMEOUT in a status word on the device,
 * stop computing and return, leaving C unspecified.  b2_device_status synchronises `cuda_stream`,
 * returns that word (B2_OK when nothing happened) and clears it; B2_ERR_LAUNCH when the
 * synchronisation or the copy fails.  It is the only call of this library that blocks besides
 * the host-buffer forms.
 */
int b2_device_status(void* cuda_stream);
/*
 * Self-test of that mechanism: enqueues a one-warp kernel that waits, with a bound of a few
 * thousand polls, on a barrier nothing completes, so the next b2_device_status returns
 * B2_ERR_TIMEOUT.  Nothing faults or hangs.  Returns 0 or B2_ERR_LAUNCH.
 */
int b2_selftest_wait_timeout(void* cuda_stream);

/* dtype codes for the query calls */
#define B2_F64 0
#define B2_F32 1

/* Number of kernel variants for a dtype, and a static, NUL-terminated description of one
 * ("dmma_128x128x16_s4" ...); NULL when out of range. */
int b2_variant_count(int dtype);
const char* b2_variant_name(int dtype, int variant);

/*
 * Writes a NUL-terminated JSON object describing what the selector would launch for this
 * problem (variant, CTA tile, kc, stages, micro-kernel, grid, and "k_split": over how many CTAs of a
 * thread-block cluster the k-loop of each tile is divided, 1 = not divided; "grid" counts all CTAs) into
 * json_out (HOST memory, capacity cap bytes).  Returns 0, a negative argument index as above (dtype is
 * argument 1 here, the rest shift by one), or B2_ERR_WORKSPACE when cap is too small.
 * Nothing is launched.  The answer is the one for a beta other than 0 and 1; with beta 0 or 1 and
 * 16-byte aligned columns of C an fp32 update with k <= 1024 on enough tiles goes to the TMA-staged
 * kernel instead (its tiles then leave through shared memory).  The tile derivation follows the paper's register-limit formula
 * (Section 5, "Limits imposed by registers") and pipeline-throughput estimate (Section 4).
 */
int b2_gemm_query_config(int dtype, char transa, char transb, int64_t m, int64_t n, int64_t k, int64_t lda,
                         int64_t ldb, int64_t ldc, char* json_out, size_t cap);

/*
 * Complex double GEMM (interleaved re,im; column-major; leading dimensions in complex
 * elements) built from four real-kernel launches ("4M"): the paper names complex GEMM only
 * as a consumer of the real kernel (Abstract).  With A' = alpha*A rounded once per component,
 *     Cr = A'r*Br - A'i*Bi + (beta*C)r,   Ci = A'r*Bi + A'i*Br + (beta*C)i.
 * alpha and beta point to HOST {re, im} pairs.  transa/transb accept N, T and C (conjugate
 * transpose: the operand's imaginary plane is negated while it is split, then the real
 * kernels see a plain transpose).  workspace is DEVICE memory of at least
 * b2_zgemm4m_workspace_bytes(...) bytes, 256-byte aligned, owned by the caller; its contents
 * are overwritten.  Argument numbering as above with workspace = 14.
 */
size_t b2_zgemm4m_workspace_bytes(char transa, char transb, int64_t m, int64_t n, int64_t k);
int b2_zgemm4m(char transa, char transb, int64_t m, int64_t n, int64_t k, const double alpha[2], const void* A,
               int64_t lda, const void* B, int64_t ldb, const double beta[2], void* C, int64_t ldc,
               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same operation from THREE real products ("3M") instead of four:
 *     T1 = A'r*Br,  T2 = A'i*Bi,  T3 = (A'r + A'i)*(Br + Bi),
 *     Cr = ((beta*C)r + T1) - T2,   Ci = (((beta*C)i - T1) - T2) + T3.
 * A quarter less arithmetic; the imaginary part is a difference of larger numbers, so each
 * component's error is bounded relative to sum_p (|Ar|+|Ai|)_ip (|Br|+|Bi|)_pj rather than to
 * the component's own products (not in the paper, which names complex GEMM only as a
 * consumer of the real kernel).  Arguments, transposes, quick returns, error returns and
 * workspace rules as for b2_zgemm4m, with b2_zgemm3m_workspace_bytes(...) bytes (nine planes).
 */
size_t b2_zgemm3m_workspace_bytes(char transa, char transb, int64_t m, int64_t n, int64_t k);
int b2_zgemm3m(char transa, char transb, int64_t m, int64_t n, int64_t k, const double alpha[2], const void* A,
               int64_t lda, const void* B, int64_t ldb, const double beta[2], void* C, int64_t ldc,
               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * b2_zgemm4m for callers that cannot allocate device memory.  (The paper has no counterpart;
 * this is a convenience of the library.)
 *
 * Some callers have no way to obtain a workspace: code that runs where cudaMalloc is off
 * limits (inside a latency-critical loop that must not take the allocator's lock, in a
 * plug-in whose host forbids allocation, after the application has handed all device memory
 * to its own pool).  For them the six real planes of the 4M scheme live in a scratch array
 * that is part of the library image: B2_ZGEMM4M_STATIC_BYTES bytes of device memory on every
 * GPU that loads the library, held until the process exits.  The caller passes only the
 * operands; same arguments, semantics and return values as b2_zgemm4m otherwise.
 *
 *   - Limit: b2_zgemm4m_workspace_bytes(transa, transb, m, n, k) must not exceed
 *     B2_ZGEMM4M_STATIC_BYTES (6 MiB: e.g. m = n = k = 256 needs 3 MiB, 360^3 just fits).
 *     Larger problems return B2_ERR_STATIC_LIMIT and launch nothing.  The limit applies after
 *     the argument checks and the quick returns, i.e. only to calls that really split planes:
 *     an illegal argument still returns -i, and m == 0, n == 0, alpha == 0 or k == 0 behave as
 *     in b2_zgemm4m whatever the sizes.
 *   - The call allocates and frees nothing, neither directly nor through a library.
 *   - The first call on each device looks up the array's device address (the device must be
 *     current); make that first call outside any stream capture.  Host threads that make it
 *     together each look the address up and store the same value.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.
 *     Nothing in it has to start at zero (every plane element is written before it is read
 *     within a call), but two calls that overlap on the GPU -- different streams, or
 *     different host threads -- race on it: serialise them.
 */
#define B2_ZGEMM4M_STATIC_BYTES (6u << 20)
int b2_zgemm4m_static(char transa, char transb, int64_t m, int64_t n, int64_t k, const double alpha[2],
                      const void* A, int64_t lda, const void* B, int64_t ldb, const double beta[2], void* C,
                      int64_t ldc, void* cuda_stream);

/*
 * Symmetric rank-k update on the GEMM kernel (the paper names the level-3 BLAS as consumers of its kernel,
 * Abstract and Introduction; the definition is the BLAS one):
 *     trans = N:  C := alpha*A*A^T + beta*C,  A is n x k;      trans = T (or C):  C := alpha*A^T*A + beta*C,  A is k x n.
 * Only the triangle of the n x n matrix C named by uplo ('L': i >= j, 'U': i <= j) is read or written; tiles of
 * the other triangle are not computed.  Device pointers, column-major, conventions as b2_dgemm.  Argument
 * numbering for -i: uplo 1, trans 2, n 3, k 4, alpha 5, A 6, lda 7, beta 8, C 9, ldc 10.
 * lda >= max(1, trans==N ? n : k), ldc >= max(1, n).  alpha == 0 or k == 0 scales the triangle by beta.
 */
int b2_dsyrk(char uplo, char trans, int64_t n, int64_t k, double alpha, const double* A, int64_t lda, double beta,
             double* C, int64_t ldc, void* cuda_stream);
int b2_ssyrk(char uplo, char trans, int64_t n, int64_t k, float alpha, const float* A, int64_t lda, float beta,
             float* C, int64_t ldc, void* cuda_stream);

/*
 * Strided-batched GEMM: `batch` independent problems C_b := alpha*op(A_b)*op(B_b) + beta*C_b of one shape, where
 * A_b = A + b*stride_a, B_b = B + b*stride_b, C_b = C + b*stride_c (strides in elements; stride_a / stride_b may
 * be 0 to share an operand; for batch > 1 stride_c must be at least ldc*(n-1) + m so that results do not overlap).
 * One launch covers up to 65535 problems (the batch index is the grid's second dimension).  Conventions as
 * b2_dgemm.  Argument numbering for -i: transa 1, transb 2, m 3, n 4, k 5, alpha 6, A 7, lda 8, stride_a 9, B 10,
 * ldb 11, stride_b 12, beta 13, C 14, ldc 15, stride_c 16, batch 17.
 */
int b2_dgemm_strided_batched(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha, const double* A,
                             int64_t lda, int64_t stride_a, const double* B, int64_t ldb, int64_t stride_b,
                             double beta, double* C, int64_t ldc, int64_t stride_c, int64_t batch, void* cuda_stream);
int b2_sgemm_strided_batched(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                             int64_t lda, int64_t stride_a, const float* B, int64_t ldb, int64_t stride_b, float beta,
                             float* C, int64_t ldc, int64_t stride_c, int64_t batch, void* cuda_stream);

/*
 * Triangular level-3 routines on the GEMM kernel (the paper names the level-3 BLAS as consumers of its kernel,
 * Abstract and Introduction; the definitions are the BLAS ones).  A is triangular of order m (side 'L') or n
 * (side 'R'); only the triangle named by uplo ('L'/'U') is read, and with diag = 'U' its diagonal is taken as 1
 * and not read.  op(A) = A for transa 'N', A^T for 'T' (or 'C').
 *     b2_dtrmm:  B := alpha*op(A)*B   (side 'L')   or   B := alpha*B*op(A)   (side 'R')
 *     b2_dtrsm:  solve op(A)*X = alpha*B (side 'L') or X*op(A) = alpha*B (side 'R');  X overwrites B
 * B is m x n, column-major, DEVICE memory, updated in place; A is DEVICE memory and is not modified.  alpha == 0
 * sets B to zero without reading A.  No singularity test is made (a zero on the diagonal divides by zero).
 * Method: recursive halving of the triangle puts all but the diagonal blocks of order <= 128 into calls of the
 * GEMM kernel; a diagonal block is handled by a substitution / product kernel in which a warp holds four
 * right-hand sides and walks the block's 32 x 32 sub-blocks in dependency order.
 * The order of summation therefore differs from column-by-column substitution; results satisfy the componentwise
 * residual bound of substitution, |op(A)*X - alpha*B| <= c*na*u*(|op(A)||X| + |alpha*B|), and are exact whenever
 * all intermediate values are exactly representable.
 * Argument numbering for -i: side 1, uplo 2, transa 3, diag 4, m 5, n 6, alpha 7, A 8, lda 9, B 10, ldb 11.
 * Work is enqueued on cuda_stream; nothing is allocated.
 */
int b2_dtrmm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, double alpha, const double* A,
             int64_t lda, double* B, int64_t ldb, void* cuda_stream);
int b2_strmm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, float alpha, const float* A,
             int64_t lda, float* B, int64_t ldb, void* cuda_stream);
int b2_dtrsm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, double alpha, const double* A,
             int64_t lda, double* B, int64_t ldb, void* cuda_stream);
int b2_strsm(char side, char uplo, char transa, char diag, int64_t m, int64_t n, float alpha, const float* A,
             int64_t lda, float* B, int64_t ldb, void* cuda_stream);

/*
 * Split-K GEMM for small m*n with long k.  One CTA per C tile leaves most SMs idle when m*n is small, however
 * long k is; here k is cut into `splits` contiguous chunks (whole 16-deep slabs), the chunks' partial products
 * are computed by one batched launch of the GEMM kernel into workspace planes, and a second kernel stores
 * C = alpha*(P_0 + P_1 + ... ) + beta*C with the planes added in ascending chunk order.  The result therefore
 * does not depend on scheduling (same bits on every run); it is the plain GEMM definition with a different,
 * fixed summation order (the paper, Section 2.1, fixes no order), so the b2_dgemm error bound applies and
 * integer-valued problems are bit-exact.
 *   splits     0 = chosen by the library (b2_gemm_splitk_auto: as many chunks as it takes to fill the SMs with
 *              64 x 64 tiles, each chunk at least 256 deep, at most 64); 1 = plain b2_dgemm; > k is cut to k,
 *              > 65535 to 65535.
 *   workspace  DEVICE memory, 256-byte aligned, at least b2_gemm_splitk_workspace_bytes(dtype, m, n, k, splits)
 *              bytes (dtype 0 = fp64, 1 = fp32; 0 bytes when the call degenerates to the plain GEMM);
 *              owned by the caller, overwritten.
 * Other arguments, quick returns and error numbering as b2_dgemm; splits < 0 returns -14; a missing, misaligned or
 * short workspace returns B2_ERR_WORKSPACE and launches nothing.
 */
int b2_gemm_splitk_auto(int64_t m, int64_t n, int64_t k);
size_t b2_gemm_splitk_workspace_bytes(int dtype, int64_t m, int64_t n, int64_t k, int splits);
int b2_dgemm_splitk(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha, const double* A,
                    int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc, int splits,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);
int b2_sgemm_splitk(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                    int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc, int splits,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * fp32 GEMM on the tensor cores in TF32 -- separate entry points because TF32 changes results (b2_sgemm
 * never uses it).  The paper has no counterpart; the operation is the same BLAS GEMM with the products taken
 * in the TF32 format (1 sign, 8 exponent, 10 mantissa bits) and accumulated in fp32:
 *   b2_sgemm_tf32x1   both operands rounded to nearest TF32 (ties away from zero): element error about
 *                     2^-10 * (|alpha| |A||B|)_ij;
 *   b2_sgemm_tf32x3   each operand split into a TF32 head and tail, the three leading products added
 *                     (head*head + head*tail + tail*head): back at fp32 accuracy, three times the work.
 * Same arguments, quick returns and error codes as b2_sgemm, plus a DEVICE workspace of at least
 * b2_sgemm_tf32_workspace_bytes(terms, m, n, k) bytes (terms = 1 or 3), 256-byte aligned, owned by the caller
 * and overwritten (it receives the packed, rounded K-major panels of op(A) and op(B)); argument 14.
 * Any alignment and leading dimension of A, B, C is accepted; m and n up to 65535*64 and 3*k below 2^31
 * (beyond that B2_ERR_VARIANT, nothing launched).  Bounded device-side waits: b2_device_status.
 */
size_t b2_sgemm_tf32_workspace_bytes(int terms, int64_t m, int64_t n, int64_t k);
int b2_sgemm_tf32x1(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                    int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc, void* workspace,
                    size_t workspace_bytes, void* cuda_stream);
int b2_sgemm_tf32x3(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                    int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc, void* workspace,
                    size_t workspace_bytes, void* cuda_stream);

/*
 * Host-buffer forms: A, B, C are HOST pointers (pinned memory makes the copies asynchronous),
 * dev_workspace is DEVICE memory of at least b2_gemm_host_workspace_bytes(...) bytes owned by
 * the caller.  The call copies the referenced parts of A and B (and C when beta != 0) to the
 * device, runs the kernels of b2_dgemm / b2_sgemm, copies the m x n result back into C and
 * synchronises the stream before returning.  Copies and compute are pipelined on two helper streams
 * that the library creates on its first such call on a device and keeps (no device memory is
 * allocated); these calls are serialised among host threads.  Problems with k < 2048 or fewer than
 * 2^22 elements of C are pipelined over column panels of C, each panel one b2_dgemm / b2_sgemm
 * call: the same bits as the device form.  Larger ones travel and are multiplied chunk by chunk
 * along k, so that the multiplication starts when an eighth of A and B has arrived, and finish
 * column panel by column panel, so that the copy back overlaps it: C = (...((alpha A_1 B_1) +
 * alpha A_2 B_2) + ...) + beta C, the same error bound as the single call, exact on integer
 * data, not the same rounding otherwise; their workspace holds a second buffer of C's size.
 * Argument numbering as b2_dgemm, workspace = 14.
 */
size_t b2_gemm_host_workspace_bytes(int dtype, char transa, char transb, int64_t m, int64_t n, int64_t k);
int b2_dgemm_host(char transa, char transb, int64_t m, int64_t n, int64_t k, double alpha, const double* A,
                  int64_t lda, const double* B, int64_t ldb, double beta, double* C, int64_t ldc,
                  void* dev_workspace, size_t workspace_bytes, void* cuda_stream);
int b2_sgemm_host(char transa, char transb, int64_t m, int64_t n, int64_t k, float alpha, const float* A,
                  int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                  void* dev_workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Pipeline-throughput probe (Section 4, "Estimating throughput": the estimate needs each
 * pipeline's rate).  Launches `ctas` CTAs of `threads_per_cta` threads that each issue
 * `iters` rounds of independent register-resident multiply-adds of the given kind and
 * returns.  scratch is DEVICE memory of at least 64 + 8*ctas bytes; after the stream has
 * drained, the int64 at byte offset 64 + 8*b holds the SM clock cycles CTA b spent in the
 * loop.  *fma_per_thread_iter (HOST) receives the multiply-adds one thread performs per round,
 * so rate = threads * iters * (*fma_per_thread_iter) / cycles.  Returns 0, -i for a bad
 * i-th argument, or B2_ERR_LAUNCH.
 */
#define B2_PROBE_DFMA 0
#define B2_PROBE_FFMA 1
#define B2_PROBE_DMMA_M8N8K4 2
#define B2_PROBE_DMMA_M16N8K4 3
#define B2_PROBE_DMMA_M16N8K8 4
#define B2_PROBE_DMMA_M16N8K16 5
#define B2_PROBE_FFMA2 6 /* packed fp32 pair multiply-add, fma.rn.f32x2 */
/*
 * Instruction-mix kinds: one round is one 16-deep slab of a GEMM micro-kernel's inner loop -- per k the
 * shared-memory fragment loads and the multiply-adds of one rank-1 update of the CTA tile, the code the GEMM
 * kernels run -- over slabs that stay in shared memory (no global traffic, no staging).  threads_per_cta must
 * be the micro-kernel's CTA size (128, but 64 for the 4 x 4 kind; -2 otherwise); the CTAs per SM are the caller's choice
 * through `ctas`.  OR-ing B2_PROBE_WITH_BARRIER adds the one CTA-wide barrier per slab of the cp.async-staged
 * kernels.  The rate such a probe reaches is the ceiling of that instruction mix at that residency.
 */
#define B2_PROBE_MIX_FFMA2_8X8 7  /* fp32 128 x 64 tile, 8 x 8 per thread: 32 fma.rn.f32x2 + 4 ld.shared.v4 per k */
#define B2_PROBE_MIX_FFMA2_16X8 8 /* fp32 128 x 128 tile, 16 x 8 per thread: 64 fma.rn.f32x2 + 6 ld.shared.v4 per k */
#define B2_PROBE_MIX_DMMA_64X64 9 /* fp64 64 x 64 tile, 32 x 32 per warp: 8 mma.m16n8k4 + 6 fragment loads per 4 k */
#define B2_PROBE_MIX_FFMA_8X8 10  /* fp32 128 x 64 tile, 8 x 8 per thread, scalar: 64 fma.rn.f32 + 4 ld.shared.v4 per k */
#define B2_PROBE_MIX_FFMA2_4X4 11 /* fp32 32 x 32 tile of 64 threads, 4 x 4 per thread: 8 fma.rn.f32x2 + 2 ld.shared.v4 */
#define B2_PROBE_MIX_DFMA_8X8 12  /* fp64 128 x 64 tile, 8 x 8 per thread: 64 fma.rn.f64 + 8 ld.shared.v2 per k */
#define B2_PROBE_WITH_BARRIER 0x100
int b2_pipe_probe(int kind, int threads_per_cta, int ctas, int64_t iters, void* scratch, size_t scratch_bytes,
                  double* fma_per_thread_iter, void* cuda_stream);

/*
 * The paper's analytical model (host-only calls; nothing is launched, no GPU is needed).
 *
 * b2_model_throughput: Section 4 ("Little's Law").  Pipelines i = 0..npipes-1 retire rate[i]
 *   instructions per cycle; an instruction mix puts jobs[i] instructions on pipeline i per outer
 *   product.  Returns outer products per cycle = min_i rate[i] / jobs[i] over pipelines with
 *   jobs[i] > 0 (infinity when there is none), or -1 for invalid input (npipes <= 0, null
 *   pointers, rate <= 0, jobs < 0).  rate and jobs are HOST arrays.
 * b2_model_stalled_throughput: Section 4 ("Estimating throughput").  A pipeline whose n_dependent
 *   instructions of latency `latency` cannot be overlapped needs W = jobs + n_dependent*latency
 *   cycles; returns 1/W, or -1 for invalid input.
 * b2_model_register_updates: Section 5 ("Limits imposed by registers").  Stores
 *   floor((r_total - mr*nr/v - r_a) / r_r) in *n_updates (HOST); returns 0, -1 for non-positive
 *   sizes, -7 for a null output.
 * b2_model_predict_variant: the Section 4 estimate applied to one sub-partition of a B200 SM
 *   (pipelines: issue, FP64 FMA, FP64 tensor, FP32 FMA, shared-memory wavefronts; rates from
 *   b2_pipe_probe) for kernel variant `variant` of `dtype`.  Stores the predicted fraction of the
 *   arithmetic pipe's peak in *fraction: min(pipeline estimate, L2 feed) x latency coverage (the
 *   paper's sizing rule of Section 4 read as Little's law over all warps of a scheduler).  When
 *   json_out is not NULL it receives a JSON object with the jobs per pipeline per rank-1 update, the
 *   clocks each pipeline needs, the three factors, registers and resident CTAs, the prediction and
 *   the measured steady-state fraction (HOST buffer of cap bytes).  Returns 0, -1/-2/-3 for a bad
 *   dtype / variant / null fraction, B2_ERR_WORKSPACE when cap is too small.
 */
double b2_model_throughput(int npipes, const double* rate, const double* jobs);
double b2_model_stalled_throughput(double jobs, int n_dependent, double latency);
int b2_model_register_updates(int r_total, int mr, int nr, int v, int r_a, int r_r, int* n_updates);
int b2_model_predict_variant(int dtype, int variant, double* fraction, char* json_out, size_t cap);
/*
 * b2_model_enumerate: Section 5.1 ("A Work Flow for Kernel Generation": enumerate the ways to compute the outer
 *   product, estimate each with the model of Section 4, keep the best) for the SM.  Candidates are micro-kernel
 *   kind (dtype 0: DMMA, DFMA; dtype 1: packed-pair and scalar FFMA) x warp tile x warp grid of a CTA x ring
 *   stages; a candidate is kept when it fits the register limit of Section 5 restated for a thread (accumulators
 *   + R_A + at least two unit updates' fragments <= 255, and the SM's register file and shared memory for at
 *   least one CTA; the limits are queried from the current device, B200 values without one).  Each is scored
 *   with predicted fraction = min(pipeline estimate, L2 feed) x latency coverage at the residency it reaches.
 *   json_out (HOST, cap bytes) receives {"dtype", "candidates", "ranked": [...]} with the best `top` candidates in
 *   rank order and, whatever their rank, the candidates that exist as variants of this library ("built_as").
 *   Returns 0, -1 / -2 / -3 for a bad dtype / top <= 0 / null buffer, B2_ERR_WORKSPACE when cap is too small.
 */
int b2_model_enumerate(int dtype, int top, char* json_out, size_t cap);

/* Static, NUL-terminated text for a return value of any call above. */
const char* b2_strerror(int status);
/* Static, NUL-terminated library version. */
const char* b2_version(void);

#ifdef __cplusplus
}
#endif
#endif /* B2GEMM_H_ */
