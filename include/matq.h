/*
 * matq.h — C ABI of the B200 (sm_100a) library for the nested
 * int8 -> int4 -> int2 weight path of Matryoshka Quantization (MatQuant).
 *
 * Notation (the paper's): W is a weight matrix with N output channels (rows)
 * and K input features, stored row-major as bf16; c = 8 is the width of the
 * base code; r (1 <= r <= c) is the width sliced out of it; alpha and z are
 * the per-output-channel scale and (real-valued) zero point of Eq. 1; x are
 * bf16 activations; y are fp32 outputs.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers owned by the caller unless the comment says
 *     "host".  The library never allocates, frees or keeps a pointer (the one
 *     exception, entry point (5), keeps the address of its own built-in array:
 *     see there).
 *   - `stream` is a cudaStream_t passed as void*.  Work is enqueued on it and
 *     the call returns without synchronising.
 *   - The return value is a status (MATQ_OK = 0).  Argument errors are found on
 *     the host before anything is launched.  Errors that depend on the data
 *     (non-finite weight, overflow list too small) are written by the kernels
 *     into `dev_status` (device int32, nullable; first error wins; the caller
 *     zeroes it) and never trap.
 *   - 16-byte alignment of the matrix pointers and the row-length multiples
 *     stated per call select the vectorised kernels; other shapes are either
 *     served by slower generic kernels or rejected with MATQ_ERR_SHAPE /
 *     MATQ_ERR_ALIGNMENT as stated.
 *   - Thread-safe: calls from several host threads need no locking.  The only
 *     state the library keeps is write-once per device (each kernel's opt-in to
 *     its largest shared-memory size, the address of (5)'s array); (5)'s array
 *     itself is shared by all calls of (5) on a GPU, see there.
 */
#ifndef MATQ_H_
#define MATQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum matq_status {
    MATQ_OK = 0,
    MATQ_ERR_INVALID_ARG = 1,  /* null pointer, negative size, inconsistent optional arguments */
    MATQ_ERR_UNSUPPORTED = 2,  /* c != 8, r outside [1, c], r not packable for this call */
    MATQ_ERR_SHAPE = 3,        /* K (or ld*) is not a multiple the call requires */
    MATQ_ERR_ALIGNMENT = 4,    /* pointer not aligned as the call requires */
    MATQ_ERR_WORKSPACE = 5,    /* workspace missing or too small */
    MATQ_ERR_CUDA = 6,         /* a CUDA runtime call failed (launch error, no sm_100 device) */
    /* written to dev_status by kernels */
    MATQ_ERR_NONFINITE = 8,    /* a weight is NaN or +-Inf */
    MATQ_ERR_CAPACITY = 9,     /* extra-precision overflow list does not fit ovf_capacity */
    MATQ_ERR_TIMEOUT = 10      /* a bounded device-side wait gave up */
};

/* Where matq_gemm_multi takes the weights from. */
enum matq_src_kind {
    MATQ_SRC_BF16 = 0,    /* bf16 W [N, K]; Eq. 1 is applied on the fly, alpha / zero are outputs */
    MATQ_SRC_CODES8 = 1,  /* uint8 codes q [N, K]; alpha / zero are inputs */
    MATQ_SRC_PACKED = 2   /* one packed r-bit plane (+ optional overflow list); n_r must be 1 */
};

/* matq_gemv flags */
enum matq_gemv_flags {
    MATQ_GEMV_AUTO = 0,        /* library picks the kernel */
    MATQ_GEMV_CUDA_CORE = 1,   /* fp32 FMA path */
    MATQ_GEMV_TENSOR = 2,      /* warp-level tensor-core path (mma.sync, bf16 x bf16 -> fp32) */
    MATQ_GEMV_TCGEN05 = 3,     /* tcgen05.mma path: unpacked weights as the TMEM A operand */
    MATQ_GEMV_TENSOR_INT8 = 4, /* warp-level integer tensor-core path (mma.sync, u8 x u8 -> s32) for B = 1 and
                                  K <= 32768: the fields enter as exact 8-bit integers, the activations as the
                                  four bytes of a block-scaled 30-bit integer, sums are exact; anything else
                                  runs the bf16 kernel.  MATQ_GEMV_AUTO takes this path when it applies. */
    MATQ_GEMV_STREAM = 5,      /* persistent integer tensor-core kernel (B = 1, K <= 32768): one CTA per SM, the plane
                                  streamed by bulk copies into a ring in shared memory; the kernel behind
                                  matq_gemv_grouped, here with a list of one */
    MATQ_GEMV_PATH_MASK = 0xff,
    MATQ_GEMV_TEST_STALL = 0x8000, /* matq_gemv_grouped only, for testing the error path: the kernel's producer issues no
                                  copies, so every wait for data runs out (after about a millisecond instead of two
                                  seconds); the call then reports MATQ_ERR_TIMEOUT through dev_status, writes no output
                                  and returns, and the next call on the same stream works as usual */
    MATQ_GEMV_PDL = 0x100      /* launch with programmatic stream serialisation: the kernel starts
                                  fetching weights (plane, alpha, zero, overflow lists) while the previous
                                  kernel in the stream drains and waits for it only before reading x.
                                  Only valid when that previous kernel does not write those weights. */
};

const char *matq_status_string(int status);
int matq_version(void);

/* Bytes per row of a packed r-bit plane: K * r / 8 for r in {8, 4, 2} and K a
 * multiple of 8 / r; -1 otherwise. */
int64_t matq_packed_row_bytes(int64_t K, int r);

/*
 * (1) MinMax quantisation, Eq. 1, one (alpha, z) per output channel:
 *       alpha_n = (max_k W[n,k] - min_k W[n,k]) / (2^c - 1),  z_n = -min_k W[n,k] / alpha_n,
 *       q[n,k]  = clamp(round_half_up(W[n,k] / alpha_n + z_n), 0, 2^c - 1)
 *     with the result of IEEE binary32 arithmetic, one correctly rounded operation
 *     per step in the order written (true division, separate sum): the codes are
 *     defined bit for bit.  (The kernels may reach those bits by other instruction
 *     sequences that reproduce every rounding.)  A constant row gets alpha = 1,
 *     z = -W[n,0], codes 0.
 *   W      in   bf16 [N, K], row stride ldw elements (ldw >= K)
 *   q      out  uint8 [N, K] contiguous; may be NULL when only alpha / zero are wanted
 *   alpha  out  fp32 [N]
 *   zero   out  fp32 [N]
 *   A NaN / Inf weight sets dev_status = MATQ_ERR_NONFINITE; that row's outputs are unspecified.
 *   Fast paths: W 16-byte aligned, q 8-byte aligned, K % 8 == 0, ldw % 8 == 0, K <= 16384 (rows held in
 *   registers); W and q 16-byte aligned, K % 16 == 0, ldw % 8 == 0, K <= 65536 (rows held in shared memory).
 *   Any other shape runs a scalar kernel.  c must be 8.
 */
int matq_quantize(const void *W, int64_t N, int64_t K, int64_t ldw, int c,
                  uint8_t *q, float *alpha, float *zero,
                  int32_t *dev_status, void *stream);

/*
 * (1b) MinMax quantisation with OmniQuant's two clipping scales per output channel (Section 3.1, Eq. 3):
 *       alpha_n = (gamma_n max_k W[n,k] - beta_n min_k W[n,k]) / (2^c - 1),  z_n = -beta_n min_k W[n,k] / alpha_n,
 *       q[n,k]  = clamp(round_half_up(W[n,k] / alpha_n + z_n), 0, 2^c - 1)
 *     in IEEE binary32, one correctly rounded operation per step in the order written (the two products, their
 *     difference, the division by 2^c - 1, the division for z, then per weight as in Eq. 1).  Scales below 1 clip
 *     the range: weights outside it saturate at 0 or 2^c - 1, which is what fills the top bucket that the
 *     extra-precision slice (Eq. 8) keeps.  gamma_n max - beta_n min <= 0 gives alpha = 1, z = -beta_n min.
 *   gamma, beta  in  fp32 [N] device pointers; either may be NULL (= 1 for every row; both NULL is matq_quantize)
 *   A non-finite weight or scale sets dev_status = MATQ_ERR_NONFINITE; that row's outputs are unspecified.
 *   Everything else (W, q, alpha, zero, shapes, alignment, errors) as for matq_quantize.  How gamma and beta are
 *   learned is outside this library.
 */
int matq_quantize_clip(const void *W, int64_t N, int64_t K, int64_t ldw, int c,
                       const float *gamma, const float *beta,
                       uint8_t *q, float *alpha, float *zero,
                       int32_t *dev_status, void *stream);

/*
 * (2) MSB slicing S(q, r) of Eq. 6 (extra_precision = 0) or of the Errata's
 *     Eq. 8 (extra_precision = 1), then packing.  With sh = c - r:
 *       k      = min((q + 2^(sh-1)) >> sh, 2^r - 1)      (k = q when sh = 0)
 *       S(q,r) = k << sh
 *     Plane format: for r in {8, 4, 2}, byte j of a row holds the fields k of
 *     elements j*(8/r) + i, i = 0 .. 8/r - 1, field i in bits [i*r, (i+1)*r).
 *     Rows are contiguous, K*r/8 bytes each.  Slices are always taken from the
 *     c-bit code (Section 3.2), never from another slice.
 *   q                in   uint8 [N, K] contiguous
 *   packed           out  uint8 [N, K*r/8]; NULL allowed (then only the other outputs are written);
 *                         non-NULL requires r in {8, 4, 2} and K % (8/r) == 0
 *   sliced_unpacked  out  uint8 [N, K] = S(q, r) of Eq. 6, any 1 <= r <= 8; NULL allowed
 *                         (an interpolated precision such as r = 6 or 3, Section 5.1, is served in decode by passing
 *                         this array to matq_gemv as an r = 8 plane: dequantisation is alpha * (S - z) either way)
 *   Extra precision (Eq. 8 keeps bucket 2^r): the plane holds the CLAMPED field,
 *   so it is byte-identical to the standard plane, and the elements whose Eq. 8
 *   value is one bucket higher (exactly those with q >= 2^c - 2^(sh-1)) are listed:
 *   ovf_row_ptr      out  int32 [N + 1]; row n's entries are ovf_col[ovf_row_ptr[n] .. ovf_row_ptr[n+1])
 *   ovf_col          out  uint16 [ovf_capacity] column indices, ascending within a row (needs K <= 65536)
 *   ovf_count        out  int64 [1] (device): total number of overflow elements, written even when
 *                         it exceeds ovf_capacity; then dev_status = MATQ_ERR_CAPACITY and ovf_col is unspecified
 *   All three are required iff extra_precision != 0 and r < c; otherwise they are ignored
 *   (ovf_count, if non-NULL, is set to 0).  The result is deterministic.
 */
int matq_slice_pack(const uint8_t *q, int64_t N, int64_t K, int c, int r, int extra_precision,
                    uint8_t *packed, uint8_t *sliced_unpacked,
                    int32_t *ovf_row_ptr, uint16_t *ovf_col, int64_t ovf_capacity, int64_t *ovf_count,
                    int32_t *dev_status, void *stream);

/*
 * (2b) The int4 and the int2 plane of a nested model from ONE read of its int8 codes (Section 3.2: every nested
 *      precision is a slice of the same c-bit code): exactly matq_slice_pack(r = 4) into packed4 (Eq. 6) and
 *      matq_slice_pack(r = 2, extra_precision) into packed2 with its overflow lists (Eq. 6, or Eq. 8's base plane and
 *      lists), bit for bit, at 1.75 instead of 2.75 bytes of HBM traffic per weight.  One kernel when K % 16 == 0,
 *      K <= 16384, N * K < 2^31, the buffers are 16-byte aligned and extra_precision is set; two calls otherwise.
 *   packed4   out  uint8 [N, K / 2]        packed2   out  uint8 [N, K / 4]       (K % 4 == 0)
 *   the overflow arguments, dev_status and the error behaviour are those of matq_slice_pack for r = 2.
 */
int matq_slice_pack_nested(const uint8_t *q, int64_t N, int64_t K, int c, uint8_t *packed4, uint8_t *packed2,
                           int extra_precision,
                           int32_t *ovf_row_ptr, uint16_t *ovf_col, int64_t ovf_capacity, int64_t *ovf_count,
                           int32_t *dev_status, void *stream);

/*
 * (3) Decode-time weight-only quantised linear layer on a packed r-bit plane:
 *       y[b,n] = sum_k x[b,k] * alpha_n * (S[n,k] - z_n),   S = k << (c - r)
 *     (dequantisation alpha * (S - z) with the same alpha, z at every r, since
 *     Eq. 6 returns values on the c-bit grid).  When the overflow list is given,
 *     S[n,j] is one bucket (2^(c-r)) higher at the listed columns j (Eq. 8).
 *   packed       in   uint8 [N, K*r/8], r in {8, 4, 2}, 16-byte aligned, K % 128 == 0
 *   alpha, zero  in   fp32 [N]
 *   ovf_row_ptr, ovf_col  in   both NULL or both given (format as in matq_slice_pack)
 *   x            in   bf16 [B, K], row stride ldx elements, 1 <= B <= 16, 16-byte aligned, ldx % 8 == 0
 *   y            out  fp32 [B, N], row stride ldy elements
 *   workspace         device scratch of at least matq_gemv_workspace_bytes(...) bytes (may be NULL if that is 0)
 *   flags             matq_gemv_flags; 0 (MATQ_GEMV_AUTO) is the only value a caller needs, MATQ_GEMV_PDL an optimisation for
 *                     chains of calls, the path values exist for tests and measurements
 *   Results differ from an fp64 evaluation by rounding only.  B = 1 (and K <= 32768) sums exact integer
 *   products of the fields with the activations scaled to 30-bit integers by a power of two taken from
 *   max |x| (an activation below 2^-22 of the largest is rounded to an absolute 2^-24 of the largest at worst),
 *   then applies alpha and z in fp32; other batches accumulate bf16 x bf16 products in fp32.
 *   MATQ_GEMV_STREAM with B > 1 (dense rows: ldx == K, ldy == N; no lists) takes the batched integer kernel
 *   described under (3b).
 */
size_t matq_gemv_workspace_bytes(int64_t N, int64_t K, int r, int B);
int matq_gemv(const uint8_t *packed, int64_t N, int64_t K, int c, int r,
              const float *alpha, const float *zero,
              const int32_t *ovf_row_ptr, const uint16_t *ovf_col,
              const void *x, int B, int64_t ldx, float *y, int64_t ldy,
              void *workspace, size_t workspace_bytes, unsigned flags,
              int32_t *dev_status, void *stream);

/*
 * (3b) Several decode GEMVs in ONE launch.  A decoder layer multiplies the same activation vector with
 *      several weight matrices (the query, key and value projections; the gate and up projections of the FFN,
 *      Sections 1 and 5.3), a Mix'n'Match model (Section 3.2.1, Appendix B) gives every layer its own r, and each
 *      plane is only a few megabytes, i.e. a few microseconds of HBM time: a launch per plane is bound by launch
 *      latency, not by the weight traffic that Section 1 names as the cost of decoding.  This call takes a list of
 *      independent problems, each a matq_gemv,
 *        y_i[b,n] = sum_k x_i[b,k] * alpha_i[n] * (S_i[n,k] - z_i[n])    (+ Eq. 8's extra bucket where a list is given),
 *      and runs them with persistent kernels whose CTAs share the list's bytes evenly, whatever the shapes.
 *      Problems may share x or not, may differ in N, K, r and B, and must not depend on one another (no y_i may be
 *      an x_j of the same call).  With one vector per problem (B <= 1) the results are those of matq_gemv's integer
 *      path (exact integer sums, reproducible: a problem gives the same bits alone, in any list and however the list
 *      is split over CTAs).
 *      Batches (2 <= B <= 16, no lists): the plane is read from HBM once for up to 16 vectors (8 at r = 2).  The
 *      sums are exact integers again; what is rounded is the activation, relative to the largest magnitude of ITS
 *      vector.  B = 2, and every batch at r = 2: a 22-bit integer, and a field that sits s bits up in its byte meets its
 *      activation divided by 2^s, so the rounding step is 2^-22 (r = 8), 2^-18 (r = 4), 2^-16 (r = 2) of twice the
 *      vector's largest magnitude (about 1e-6, 2e-5, 6e-5 of rms(y) for Gaussian activations).  B >= 3 at r = 8 and
 *      r = 4: a 15-bit integer and its sign (two signed base-256 digits, four vectors per 8-column MMA instead of
 *      two), a rounding step of 2^-14 of the power of two at or below the vector's largest magnitude (2^-13 when that
 *      magnitude's bf16 significand is all ones), the same for both fields: about 4e-5 of rms(y) for Gaussian
 *      activations, below what the 8-bit significands of the bf16 inputs themselves resolve, and well inside the
 *      1e-2 rms(y) of the tensor-core paths.  In either form a vector whose largest element is thousands of times its
 *      typical one loses accordingly; such vectors belong in problems of their own (B = 1: 30-bit activations) or in
 *      matq_gemv's default path (bf16 products).  A batch that does not fit one launch's shared memory (at K = 9216:
 *      more than 4 vectors) is cut into problems that share the plane; r = 2 batches need K % 256 == 0.
 *   problems   in   HOST array of n_problems descriptors; the pointers inside are DEVICE pointers:
 *                     packed uint8 [N, K*r/8] 16-byte aligned, alpha / zero fp32 [N], ovf_row_ptr / ovf_col both NULL
 *                     or both given (B <= 1 only), x bf16 [K] (or [B, K], rows K apart) 16-byte aligned, y fp32 [N]
 *                     (or [B, N], rows N apart).  r in {8, 4, 2}, K % 128 == 0, K <= 32768.
 *                     A problem with N == 0 is skipped.  The array is read during the call only.
 *   n_problems      any number >= 0; up to 128 problems share a launch, longer lists take several; single vectors
 *                   and batches that need 1, 2 or 4 column groups (of two or of four vectors) go to launches of
 *                   their own
 *   flags           0 or MATQ_GEMV_PDL (MATQ_GEMV_TEST_STALL for tests of the error path; meaning of PDL as for matq_gemv: no plane, alpha, zero or list of the call is
 *                   written by the previous kernel of the stream)
 *   A wait inside the kernel that does not end within about two seconds sets dev_status = MATQ_ERR_TIMEOUT; the
 *   outputs are then unspecified and the kernel still returns.
 */
typedef struct matq_gemv_problem {
    const uint8_t *packed;
    int64_t N, K;
    int r;
    const float *alpha;
    const float *zero;
    const int32_t *ovf_row_ptr;
    const uint16_t *ovf_col;
    const void *x;
    float *y;
    int64_t B;                   /* activation vectors: 0 or 1 = one (x bf16 [K], y fp32 [N]); 2 .. 16 = x bf16 [B, K], y fp32 [B, N], dense rows */
} matq_gemv_problem;
int matq_gemv_grouped(const matq_gemv_problem *problems, int n_problems, int c, unsigned flags,
                      int32_t *dev_status, void *stream);
/* Number of kernel launches matq_gemv_grouped makes for this list (host only, launches nothing); -1 for a list it would refuse. */
int matq_gemv_grouped_launches(const matq_gemv_problem *problems, int n_problems);

/*
 * (4) Multi-precision dense forward of MatQuant co-training (Eq. 7): for every
 *     r in rs, Y_r = X . dequant(S(Q(W, c), r))^T, all precisions from one pass
 *     over the weights.  The integer fields enter the tensor cores exactly as
 *     bf16 (0 .. 255 are exact) with fp32 accumulation; alpha and z * sum_k x
 *     are applied per channel afterwards:
 *       Y_r[m,n] = alpha_n * ( 2^(c-r) * sum_k X[m,k] k_r[n,k]  -  z_n * sum_k X[m,k] ).
 *   Wsrc         in   per src_kind (matq_src_kind)
 *   alpha, zero  out for MATQ_SRC_BF16, in otherwise; fp32 [N]
 *   extra_precision   slice with Eq. 8 instead of Eq. 6 (for MATQ_SRC_PACKED: apply the overflow list)
 *   X            in   bf16 [M, K], row stride ldx
 *   rs           in   HOST array of n_r distinct precisions (1 <= n_r <= 3), e.g. {8, 4, 2}
 *   Y            in   HOST array of n_r device pointers, each fp32 [M, N] with row stride ldy
 *   workspace         device scratch of at least matq_gemm_multi_workspace_bytes(...) bytes
 *   Requires K % 64 == 0, N % 8 == 0, 16-byte aligned pointers.
 */
size_t matq_gemm_multi_workspace_bytes(int src_kind, int64_t M, int64_t N, int64_t K, int n_r);
int matq_gemm_multi(int src_kind, const void *Wsrc, int64_t N, int64_t K, int c,
                    float *alpha, float *zero, int extra_precision,
                    const int32_t *ovf_row_ptr, const uint16_t *ovf_col,
                    const void *X, int64_t M, int64_t ldx,
                    const int *rs, int n_r, float *const *Y, int64_t ldy,
                    void *workspace, size_t workspace_bytes,
                    int32_t *dev_status, void *stream);

/*
 * (4b) The objective of MatQuant co-training for one linear layer (Eq. 7 with the L2 reconstruction loss of Eq. 5):
 *       L_r   = sum_{m,n} ( Yt[m,n] - Y_r[m,n] )^2   for every r in rs, Y_r as in matq_gemm_multi,
 *       total = sum_i lambda[i] * L_{rs[i]}
 *     computed in the epilogue of the same tensor-core pass: the n_r outputs are compared with the target while they
 *     are still in tensor memory and are never written to HBM (for R = {8, 4, 2} that is 12 bytes per output element
 *     not stored).  No 1/N: the caller divides by its sample count.
 *   lambda  in   HOST array of n_r loss weights (Eq. 7's lambda_r)
 *   teacher in   HOST array of n_r ints or NULL (co-distillation, Section 5.2): -1 = precision i is compared with Yt;
 *                j in [0, n_r), j != i = it is compared with Y_{rs[j]}, the output of that (higher-precision) nested
 *                model, instead; 256 + j = with both, the two squared errors added.  NULL = all -1.
 *   Yt      in   fp32 [M, N] target, row stride ldt elements (e.g. the bf16 layer's output F(W_F, X))
 *   loss    out  DEVICE double [n_r + 1]: L_{rs[0]}, ..., L_{rs[n_r-1]}, total.  Per-thread and per-CTA sums are fp32,
 *                the sum over CTAs is double, all in a fixed order: results are reproducible run to run.
 *   workspace    at least matq_gemm_multi_loss_workspace_bytes(...) bytes, 256-byte aligned
 *   Everything else as for matq_gemm_multi.
 */
size_t matq_gemm_multi_loss_workspace_bytes(int src_kind, int64_t M, int64_t N, int64_t K, int n_r);
int matq_gemm_multi_loss(int src_kind, const void *Wsrc, int64_t N, int64_t K, int c,
                         float *alpha, float *zero, int extra_precision,
                         const int32_t *ovf_row_ptr, const uint16_t *ovf_col,
                         const void *X, int64_t M, int64_t ldx,
                         const int *rs, int n_r, const float *lambda, const int *teacher,
                         const float *Yt, int64_t ldt, double *loss,
                         void *workspace, size_t workspace_bytes,
                         int32_t *dev_status, void *stream);

/*
 * (5) matq_gemm_multi without a workspace argument.  The paper has no counterpart to this call: it exists for
 *     callers that cannot obtain device memory when they call the library (a serving loop whose memory was divided
 *     up at start-up and that must not call cudaMalloc on the request path, because that call synchronises the
 *     device and can fail under fragmentation; a plug-in inside another framework's memory pool).  The scratch
 *     that matq_gemm_multi takes from its workspace comes from an array built into the library's device image:
 *     matq_gemm_multi_static_max_bytes() bytes (16 MiB) on every GPU that loads the library, held until exit.
 *   Arguments and results are those of matq_gemm_multi.  Nothing is allocated or freed by this call.
 *   MATQ_ERR_WORKSPACE is returned, before anything is launched, when
 *     matq_gemm_multi_workspace_bytes(src_kind, M, N, K, n_r) > matq_gemm_multi_static_max_bytes().
 *   The first call on each device looks up the array's device address (that device must be current) and should be
 *   made before any stream capture begins.  The address is kept for the life of the process: after a cudaDeviceReset
 *   it is stale, and this entry point must not be used on that device again.  All calls on a GPU share the array and it keeps the previous call's
 *   contents; none of it needs to start at zero, but calls that overlap on the GPU race on it and must be ordered
 *   by the caller (one stream, or events between streams).
 */
size_t matq_gemm_multi_static_max_bytes(void);
int matq_gemm_multi_static(int src_kind, const void *Wsrc, int64_t N, int64_t K, int c,
                           float *alpha, float *zero, int extra_precision,
                           const int32_t *ovf_row_ptr, const uint16_t *ovf_col,
                           const void *X, int64_t M, int64_t ldx,
                           const int *rs, int n_r, float *const *Y, int64_t ldy,
                           int32_t *dev_status, void *stream);

/*
 * Testing hook for the error path of the dense forward (matq_gemm_multi, matq_gemm_multi_loss,
 * matq_gemm_multi_static).  While `on` is non-zero, the tensor-core kernel of every such call issues none of its copies,
 * and its waits give up after about a millisecond instead of about two seconds (every wait of that kernel is bounded in
 * SM clock cycles).  Such a call returns MATQ_OK, reports MATQ_ERR_TIMEOUT through dev_status, stores nothing to Y
 * (loss mode: the loss it writes is meaningless) and frees its tensor memory; alpha, zero and the workspace are written
 * as usual.  The setting is process-wide and is read when a call is made: do not change it while another thread is
 * inside one of these calls.  Returns the previous setting.  No copy is in flight when such a kernel exits, and the next
 * call with the hook off works as usual.
 */
int matq_gemm_multi_test_stall(int on);

/*
 * Testing hook for the one device-side wait of matq_slice_pack / matq_slice_pack_nested with extra_precision: the
 * look-back of the one-pass kernel, in which a tile of rows waits for the overflow counts of the tiles before it.  While
 * `on` is non-zero, the first tile never publishes its count and a look-back gives up after 2^8 polls instead of 2^20;
 * every later tile then meets "nothing yet" until its limit, or the mark of a tile that has already given up.  Such a
 * call returns MATQ_OK and reports MATQ_ERR_TIMEOUT through dev_status; the planes are complete, ovf_row_ptr, ovf_col and
 * ovf_count are not.  Process-wide like the hook above; returns the previous setting.  Shapes that the one-pass kernel
 * does not take (K % 16 != 0, K > 16384, 2^31 codes or more) have no device-side wait and ignore it.
 */
int matq_slice_pack_test_stall(int on);

#ifdef __cplusplus
}
#endif
#endif /* MATQ_H_ */
