/*
 * matq_ref — plain CPU oracle for the nested int8 -> int4 -> int2 weight path
 * of Matryoshka Quantization.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct
 * definition the CUDA library is checked against.  It shares no code, header,
 * table or helper with the CUDA path and must never be called from it; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Every function writes the paper's definition out step by step:
 *   quantize     Eq. 1   (MinMax, one (alpha, z) per output channel = row of W)
 *   slice        Eq. 6   (rounded, clamped MSB slice on the c-bit grid)
 *   slice (E.P.) Eq. 8   (Errata: the same without the clamp, 2^r + 1 levels)
 *   pack         the paper gives no format; see "Packed format" below
 *   gemv / gemm  y = x . dequant(S(q, r))^T with dequant(S) = alpha * (S - z),
 *                the forward F(S(Q(theta, c), r), x) of Eq. 7, in fp64
 *
 * Readings taken where the paper is silent (all listed again in the design notes):
 *   - The rounding brackets in Eq. 1 and Eq. 6 round half UP.  Appendix A
 *     explains the rounding of Eq. 6 as "add the (r+1)-th most significant
 *     bit", which is floor(v + 1/2); the same symbol in Eq. 1 gets the same
 *     function.
 *   - Eq. 1 is evaluated in IEEE binary32, one correctly rounded operation per
 *     step, in the order written below, with a true division (no reciprocal,
 *     no fused multiply-add).  z is real-valued (Eq. 1 does not round it).
 *   - max(w) == min(w): alpha := 1, z := -min(w); all codes are 0 and the
 *     dequantised value is the constant itself.
 *   - 1 <= r <= c; r == c is the identity.  Slices are always taken from the
 *     c-bit code, never from another slice (Section 3.2).
 *
 * Packed format (this library's; the Errata only says the extra bits "can be
 * packed into int2/int4"): for r in {8, 4, 2}, byte j of a row holds the
 * fields k = S(q, r) / 2^(c-r) of elements j*(8/r) + i, i = 0 .. 8/r - 1, field
 * i in bits [i*r, (i+1)*r).  Rows are contiguous, K*r/8 bytes each.  An
 * extra-precision model stores the CLAMPED field in the plane (so the plane
 * is byte-identical to the standard one) plus, per row, the ascending column
 * indices of the elements whose Eq. 8 value lies one bucket above the clamp
 * ("+2^(c-r)" corrections): ovf_row_ptr[N+1], ovf_col[nnz].
 *
 * Build: gcc -O2 -std=c11 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum {
    MATQ_REF_OK = 0,
    MATQ_REF_ERR_INVALID_ARG = 1,
    MATQ_REF_ERR_UNSUPPORTED = 2,
    MATQ_REF_ERR_SHAPE = 3,
    MATQ_REF_ERR_NONFINITE = 8,
    MATQ_REF_ERR_CAPACITY = 9
};

enum { MATQ_REF_SRC_BF16 = 0, MATQ_REF_SRC_CODES8 = 1, MATQ_REF_SRC_PACKED = 2 };

int matq_ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* bf16 -> binary32 is exact: the 16 bits are the top half of the float. */
static float bf16_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* floor(u + 1/2) without forming u + 1/2 (which could round): u - floor(u) is
 * exact in binary32 for |u| < 2^23. */
static float round_half_up(float u)
{
    float fl = floorf(u);
    float frac = u - fl;
    return (frac >= 0.5f) ? fl + 1.0f : fl;
}

/* ------------------------------------------------------------------ Eq. 1 */
/* W: bf16 bits [N, K], row stride ldw elements.  q: uint8 [N, K] (may be
 * NULL).  alpha, zero: fp32 [N].  A non-finite weight anywhere makes the call
 * return MATQ_REF_ERR_NONFINITE (the row's outputs are then unspecified). */
int matq_ref_quantize(const uint16_t *W, int64_t N, int64_t K, int64_t ldw, int c,
                      uint8_t *q, float *alpha, float *zero)
{
    if (!W || !alpha || !zero || N < 0 || K <= 0 || ldw < K) return MATQ_REF_ERR_INVALID_ARG;
    if (c != 8) return MATQ_REF_ERR_UNSUPPORTED;
    const float qmax = (float)((1 << c) - 1);
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int64_t n = 0; n < N; ++n) {
        const uint16_t *row = W + n * ldw;
        float mn = bf16_to_float(row[0]);
        float mx = mn;
        int nonfinite = 0;
        for (int64_t k = 0; k < K; ++k) {
            float w = bf16_to_float(row[k]);
            if (!isfinite(w)) nonfinite = 1;
            if (w < mn) mn = w;
            if (w > mx) mx = w;
        }
        if (nonfinite) { bad |= 1; continue; }
        float range = mx - mn;
        float a = (range > 0.0f) ? range / qmax : 1.0f;
        float z = (-mn) / a;
        alpha[n] = a;
        zero[n] = z;
        if (!q) continue;
        for (int64_t k = 0; k < K; ++k) {
            float w = bf16_to_float(row[k]);
            float t = w / a;
            float u = t + z;
            float r = round_half_up(u);
            if (r < 0.0f) r = 0.0f;
            if (r > qmax) r = qmax;
            q[n * K + k] = (uint8_t)r;
        }
    }
    return bad ? MATQ_REF_ERR_NONFINITE : MATQ_REF_OK;
}

/* ------------------------------------------------------------------ Eq. 3 */
/* MinMax quantisation with OmniQuant's two clipping scales (Section 3.1, Eq. 3):
 *   alpha = (gamma * max(w) - beta * min(w)) / (2^c - 1),  z = -beta * min(w) / alpha,
 *   Q = clamp(round(w / alpha + z), 0, 2^c - 1),
 * gamma and beta per output channel (NULL = 1 for every row, which is Eq. 1).
 * Every step is one fp32 operation, in the order written: the two products,
 * their difference, the division by 2^c - 1, the division for z, then per weight
 * the division, the sum, round half up and the clamp.  A range that is not
 * positive gives alpha = 1 (the reading taken for a constant row in Eq. 1).
 * A non-finite weight, gamma or beta makes the call return
 * MATQ_REF_ERR_NONFINITE (that row's outputs are then unspecified). */
int matq_ref_quantize_clip(const uint16_t *W, int64_t N, int64_t K, int64_t ldw, int c,
                           const float *gamma, const float *beta,
                           uint8_t *q, float *alpha, float *zero)
{
    if (!W || !alpha || !zero || N < 0 || K <= 0 || ldw < K) return MATQ_REF_ERR_INVALID_ARG;
    if (c != 8) return MATQ_REF_ERR_UNSUPPORTED;
    const float qmax = (float)((1 << c) - 1);
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int64_t n = 0; n < N; ++n) {
        const uint16_t *row = W + n * ldw;
        float mn = bf16_to_float(row[0]);
        float mx = mn;
        int nonfinite = 0;
        for (int64_t k = 0; k < K; ++k) {
            float w = bf16_to_float(row[k]);
            if (!isfinite(w)) nonfinite = 1;
            if (w < mn) mn = w;
            if (w > mx) mx = w;
        }
        const float g = gamma ? gamma[n] : 1.0f;
        const float b = beta ? beta[n] : 1.0f;
        if (!isfinite(g) || !isfinite(b)) nonfinite = 1;
        if (nonfinite) { bad |= 1; continue; }
        float hi = g * mx;
        float lo = b * mn;
        float range = hi - lo;
        float a = (range > 0.0f) ? range / qmax : 1.0f;
        float z = (-lo) / a;
        alpha[n] = a;
        zero[n] = z;
        if (!q) continue;
        for (int64_t k = 0; k < K; ++k) {
            float w = bf16_to_float(row[k]);
            float t = w / a;
            float u = t + z;
            float r = round_half_up(u);
            if (r < 0.0f) r = 0.0f;
            if (r > qmax) r = qmax;
            q[n * K + k] = (uint8_t)r;
        }
    }
    return bad ? MATQ_REF_ERR_NONFINITE : MATQ_REF_OK;
}

/* ------------------------------------------------------- Eq. 6 and Eq. 8 */
/* Value of S(q, r) on the c-bit grid, 0 .. 2^c (2^c only with Eq. 8).
 * floor(q / 2^sh + 1/2) on integers is (q + 2^(sh-1)) >> sh. */
static unsigned slice_value(unsigned q, int c, int r, int extra_precision)
{
    int sh = c - r;
    if (sh == 0) return q;
    unsigned k = (q + (1u << (sh - 1))) >> sh;
    unsigned kmax = (1u << r) - 1u;
    if (!extra_precision && k > kmax) k = kmax;
    return k << sh;
}

/* S: uint16 [n] because Eq. 8 can return 2^c = 256. */
int matq_ref_slice(const uint8_t *q, int64_t n, int c, int r, int extra_precision, uint16_t *S)
{
    if (!q || !S || n < 0) return MATQ_REF_ERR_INVALID_ARG;
    if (c != 8 || r < 1 || r > c) return MATQ_REF_ERR_UNSUPPORTED;
    for (int64_t i = 0; i < n; ++i) S[i] = (uint16_t)slice_value(q[i], c, r, extra_precision);
    return MATQ_REF_OK;
}

/* ------------------------------------------------------------ slice + pack */
/* packed: uint8 [N, K*r/8] (r in {8,4,2}; may be NULL for other r).
 * sliced_unpacked: uint8 [N, K] = Eq. 6 value (clamped), may be NULL.
 * With extra_precision and r < c: ovf_row_ptr int32 [N+1], ovf_col uint16
 * [ovf_capacity], *ovf_count = total overflow elements (always written). */
int matq_ref_slice_pack(const uint8_t *q, int64_t N, int64_t K, int c, int r, int extra_precision,
                        uint8_t *packed, uint8_t *sliced_unpacked,
                        int32_t *ovf_row_ptr, uint16_t *ovf_col, int64_t ovf_capacity,
                        int64_t *ovf_count)
{
    if (!q || N < 0 || K <= 0) return MATQ_REF_ERR_INVALID_ARG;
    if (c != 8 || r < 1 || r > c) return MATQ_REF_ERR_UNSUPPORTED;
    const int packable = (r == 8 || r == 4 || r == 2);
    if (packed && !packable) return MATQ_REF_ERR_UNSUPPORTED;
    const int per_byte = packable ? 8 / r : 1;
    if (packed && (K % per_byte) != 0) return MATQ_REF_ERR_SHAPE;
    const int sh = c - r;
    const int want_ovf = extra_precision && sh > 0;
    if (want_ovf && (!ovf_row_ptr || !ovf_count || K > 65536)) return MATQ_REF_ERR_INVALID_ARG;

    if (sliced_unpacked)
        for (int64_t i = 0; i < N * K; ++i) sliced_unpacked[i] = (uint8_t)slice_value(q[i], c, r, 0);

    if (packed) {
        const int64_t row_bytes = K / per_byte;
        for (int64_t n = 0; n < N; ++n)
            for (int64_t j = 0; j < row_bytes; ++j) {
                unsigned byte = 0;
                for (int i = 0; i < per_byte; ++i) {
                    unsigned field = slice_value(q[n * K + j * per_byte + i], c, r, 0) >> sh;
                    byte |= field << (i * r);
                }
                packed[n * row_bytes + j] = (uint8_t)byte;
            }
    }

    if (want_ovf) {
        int64_t nnz = 0;
        for (int64_t n = 0; n < N; ++n) {
            ovf_row_ptr[n] = (int32_t)nnz;
            for (int64_t k = 0; k < K; ++k) {
                unsigned s_ep = slice_value(q[n * K + k], c, r, 1);
                unsigned s = slice_value(q[n * K + k], c, r, 0);
                if (s_ep != s) {
                    if (ovf_col && nnz < ovf_capacity) ovf_col[nnz] = (uint16_t)k;
                    ++nnz;
                }
            }
        }
        ovf_row_ptr[N] = (int32_t)nnz;
        *ovf_count = nnz;
        if (nnz > ovf_capacity) return MATQ_REF_ERR_CAPACITY;
    } else if (ovf_count) {
        *ovf_count = 0;
    }
    return MATQ_REF_OK;
}

/* Inverse of the plane format: fields[n, k] = k_r in [0, 2^r - 1]. */
int matq_ref_unpack(const uint8_t *packed, int64_t N, int64_t K, int r, uint8_t *fields)
{
    if (!packed || !fields || N < 0 || K <= 0) return MATQ_REF_ERR_INVALID_ARG;
    if (!(r == 8 || r == 4 || r == 2)) return MATQ_REF_ERR_UNSUPPORTED;
    const int per_byte = 8 / r;
    if (K % per_byte) return MATQ_REF_ERR_SHAPE;
    const int64_t row_bytes = K / per_byte;
    const unsigned mask = (1u << r) - 1u;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            unsigned byte = packed[n * row_bytes + k / per_byte];
            fields[n * K + k] = (uint8_t)((byte >> ((k % per_byte) * r)) & mask);
        }
    return MATQ_REF_OK;
}

/* --------------------------------------------------------------- matmuls */
/* y[m, n] = sum_k x[m, k] * alpha[n] * (S[n, k] - zero[n]), fp64, k ascending.
 * S: uint16 [N, K] values on the c-bit grid (0 .. 2^c). */
static void matmul_dequant(const uint16_t *S, int64_t N, int64_t K,
                           const float *alpha, const float *zero,
                           const uint16_t *X, int64_t M, int64_t ldx, double *Y, int64_t ldy)
{
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const double a = (double)alpha[n];
        const double z = (double)zero[n];
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double w_hat = a * ((double)S[n * K + k] - z);
                acc += (double)bf16_to_float(X[m * ldx + k]) * w_hat;
            }
            Y[m * ldy + n] = acc;
        }
    }
}

/* Decode-time linear layer from a packed r-bit plane (+ optional E.P. list).
 * x: bf16 bits [B, K] (row stride ldx); y: fp64 [B, N] (row stride ldy). */
int matq_ref_gemv(const uint8_t *packed, int64_t N, int64_t K, int c, int r,
                  const float *alpha, const float *zero,
                  const int32_t *ovf_row_ptr, const uint16_t *ovf_col,
                  const uint16_t *x, int64_t B, int64_t ldx, double *y, int64_t ldy,
                  uint16_t *S_scratch /* uint16 [N, K], caller-provided */)
{
    if (!packed || !alpha || !zero || !x || !y || !S_scratch) return MATQ_REF_ERR_INVALID_ARG;
    if (c != 8 || !(r == 8 || r == 4 || r == 2)) return MATQ_REF_ERR_UNSUPPORTED;
    const int per_byte = 8 / r;
    if (K % per_byte) return MATQ_REF_ERR_SHAPE;
    if ((ovf_row_ptr == NULL) != (ovf_col == NULL)) return MATQ_REF_ERR_INVALID_ARG;
    const int sh = c - r;
    const int64_t row_bytes = K / per_byte;
    const unsigned mask = (1u << r) - 1u;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) {
            unsigned byte = packed[n * row_bytes + k / per_byte];
            unsigned field = (byte >> ((k % per_byte) * r)) & mask;
            S_scratch[n * K + k] = (uint16_t)(field << sh);
        }
        if (ovf_row_ptr)
            for (int32_t p = ovf_row_ptr[n]; p < ovf_row_ptr[n + 1]; ++p)
                S_scratch[n * K + ovf_col[p]] += (uint16_t)(1u << sh);
    }
    matmul_dequant(S_scratch, N, K, alpha, zero, x, B, ldx, y, ldy);
    return MATQ_REF_OK;
}

/* Multi-precision forward: Y_r = X . dequant(S(q, r))^T for every r in rs.
 * src_kind BF16: Wsrc = bf16 bits [N, K]; alpha/zero are OUTPUTS of Eq. 1.
 * src_kind CODES8: Wsrc = uint8 codes [N, K]; alpha/zero inputs.
 * src_kind PACKED: n_r == 1, Wsrc = packed plane of rs[0] (+ overflow list).
 * q_scratch: uint8 [N, K]; S_scratch: uint16 [N, K]. */
int matq_ref_gemm_multi(int src_kind, const void *Wsrc, int64_t N, int64_t K, int c,
                        float *alpha, float *zero, int extra_precision,
                        const int32_t *ovf_row_ptr, const uint16_t *ovf_col,
                        const uint16_t *X, int64_t M, int64_t ldx,
                        const int *rs, int n_r, double *const *Y, int64_t ldy,
                        uint8_t *q_scratch, uint16_t *S_scratch)
{
    if (!Wsrc || !alpha || !zero || !X || !rs || !Y || n_r < 1 || !S_scratch)
        return MATQ_REF_ERR_INVALID_ARG;
    if (c != 8) return MATQ_REF_ERR_UNSUPPORTED;
    if (src_kind == MATQ_REF_SRC_PACKED) {
        if (n_r != 1) return MATQ_REF_ERR_INVALID_ARG;
        return matq_ref_gemv((const uint8_t *)Wsrc, N, K, c, rs[0], alpha, zero,
                             extra_precision ? ovf_row_ptr : NULL, extra_precision ? ovf_col : NULL,
                             X, M, ldx, Y[0], ldy, S_scratch);
    }
    const uint8_t *q;
    if (src_kind == MATQ_REF_SRC_BF16) {
        if (!q_scratch) return MATQ_REF_ERR_INVALID_ARG;
        int st = matq_ref_quantize((const uint16_t *)Wsrc, N, K, K, c, q_scratch, alpha, zero);
        if (st) return st;
        q = q_scratch;
    } else if (src_kind == MATQ_REF_SRC_CODES8) {
        q = (const uint8_t *)Wsrc;
    } else {
        return MATQ_REF_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n_r; ++i) {
        int st = matq_ref_slice(q, N * K, c, rs[i], extra_precision, S_scratch);
        if (st) return st;
        matmul_dequant(S_scratch, N, K, alpha, zero, X, M, ldx, Y[i], ldy);
    }
    return MATQ_REF_OK;
}
