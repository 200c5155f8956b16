/*
 * fp64 CPU oracle for single-token multiquery attention over a KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA library is
 * checked against; it is never part of the product path and shares no code,
 * header, table or helper with it.  Only the tests, the smoke check and the
 * CPU-baseline leg of the benchmark may load it.
 *
 * What it follows: "Efficiently Scaling Transformer Inference", Section 3.3
 * ("Partitioning the attention layer"): multiquery attention emits n_heads
 * query heads but a single key head and a single value head that every query
 * head shares; in the generate phase there is one query token per sequence and
 * the KV cache holds all earlier tokens (same section, paragraph on
 * autoregressive generation).  The paper states attention by reference to the
 * standard scaled dot-product softmax form, so the definition is written out
 * here in plain index order, in double precision, with no blocking, no
 * running maximum across tiles and no base-2 rewriting (Section 3.5 mentions
 * base-2 softmax only as an implementation speed-up; it is the same function).
 *
 * Readings where the paper is silent (all listed in the design notes):
 *   - one query position per sequence, hence no causal mask;
 *   - `scale` is supplied by the caller and applied to the double logit;
 *   - lengths[b] counts the valid cache rows and is clamped into [0, Lmax];
 *   - a sequence of length 0 yields an all-zero output row;
 *   - rows at or beyond lengths[b] are never read.
 *
 * Pins (tests/test_oracle_pins.py): softmax rows sum to 1; length 1 returns
 * v_0 bit-exactly; constant V returns the constant; closed forms for length 2,
 * zero query and one dominant logit; invariance under joint row permutation,
 * key shift and row duplication; brute-force multihead attention with K/V
 * replicated per head; a library float64 attention routine; the split/merge
 * identity.  The paper prints no numeric attention output, so element values
 * are pinned by those independent routes rather than by a printed example:
 * by the paper alone this is "parity unpinned".
 *
 * Inputs are bf16 bit patterns (uint16) widened exactly to double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_bits_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static inline int clamp_len(int32_t len, int Lmax)
{
    if (len < 0) return 0;
    if (len > Lmax) return Lmax;
    return (int)len;
}

static int bad_shape(int B, int H, int D, int Lmax)
{
    return B <= 0 || H <= 0 || D <= 0 || Lmax <= 0;
}

/* Scaled logits of query head (b,h) against cache rows [l0, l1) of sequence b:
 * s[l - l0] = scale * sum_d q[b,h,d] * k[b,l,d]  (Section 3.3: every query
 * head of a sequence meets the same single key head). */
static void logits_row(const uint16_t* q, const uint16_t* k, int b, int h,
                       int H, int D, int Lmax, int l0, int l1, double scale,
                       double* s)
{
    const uint16_t* qv = q + ((size_t)b * H + h) * D;
    for (int l = l0; l < l1; ++l) {
        const uint16_t* kv = k + ((size_t)b * Lmax + l) * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += bf16_bits_to_double(qv[d]) * bf16_bits_to_double(kv[d]);
        s[l - l0] = scale * acc;
    }
}

/*
 * out[b,h,:] = sum_l softmax_l(scale * q[b,h,:] . k[b,l,:]) * v[b,l,:]
 * over l in [0, lengths[b]).  Host pointers.  Returns 0, or -1 on a bad shape
 * or allocation failure.  The result does not depend on num_threads: threads
 * split the (b,h) pairs and each output row is summed in index order.
 */
int mqa_decode_ref_f64(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                       const int32_t* lengths, double* out,
                       int B, int H, int D, int Lmax, float scale,
                       int num_threads)
{
    if (!q || !k || !v || !lengths || !out || bad_shape(B, H, D, Lmax)) return -1;
    const double sc = (double)scale;
    int failed = 0;
    if (num_threads < 1) num_threads = 1;
#ifdef _OPENMP
#pragma omp parallel num_threads(num_threads)
#endif
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)Lmax);
        if (!s) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            failed = 1;
        }
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
        for (long bh = 0; bh < (long)B * H; ++bh) {
            if (!s) continue;
            const int b = (int)(bh / H), h = (int)(bh % H);
            const int n = clamp_len(lengths[b], Lmax);
            double* o = out + ((size_t)b * H + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (n == 0) continue;
            logits_row(q, k, b, h, H, D, Lmax, 0, n, sc, s);
            double m = s[0];
            for (int l = 1; l < n; ++l) if (s[l] > m) m = s[l];
            double Z = 0.0;
            for (int l = 0; l < n; ++l) { s[l] = exp(s[l] - m); Z += s[l]; }
            for (int l = 0; l < n; ++l) {
                const uint16_t* vv = v + ((size_t)b * Lmax + l) * D;
                const double p = s[l];
                for (int d = 0; d < D; ++d) o[d] += p * bf16_bits_to_double(vv[d]);
            }
            for (int d = 0; d < D; ++d) o[d] /= Z;
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/*
 * Softmax weights themselves: w[b,h,l] for l < lengths[b], 0 beyond.
 * w is [B,H,Lmax] doubles.  For small inputs (the pins).
 */
int mqa_ref_weights_f64(const uint16_t* q, const uint16_t* k,
                        const int32_t* lengths, double* w,
                        int B, int H, int D, int Lmax, float scale)
{
    if (!q || !k || !lengths || !w || bad_shape(B, H, D, Lmax)) return -1;
    const double sc = (double)scale;
    for (int b = 0; b < B; ++b) {
        const int n = clamp_len(lengths[b], Lmax);
        for (int h = 0; h < H; ++h) {
            double* row = w + ((size_t)b * H + h) * Lmax;
            for (int l = 0; l < Lmax; ++l) row[l] = 0.0;
            if (n == 0) continue;
            logits_row(q, k, b, h, H, D, Lmax, 0, n, sc, row);
            double m = row[0];
            for (int l = 1; l < n; ++l) if (row[l] > m) m = row[l];
            double Z = 0.0;
            for (int l = 0; l < n; ++l) { row[l] = exp(row[l] - m); Z += row[l]; }
            for (int l = 0; l < n; ++l) row[l] /= Z;
        }
    }
    return 0;
}

/*
 * One split of one sequence: over cache rows [l0, l1) (clipped to the valid
 * length) of sequence b, for every head h, the three quantities a split of
 * the sequence axis hands to the merge step:
 *   m[h]   = max_l s[l]                     (natural-log domain; -inf if empty)
 *   z[h]   = sum_l exp(s[l] - m[h])         (0 if empty)
 *   acc[h,:] = sum_l exp(s[l] - m[h]) v[l,:]  (unnormalised; 0 if empty)
 * Used only to pin the merge formula against the plain definition.
 */
int mqa_ref_partial_f64(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                        const int32_t* lengths, int b, int l0, int l1,
                        double* m, double* z, double* acc,
                        int B, int H, int D, int Lmax, float scale)
{
    if (!q || !k || !v || !lengths || !m || !z || !acc || bad_shape(B, H, D, Lmax)) return -1;
    if (b < 0 || b >= B) return -1;
    const double sc = (double)scale;
    const int n = clamp_len(lengths[b], Lmax);
    if (l0 < 0) l0 = 0;
    if (l1 > n) l1 = n;
    double* s = (double*)malloc(sizeof(double) * (size_t)Lmax);
    if (!s) return -1;
    for (int h = 0; h < H; ++h) {
        double* o = acc + (size_t)h * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (l1 <= l0) { m[h] = -INFINITY; z[h] = 0.0; continue; }
        logits_row(q, k, b, h, H, D, Lmax, l0, l1, sc, s);
        const int cnt = l1 - l0;
        double mx = s[0];
        for (int i = 1; i < cnt; ++i) if (s[i] > mx) mx = s[i];
        double Z = 0.0;
        for (int i = 0; i < cnt; ++i) {
            const double p = exp(s[i] - mx);
            Z += p;
            const uint16_t* vv = v + ((size_t)b * Lmax + (l0 + i)) * D;
            for (int d = 0; d < D; ++d) o[d] += p * bf16_bits_to_double(vv[d]);
        }
        m[h] = mx; z[h] = Z;
    }
    free(s);
    return 0;
}

/*
 * Log-sum-exp merge of S partial results of one (sequence, head):
 *   M = max_s m_s;  out = sum_s e^{m_s-M} acc_s / sum_s e^{m_s-M} z_s.
 * Splits with z_s == 0 (no valid rows) are skipped; if all are empty the
 * output row is zero.  m,z are [S]; acc is [S,D]; out is [D].
 */
int mqa_ref_merge_f64(const double* m, const double* z, const double* acc,
                      int S, int D, double* out)
{
    if (!m || !z || !acc || !out || S <= 0 || D <= 0) return -1;
    double M = -INFINITY;
    for (int s = 0; s < S; ++s) if (z[s] > 0.0 && m[s] > M) M = m[s];
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (M == -INFINITY) return 0;
    double Z = 0.0;
    for (int s = 0; s < S; ++s) {
        if (!(z[s] > 0.0)) continue;
        const double w = exp(m[s] - M);
        Z += w * z[s];
        for (int d = 0; d < D; ++d) out[d] += w * acc[(size_t)s * D + d];
    }
    for (int d = 0; d < D; ++d) out[d] /= Z;
    return 0;
}

/*
 * Attention with KVH key/value heads per sequence (Section 4.2 compares multihead attention, KVH = H,
 * with multiquery attention, KVH = 1).  Query head h reads key/value head g = h / (H/KVH).
 * Layouts: q [B,H,D], k and v [B,KVH,Lmax,D], lengths [B], out [B,H,D].  The plain definition again,
 * written with its own index arithmetic (it does not call the multiquery routine above).
 */
int gqa_decode_ref_f64(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                       const int32_t* lengths, double* out,
                       int B, int H, int KVH, int D, int Lmax, float scale)
{
    if (!q || !k || !v || !lengths || !out || bad_shape(B, H, D, Lmax) || KVH <= 0 || H % KVH != 0) return -1;
    const double sc = (double)scale;
    const int per = H / KVH;
    double* s = (double*)malloc(sizeof(double) * (size_t)Lmax);
    if (!s) return -1;
    for (int b = 0; b < B; ++b) {
        const int n = clamp_len(lengths[b], Lmax);
        for (int h = 0; h < H; ++h) {
            const int g = h / per;
            const uint16_t* qv = q + ((size_t)b * H + h) * D;
            const uint16_t* kh = k + (((size_t)b * KVH + g) * Lmax) * D;
            const uint16_t* vh = v + (((size_t)b * KVH + g) * Lmax) * D;
            double* o = out + ((size_t)b * H + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (n == 0) continue;
            double m = -INFINITY;
            for (int l = 0; l < n; ++l) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += bf16_bits_to_double(qv[d]) * bf16_bits_to_double(kh[(size_t)l * D + d]);
                s[l] = sc * acc;
                if (s[l] > m) m = s[l];
            }
            double Z = 0.0;
            for (int l = 0; l < n; ++l) { s[l] = exp(s[l] - m); Z += s[l]; }
            for (int l = 0; l < n; ++l)
                for (int d = 0; d < D; ++d) o[d] += s[l] * bf16_bits_to_double(vh[(size_t)l * D + d]);
            for (int d = 0; d < D; ++d) o[d] /= Z;
        }
    }
    free(s);
    return 0;
}

int mqa_ref_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
