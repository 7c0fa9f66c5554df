/*
 * Float64 CPU oracle for Cartridge decode attention.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA path is checked against.  It is never
 * linked into, imported by, or called from the product library; only tests, the smoke check and
 * the benchmark's CPU-baseline leg may use it.  It shares no code with the CUDA path.
 *
 * What it computes (paper Eq. 1 evaluated at the last position i, Sec. 2.3; the Cartridge KV-cache
 * layout of Sec. 3.2; served as a cached prefix of p tokens, Sec. 3.3; composition by concatenation, Sec. 3.1
 * and Sec. 5.4): for request b whose KV cache is the concatenation, in order, of its segments
 * (zero or more Cartridges followed by the request's own suffix), for query head h reading KV head
 * g = h div (Hq/Hkv):
 *
 *     K* = concat_s K_s[g]        V* = concat_s V_s[g]           (explicit copies, n rows of D)
 *     t_j  = scale * <q[b,h], K*_j>                               j = 1..n
 *     M    = max_j t_j
 *     lse  = M + ln sum_j exp(t_j - M)
 *     o    = sum_j exp(t_j - lse) V*_j
 *
 * All arithmetic is IEEE double on the exact values of the bf16 inputs.  No blocking, no fusion,
 * no online rescaling: every score is stored, then the maximum, then the sum, then the output.
 *
 * Parity pins (tests/test_oracle_pins.py): exact-rational brute force on tiny inputs, closed forms
 * (one token, identical keys, q = 0, one-hot keys at large scale, key shift, cache duplication),
 * invariants (LSE merge of parts, composition = concatenation, permutation, convexity, GQA head
 * swap) and a float64 library softmax-attention cross-check.  The paper prints no numeric example
 * of attention, so no paper-printed values exist to pin against.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE binary32: widen by appending 16 zero bits. */
static double bf16_to_double(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

int cart_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * One layer of decode attention for a batch.
 *
 *   B, Hq, Hkv, D   batch, query heads, KV heads (Hq % Hkv == 0), head dimension
 *   scale           softmax scale applied to the raw dot product
 *   q               [B][Hq][D] bf16 bit patterns
 *   seg_begin       [B+1] offsets: request b owns segments seg_begin[b] .. seg_begin[b+1]-1, in
 *                   cache order (Cartridges first, suffix last)
 *   seg_k, seg_v    per segment: pointer to this layer's block, element (g, j, d) at
 *                   g*seg_head_stride + j*D + d  (bf16 bit patterns)
 *   seg_n           per segment: number of KV tokens (may be 0)
 *   seg_head_stride per segment: elements between consecutive KV heads (>= seg_n*D; larger when a
 *                   suffix buffer has spare capacity)
 *   out             [B][Hq][D] double
 *   lse             [B][Hq] double, natural log of the sum of exp of the scaled scores
 *
 * Returns 0 on success, 1 on a bad shape, 2 if some request has an empty cache, 3 on allocation
 * failure.
 */
int cart_oracle_decode_layer(int B, int Hq, int Hkv, int D, double scale,
                             const uint16_t *q,
                             const int32_t *seg_begin,
                             const uint16_t *const *seg_k,
                             const uint16_t *const *seg_v,
                             const int64_t *seg_n,
                             const int64_t *seg_head_stride,
                             double *out, double *lse)
{
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return 1;
    const int G = Hq / Hkv;
    for (int b = 0; b < B; ++b) {
        int64_t n = 0;
        for (int s = seg_begin[b]; s < seg_begin[b + 1]; ++s) {
            if (seg_n[s] < 0) return 1;
            n += seg_n[s];
        }
        if (n == 0) return 2;
    }

    int status = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int g = 0; g < Hkv; ++g) {
            int64_t n = 0;
            for (int s = seg_begin[b]; s < seg_begin[b + 1]; ++s) n += seg_n[s];

            /* The explicitly concatenated cache [Cartridge(s) ; suffix] of this KV head. */
            double *Kcat = (double *)malloc((size_t)n * D * sizeof(double));
            double *Vcat = (double *)malloc((size_t)n * D * sizeof(double));
            double *t = (double *)malloc((size_t)n * sizeof(double));
            if (!Kcat || !Vcat || !t) {
#pragma omp atomic write
                status = 3;
                free(Kcat); free(Vcat); free(t);
                continue;
            }
            int64_t row = 0;
            for (int s = seg_begin[b]; s < seg_begin[b + 1]; ++s) {
                const uint16_t *ks = seg_k[s] + (int64_t)g * seg_head_stride[s];
                const uint16_t *vs = seg_v[s] + (int64_t)g * seg_head_stride[s];
                for (int64_t j = 0; j < seg_n[s]; ++j, ++row)
                    for (int d = 0; d < D; ++d) {
                        Kcat[row * D + d] = bf16_to_double(ks[j * D + d]);
                        Vcat[row * D + d] = bf16_to_double(vs[j * D + d]);
                    }
            }

            for (int i = 0; i < G; ++i) {
                const int h = g * G + i;
                const uint16_t *qh = q + ((int64_t)b * Hq + h) * D;
                double M = -INFINITY;
                for (int64_t j = 0; j < n; ++j) {
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += bf16_to_double(qh[d]) * Kcat[j * D + d];
                    t[j] = scale * dot;
                    if (t[j] > M) M = t[j];
                }
                double sum = 0.0;
                for (int64_t j = 0; j < n; ++j) sum += exp(t[j] - M);
                const double L = M + log(sum);
                double *o = out + ((int64_t)b * Hq + h) * D;
                for (int d = 0; d < D; ++d) o[d] = 0.0;
                for (int64_t j = 0; j < n; ++j) {
                    const double w = exp(t[j] - L);
                    for (int d = 0; d < D; ++d) o[d] += w * Vcat[j * D + d];
                }
                lse[(int64_t)b * Hq + h] = L;
            }
            free(Kcat); free(Vcat); free(t);
        }
    }
    return status;
}
