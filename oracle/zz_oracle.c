/*
 * CPU oracle for the ZigzagAttention inference hot path.  TEST INFRASTRUCTURE ONLY:
 * it is used by the tests, by the smoke check and by the timed CPU-baseline leg of
 * the benchmark; the product (the CUDA library) never calls, links or imports it,
 * and it shares no code, header, table or helper with the CUDA path.
 *
 * Everything here is the plain definition written out, in fp64 on the bf16 input
 * values widened exactly: no tiling, no online softmax, no reordering.
 *
 * What it computes (citations are to the paper):
 *   - "full attention" of a retrieval head and "streaming attention" of a
 *     streaming head (Section 2.1, the two terms of Eq. 1; Eq. 1 with alpha = 1
 *     is the former and alpha = 0 the latter).  Streaming attention attends to the
 *     sink tokens plus a recent window, the remaining KV being waived
 *     (Introduction, the paragraph on DuoAttention; sink/window sizes are the two
 *     hyper-parameters fixed in Section 3.3).
 *   - the prefill and decoding phases over a KV cache (Introduction, second
 *     paragraph): a prefill call evaluates rows t = P .. P+C-1, a decode step the
 *     single row t = N-1 after the new token has been appended.
 *   - the per-layer exclusive assignment (Section 2.2, first paragraph) is the
 *     special case in which every KV head of the layer has the same kind; the
 *     mixed-head (DuoAttention-style) layer is the general case, kind per KV head.
 *
 * Readings where the paper is silent (also listed in the design notes):
 *   - visible set of a streaming head for the query at absolute position t:
 *       V(t) = { j : 0 <= j <= t  and  ( j < S  or  t - j < W ) }
 *     i.e. the window of W keys includes the current token;
 *   - the streaming KV store is a ring of S+W slots: slot(t) = t for t < S,
 *     otherwise S + ((t - S) mod W); pos[slot] holds the token index or -1;
 *   - query head h uses KV head floor(h / G), G = Hq / Hkv;
 *   - natural-base softmax with an explicit scale factor.
 *
 * Pins (see tests): brute force with an explicit score/mask matrix written
 * differently (numpy, long double, no max subtraction); rows of the softmax sum to
 * one; q = 0 gives the arithmetic mean of the visible values; a dominant key
 * selects its value; S+W >= N equals full attention bit for bit; S=0, W=1 gives
 * v_t; |V(t)| = min(t+1, S+W); decode step t == prefill row t; chunked == single
 * shot; ring route == full-history route; occupied ring positions; invariance
 * under slot permutation; GQA replication; mixed layer == per-head kinds.
 * Layer-mask choice (Eq. 5, at the end of this file): a hand-worked example (tests/golden),
 * the same objective written per layer in numpy over itertools subsets, the already-exclusive
 * split costing nothing, omega = 0 reducing to the least retrieval mass, head-order invariance.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ZZO_OK 0
#define ZZO_BAD_ARG (-1)

static double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* V(t) membership.  kind: 1 = retrieval (full attention), 0 = streaming. */
int zzo_visible(int kind, int64_t j, int64_t t, int64_t S, int64_t W) {
    if (j < 0 || j > t) return 0;
    if (kind) return 1;
    return (j < S) || (t - j < W);
}

/* |V(t)| counted one key at a time. */
int64_t zzo_visible_count(int kind, int64_t t, int64_t S, int64_t W) {
    int64_t n = 0;
    for (int64_t j = 0; j <= t; ++j) n += zzo_visible(kind, j, t, S, W);
    return n;
}

/* Ring slot of token t (streaming KV store). */
int64_t zzo_slot(int64_t t, int64_t S, int64_t W) {
    if (t < S) return t;
    return S + ((t - S) % W);
}

/*
 * Attention rows from the full K/V history.
 *   q        [n_rows][Hq][D]   bf16 bits, row i is the query at absolute position t_rows[i]
 *   k, v     [n_hist][Hkv][D]  bf16 bits, token j at index j (the whole history, nothing waived)
 *   kv_kind  [Hkv]             1 = retrieval KV head, 0 = streaming KV head
 *   out      [n_rows][Hq][D]   fp64
 *   p_sum    NULL or [n_rows][Hq]: the sum of the softmax weights of the row (should be 1)
 * For each (row, head): s_j = scale * <q, k_j> over j in V(t); m = max s_j;
 * p_j = exp(s_j - m) / sum_i exp(s_i - m); o = sum_j p_j v_j.
 */
int zzo_attn_rows(const uint16_t* q, const int64_t* t_rows, int64_t n_rows,
                  const uint16_t* k, const uint16_t* v, int64_t n_hist,
                  int Hq, int Hkv, int D, const uint8_t* kv_kind,
                  int64_t S, int64_t W, double scale, double* out, double* p_sum) {
    if (!q || !t_rows || !k || !v || !kv_kind || !out) return ZZO_BAD_ARG;
    if (Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0 || n_rows < 0) return ZZO_BAD_ARG;
    if (S < 0 || W < 1) return ZZO_BAD_ARG;
    for (int64_t i = 0; i < n_rows; ++i)
        if (t_rows[i] < 0 || t_rows[i] >= n_hist) return ZZO_BAD_ARG;
    const int G = Hq / Hkv;
    const int64_t units = n_rows * (int64_t)Hq;
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)(n_hist > 0 ? n_hist : 1));
#pragma omp for schedule(dynamic, 1)
        for (int64_t u = 0; u < units; ++u) {
            const int64_t i = u / Hq;
            const int h = (int)(u % Hq);
            const int g = h / G;
            const int kind = kv_kind[g] ? 1 : 0;
            const int64_t t = t_rows[i];
            const uint16_t* qrow = q + ((size_t)i * Hq + h) * D;
            /* scores and their maximum over the visible set */
            double m = -INFINITY;
            for (int64_t j = 0; j <= t; ++j) {
                if (!zzo_visible(kind, j, t, S, W)) continue;
                const uint16_t* krow = k + ((size_t)j * Hkv + g) * D;
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += bf16_to_f64(qrow[d]) * bf16_to_f64(krow[d]);
                s[j] = scale * dot;
                if (s[j] > m) m = s[j];
            }
            /* normaliser */
            double denom = 0.0;
            for (int64_t j = 0; j <= t; ++j) {
                if (!zzo_visible(kind, j, t, S, W)) continue;
                denom += exp(s[j] - m);
            }
            /* weighted sum of the values */
            double* orow = out + ((size_t)i * Hq + h) * D;
            for (int d = 0; d < D; ++d) orow[d] = 0.0;
            double psum = 0.0;
            for (int64_t j = 0; j <= t; ++j) {
                if (!zzo_visible(kind, j, t, S, W)) continue;
                const double p = exp(s[j] - m) / denom;
                psum += p;
                const uint16_t* vrow = v + ((size_t)j * Hkv + g) * D;
                for (int d = 0; d < D; ++d) orow[d] += p * bf16_to_f64(vrow[d]);
            }
            if (p_sum) p_sum[(size_t)i * Hq + h] = psum;
        }
        free(s);
    }
    return ZZO_OK;
}

/*
 * Streaming KV store: append C tokens one at a time to a ring of S+W slots.
 *   ring_k, ring_v [Hkv][S+W][D]  bf16 bits (canonical export order)
 *   pos            [S+W]          token index held by the slot, -1 = empty
 *   len            in/out         tokens appended so far
 *   k_new, v_new   [C][Hkv][D]
 * Token t goes to slot(t); whatever was there (token t - W) is thereby evicted.
 */
int zzo_ring_append(uint16_t* ring_k, uint16_t* ring_v, int32_t* pos, int64_t* len,
                    const uint16_t* k_new, const uint16_t* v_new, int64_t C,
                    int Hkv, int D, int64_t S, int64_t W) {
    if (!ring_k || !ring_v || !pos || !len || (C > 0 && (!k_new || !v_new))) return ZZO_BAD_ARG;
    if (Hkv <= 0 || D <= 0 || S < 0 || W < 1 || C < 0) return ZZO_BAD_ARG;
    const int64_t R = S + W;
    for (int64_t i = 0; i < C; ++i) {
        const int64_t t = *len;
        const int64_t sl = zzo_slot(t, S, W);
        for (int g = 0; g < Hkv; ++g) {
            memcpy(ring_k + ((size_t)g * R + sl) * D, k_new + ((size_t)i * Hkv + g) * D,
                   sizeof(uint16_t) * (size_t)D);
            memcpy(ring_v + ((size_t)g * R + sl) * D, v_new + ((size_t)i * Hkv + g) * D,
                   sizeof(uint16_t) * (size_t)D);
        }
        pos[sl] = (int32_t)t;
        *len = t + 1;
    }
    return ZZO_OK;
}

/*
 * Retrieval KV store: slot j holds token j.
 *   cache_k, cache_v [Hkv][cap][D]; len in/out; returns ZZO_BAD_ARG on overflow
 *   (and leaves everything unchanged).
 */
int zzo_full_append(uint16_t* cache_k, uint16_t* cache_v, int64_t cap, int64_t* len,
                    const uint16_t* k_new, const uint16_t* v_new, int64_t C, int Hkv, int D) {
    if (!cache_k || !cache_v || !len || (C > 0 && (!k_new || !v_new))) return ZZO_BAD_ARG;
    if (*len + C > cap || C < 0) return ZZO_BAD_ARG;
    for (int64_t i = 0; i < C; ++i) {
        const int64_t t = *len;
        for (int g = 0; g < Hkv; ++g) {
            memcpy(cache_k + ((size_t)g * cap + t) * D, k_new + ((size_t)i * Hkv + g) * D,
                   sizeof(uint16_t) * (size_t)D);
            memcpy(cache_v + ((size_t)g * cap + t) * D, v_new + ((size_t)i * Hkv + g) * D,
                   sizeof(uint16_t) * (size_t)D);
        }
        *len = t + 1;
    }
    return ZZO_OK;
}

/*
 * One attention row computed from a slot store (ring or retrieval cache) instead
 * of the history: every slot with pos >= 0 holds token pos[slot]; the key takes
 * part iff pos[slot] is in V(t).  Slots are visited in physical order.
 *   q [Hq][D]; store_k, store_v [Hkv][n_slots][D]; pos [n_slots]; out [Hq][D] fp64
 */
int zzo_attn_from_slots(const uint16_t* q, int64_t t, const uint16_t* store_k,
                        const uint16_t* store_v, const int32_t* pos, int64_t n_slots,
                        int Hq, int Hkv, int D, const uint8_t* kv_kind,
                        int64_t S, int64_t W, double scale, double* out) {
    if (!q || !store_k || !store_v || !pos || !kv_kind || !out) return ZZO_BAD_ARG;
    if (Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return ZZO_BAD_ARG;
    const int G = Hq / Hkv;
    double* s = (double*)malloc(sizeof(double) * (size_t)(n_slots > 0 ? n_slots : 1));
    for (int h = 0; h < Hq; ++h) {
        const int g = h / G;
        const int kind = kv_kind[g] ? 1 : 0;
        const uint16_t* qrow = q + (size_t)h * D;
        double m = -INFINITY;
        for (int64_t sl = 0; sl < n_slots; ++sl) {
            if (pos[sl] < 0 || !zzo_visible(kind, pos[sl], t, S, W)) continue;
            const uint16_t* krow = store_k + ((size_t)g * n_slots + sl) * D;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += bf16_to_f64(qrow[d]) * bf16_to_f64(krow[d]);
            s[sl] = scale * dot;
            if (s[sl] > m) m = s[sl];
        }
        double denom = 0.0;
        for (int64_t sl = 0; sl < n_slots; ++sl) {
            if (pos[sl] < 0 || !zzo_visible(kind, pos[sl], t, S, W)) continue;
            denom += exp(s[sl] - m);
        }
        double* orow = out + (size_t)h * D;
        for (int d = 0; d < D; ++d) orow[d] = 0.0;
        for (int64_t sl = 0; sl < n_slots; ++sl) {
            if (pos[sl] < 0 || !zzo_visible(kind, pos[sl], t, S, W)) continue;
            const double p = exp(s[sl] - m) / denom;
            const uint16_t* vrow = store_v + ((size_t)g * n_slots + sl) * D;
            for (int d = 0; d < D; ++d) orow[d] += p * bf16_to_f64(vrow[d]);
        }
    }
    free(s);
    return ZZO_OK;
}

int zzo_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Layer-mask choice by exhaustive enumeration (Section 2.2, Eq. 5), as the paper describes it:
 * every subset of p streaming layers is examined one by one and the one of minimum cost kept.
 *   alpha            [L][H]  head importances
 *   head_is_retr     [L][H]  the quantile split the transition starts from (1 = retrieval head)
 *   p                        number of all-streaming layers
 *   omega                    scaling factor of the third case
 *   best_is_retr     [L]     out: 1 = retrieval layer, for the first subset (in increasing binary
 *                            order of the streaming-layer bit mask) that attains the minimum
 *   best_cost, second_cost   out: the minimum and the smallest cost of any other subset
 * Per head (i, j), with the layer's new kind k_i:  0 if the head keeps its kind;  alpha_ij if a
 * retrieval head becomes a streaming head;  -omega * alpha_ij if a streaming head becomes a
 * retrieval head.  L <= 24.
 */
int zzo_layer_mask_enumerate(const double* alpha, const uint8_t* head_is_retr, int L, int H, int p,
                             double omega, uint8_t* best_is_retr, double* best_cost, double* second_cost) {
    if (!alpha || !head_is_retr || !best_is_retr || !best_cost || !second_cost) return ZZO_BAD_ARG;
    if (L < 1 || L > 24 || H < 1 || p < 0 || p > L) return ZZO_BAD_ARG;
    double best = INFINITY, second = INFINITY;
    uint32_t best_mask = 0;
    for (uint32_t mask = 0; mask < (1u << L); ++mask) {          /* bit i set: layer i becomes streaming */
        int bits = 0;
        for (int i = 0; i < L; ++i) bits += (mask >> i) & 1u;
        if (bits != p) continue;
        double cost = 0.0;
        for (int i = 0; i < L; ++i) {
            const int layer_streaming = (mask >> i) & 1u;
            for (int j = 0; j < H; ++j) {
                const int was_retr = head_is_retr[i * H + j] ? 1 : 0;
                double hat;
                if (was_retr && layer_streaming) hat = alpha[i * H + j];                 /* o(1) */
                else if (!was_retr && !layer_streaming) hat = -omega * alpha[i * H + j]; /* o(2) */
                else hat = 0.0;                                                          /* o(0) */
                cost += hat;
            }
        }
        if (cost < best) { second = best; best = cost; best_mask = mask; }
        else if (cost < second) second = cost;
    }
    for (int i = 0; i < L; ++i) best_is_retr[i] = ((best_mask >> i) & 1u) ? 0 : 1;
    *best_cost = best;
    *second_cost = second;
    return ZZO_OK;
}

/* Quantile split (Section 2.1, last paragraph): the n_streaming heads of smallest alpha become
 * streaming heads; among equal alphas the earlier (layer, head) first.  Selection by repeated
 * minimum search, no sort. */
int zzo_quantile_split(const double* alpha, int n, int n_streaming, uint8_t* is_retr) {
    if (!alpha || !is_retr || n < 1 || n_streaming < 0 || n_streaming > n) return ZZO_BAD_ARG;
    for (int i = 0; i < n; ++i) is_retr[i] = 1;
    for (int r = 0; r < n_streaming; ++r) {
        int arg = -1;
        for (int i = 0; i < n; ++i)
            if (is_retr[i] && (arg < 0 || alpha[i] < alpha[arg])) arg = i;
        is_retr[arg] = 0;
    }
    return ZZO_OK;
}

/* ---------------------------------------------------------------------------------------------
 * FP8 storage of retrieval KV rows (the paper has no such variant; this is the reading the
 * library documents, written out as its definition).
 *
 * A row is the 128 (in general D) bf16 values of one token and one KV head.  It is stored as
 * D codes in the OCP 8-bit floating-point format E4M3 (1 sign, 4 exponent bits of bias 7, 3
 * mantissa bits; no infinities; largest finite magnitude 448 = 1.75 * 2^8; S.1111.111 is NaN)
 * and one scale byte e (an exponent-only number, value 2^(e - 127)):
 *     amax = max_d |x_d|;  write amax = m * 2^k with 1 <= m < 2 (k taken from the exponent field
 *     of the bf16 bits; a zero or subnormal amax counts as k = -127);
 *     e = clamp(k + 127 - 8 + (m > 1.75 ? 1 : 0), 1, 254): the smallest power of two with
 *     amax / 2^(e-127) <= 448, so nothing saturates;
 *     code_d = E4M3 nearest to x_d / 2^(e-127), ties to the even code, magnitudes beyond 448
 *     (only possible through the clamp) to 448.
 * The stored value of the element is value(code_d) * 2^(e-127), exactly.
 * --------------------------------------------------------------------------------------------- */

/* value of one E4M3 code (NaN codes are never produced; they decode to 0 here) */
double zzo_e4m3_value(uint8_t c) {
    const int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return 0.0;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

/* nearest E4M3 code of y, ties to even, saturating at +-448 */
uint8_t zzo_e4m3_encode(double y) {
    const uint8_t sign = (y < 0.0 || (y == 0.0 && signbit(y))) ? 0x80 : 0x00;
    double a = fabs(y);
    if (!(a == a)) return (uint8_t)(sign | 0x7E);
    if (a >= 448.0) return (uint8_t)(sign | 0x7E);
    if (a == 0.0) return sign;
    int ex;
    (void)frexp(a, &ex);                /* a = f * 2^ex, 0.5 <= f < 1  ->  floor(log2 a) = ex - 1 */
    int e = ex - 1;
    if (e < -6) e = -6;                 /* subnormal range shares the quantum of the smallest normal */
    const double quantum = ldexp(1.0, e - 3);
    double n = nearbyint(a / quantum);  /* default rounding mode: to nearest, ties to even */
    if (n >= 16.0) { n = 8.0; e += 1; }
    int biased, mant;
    if (n >= 8.0) { biased = e + 7; mant = (int)n - 8; }
    else { biased = 0; mant = (int)n; } /* only reachable with e == -6 */
    if (biased > 15 || (biased == 15 && mant == 7)) return (uint8_t)(sign | 0x7E);
    return (uint8_t)(sign | (biased << 3) | mant);
}

/* scale byte of a row of D bf16 values */
uint8_t zzo_fp8_scale_byte(const uint16_t* row, int D) {
    unsigned amax = 0;
    for (int d = 0; d < D; ++d) {
        const unsigned a = row[d] & 0x7FFFu;
        if (a > amax) amax = a;
    }
    const int k_biased = (int)(amax >> 7);          /* exponent field: k + 127 (0 for zero / subnormal) */
    const int mant = (int)(amax & 0x7F);            /* m = 1 + mant / 128; 1.75 <-> 0x60 */
    int e = k_biased - 8 + (mant > 0x60 ? 1 : 0);
    if (e < 1) e = 1;
    if (e > 254) e = 254;
    return (uint8_t)e;
}

/* rows [n][D] bf16 bits -> codes [n][D], scale bytes [n] */
int zzo_fp8_quantize_rows(const uint16_t* x, int64_t n, int D, uint8_t* codes, uint8_t* scale) {
    if (!x || !codes || !scale || n < 0 || D <= 0) return ZZO_BAD_ARG;
    for (int64_t r = 0; r < n; ++r) {
        const uint16_t* row = x + (size_t)r * D;
        const uint8_t e = zzo_fp8_scale_byte(row, D);
        scale[r] = e;
        for (int d = 0; d < D; ++d)
            codes[(size_t)r * D + d] = zzo_e4m3_encode(ldexp(bf16_to_f64(row[d]), 127 - (int)e));
    }
    return ZZO_OK;
}

/* stored values as fp64: out[r][d] = value(code) * 2^(scale - 127) */
int zzo_fp8_dequantize_rows(const uint8_t* codes, const uint8_t* scale, int64_t n, int D, double* out) {
    if (!codes || !scale || !out || n < 0 || D <= 0) return ZZO_BAD_ARG;
    for (int64_t r = 0; r < n; ++r)
        for (int d = 0; d < D; ++d)
            out[(size_t)r * D + d] = ldexp(zzo_e4m3_value(codes[(size_t)r * D + d]), (int)scale[r] - 127);
    return ZZO_OK;
}
