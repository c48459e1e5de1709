/*
 * swaa_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain, slow, float64 CPU statement of the attention that the SWAA method
 * computes: causal softmax attention under a per-layer mask policy.  It exists
 * so that the GPU library can be checked against something written directly
 * from the paper's definition.  It shares no code with the GPU path and is
 * only ever called by tests, the smoke check and the benchmark's CPU-baseline
 * leg.
 *
 * What the paper fixes (all in prose; it prints no formula):
 *   - Sec. 1 / App. A: sliding window attention restricts each token to a
 *     fixed-size local window of earlier tokens (causal), cost O(N*W).
 *   - Sec. 3.2.1 "Keep First k Tokens" and the Fig. 1(b) caption: a token
 *     attends to its local window AND the first k tokens (a union).
 *   - Sec. 3.1.1 "FA Decode" and the Fig. 1(a) caption: a generated token
 *     attends to every earlier token of the whole context.
 *   - Sec. 3.1.2 "Interleaving FA/SWA layers": some layers keep full causal
 *     attention.
 *   - Sec. 4.1.2: SWA equals full attention when the context fits the window.
 *
 * Readings taken where the paper is silent:
 *   - the window holds W keys INCLUDING the query's own position:
 *        visible(i, j) = j <= i  and ( is_full  or  j > i - W  or  j < S )
 *   - sink positions are relative to the start of each packed sequence;
 *   - grouped-query attention: query head h reads key/value head h / (Hq/Hkv);
 *   - the softmax scale is an argument (callers pass 1/sqrt(D));
 *   - decode: the cache already holds the current token, the query sits at
 *     position len-1.
 *
 * Every row is computed by the textbook two-pass softmax over exactly the
 * visible keys; keys that are not visible are never read.  No tiling, no
 * running maximum, no reordering.  Inputs are float32 arrays that hold the
 * bf16 input values exactly; all arithmetic is double.
 *
 * Pins (tests/test_oracle_pins.py): brute-force set enumeration on tiny
 * inputs, the closed-form visible-pair count, W >= L == full causal (Sec.
 * 4.1.2) == a library float64 softmax-attention, W=1/S=0 returns V, Q=0
 * returns the mean of the visible V rows, rows of probabilities sum to 1,
 * decode == last prefill row.  No value printed by the paper exists to
 * compare against (it prints none for this path).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Sec. 3.2.1 (window AND first k), Sec. 1 (causal local window), Sec. 3.1.1/3.1.2 (full). */
int swaa_oracle_visible(int64_t i, int64_t j, int64_t W, int64_t S, int is_full) {
    if (j < 0 || j > i) return 0;   /* causal */
    if (is_full) return 1;          /* FA layer or FA decode */
    if (j > i - W) return 1;        /* inside the window of W keys ending at i */
    if (j < S) return 1;            /* one of the first S (sink) tokens */
    return 0;
}

/* Number of visible (i, j) pairs of one sequence of length L, by direct enumeration. */
int64_t swaa_oracle_count_pairs(int64_t L, int64_t W, int64_t S, int is_full) {
    int64_t n = 0;
    for (int64_t i = 0; i < L; ++i)
        for (int64_t j = 0; j <= i; ++j)
            n += swaa_oracle_visible(i, j, W, S, is_full);
    return n;
}

/*
 * One output row.  q: D values of the query at position i of its sequence.
 * k, v: position 0 of the same sequence and key/value head; consecutive
 * positions are kv_stride floats apart.  Writes out[D]; *lse = log of the sum
 * of exp(score) over visible keys; *psum = sum of the normalised probabilities
 * (should be 1); *nvis = how many keys were visible.  `scores` is scratch of at
 * least i+1 doubles.
 */
static void oracle_row(const float* q, const float* k, const float* v, int64_t i, int64_t kv_stride, int D,
                       int64_t W, int64_t S, int is_full, double scale, double* out, double* lse, double* psum,
                       int64_t* nvis, double* scores) {
    double m = -INFINITY;
    int64_t cnt = 0;
    for (int64_t j = 0; j <= i; ++j) {
        if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
        const float* kj = k + j * kv_stride;
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += (double)q[d] * (double)kj[d];
        s *= scale;
        scores[j] = s;
        if (s > m) m = s;
        ++cnt;
    }
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    double denom = 0.0;
    for (int64_t j = 0; j <= i; ++j) {
        if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
        denom += exp(scores[j] - m);
    }
    double ps = 0.0;
    for (int64_t j = 0; j <= i; ++j) {
        if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
        double p = exp(scores[j] - m) / denom;
        ps += p;
        const float* vj = v + j * kv_stride;
        for (int d = 0; d < D; ++d) out[d] += p * (double)vj[d];
    }
    if (lse) *lse = m + log(denom);
    if (psum) *psum = ps;
    if (nvis) *nvis = cnt;
}

/*
 * Packed variable-length prefill (self attention, one cu_seqlens for q and k).
 *   q   [T, Hq, D], k, v [T, Hkv, D]  float32 (bf16 values), token-major.
 *   cu_seqlens [B+1], cu[0] = 0, cu[B] = T.
 * Computes n_rows rows chosen by (row_t[r], row_h[r]) = (packed token index,
 * query head); with row_t == NULL every (t, h) is computed in t-major order and
 * n_rows must be T*Hq.  out is [n_rows, D] double; lse, psum, nvis are
 * [n_rows] (each may be NULL).  Returns 0, or -1 on inconsistent arguments.
 */
int swaa_oracle_prefill(const float* q, const float* k, const float* v, const int32_t* cu_seqlens, int B, int Hq,
                        int Hkv, int D, int64_t W, int64_t S, int is_full, double scale, int64_t n_rows,
                        const int64_t* row_t, const int32_t* row_h, double* out, double* lse, double* psum,
                        int64_t* nvis) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return -1;
    if (!is_full && W < 1) return -1;
    if (S < 0) return -1;
    const int G = Hq / Hkv;
    const int64_t T = B > 0 ? cu_seqlens[B] : 0;
    int64_t max_len = 0;
    for (int b = 0; b < B; ++b) {
        int64_t len = (int64_t)cu_seqlens[b + 1] - cu_seqlens[b];
        if (len < 0) return -1;
        if (len > max_len) max_len = len;
    }
    if (row_t == NULL && n_rows != T * Hq) return -1;
    int bad = 0;
#pragma omp parallel
    {
        double* scores = (double*)malloc(sizeof(double) * (size_t)(max_len > 0 ? max_len : 1));
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < n_rows; ++r) {
            int64_t t = row_t ? row_t[r] : r / Hq;
            int h = row_t ? row_h[r] : (int)(r % Hq);
            if (t < 0 || t >= T || h < 0 || h >= Hq) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            int b = 0;
            while (!(cu_seqlens[b] <= t && t < cu_seqlens[b + 1])) ++b; /* sequence that owns token t */
            int64_t start = cu_seqlens[b];
            int64_t i = t - start; /* position inside its own sequence */
            int hk = h / G;
            oracle_row(q + (t * Hq + h) * (int64_t)D, k + (start * Hkv + hk) * (int64_t)D,
                       v + (start * Hkv + hk) * (int64_t)D, i, (int64_t)Hkv * D, D, W, S, is_full, scale,
                       out + r * D, lse ? lse + r : NULL, psum ? psum + r : NULL, nvis ? nvis + r : NULL, scores);
        }
        free(scores);
    }
    return bad ? -1 : 0;
}

/*
 * Chunked prefill: the queries of sequence b are the LAST len_q tokens of a context of len_k >= len_q
 * tokens whose keys and values are all given (Sec. 3.1.1 / Fig. 1a: later tokens attend to the stored
 * context; a serving engine feeds a long prompt in chunks).  Query i of the chunk sits at position
 * len_k - len_q + i of its sequence and sees the keys the mask policy allows for that position.
 *   q [Tq, Hq, D] packed by cu_q [B+1]; k, v [Tk, Hkv, D] packed by cu_k [B+1]; float32 (bf16 values).
 * Rows are chosen as in swaa_oracle_prefill, row_t being a packed QUERY token index.
 * is_full_seq (nullable, [B]): a mask policy per sequence, for a batch that mixes sequences in different phases
 * (Fig. 1a: prefill tokens under the SWA mask next to generated tokens under full attention); when given it
 * replaces is_full, sequence b being full causal iff is_full_seq[b] != 0.
 * Returns 0, or -1 on inconsistent arguments (also len_q > len_k).
 */
int swaa_oracle_prefill_chunked(const float* q, const float* k, const float* v, const int32_t* cu_q,
                                const int32_t* cu_k, int B, int Hq, int Hkv, int D, int64_t W, int64_t S,
                                int is_full, const uint8_t* is_full_seq, double scale, int64_t n_rows,
                                const int64_t* row_t, const int32_t* row_h, double* out, double* lse, double* psum,
                                int64_t* nvis) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return -1;
    if ((!is_full || is_full_seq) && W < 1) return -1;
    if (S < 0) return -1;
    const int G = Hq / Hkv;
    const int64_t Tq = B > 0 ? cu_q[B] : 0;
    int64_t max_len = 0;
    for (int b = 0; b < B; ++b) {
        int64_t lq = (int64_t)cu_q[b + 1] - cu_q[b], lk = (int64_t)cu_k[b + 1] - cu_k[b];
        if (lq < 0 || lk < lq) return -1;
        if (lk > max_len) max_len = lk;
    }
    if (row_t == NULL && n_rows != Tq * Hq) return -1;
    int bad = 0;
#pragma omp parallel
    {
        double* scores = (double*)malloc(sizeof(double) * (size_t)(max_len > 0 ? max_len : 1));
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < n_rows; ++r) {
            int64_t t = row_t ? row_t[r] : r / Hq;
            int h = row_t ? row_h[r] : (int)(r % Hq);
            if (t < 0 || t >= Tq || h < 0 || h >= Hq) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            int b = 0;
            while (!(cu_q[b] <= t && t < cu_q[b + 1])) ++b; /* sequence that owns query token t */
            int64_t lq = (int64_t)cu_q[b + 1] - cu_q[b], lk = (int64_t)cu_k[b + 1] - cu_k[b];
            int64_t i = (lk - lq) + (t - cu_q[b]); /* position of the query inside its sequence */
            int64_t kstart = cu_k[b];
            int hk = h / G;
            const int full_b = is_full_seq ? (is_full_seq[b] != 0) : is_full;
            oracle_row(q + (t * Hq + h) * (int64_t)D, k + (kstart * Hkv + hk) * (int64_t)D,
                       v + (kstart * Hkv + hk) * (int64_t)D, i, (int64_t)Hkv * D, D, W, S, full_b, scale,
                       out + r * D, lse ? lse + r : NULL, psum ? psum + r : NULL, nvis ? nvis + r : NULL, scores);
        }
        free(scores);
    }
    return bad ? -1 : 0;
}

/*
 * Decode: one query token per sequence against a dense cache.
 *   q [B, Hq, D]; kcache, vcache [B, Lmax, Hkv, D]; seqlens [B] counts the valid
 *   cache entries INCLUDING the current token, so the query's position is
 *   seqlens[b]-1 (Sec. 3.1.1: with is_full it sees the whole context).
 * out [B, Hq, D] double; lse, psum, nvis [B, Hq] (nullable).
 */
int swaa_oracle_decode(const float* q, const float* kcache, const float* vcache, const int32_t* seqlens, int B,
                       int64_t Lmax, int Hq, int Hkv, int D, int64_t W, int64_t S, int is_full, double scale,
                       double* out, double* lse, double* psum, int64_t* nvis) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return -1;
    if (!is_full && W < 1) return -1;
    if (S < 0) return -1;
    const int G = Hq / Hkv;
    for (int b = 0; b < B; ++b)
        if (seqlens[b] < 1 || seqlens[b] > Lmax) return -1;
#pragma omp parallel
    {
        double* scores = (double*)malloc(sizeof(double) * (size_t)(Lmax > 0 ? Lmax : 1));
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < (int64_t)B * Hq; ++r) {
            int b = (int)(r / Hq), h = (int)(r % Hq), hk = h / G;
            int64_t i = (int64_t)seqlens[b] - 1;
            oracle_row(q + r * D, kcache + ((int64_t)b * Lmax * Hkv + hk) * D,
                       vcache + ((int64_t)b * Lmax * Hkv + hk) * D, i, (int64_t)Hkv * D, D, W, S, is_full, scale,
                       out + r * D, lse ? lse + r : NULL, psum ? psum + r : NULL, nvis ? nvis + r : NULL, scores);
        }
        free(scores);
    }
    return 0;
}

/*
 * Decode with the cache of every sequence cut along the context (App. A: the full-context cache must be retained
 * under FA decode, which is what makes splitting it over several devices attractive).  One shard holds the
 * entries at positions [pos0, pos0 + Lshard) of every sequence: kshard, vshard [B, Lshard, Hkv, D], entry p at row
 * p - pos0.  seqlens [B] are the TOTAL lengths; the query sits at position seqlens[b] - 1 and sees the keys the
 * mask policy allows for that position (Sec. 3.1.1, 3.2.1), of which this shard contributes those it holds.
 * part [B, Hq, D + 2] double: (m, l, o[D]) with m = max of the visible scores of the shard, l = sum exp(s - m),
 * o = sum exp(s - m) v.  A shard that holds no visible key of a row gives (-inf, 0, 0...).  nvis [B, Hq] (nullable).
 */
int swaa_oracle_decode_partial(const float* q, const float* kshard, const float* vshard, const int32_t* seqlens, int B,
                               int64_t Lshard, int64_t pos0, int Hq, int Hkv, int D, int64_t W, int64_t S,
                               int is_full, double scale, double* part, int64_t* nvis) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0 || Lshard < 0 || pos0 < 0) return -1;
    if (!is_full && W < 1) return -1;
    if (S < 0) return -1;
    const int G = Hq / Hkv;
    for (int b = 0; b < B; ++b)
        if (seqlens[b] < 1) return -1;
#pragma omp parallel
    {
        double* scores = (double*)malloc(sizeof(double) * (size_t)(Lshard > 0 ? Lshard : 1));
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < (int64_t)B * Hq; ++r) {
            const int b = (int)(r / Hq), h = (int)(r % Hq), hk = h / G;
            const int64_t i = (int64_t)seqlens[b] - 1;
            const float* qi = q + r * D;
            double* pr = part + r * (D + 2);
            double m = -INFINITY;
            int64_t cnt = 0;
            for (int64_t jl = 0; jl < Lshard; ++jl) {
                if (!swaa_oracle_visible(i, pos0 + jl, W, S, is_full)) continue;
                const float* kj = kshard + (((int64_t)b * Lshard + jl) * Hkv + hk) * D;
                double sdot = 0.0;
                for (int d = 0; d < D; ++d) sdot += (double)qi[d] * (double)kj[d];
                scores[jl] = sdot * scale;
                if (scores[jl] > m) m = scores[jl];
                ++cnt;
            }
            double l = 0.0;
            for (int d = 0; d < D; ++d) pr[2 + d] = 0.0;
            for (int64_t jl = 0; jl < Lshard; ++jl) {
                if (!swaa_oracle_visible(i, pos0 + jl, W, S, is_full)) continue;
                const double e = exp(scores[jl] - m);
                const float* vj = vshard + (((int64_t)b * Lshard + jl) * Hkv + hk) * D;
                l += e;
                for (int d = 0; d < D; ++d) pr[2 + d] += e * (double)vj[d];
            }
            pr[0] = m;
            pr[1] = l;
            if (nvis) nvis[r] = cnt;
        }
        free(scores);
    }
    return 0;
}

/*
 * Log-sum-exp combine of P partial results per row (the cross-split merge of a split-K decode, here across
 * shards): M = max_s m_s, out = sum_s e^(m_s - M) o_s / sum_s e^(m_s - M) l_s; shards with l_s = 0 are skipped;
 * a row for which every shard is empty gives zeros.  part [P, n_rows, D + 2], out [n_rows, D].
 */
int swaa_oracle_decode_combine(const double* part, int P, int64_t n_rows, int D, double* out) {
    if (P < 1 || n_rows < 0 || D <= 0) return -1;
    for (int64_t r = 0; r < n_rows; ++r) {
        double M = -INFINITY;
        for (int s = 0; s < P; ++s) {
            const double* pr = part + ((int64_t)s * n_rows + r) * (D + 2);
            if (pr[1] > 0.0 && pr[0] > M) M = pr[0];
        }
        double den = 0.0;
        for (int d = 0; d < D; ++d) out[r * D + d] = 0.0;
        for (int s = 0; s < P; ++s) {
            const double* pr = part + ((int64_t)s * n_rows + r) * (D + 2);
            if (!(pr[1] > 0.0)) continue;
            const double w = exp(pr[0] - M);
            den += w * pr[1];
            for (int d = 0; d < D; ++d) out[r * D + d] += w * pr[2 + d];
        }
        if (den > 0.0)
            for (int d = 0; d < D; ++d) out[r * D + d] /= den;
    }
    return 0;
}

/*
 * Context-parallel prefill: one participant owns a contiguous stretch of every sequence (App. A: SWA prefill is
 * O(N * W), and a token only needs the W - 1 keys before it plus the first k tokens, Sec. 3.2.1, so a stretch can
 * be processed from local data once a halo of earlier keys and the sink rows have been brought in).
 *   k_local, v_local [Tk, Hkv, D] packed by cu_k: for sequence b the keys at positions key_pos0[b] ..
 *       key_pos0[b] + len_k - 1 (halo followed by the owned stretch);
 *   q [Tq, Hq, D] packed by cu_q: the queries of the LAST len_q of those positions;
 *   sink_k, sink_v [B, sink_rows, Hkv, D]: the keys at positions 0 .. sink_rows - 1 of every sequence.
 * A query at position i sees the positions the mask policy allows; each is taken from the local keys when
 * p >= key_pos0[b], else from the sink rows when p < min(S, sink_rows); a visible position available from
 * neither (halo too short) is an error (-2).  Keys are visited in increasing position, exactly as
 * swaa_oracle_prefill visits them.  Rows chosen as in swaa_oracle_prefill_chunked.
 */
int swaa_oracle_prefill_cp(const float* q, const float* k_local, const float* v_local, const float* sink_k,
                           const float* sink_v, const int32_t* cu_q, const int32_t* cu_k, const int64_t* key_pos0,
                           int B, int64_t sink_rows, int Hq, int Hkv, int D, int64_t W, int64_t S, int is_full,
                           double scale, int64_t n_rows, const int64_t* row_t, const int32_t* row_h, double* out,
                           double* lse, int64_t* nvis) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0 || sink_rows < 0) return -1;
    if (!is_full && W < 1) return -1;
    if (S < 0) return -1;
    const int G = Hq / Hkv;
    const int64_t Tq = B > 0 ? cu_q[B] : 0;
    int64_t max_pos = 0;
    for (int b = 0; b < B; ++b) {
        int64_t lq = (int64_t)cu_q[b + 1] - cu_q[b], lk = (int64_t)cu_k[b + 1] - cu_k[b];
        if (lq < 0 || lk < lq || key_pos0[b] < 0) return -1;
        if (key_pos0[b] + lk > max_pos) max_pos = key_pos0[b] + lk;
    }
    if (row_t == NULL && n_rows != Tq * Hq) return -1;
    int bad = 0;
#pragma omp parallel
    {
        double* scores = (double*)malloc(sizeof(double) * (size_t)(max_pos > 0 ? max_pos : 1));
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < n_rows; ++r) {
            const int64_t t = row_t ? row_t[r] : r / Hq;
            const int h = row_t ? row_h[r] : (int)(r % Hq);
            if (t < 0 || t >= Tq || h < 0 || h >= Hq) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            int b = 0;
            while (!(cu_q[b] <= t && t < cu_q[b + 1])) ++b;
            const int64_t lq = (int64_t)cu_q[b + 1] - cu_q[b], lk = (int64_t)cu_k[b + 1] - cu_k[b];
            const int64_t p0 = key_pos0[b];
            const int64_t i = p0 + (lk - lq) + (t - cu_q[b]);
            const int hk = h / G;
            const float* qi = q + (t * Hq + h) * (int64_t)D;
            double m = -INFINITY;
            int64_t cnt = 0;
            int missing = 0;
            for (int64_t p = 0; p <= i; ++p) {
                if (!swaa_oracle_visible(i, p, W, S, is_full)) continue;
                const float* kp;
                if (p >= p0) kp = k_local + ((cu_k[b] + (p - p0)) * Hkv + hk) * (int64_t)D;
                else if (p < S && p < sink_rows) kp = sink_k + (((int64_t)b * sink_rows + p) * Hkv + hk) * D;
                else { missing = 1; break; }
                double sdot = 0.0;
                for (int d = 0; d < D; ++d) sdot += (double)qi[d] * (double)kp[d];
                scores[p] = sdot * scale;
                if (scores[p] > m) m = scores[p];
                ++cnt;
            }
            if (missing) {
#pragma omp atomic write
                bad = 2;
                continue;
            }
            double denom = 0.0;
            for (int64_t p = 0; p <= i; ++p)
                if (swaa_oracle_visible(i, p, W, S, is_full)) denom += exp(scores[p] - m);
            double* orow = out + r * D;
            for (int d = 0; d < D; ++d) orow[d] = 0.0;
            for (int64_t p = 0; p <= i; ++p) {
                if (!swaa_oracle_visible(i, p, W, S, is_full)) continue;
                const double pr = exp(scores[p] - m) / denom;
                const float* vp = p >= p0 ? v_local + ((cu_k[b] + (p - p0)) * Hkv + hk) * (int64_t)D
                                          : sink_v + (((int64_t)b * sink_rows + p) * Hkv + hk) * D;
                for (int d = 0; d < D; ++d) orow[d] += pr * (double)vp[d];
            }
            if (lse) lse[r] = m + log(denom);
            if (nvis) nvis[r] = cnt;
        }
        free(scores);
    }
    return bad == 0 ? 0 : -bad;
}

/*
 * Gradients of the packed self-attention prefill with respect to q, k, v for an upstream gradient dout
 * (Sec. 3.2.2: fine-tuning under the SWA mask).  From out_i = sum_j p_ij v_j, p = softmax over the visible keys
 * of s_ij = scale * q_i.k_j:
 *     dv_j += p_ij dout_i;   dp_ij = dout_i . v_j;   ds_ij = p_ij (dp_ij - sum_j' p_ij' dp_ij');
 *     dq_i = scale * sum_j ds_ij k_j;   dk_j += scale * ds_ij q_i     (dk, dv summed over the heads of a group).
 * Two plain passes: rows (softmax statistics and dq), then keys (dk, dv from the rows that see them).
 *   q, dout [T, Hq, D]; k, v [T, Hkv, D] float32 (bf16 values); dq [T, Hq, D], dk, dv [T, Hkv, D] double.
 * out_given (nullable, [T, Hq, D] float32): since out_i = sum_j p_ij v_j, the row term sum_j' p_ij' dp_ij' equals
 * dout_i . out_i.  With out_given == NULL it is computed from the probabilities (the exact gradient).  With a
 * tensor given, dout_i . out_given_i is used instead: the gradient as a function of a stored (e.g. rounded) forward
 * output, which is what an entry point that receives `out` as an argument computes.
 * Returns 0, or -1 on inconsistent arguments.
 */
int swaa_oracle_prefill_backward(const float* q, const float* k, const float* v, const float* dout,
                                 const float* out_given, const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D,
                                 int64_t W, int64_t S, int is_full, double scale, double* dq, double* dk, double* dv) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return -1;
    if (!is_full && W < 1) return -1;
    if (S < 0) return -1;
    const int G = Hq / Hkv;
    const int64_t T = B > 0 ? cu_seqlens[B] : 0;
    int64_t max_len = 0;
    for (int b = 0; b < B; ++b) {
        int64_t len = (int64_t)cu_seqlens[b + 1] - cu_seqlens[b];
        if (len < 0) return -1;
        if (len > max_len) max_len = len;
    }
    /* per (token, head): row maximum m, denominator den, and sum_j p_ij dp_ij */
    double* rm = (double*)malloc(sizeof(double) * (size_t)(T * Hq > 0 ? T * Hq : 1));
    double* rden = (double*)malloc(sizeof(double) * (size_t)(T * Hq > 0 ? T * Hq : 1));
    double* rdot = (double*)malloc(sizeof(double) * (size_t)(T * Hq > 0 ? T * Hq : 1));
#pragma omp parallel
    {
        double* sc = (double*)malloc(sizeof(double) * (size_t)(max_len > 0 ? max_len : 1));
        double* dp = (double*)malloc(sizeof(double) * (size_t)(max_len > 0 ? max_len : 1));
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < T * Hq; ++r) {
            const int64_t t = r / Hq;
            const int h = (int)(r % Hq), hk = h / G;
            int b = 0;
            while (!(cu_seqlens[b] <= t && t < cu_seqlens[b + 1])) ++b;
            const int64_t s0 = cu_seqlens[b], i = t - s0;
            const float* qi = q + r * D;
            const float* gi = dout + r * D;
            double m = -INFINITY;
            for (int64_t j = 0; j <= i; ++j) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                const float* kj = k + ((s0 + j) * Hkv + hk) * (int64_t)D;
                const float* vj = v + ((s0 + j) * Hkv + hk) * (int64_t)D;
                double s = 0.0, d = 0.0;
                for (int c = 0; c < D; ++c) {
                    s += (double)qi[c] * (double)kj[c];
                    d += (double)gi[c] * (double)vj[c];
                }
                sc[j] = s * scale;
                dp[j] = d;
                if (sc[j] > m) m = sc[j];
            }
            double den = 0.0, dot = 0.0;
            for (int64_t j = 0; j <= i; ++j) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                den += exp(sc[j] - m);
            }
            if (out_given) {
                const float* oi = out_given + (t * Hq + h) * (int64_t)D;
                for (int c = 0; c < D; ++c) dot += (double)gi[c] * (double)oi[c];
            } else {
                for (int64_t j = 0; j <= i; ++j) {
                    if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                    dot += exp(sc[j] - m) / den * dp[j];
                }
            }
            rm[r] = m;
            rden[r] = den;
            rdot[r] = dot;
            double* dqi = dq + r * D;
            for (int c = 0; c < D; ++c) dqi[c] = 0.0;
            for (int64_t j = 0; j <= i; ++j) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                const double ds = exp(sc[j] - m) / den * (dp[j] - dot);
                const float* kj = k + ((s0 + j) * Hkv + hk) * (int64_t)D;
                for (int c = 0; c < D; ++c) dqi[c] += scale * ds * (double)kj[c];
            }
        }
        free(sc);
        free(dp);
        /* keys: every (token, kv head) collects from the rows and heads that see it */
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < T * Hkv; ++r) {
            const int64_t t = r / Hkv;
            const int hk = (int)(r % Hkv);
            int b = 0;
            while (!(cu_seqlens[b] <= t && t < cu_seqlens[b + 1])) ++b;
            const int64_t s0 = cu_seqlens[b], len = cu_seqlens[b + 1] - s0, j = t - s0;
            const float* kj = k + r * D;
            const float* vj = v + r * D;
            double* dkj = dk + r * D;
            double* dvj = dv + r * D;
            for (int c = 0; c < D; ++c) dkj[c] = dvj[c] = 0.0;
            for (int64_t i = j; i < len; ++i) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                for (int h = hk * G; h < (hk + 1) * G; ++h) {
                    const int64_t ri = (s0 + i) * Hq + h;
                    const float* qi = q + ri * D;
                    const float* gi = dout + ri * D;
                    double s = 0.0, d = 0.0;
                    for (int c = 0; c < D; ++c) {
                        s += (double)qi[c] * (double)kj[c];
                        d += (double)gi[c] * (double)vj[c];
                    }
                    const double p = exp(s * scale - rm[ri]) / rden[ri];
                    const double ds = p * (d - rdot[ri]);
                    for (int c = 0; c < D; ++c) {
                        dvj[c] += p * (double)gi[c];
                        dkj[c] += scale * ds * (double)qi[c];
                    }
                }
            }
        }
    }
    free(rm);
    free(rden);
    free(rdot);
    return 0;
}

/*
 * The same gradients for chosen rows and keys only, so that a long sequence can be checked without the
 * O(L * W) cost of every row (Sec. 3.2.2; formulas as in swaa_oracle_prefill_backward, nothing else changes):
 *   dq for the n_q (packed token, query head) pairs (qrow_t[r], qrow_h[r])      -> dq_out [n_q, D]
 *   dk, dv for the n_k (packed token, key/value head) pairs (key_t[r], key_hk[r]) -> dk_out, dv_out [n_k, D]
 * A key's gradient needs the softmax statistics (maximum, denominator, sum_j p_ij dp_ij) of every row that
 * sees it, for all query heads of its group; those are computed once for exactly the rows that some chosen key
 * needs, each by the same two plain passes over its visible keys, and then used by the key loop.
 * out_given as in swaa_oracle_prefill_backward.
 * Returns 0, or -1 on inconsistent arguments.
 */
int swaa_oracle_prefill_backward_rows(const float* q, const float* k, const float* v, const float* dout,
                                      const float* out_given, const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D, int64_t W, int64_t S,
                                      int is_full, double scale, int64_t n_q, const int64_t* qrow_t,
                                      const int32_t* qrow_h, double* dq_out, int64_t n_k, const int64_t* key_t,
                                      const int32_t* key_hk, double* dk_out, double* dv_out) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0) return -1;
    if (!is_full && W < 1) return -1;
    if (S < 0 || n_q < 0 || n_k < 0) return -1;
    const int G = Hq / Hkv;
    const int64_t T = B > 0 ? cu_seqlens[B] : 0;
    int64_t max_len = 0;
    for (int b = 0; b < B; ++b) {
        int64_t len = (int64_t)cu_seqlens[b + 1] - cu_seqlens[b];
        if (len < 0) return -1;
        if (len > max_len) max_len = len;
    }
    for (int64_t r = 0; r < n_q; ++r)
        if (qrow_t[r] < 0 || qrow_t[r] >= T || qrow_h[r] < 0 || qrow_h[r] >= Hq) return -1;
    for (int64_t r = 0; r < n_k; ++r)
        if (key_t[r] < 0 || key_t[r] >= T || key_hk[r] < 0 || key_hk[r] >= Hkv) return -1;
    /* which (token, kv head) rows does some chosen key need the statistics of? */
    unsigned char* need = (unsigned char*)calloc((size_t)(T * Hkv > 0 ? T * Hkv : 1), 1);
    for (int64_t r = 0; r < n_k; ++r) {
        const int64_t t = key_t[r];
        int b = 0;
        while (!(cu_seqlens[b] <= t && t < cu_seqlens[b + 1])) ++b;
        const int64_t s0 = cu_seqlens[b], len = cu_seqlens[b + 1] - s0, j = t - s0;
        for (int64_t i = j; i < len; ++i)
            if (swaa_oracle_visible(i, j, W, S, is_full)) need[(s0 + i) * Hkv + key_hk[r]] = 1;
    }
    double* rm = (double*)malloc(sizeof(double) * (size_t)(T * Hq > 0 ? T * Hq : 1));
    double* rden = (double*)malloc(sizeof(double) * (size_t)(T * Hq > 0 ? T * Hq : 1));
    double* rdot = (double*)malloc(sizeof(double) * (size_t)(T * Hq > 0 ? T * Hq : 1));
#pragma omp parallel
    {
        double* sc = (double*)malloc(sizeof(double) * (size_t)(max_len > 0 ? max_len : 1));
        double* dp = (double*)malloc(sizeof(double) * (size_t)(max_len > 0 ? max_len : 1));
        /* pass A: statistics of the needed rows (r < T*Hq), then dq of the chosen rows (r >= T*Hq) */
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < T * Hq + n_q; ++r) {
            const int chosen = r >= T * Hq;
            const int64_t t = chosen ? qrow_t[r - T * Hq] : r / Hq;
            const int h = chosen ? qrow_h[r - T * Hq] : (int)(r % Hq);
            const int hk = h / G;
            if (!chosen && !need[t * Hkv + hk]) continue;
            int b = 0;
            while (!(cu_seqlens[b] <= t && t < cu_seqlens[b + 1])) ++b;
            const int64_t s0 = cu_seqlens[b], i = t - s0;
            const float* qi = q + (t * Hq + h) * (int64_t)D;
            const float* gi = dout + (t * Hq + h) * (int64_t)D;
            double m = -INFINITY;
            for (int64_t j = 0; j <= i; ++j) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                const float* kj = k + ((s0 + j) * Hkv + hk) * (int64_t)D;
                const float* vj = v + ((s0 + j) * Hkv + hk) * (int64_t)D;
                double s = 0.0, d = 0.0;
                for (int c = 0; c < D; ++c) {
                    s += (double)qi[c] * (double)kj[c];
                    d += (double)gi[c] * (double)vj[c];
                }
                sc[j] = s * scale;
                dp[j] = d;
                if (sc[j] > m) m = sc[j];
            }
            double den = 0.0, dot = 0.0;
            for (int64_t j = 0; j <= i; ++j) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                den += exp(sc[j] - m);
            }
            if (out_given) {
                const float* oi = out_given + (t * Hq + h) * (int64_t)D;
                for (int c = 0; c < D; ++c) dot += (double)gi[c] * (double)oi[c];
            } else {
                for (int64_t j = 0; j <= i; ++j) {
                    if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                    dot += exp(sc[j] - m) / den * dp[j];
                }
            }
            if (!chosen) {
                rm[r] = m;
                rden[r] = den;
                rdot[r] = dot;
                continue;
            }
            double* dqi = dq_out + (r - T * Hq) * D;
            for (int c = 0; c < D; ++c) dqi[c] = 0.0;
            for (int64_t j = 0; j <= i; ++j) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                const double ds = exp(sc[j] - m) / den * (dp[j] - dot);
                const float* kj = k + ((s0 + j) * Hkv + hk) * (int64_t)D;
                for (int c = 0; c < D; ++c) dqi[c] += scale * ds * (double)kj[c];
            }
        }
        free(sc);
        free(dp);
        /* pass B: the chosen keys collect from the rows and heads that see them */
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_k; ++r) {
            const int64_t t = key_t[r];
            const int hk = key_hk[r];
            int b = 0;
            while (!(cu_seqlens[b] <= t && t < cu_seqlens[b + 1])) ++b;
            const int64_t s0 = cu_seqlens[b], len = cu_seqlens[b + 1] - s0, j = t - s0;
            const float* kj = k + (t * Hkv + hk) * (int64_t)D;
            const float* vj = v + (t * Hkv + hk) * (int64_t)D;
            double* dkj = dk_out + r * D;
            double* dvj = dv_out + r * D;
            for (int c = 0; c < D; ++c) dkj[c] = dvj[c] = 0.0;
            for (int64_t i = j; i < len; ++i) {
                if (!swaa_oracle_visible(i, j, W, S, is_full)) continue;
                for (int h = hk * G; h < (hk + 1) * G; ++h) {
                    const int64_t ri = (s0 + i) * Hq + h;
                    const float* qi = q + ri * D;
                    const float* gi = dout + ri * D;
                    double s = 0.0, d = 0.0;
                    for (int c = 0; c < D; ++c) {
                        s += (double)qi[c] * (double)kj[c];
                        d += (double)gi[c] * (double)vj[c];
                    }
                    const double p = exp(s * scale - rm[ri]) / rden[ri];
                    const double ds = p * (d - rdot[ri]);
                    for (int c = 0; c < D; ++c) {
                        dvj[c] += p * (double)gi[c];
                        dkj[c] += scale * ds * (double)qi[c];
                    }
                }
            }
        }
    }
    free(need);
    free(rm);
    free(rden);
    free(rdot);
    return 0;
}

/*
 * Layer schedule (Sec. 3.1.2 fixed-interval FA layers; Sec. 3.1.1 FA decode;
 * Table 1 columns "FA layers" and "FA decode").  Layers fa_start, fa_start +
 * fa_step, ... keep full attention (fa_step == 0: none).  phase 0 = prefill,
 * 1 = decode.  With fa_decode every layer is full in the decode phase.
 */
int swaa_oracle_layer_is_full(int layer, int fa_start, int fa_step, int fa_decode, int phase) {
    int in_list = 0;
    if (fa_step > 0)
        for (int l = fa_start; l <= layer; l += fa_step)
            if (l == layer) in_list = 1;
    if (in_list) return 1;
    if (phase == 1 && fa_decode) return 1;
    return 0;
}

/*
 * The same with an explicit set of FA layers (App. "Results of LightTransfer": the FA layers are chosen per layer
 * by a lazy ratio instead of at a fixed interval): fa_mask[layer] != 0 marks an FA layer.
 */
int swaa_oracle_layer_is_full_mask(int layer, const uint8_t* fa_mask, int fa_decode, int phase) {
    if (fa_mask[layer]) return 1;
    if (phase == 1 && fa_decode) return 1;
    return 0;
}

/*
 * Layer selection by lazy ratio (App. "Results of LightTransfer"): the n_lazy layers with the HIGHEST ratio are the
 * "lazy" ones (those that could take SWA), the rest "non-lazy".  fa_on_lazy == 0 gives full attention to the
 * non-lazy layers (the method as proposed), != 0 to the lazy ones (the variant the paper also evaluates).  Equal
 * ratios: the layer with the lower index counts as the lazier.  Plain selection: n_lazy passes, each taking the
 * largest remaining ratio.  fa_mask_out [n_layers].
 */
int swaa_oracle_select_fa_layers(const double* ratio, int n_layers, int n_lazy, int fa_on_lazy, uint8_t* fa_mask_out) {
    if (n_layers < 0 || n_lazy < 0 || n_lazy > n_layers) return -1;
    uint8_t* lazy = (uint8_t*)calloc((size_t)(n_layers > 0 ? n_layers : 1), 1);
    for (int pass = 0; pass < n_lazy; ++pass) {
        int best = -1;
        for (int l = 0; l < n_layers; ++l)
            if (!lazy[l] && (best < 0 || ratio[l] > ratio[best])) best = l;
        lazy[best] = 1;
    }
    for (int l = 0; l < n_layers; ++l) fa_mask_out[l] = (uint8_t)(fa_on_lazy ? lazy[l] : !lazy[l]);
    free(lazy);
    return 0;
}

int swaa_oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
