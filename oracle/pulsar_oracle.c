/*
 * Pulsar Attention context-encoding oracle: plain, slow, float64 CPU code.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker the CUDA library is
 * compared against; it shares no code, header, table or helper with the CUDA
 * path and the product never calls it.  Each function writes out the paper's
 * definition of the operation directly:
 *
 *   oracle_maxidf_select   Section 3.1 Eq. 2-3, Algorithm 1 lines 3 and 6,
 *                          Appendix C.1 (Eq. 5) and C.5 (Eq. 9), Eq. 4 / Eq. 14
 *   oracle_phase1_attn     Eq. 1 applied to the assembled input of Eq. 4
 *                          (Algorithm 1 lines 7-8), block rows only
 *   oracle_phase2_attn     Section 3.2 / Appendix H: one softmax over the
 *                          concatenated retained KV, plus per-block partials
 *   oracle_lse_merge       Appendix H Eq. 12-13, applied iteratively
 *   oracle_chunk_select    Appendix C: the TF-IDF (Eq. 6), BM25 (Eq. 7), type-token (Eq. 8) and
 *                          Max-IDF (Eq. 9) chunk scores with the same top-k and prefix list
 *   oracle_assemble_positions, oracle_rope_apply   Appendix E: position ids of the assembled
 *                          inputs (sparse / contiguous) and the rotary embedding they feed
 *   oracle_generate_step   Algorithm 1 lines 11-16: append KV(q) to the generation shard,
 *                          attend to context + shard (causal within the shard)
 *
 * Readings taken where the paper is silent: natural logarithm; N = number of
 * logical blocks; equal chunk scores are ranked by the lower chunk index;
 * duplicates between the sink and the first summary are kept (each occurrence
 * counts once); query head h reads KV head h / (Hq/Hkv); softmax scale
 * 1/sqrt(d) unless the caller gives one; LSE is the natural log of the sum of
 * exponentials of the scaled logits.
 *
 * Parity pins (tests, CPU only): brute-force selection on tiny inputs, needle
 * property, Table 6 lengths, dense attention with a materialised multiplicity
 * mask, library causal attention for block 0, single softmax over all keys for
 * Phase 2.  Parity unpinned (no statement in the paper): the tie-break rule
 * and the keeping of duplicates; both are the readings above.
 *
 * bf16 inputs arrive as raw 16-bit patterns and are widened exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------ */
/* Selection                                                                 */
/* ------------------------------------------------------------------------ */

/*
 * df(t)  = number of blocks that contain token t          (Section 3.1)
 * IDF(t) = ln(N / max(df(t), 1)),  N = number of blocks    (Eq. 3 / Eq. 5)
 * score(chunk) = max over its tokens of IDF                (Eq. 2 / Eq. 9)
 * Sigma_b = the k best chunks of block b, in positional order (Alg. 1 l.6)
 * prefix  = [sink | Sigma_0 | ... | Sigma_{B-2}], block i uses its first
 *           prefix_len[i] entries: 0 for i = 0, else sink + the tokens of
 *           Sigma_0 .. Sigma_{i-1}, which is sink + i*k*chunk when every selected
 *           chunk is a whole one (Eq. 4, Eq. 14)
 *
 * Lengths that do not divide (the paper cuts the tokenised context "into blocks
 * of size" n_b and each block into chunks of m tokens, and says no more; the
 * reading taken): the B = ceil(L / n_b) blocks are consecutive runs of n_b
 * tokens, the last one holding the L - (B-1) n_b tokens that remain; a block of
 * len tokens has ceil(len / m) chunks, the last one holding the tokens that
 * remain and scored on those; a block with fewer than k chunks contributes all
 * of them; the sink is the first min(sink, |B_0|) tokens.
 *
 * C = ceil(block_size / chunk) chunk slots per block.  Outputs (any may be NULL):
 * sel_chunks [B*k] (a block's chosen chunks ascending, then -1 up to k),
 * prefix_idx [sink+(B-1)*k*chunk] (entries past the last used one are -1),
 * prefix_len [B], df_out [vocab], idf_out [vocab], score_out [B*C] (-inf for a
 * slot without a chunk).
 * Returns 0, or -1 on a shape that the definition does not cover.
 */
int oracle_maxidf_select(const uint32_t *token_ids, int64_t L, int32_t vocab_size,
                         int32_t block_size, int32_t chunk, int32_t k, int32_t sink,
                         int32_t *sel_chunks, int32_t *prefix_idx, int32_t *prefix_len,
                         uint32_t *df_out, double *idf_out, double *score_out) {
    if (L <= 0 || block_size <= 0 || chunk <= 0 || vocab_size <= 0) return -1;
    const int64_t B = (L + block_size - 1) / block_size;
    const int64_t C = (block_size + chunk - 1) / chunk;
    if (k < 0 || k > C || sink < 0 || sink > block_size) return -1;
    for (int64_t p = 0; p < L; ++p)
        if (token_ids[p] >= (uint32_t)vocab_size) return -1;

    uint32_t *df = (uint32_t *)calloc((size_t)vocab_size, sizeof(uint32_t));
    int64_t *last_block = (int64_t *)malloc((size_t)vocab_size * sizeof(int64_t));
    double *idf = (double *)malloc((size_t)vocab_size * sizeof(double));
    double *score = (double *)malloc((size_t)C * sizeof(double));
    char *taken = (char *)malloc((size_t)C);
    if (!df || !last_block || !idf || !score || !taken) return -2;

    /* document frequency: a block counts once however often the token occurs */
    for (int64_t t = 0; t < vocab_size; ++t) last_block[t] = -1;
    for (int64_t p = 0; p < L; ++p) {
        const int64_t b = p / block_size;
        uint32_t t = token_ids[p];
        if (last_block[t] != b) { last_block[t] = b; df[t] += 1; }
    }
    for (int64_t t = 0; t < vocab_size; ++t) {
        uint32_t f = df[t] > 1 ? df[t] : 1;
        idf[t] = log((double)B / (double)f);
    }

    const int64_t cap = sink + (B - 1) * (int64_t)k * chunk;      /* room in prefix_idx */
    const int64_t len0 = L < block_size ? L : block_size;
    int64_t used = sink < len0 ? sink : len0;                     /* entries written so far */
    if (prefix_idx) for (int64_t j = 0; j < used; ++j) prefix_idx[j] = (int32_t)j;

    for (int64_t b = 0; b < B; ++b) {
        const int64_t lo = b * block_size;
        const int64_t hi = lo + block_size < L ? lo + block_size : L;
        const int64_t Cb = (hi - lo + chunk - 1) / chunk;         /* chunks this block has */
        if (prefix_len) prefix_len[b] = b == 0 ? 0 : (int32_t)used;
        for (int64_t c = 0; c < C; ++c) {
            double s = -INFINITY;
            for (int64_t p = lo + c * chunk; p < lo + (c + 1) * chunk && p < hi; ++p) {
                double v = idf[token_ids[p]];
                if (v > s) s = v;
            }
            score[c] = s;
            if (score_out) score_out[b * C + c] = s;
        }
        /* top-k: take the best remaining chunk k times; a strict comparison
           scanning upward leaves equal scores to the lower index */
        memset(taken, 0, (size_t)C);
        for (int32_t j = 0; j < k && j < Cb; ++j) {
            int64_t best = -1;
            for (int64_t c = 0; c < Cb; ++c)
                if (!taken[c] && (best < 0 || score[c] > score[best])) best = c;
            if (best >= 0) taken[best] = 1;
        }
        /* positional order */
        int32_t j = 0;
        for (int64_t c = 0; c < Cb; ++c) {
            if (!taken[c]) continue;
            if (sel_chunks) sel_chunks[b * k + j] = (int32_t)c;
            if (b < B - 1)
                for (int64_t p = lo + c * chunk; p < lo + (c + 1) * chunk && p < hi; ++p) {
                    if (prefix_idx) prefix_idx[used] = (int32_t)p;
                    ++used;
                }
            ++j;
        }
        for (; j < k; ++j)
            if (sel_chunks) sel_chunks[b * k + j] = -1;
    }
    if (prefix_idx) for (int64_t j = used; j < cap; ++j) prefix_idx[j] = -1;

    if (df_out) memcpy(df_out, df, (size_t)vocab_size * sizeof(uint32_t));
    if (idf_out) memcpy(idf_out, idf, (size_t)vocab_size * sizeof(double));
    free(df); free(last_block); free(idf); free(score); free(taken);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Attention over an explicit key list                                       */
/* ------------------------------------------------------------------------ */

/* softmax(q.k_j * scale) V over keys key[0..n) of KV head kv; out[d], *lse.
   z is caller scratch of n doubles. */
static void attend_list(const double *q, const float *Kf, const float *Vf,
                        const int64_t *key, int64_t n, int32_t Hkv, int32_t kv,
                        int32_t d, double scale, double *z, double *out, double *lse) {
    double zmax = -INFINITY;
    for (int64_t j = 0; j < n; ++j) {
        const float *kr = Kf + ((size_t)key[j] * Hkv + kv) * d;
        double acc = 0.0;
        for (int32_t e = 0; e < d; ++e) acc += q[e] * (double)kr[e];
        z[j] = acc * scale;
        if (z[j] > zmax) zmax = z[j];
    }
    double denom = 0.0;
    for (int32_t e = 0; e < d; ++e) out[e] = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        double w = exp(z[j] - zmax);
        denom += w;
        const float *vr = Vf + ((size_t)key[j] * Hkv + kv) * d;
        for (int32_t e = 0; e < d; ++e) out[e] += w * (double)vr[e];
    }
    for (int32_t e = 0; e < d; ++e) out[e] /= denom;
    *lse = zmax + log(denom);
}

static float *widen(const uint16_t *x, size_t n) {
    float *f = (float *)malloc(n * sizeof(float));
    if (!f) return NULL;
    for (size_t i = 0; i < n; ++i) f[i] = (float)bf16_to_double(x[i]);
    return f;
}

/*
 * Phase 1 (Eq. 1 over Input_i of Eq. 4).  Query row at global position
 * p = i*block_size + r, head h, sees the keys prefix_idx[0 .. prefix_len[i])
 * followed by the block's own rows i*block_size .. p (causal).  A key that is
 * listed twice is attended twice.
 *
 * Q [L,Hq,d], K,V [L,Hkv,d] bf16 bit patterns.  rows: n_rows global query
 * positions to compute (NULL = all L, in order).  O [n_rows,Hq,d] and
 * LSE [n_rows,Hq] in float64.  scale <= 0 selects 1/sqrt(d).
 */
int oracle_phase1_attn(const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                       int64_t L, int32_t Hq, int32_t Hkv, int32_t d, int32_t block_size,
                       const int32_t *prefix_idx, const int32_t *prefix_len,
                       int32_t prefix_total, double scale,
                       const int64_t *rows, int64_t n_rows, double *O, double *LSE) {
    if (L <= 0 || block_size <= 0 || Hkv <= 0 || Hq % Hkv || d <= 0) return -1;
    const int64_t B = (L + block_size - 1) / block_size;      /* the last block may be shorter */
    for (int64_t i = 0; i < B; ++i) {
        if (prefix_len[i] < 0 || prefix_len[i] > prefix_total) return -1;
        for (int32_t j = 0; j < prefix_len[i]; ++j)
            if (prefix_idx[j] < 0 || prefix_idx[j] >= i * block_size) return -1;
    }
    if (!rows) n_rows = L;
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    const int32_t g = Hq / Hkv;
    float *Kf = widen(K, (size_t)L * Hkv * d);
    float *Vf = widen(V, (size_t)L * Hkv * d);
    if (!Kf || !Vf) return -2;
    int err = 0;

#pragma omp parallel
    {
        int64_t *key = (int64_t *)malloc((size_t)(prefix_total + block_size) * sizeof(int64_t));
        double *z = (double *)malloc((size_t)(prefix_total + block_size) * sizeof(double));
        double *q = (double *)malloc((size_t)d * sizeof(double));
        if (!key || !z || !q) {
#pragma omp atomic write
            err = -2;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int64_t s = 0; s < n_rows; ++s) {
                const int64_t p = rows ? rows[s] : s;
                const int64_t i = p / block_size;
                int64_t n = 0;
                for (int32_t j = 0; j < prefix_len[i]; ++j) key[n++] = prefix_idx[j];
                for (int64_t j = i * block_size; j <= p; ++j) key[n++] = j;
                for (int32_t h = 0; h < Hq; ++h) {
                    for (int32_t e = 0; e < d; ++e)
                        q[e] = bf16_to_double(Q[((size_t)p * Hq + h) * d + e]);
                    attend_list(q, Kf, Vf, key, n, Hkv, h / g, d, scale, z,
                                O + ((size_t)s * Hq + h) * d, LSE + (size_t)s * Hq + h);
                }
            }
        }
        free(key); free(z); free(q);
    }
    free(Kf); free(Vf);
    return err;
}

/*
 * Phase 2.  Every query row attends to all L = B*block_size retained keys of
 * its KV head with one softmax (the result the LSE merge must reproduce), and,
 * if part_O/part_LSE are given, to each block's block_size keys separately
 * (A_h, l_h of Algorithm 1 line 12).
 *
 * Qq [nq,Hq,d], K,V [B*block_size,Hkv,d] bf16 bit patterns.
 * O [nq,Hq,d], LSE [nq,Hq]; part_O [B,nq,Hq,d], part_LSE [B,nq,Hq] or NULL.
 */
int oracle_phase2_attn(const uint16_t *Qq, int32_t nq, const uint16_t *K, const uint16_t *V,
                       int32_t B, int32_t block_size, int32_t Hq, int32_t Hkv, int32_t d,
                       double scale, double *O, double *LSE, double *part_O, double *part_LSE) {
    if (nq <= 0 || B <= 0 || block_size <= 0 || Hkv <= 0 || Hq % Hkv || d <= 0) return -1;
    const int64_t L = (int64_t)B * block_size;
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    const int32_t g = Hq / Hkv;
    float *Kf = widen(K, (size_t)L * Hkv * d);
    float *Vf = widen(V, (size_t)L * Hkv * d);
    if (!Kf || !Vf) return -2;
    int err = 0;

#pragma omp parallel
    {
        int64_t *key = (int64_t *)malloc((size_t)L * sizeof(int64_t));
        double *z = (double *)malloc((size_t)L * sizeof(double));
        double *q = (double *)malloc((size_t)d * sizeof(double));
        if (!key || !z || !q) {
#pragma omp atomic write
            err = -2;
        } else {
            for (int64_t j = 0; j < L; ++j) key[j] = j;
#pragma omp for schedule(dynamic, 1) collapse(2)
            for (int32_t r = 0; r < nq; ++r)
                for (int32_t h = 0; h < Hq; ++h) {
                    for (int32_t e = 0; e < d; ++e)
                        q[e] = bf16_to_double(Qq[((size_t)r * Hq + h) * d + e]);
                    attend_list(q, Kf, Vf, key, L, Hkv, h / g, d, scale, z,
                                O + ((size_t)r * Hq + h) * d, LSE + (size_t)r * Hq + h);
                    if (part_O && part_LSE)
                        for (int32_t b = 0; b < B; ++b)
                            attend_list(q, Kf, Vf, key + (int64_t)b * block_size, block_size,
                                        Hkv, h / g, d, scale, z,
                                        part_O + (((size_t)b * nq + r) * Hq + h) * d,
                                        part_LSE + ((size_t)b * nq + r) * Hq + h);
                }
        }
        free(key); free(z); free(q);
    }
    free(Kf); free(Vf);
    return err;
}

/*
 * Online-softmax merge, Appendix H Eq. 12-13, folded over the parts in order:
 *   l' = l + ln(1 + e^{l_h - l}),  o' = e^{l - l'} o + e^{l_h - l'} o_h.
 * part_O [n_parts,rows,d], part_LSE [n_parts,rows] -> O [rows,d], LSE [rows].
 */
int oracle_lse_merge(const double *part_O, const double *part_LSE, int32_t n_parts,
                     int64_t rows, int32_t d, double *O, double *LSE) {
    if (n_parts <= 0 || rows < 0 || d <= 0) return -1;
    for (int64_t r = 0; r < rows; ++r) {
        double l = part_LSE[r];
        for (int32_t e = 0; e < d; ++e) O[r * d + e] = part_O[r * d + e];
        for (int32_t h = 1; h < n_parts; ++h) {
            double lh = part_LSE[(size_t)h * rows + r];
            double ln = l + log(1.0 + exp(lh - l));
            double a = exp(l - ln), bw = exp(lh - ln);
            const double *oh = part_O + ((size_t)h * rows + r) * d;
            for (int32_t e = 0; e < d; ++e) O[r * d + e] = a * O[r * d + e] + bw * oh[e];
            l = ln;
        }
        LSE[r] = l;
    }
    return 0;
}

/*
 * One generation step (Algorithm 1 lines 11-16).  The n_new newest tokens' keys and values are
 * appended to the generation shard (line 15); new token u then attends with one softmax to all
 * L context keys and to shard rows 0 .. gen_len + u (itself included), which is what the merged
 * per-shard results of lines 12-13 equal (Section 3.2).
 *
 * Qnew [n_new,Hq,d], Knew,Vnew [n_new,Hkv,d], Kctx,Vctx [L,Hkv,d], Kgen,Vgen [gen_cap,Hkv,d]
 * bf16 bit patterns; Kgen/Vgen rows [gen_len, gen_len+n_new) are overwritten.
 * O [n_new,Hq,d], LSE [n_new,Hq] float64.
 */
int oracle_generate_step(const uint16_t *Qnew, const uint16_t *Knew, const uint16_t *Vnew, int32_t n_new,
                         const uint16_t *Kctx, const uint16_t *Vctx, int64_t L,
                         uint16_t *Kgen, uint16_t *Vgen, int32_t gen_len, int32_t gen_cap,
                         int32_t Hq, int32_t Hkv, int32_t d, double scale, double *O, double *LSE) {
    if (n_new <= 0 || L <= 0 || gen_len < 0 || gen_len + n_new > gen_cap || Hkv <= 0 || Hq % Hkv || d <= 0)
        return -1;
    if (scale <= 0.0) scale = 1.0 / sqrt((double)d);
    const int32_t g = Hq / Hkv;
    const size_t row = (size_t)Hkv * d;
    memcpy(Kgen + (size_t)gen_len * row, Knew, (size_t)n_new * row * sizeof(uint16_t));
    memcpy(Vgen + (size_t)gen_len * row, Vnew, (size_t)n_new * row * sizeof(uint16_t));
    const int64_t total = L + gen_len + n_new;
    /* context rows followed by shard rows, widened */
    float *Kf = (float *)malloc((size_t)total * row * sizeof(float));
    float *Vf = (float *)malloc((size_t)total * row * sizeof(float));
    int64_t *key = (int64_t *)malloc((size_t)total * sizeof(int64_t));
    double *z = (double *)malloc((size_t)total * sizeof(double));
    double *q = (double *)malloc((size_t)d * sizeof(double));
    if (!Kf || !Vf || !key || !z || !q) return -2;
    for (size_t i = 0; i < (size_t)L * row; ++i) { Kf[i] = (float)bf16_to_double(Kctx[i]); Vf[i] = (float)bf16_to_double(Vctx[i]); }
    for (size_t i = 0; i < (size_t)(gen_len + n_new) * row; ++i) {
        Kf[(size_t)L * row + i] = (float)bf16_to_double(Kgen[i]);
        Vf[(size_t)L * row + i] = (float)bf16_to_double(Vgen[i]);
    }
    for (int64_t j = 0; j < total; ++j) key[j] = j;
    for (int32_t u = 0; u < n_new; ++u)
        for (int32_t h = 0; h < Hq; ++h) {
            for (int32_t e = 0; e < d; ++e) q[e] = bf16_to_double(Qnew[((size_t)u * Hq + h) * d + e]);
            attend_list(q, Kf, Vf, key, L + gen_len + u + 1, Hkv, h / g, d, scale, z,
                        O + ((size_t)u * Hq + h) * d, LSE + (size_t)u * Hq + h);
        }
    free(Kf); free(Vf); free(key); free(z); free(q);
    return 0;
}

/*
 * Chunk selection under any of the four scoring heuristics of Appendix C.
 *   mode 0  Max-IDF   score = max_p IDF(t_p)                               (Eq. 9)
 *   mode 1  TF-IDF    score = (1/|C|) sum_p IDF(t_p)                       (Eq. 6)
 *   mode 2  BM25      score = sum over types t of IDF_BM25(t) * tf(t)(k1+1) / (tf(t) + k1 D(C)),
 *                     D(C) = 1 - b + b |C| / lbar, k1 = 1.2, b = 0.75, lbar = mean chunk length,
 *                     IDF_BM25(t) = ln((N - df + 0.5)/(df + 0.5) + 1)      (Eq. 7)
 *   mode 3  type-token ratio ("Entropy")  score = distinct tokens / |C|    (Eq. 8)
 * IDF(t) = ln(N / max(df, 1)) (Eq. 5).  Sums run over the chunk's positions in order (BM25:
 * over its types in order of first occurrence), in float64.  Top-k, tie rule, positional order,
 * the prefix list and the treatment of lengths that do not divide are those of
 * oracle_maxidf_select: |C| is the number of tokens the chunk has (a short last chunk is scored
 * on those), lbar = L / (number of chunks in the sequence).
 * Outputs as there; score_out [B*C] float64 (-inf for a slot without a chunk).
 */
int oracle_chunk_select(const uint32_t *token_ids, int64_t L, int32_t vocab_size, int32_t block_size,
                        int32_t chunk, int32_t k, int32_t sink, int32_t mode,
                        int32_t *sel_chunks, int32_t *prefix_idx, int32_t *prefix_len, double *score_out) {
    if (L <= 0 || block_size <= 0 || chunk <= 0 || vocab_size <= 0 || mode < 0 || mode > 3) return -1;
    const int64_t B = (L + block_size - 1) / block_size, C = (block_size + chunk - 1) / chunk;
    if (k < 0 || k > C || sink < 0 || sink > block_size) return -1;
    for (int64_t p = 0; p < L; ++p)
        if (token_ids[p] >= (uint32_t)vocab_size) return -1;
    uint32_t *df = (uint32_t *)calloc((size_t)vocab_size, sizeof(uint32_t));
    int64_t *last_block = (int64_t *)malloc((size_t)vocab_size * sizeof(int64_t));
    double *score = (double *)malloc((size_t)C * sizeof(double));
    char *taken = (char *)malloc((size_t)C);
    if (!df || !last_block || !score || !taken) return -2;
    for (int64_t t = 0; t < vocab_size; ++t) last_block[t] = -1;
    for (int64_t p = 0; p < L; ++p) {
        const int64_t b = p / block_size;
        uint32_t t = token_ids[p];
        if (last_block[t] != b) { last_block[t] = b; df[t] += 1; }
    }
    const double N = (double)B, k1 = 1.2, bb = 0.75;
    /* mean chunk length over the sequence: full blocks have C chunks, the last block what it needs */
    const int64_t last_len = L - (B - 1) * block_size;
    const int64_t n_chunks = (B - 1) * C + (last_len + chunk - 1) / chunk;
    const double lbar = (double)L / (double)n_chunks;
    const int64_t cap = sink + (B - 1) * (int64_t)k * chunk;
    const int64_t len0 = L < block_size ? L : block_size;
    int64_t used = sink < len0 ? sink : len0;
    if (prefix_idx) for (int64_t j = 0; j < used; ++j) prefix_idx[j] = (int32_t)j;
    for (int64_t b = 0; b < B; ++b) {
        const int64_t lo = b * block_size;
        const int64_t hi = lo + block_size < L ? lo + block_size : L;
        const int64_t Cb = (hi - lo + chunk - 1) / chunk;
        if (prefix_len) prefix_len[b] = b == 0 ? 0 : (int32_t)used;
        for (int64_t c = 0; c < C; ++c) {
            const uint32_t *tok = token_ids + lo + c * chunk;
            int64_t len = hi - (lo + c * chunk);
            if (len > chunk) len = chunk;
            double s = 0.0;
            if (len <= 0) {
                s = -INFINITY;
            } else if (mode == 0) {
                s = -INFINITY;
                for (int64_t p = 0; p < len; ++p) {
                    uint32_t f = df[tok[p]] > 1 ? df[tok[p]] : 1;
                    double v = log(N / (double)f);
                    if (v > s) s = v;
                }
            } else if (mode == 1) {
                for (int64_t p = 0; p < len; ++p) {
                    uint32_t f = df[tok[p]] > 1 ? df[tok[p]] : 1;
                    s = s + log(N / (double)f);
                }
                s = s / (double)len;
            } else {
                const double Dc = (1.0 - bb) + bb * ((double)len / lbar);
                int32_t distinct = 0;
                for (int64_t p = 0; p < len; ++p) {
                    int first = 1;
                    for (int64_t q = 0; q < p; ++q) if (tok[q] == tok[p]) first = 0;
                    if (!first) continue;
                    ++distinct;
                    if (mode == 2) {
                        int32_t tf = 0;
                        for (int64_t q = 0; q < len; ++q) if (tok[q] == tok[p]) ++tf;
                        double f = (double)df[tok[p]];
                        double idf = log((N - f + 0.5) / (f + 0.5) + 1.0);
                        s = s + (idf * ((double)tf * (k1 + 1.0))) / ((double)tf + k1 * Dc);
                    }
                }
                if (mode == 3) s = (double)distinct / (double)len;
            }
            score[c] = s;
            if (score_out) score_out[b * C + c] = s;
        }
        memset(taken, 0, (size_t)C);
        for (int32_t j = 0; j < k && j < Cb; ++j) {
            int64_t best = -1;
            for (int64_t c = 0; c < Cb; ++c)
                if (!taken[c] && (best < 0 || score[c] > score[best])) best = c;
            if (best >= 0) taken[best] = 1;
        }
        int32_t j = 0;
        for (int64_t c = 0; c < Cb; ++c) {
            if (!taken[c]) continue;
            if (sel_chunks) sel_chunks[b * k + j] = (int32_t)c;
            if (b < B - 1)
                for (int64_t p = lo + c * chunk; p < lo + (c + 1) * chunk && p < hi; ++p) {
                    if (prefix_idx) prefix_idx[used] = (int32_t)p;
                    ++used;
                }
            ++j;
        }
        for (; j < k; ++j)
            if (sel_chunks) sel_chunks[b * k + j] = -1;
    }
    if (prefix_idx) for (int64_t j = used; j < cap; ++j) prefix_idx[j] = -1;
    free(df); free(last_block); free(score); free(taken);
    return 0;
}

/*
 * Position ids of the assembled Phase-1 inputs (Appendix E).  Input_i = [first prefix_len[i] entries
 * of the prefix list | block i] (Eq. 4), the inputs stored back to back.
 *   mode 0 (sparse, the paper's default): every token keeps its global position -- a prefix entry
 *          its prefix_idx value, row r of block i the position i*block_size + r
 *   mode 1 (contiguous): each input is renumbered 0 .. n_i - 1
 * pos_out has sum_i (prefix_len[i] + block_size) entries.  Returns that count, or -1.
 */
int64_t oracle_assemble_positions(const int32_t *prefix_idx, const int32_t *prefix_len, int32_t n_blocks,
                                  int32_t block_size, int32_t mode, int32_t *pos_out) {
    if (n_blocks <= 0 || block_size <= 0 || (mode != 0 && mode != 1)) return -1;
    int64_t at = 0;
    for (int32_t i = 0; i < n_blocks; ++i) {
        for (int32_t j = 0; j < prefix_len[i]; ++j) pos_out[at++] = mode == 0 ? prefix_idx[j] : j;
        for (int32_t r = 0; r < block_size; ++r)
            pos_out[at++] = mode == 0 ? i * block_size + r : prefix_len[i] + r;
    }
    return at;
}

/*
 * Rotary position embedding with explicit position ids (Appendix E; the rotate-half pairing of
 * the Llama family the paper runs on): for row n at position p = positions[n], head h and
 * j < d/2, with angle = p * theta^(-2j/d):
 *   y[j]       = x[j] cos(angle) - x[j + d/2] sin(angle)
 *   y[j + d/2] = x[j + d/2] cos(angle) + x[j] sin(angle)
 * X [rows, H, d] bf16 bits; Y [rows, H, d] float64 (not rounded).
 */
int oracle_rope_apply(const uint16_t *X, int64_t rows, int32_t H, int32_t d, const int32_t *positions,
                      double theta, double *Y) {
    if (rows < 0 || H <= 0 || d <= 0 || d % 2 != 0 || theta <= 0.0) return -1;
    const int32_t half = d / 2;
    for (int64_t n = 0; n < rows; ++n)
        for (int32_t j = 0; j < half; ++j) {
            const double angle = (double)positions[n] * pow(theta, -2.0 * (double)j / (double)d);
            const double c = cos(angle), sn = sin(angle);
            for (int32_t h = 0; h < H; ++h) {
                const size_t base = ((size_t)n * H + h) * d;
                const double a = bf16_to_double(X[base + j]), b = bf16_to_double(X[base + j + half]);
                Y[base + j] = a * c - b * sn;
                Y[base + j + half] = b * c + a * sn;
            }
        }
    return 0;
}
