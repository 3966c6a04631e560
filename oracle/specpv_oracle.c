/*
 * SpecPV verification hot path -- float64 CPU ORACLE.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the method
 * computes, written from the paper's definitions (Section 3.2 "Partial Verification",
 * Eq. 1-3; Section 3.3 "Rectified with Full Verification"; Algorithm 1).  It shares no code
 * with the CUDA library, is never called by the product path, and is only used by the tests,
 * the smoke check and the benchmark's CPU-baseline leg.
 *
 * Every accumulation is in double.  Inputs are the very buffers the GPU kernels read
 * (float32 or bfloat16 raw bytes, widened exactly to double), in the cache layout below.
 * No blocking, fusion or reordering beyond what a definition states; the only parallelism is
 * an OpenMP loop over independent (kv head) / (row) items.
 *
 * Layouts (all row-major, caller-owned host memory):
 *   K/V pool of ONE layer : [n_pages][Hkv][bs][d]          (dtype: 0 = float32, 1 = bfloat16)
 *   block table of one seq : [n_blocks] logical block -> page id
 *   Q                      : [M][Hq][d]      Knew/Vnew : [M][Hkv][d]
 *   tree mask              : [M][W] uint64, W = ceil(M/64); bit a of row j set <=> key a visible to j
 *   summaries              : [Hkv][nb][d] double (exact: max/min of representable values)
 *   scores                 : [Hkv][nb] double
 *
 * Readings of points the paper leaves open (also listed in the design notes); the four
 * marked (*) have no pin in the paper and are "parity unpinned" by it -- they are pinned only
 * against these readings:
 *   (*) Eq. 2 is taken as printed: max of the two FULL dot products q.Kmax and q.Kmin.
 *   (*) GQA: selection is per (layer, sequence, KV head); the reduction f of Eq. 3 runs over
 *       all G*M rows of the head group (mean, max) or, for "last", is the mean over the G
 *       heads of the single row `last_query`.
 *   (*) The budget counts sink + retrieval + local blocks; the buffer is extra.
 *   (*) Local window = the last `local_blocks` blocks including a ragged last block.
 *   Top-k ties go to the lower block index; NaN ranks below every number.
 *   Tree mask = ancestor-or-self; in a refresh the partially verified tokens form a chain in
 *   front of the tree and the tree root's parent is the chain's last token.
 *   Attention follows the semantics of scaled-dot-product attention (Section 4.1,
 *   "Implementations"): softmax(q.k * scale) over the visible keys; masked keys are skipped.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_API __attribute__((visibility("default")))

static double load_elem(const void *base, int dtype, int64_t i) {
    if (dtype == 0) {
        return (double)((const float *)base)[i];
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[i]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

static void copy_elems(void *dst, int64_t dst_i, const void *src, int64_t src_i, int64_t n, int dtype) {
    size_t es = dtype == 0 ? 4 : 2;
    memcpy((char *)dst + dst_i * es, (const char *)src + src_i * es, (size_t)n * es);
}

ORACLE_API int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------------
 * Tree mask (token-tree verification, Section 1 / Section 3.3 / Algorithm 1 "TreeDecode").
 * Rows 0..n_chain-1 : partially verified tokens, a chain (row r sees rows 0..r).
 * Rows n_chain..    : tree nodes; parents[] are tree-relative, root has parent -1 and hangs
 *                     off the chain's last row.  A node sees itself and its ancestors.
 * Returns 0, or -1 when parents[] is not a forest-free tree in topological order.
 * ------------------------------------------------------------------------------------------ */
ORACLE_API int oracle_tree_mask(const int32_t *parents, int n_tree, int n_chain, uint64_t *mask) {
    int M = n_tree + n_chain;
    int W = (M + 63) / 64;
    memset(mask, 0, (size_t)M * W * sizeof(uint64_t));
    for (int r = 0; r < n_chain; ++r)
        for (int a = 0; a <= r; ++a) mask[(size_t)r * W + a / 64] |= 1ull << (a % 64);
    for (int i = 0; i < n_tree; ++i) {
        int p = parents[i];
        if (i == 0 ? p != -1 : (p < 0 || p >= i)) return -1;
    }
    for (int i = 0; i < n_tree; ++i) {
        int row = n_chain + i;
        /* the whole chain precedes every tree node */
        for (int a = 0; a < n_chain; ++a) mask[(size_t)row * W + a / 64] |= 1ull << (a % 64);
        for (int a = i; a >= 0; a = parents[a]) {
            int col = n_chain + a;
            mask[(size_t)row * W + col / 64] |= 1ull << (col % 64);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Eq. 1: block key summaries C_i = (K_i^max, K_i^min), element-wise over the valid tokens of
 * block i, for one layer and one sequence.
 * ------------------------------------------------------------------------------------------ */
ORACLE_API void oracle_block_summaries(const void *k_pool, int dtype, int Hkv, int bs, int d,
                                       const int32_t *block_table, int seq_len,
                                       double *kmax, double *kmin) {
    int nb = (seq_len + bs - 1) / bs;
    for (int h = 0; h < Hkv; ++h)
        for (int i = 0; i < nb; ++i) {
            int n_valid = seq_len - i * bs < bs ? seq_len - i * bs : bs;
            int64_t page = block_table[i];
            for (int c = 0; c < d; ++c) {
                double mx = -INFINITY, mn = INFINITY;
                for (int t = 0; t < n_valid; ++t) {
                    double k = load_elem(k_pool, dtype, ((page * Hkv + h) * bs + t) * d + c);
                    if (k > mx) mx = k;
                    if (k < mn) mn = k;
                }
                kmax[((size_t)h * nb + i) * d + c] = mx;
                kmin[((size_t)h * nb + i) * d + c] = mn;
            }
        }
}

/* ------------------------------------------------------------------------------------------
 * Eq. 2-3: s_{i,j} = max(q_j . Kmax_i, q_j . Kmin_i), reduced over the step's query rows.
 * reduce: 0 mean, 1 max, 2 last (row `last_query`, averaged over the G heads of the group).
 * ------------------------------------------------------------------------------------------ */
ORACLE_API void oracle_block_scores_mode(const void *q, int dtype, int M, int Hq, int Hkv, int d,
                                         const double *kmax, const double *kmin, int nb,
                                         int reduce, int last_query, int score_mode, double *scores) {
    int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(static)
    for (int h = 0; h < Hkv; ++h)
        for (int i = 0; i < nb; ++i) {
            const double *bmax = kmax + ((size_t)h * nb + i) * d;
            const double *bmin = kmin + ((size_t)h * nb + i) * d;
            double acc = reduce == 1 ? -INFINITY : 0.0;
            int count = 0;
            for (int j = 0; j < M; ++j) {
                if (reduce == 2 && j != last_query) continue;
                for (int g = 0; g < G; ++g) {
                    int64_t qoff = ((int64_t)j * Hq + h * G + g) * d;
                    double dmax = 0.0, dmin = 0.0, chan = 0.0;
                    for (int c = 0; c < d; ++c) {
                        double qc = load_elem(q, dtype, qoff + c);
                        double a = qc * bmax[c], b = qc * bmin[c];
                        dmax += a;
                        dmin += b;
                        chan += a > b ? a : b;  /* channel-wise form: the maximum is taken per channel */
                    }
                    /* score_mode 0: Eq. 2 as printed (max of the two full dot products);
                     * score_mode 1: the channel-wise bound of Quest, which Section 3.2 cites as its inspiration:
                     *               sum_c max(q_c Kmax_c, q_c Kmin_c) >= q . k for every key k of the block */
                    double s = score_mode == 1 ? chan : (dmax > dmin ? dmax : dmin);
                    if (reduce == 1) { if (s > acc) acc = s; }
                    else acc += s;
                    ++count;
                }
            }
            scores[(size_t)h * nb + i] = reduce == 1 ? acc : acc / (double)count;
        }
}

ORACLE_API void oracle_block_scores(const void *q, int dtype, int M, int Hq, int Hkv, int d,
                                    const double *kmax, const double *kmin, int nb,
                                    int reduce, int last_query, double *scores) {
    oracle_block_scores_mode(q, dtype, M, Hq, Hkv, d, kmax, kmin, nb, reduce, last_query, 0, scores);
}

/* ------------------------------------------------------------------------------------------
 * Selection (Section 3.2): retained blocks = sink blocks U top-scoring retrieval blocks U
 * local blocks, ascending.  Candidates are blocks [sink, nb - local); k = budget - sink - local.
 * If nb <= budget every block is kept.  Ranking: score descending, then block index ascending;
 * NaN below everything.  Returns the count written to idx (= min(nb, budget_blocks)).
 * ------------------------------------------------------------------------------------------ */
static int ranks_before(double sa, int ia, double sb, int ib) {
    /* 1 if block (sa, ia) ranks strictly ahead of block (sb, ib) */
    int na = isnan(sa), nb_ = isnan(sb);
    if (na || nb_) {
        if (na && nb_) return ia < ib;
        return nb_; /* the number ranks ahead of the NaN */
    }
    if (sa != sb) return sa > sb;
    return ia < ib;
}

ORACLE_API int oracle_select(const double *scores, int nb, int sink_blocks, int local_blocks,
                             int budget_blocks, int32_t *idx) {
    if (nb <= budget_blocks) {
        for (int i = 0; i < nb; ++i) idx[i] = i;
        return nb;
    }
    int lo = sink_blocks, hi = nb - local_blocks; /* candidate range [lo, hi) */
    int k = budget_blocks - sink_blocks - local_blocks;
    char *keep = (char *)calloc((size_t)nb, 1);
    for (int i = 0; i < lo; ++i) keep[i] = 1;
    for (int i = hi; i < nb; ++i) keep[i] = 1;
    /* a candidate is retained iff fewer than k candidates rank ahead of it */
    for (int i = lo; i < hi; ++i) {
        int ahead = 0;
        for (int j = lo; j < hi; ++j)
            if (j != i && ranks_before(scores[j], j, scores[i], i)) ++ahead;
        if (ahead < k) keep[i] = 1;
    }
    int n = 0;
    for (int i = 0; i < nb; ++i)
        if (keep[i]) idx[n++] = i;
    free(keep);
    return n;
}

/* ------------------------------------------------------------------------------------------
 * Gather (Section 3.2, last paragraph): the partial cache is the selected blocks laid out
 * contiguously in token order, per KV head (each head has its own index list).  The partial
 * pool has the same page layout as the full pool; sequence `b` owns pages
 * [first_page, first_page + pages_per_seq).  Returns the partial length in tokens:
 * full blocks * bs, with the last selected block keeping only its valid tokens.
 * idx : [Hkv][budget_blocks] (first `count` entries valid).
 * ------------------------------------------------------------------------------------------ */
ORACLE_API int oracle_gather(const void *k_pool, const void *v_pool, int dtype, int Hkv, int bs, int d,
                             const int32_t *block_table, int seq_len,
                             const int32_t *idx, int idx_stride, int count,
                             void *pk_pool, void *pv_pool, int first_page) {
    int nb = (seq_len + bs - 1) / bs;
    int partial_len = 0;
    for (int h = 0; h < Hkv; ++h) {
        int len = 0;
        for (int s = 0; s < count; ++s) {
            int blk = idx[(size_t)h * idx_stride + s];
            int n_valid = blk == nb - 1 ? seq_len - blk * bs : bs;
            int64_t src = (((int64_t)block_table[blk]) * Hkv + h) * bs * d;
            int64_t dst = (((int64_t)first_page + s) * Hkv + h) * bs * d;
            copy_elems(pk_pool, dst, k_pool, src, (int64_t)n_valid * d, dtype);
            copy_elems(pv_pool, dst, v_pool, src, (int64_t)n_valid * d, dtype);
            len += n_valid;
        }
        partial_len = len;
    }
    return partial_len;
}

/* ------------------------------------------------------------------------------------------
 * Tree-masked GQA attention of the step's M query tokens (Algorithm 1 "TreeDecode"; attention
 * semantics of Section 4.1 "Implementations").  Row (j, n), KV head h = n / G:
 *   visible keys = the seq_len cached tokens (all precede every query) U {new token a : mask[j] bit a}
 *   out = sum_k softmax_k(q.k * scale) v_k ,   lse = log sum_k exp(q.k * scale)
 * Masked keys are skipped, so they contribute exactly zero.
 * out : [M][Hq][d] double, lse : [M][Hq] double.
 * If probs != NULL it receives the softmax weights, [M][Hq][seq_len + M] (0 for masked keys).
 * ------------------------------------------------------------------------------------------ */
ORACLE_API void oracle_tree_attention(const void *q, const void *knew, const void *vnew, int dtype,
                                      int M, int Hq, int Hkv, int d, const uint64_t *mask,
                                      const void *k_pool, const void *v_pool, int bs,
                                      const int32_t *block_table, int seq_len, double scale,
                                      double *out, double *lse, double *probs) {
    int G = Hq / Hkv;
    int W = (M + 63) / 64;
    int n_keys = seq_len + M;
#pragma omp parallel
    {
        double *logit = (double *)malloc((size_t)n_keys * sizeof(double));
        char *vis = (char *)malloc((size_t)n_keys);
        double *qrow = (double *)malloc((size_t)d * sizeof(double));
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int n = 0; n < Hq; ++n)
            for (int j = 0; j < M; ++j) {
                int h = n / G;
                for (int c = 0; c < d; ++c) qrow[c] = load_elem(q, dtype, ((int64_t)j * Hq + n) * d + c);
                /* logits of visible keys */
                double mx = -INFINITY;
                for (int t = 0; t < n_keys; ++t) {
                    int64_t koff;
                    const void *kb;
                    if (t < seq_len) {
                        vis[t] = 1;
                        kb = k_pool;
                        koff = ((((int64_t)block_table[t / bs]) * Hkv + h) * bs + t % bs) * d;
                    } else {
                        int a = t - seq_len;
                        vis[t] = (char)((mask[(size_t)j * W + a / 64] >> (a % 64)) & 1);
                        kb = knew;
                        koff = ((int64_t)a * Hkv + h) * d;
                    }
                    if (!vis[t]) continue;
                    double s = 0.0;
                    for (int c = 0; c < d; ++c) s += qrow[c] * load_elem(kb, dtype, koff + c);
                    s *= scale;
                    logit[t] = s;
                    if (s > mx) mx = s;
                }
                double denom = 0.0;
                for (int t = 0; t < n_keys; ++t)
                    if (vis[t]) denom += exp(logit[t] - mx);
                double *o = out + ((size_t)j * Hq + n) * d;
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                for (int t = 0; t < n_keys; ++t) {
                    double p = vis[t] ? exp(logit[t] - mx) / denom : 0.0;
                    if (probs) probs[((size_t)j * Hq + n) * n_keys + t] = p;
                    if (!vis[t]) continue;
                    int64_t voff;
                    const void *vb;
                    if (t < seq_len) {
                        vb = v_pool;
                        voff = ((((int64_t)block_table[t / bs]) * Hkv + h) * bs + t % bs) * d;
                    } else {
                        vb = vnew;
                        voff = ((int64_t)(t - seq_len) * Hkv + h) * d;
                    }
                    for (int c = 0; c < d; ++c) o[c] += p * load_elem(vb, dtype, voff + c);
                }
                lse[(size_t)j * Hq + n] = mx + log(denom);
            }
        free(logit);
        free(vis);
        free(qrow);
    }
}

/* ------------------------------------------------------------------------------------------
 * Commit (Section 3.2 buffer paragraph; Section 3.3): append the K/V rows `accepted[0..n)` of
 * the step (indices into Knew/Vnew) to the cache of one sequence at token positions
 * seq_len, seq_len+1, ...  Returns the new length.
 * ------------------------------------------------------------------------------------------ */
ORACLE_API int oracle_commit(const void *knew, const void *vnew, int dtype, int Hkv, int bs, int d,
                             const int32_t *accepted, int n_accepted,
                             void *k_pool, void *v_pool, const int32_t *block_table, int seq_len) {
    for (int a = 0; a < n_accepted; ++a) {
        int t = seq_len + a;
        for (int h = 0; h < Hkv; ++h) {
            int64_t src = ((int64_t)accepted[a] * Hkv + h) * d;
            int64_t dst = ((((int64_t)block_table[t / bs]) * Hkv + h) * bs + t % bs) * d;
            copy_elems(k_pool, dst, knew, src, d, dtype);
            copy_elems(v_pool, dst, vnew, src, d, dtype);
        }
    }
    return seq_len + n_accepted;
}

/* ------------------------------------------------------------------------------------------
 * Mode rule (Section 3.3, third paragraph; Algorithm 1 "SelectMode").
 * 0 = Full, 1 = Partial, 2 = Refresh.
 * ------------------------------------------------------------------------------------------ */
ORACLE_API int oracle_select_mode(int ctx_len, int budget_tokens, int n_partially_verified,
                                  int n_candidates, int buffer_tokens, int partial_initialised) {
    if (ctx_len < budget_tokens) return 0;
    if (!partial_initialised) return 2;
    if (n_partially_verified + n_candidates > buffer_tokens) return 2;
    return 1;
}

/* ==========================================================================================
 * The linear maps either side of the verification attention (Algorithm 1 "TreeDecode";
 * Section 3.3: the refresh pass computes key-value states for the partially verified and the
 * candidate tokens).  The paper names the step and leaves its arithmetic to the target model;
 * the readings taken here are those of the LLaMA / Qwen attention block:
 *   q = x Wq^T, k = x Wk^T, v = x Wv^T  (weights stored [out feature][in feature]),
 *   rotary position embedding on q and k with the half-split pairing: channel c < d/2 is
 *   paired with channel c + d/2, angle = position * theta^(-2c/d),
 *       out[c]       = in[c] cos - in[c + d/2] sin
 *       out[c + d/2] = in[c + d/2] cos + in[c] sin,
 *   position of a step token = tokens before the step + its depth in the step (a chain token's
 *   depth is its index, a tree node's depth counts from the end of the chain),
 *   o = attn Wo^T (+ residual).
 * These readings have no pin in the paper ("parity unpinned" by it); the tests pin them to
 * closed forms and to the properties that define a rotary embedding.
 * ========================================================================================== */

/* Positions of the step's rows: chain rows base, base+1, ...; tree node i at base + n_chain + depth(i). */
ORACLE_API int oracle_step_positions(const int32_t *parents, int n_tree, int n_chain, int base, int32_t *pos) {
    for (int r = 0; r < n_chain; ++r) pos[r] = base + r;
    for (int i = 0; i < n_tree; ++i) {
        int p = parents[i];
        if (i == 0 ? p != -1 : (p < 0 || p >= i)) return -1;
        int depth = 0;
        for (int a = i; parents[a] >= 0; a = parents[a]) ++depth;
        pos[n_chain + i] = base + n_chain + depth;
    }
    return 0;
}

/* y[t][f] = sum_c x[t][c] * w[f][c] (+ residual[t][f]);  x [T][n_in], w [n_out][n_in], y [T][n_out] double. */
ORACLE_API void oracle_linear(const void *x, const void *w, int dtype, int T, int n_in, int n_out,
                              const void *residual, double *y) {
#pragma omp parallel for schedule(static)
    for (int f = 0; f < n_out; ++f)
        for (int t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int c = 0; c < n_in; ++c)
                acc += load_elem(x, dtype, (int64_t)t * n_in + c) * load_elem(w, dtype, (int64_t)f * n_in + c);
            if (residual) acc += load_elem(residual, dtype, (int64_t)t * n_out + f);
            y[(int64_t)t * n_out + f] = acc;
        }
}

/* Rotary embedding in place on rows [T][H][d] of doubles, row t at position pos[t]. */
ORACLE_API void oracle_rope(double *a, int T, int H, int d, const int32_t *pos, double theta) {
    int half = d / 2;
    for (int t = 0; t < T; ++t)
        for (int h = 0; h < H; ++h) {
            double *v = a + ((int64_t)t * H + h) * d;
            for (int c = 0; c < half; ++c) {
                double angle = (double)pos[t] * pow(theta, -2.0 * (double)c / (double)d);
                double cs = cos(angle), sn = sin(angle);
                double lo = v[c], hi = v[c + half];
                v[c] = lo * cs - hi * sn;
                v[c + half] = hi * cs + lo * sn;
            }
        }
}

/* x [T][hidden], w_qkv [(Hq + 2 Hkv) d][hidden] (q heads, then k heads, then v heads) ->
 * q [T][Hq][d], k [T][Hkv][d] with the rotary embedding, v [T][Hkv][d] without. */
ORACLE_API void oracle_qkv_rope(const void *x, const void *w_qkv, int dtype, int T, int hidden, int Hq, int Hkv,
                                int d, const int32_t *pos, double theta, double *q, double *k, double *v) {
    size_t es = dtype == 0 ? 4 : 2;
    const char *w = (const char *)w_qkv;
    oracle_linear(x, w, dtype, T, hidden, Hq * d, NULL, q);
    oracle_linear(x, w + (size_t)Hq * d * hidden * es, dtype, T, hidden, Hkv * d, NULL, k);
    oracle_linear(x, w + (size_t)(Hq + Hkv) * d * hidden * es, dtype, T, hidden, Hkv * d, NULL, v);
    oracle_rope(q, T, Hq, d, pos, theta);
    oracle_rope(k, T, Hkv, d, pos, theta);
}
