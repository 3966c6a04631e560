/*
 * specpv.h -- C ABI of the SpecPV verification hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA kernels, the verification attention of SpecPV
 * (arXiv 2512.02337): tree-masked grouped-query attention of a step's draft-token tree against a
 * paged long-context KV cache, either over a small PARTIAL cache (sink blocks + top-scored
 * retrieval blocks + local window + buffer; paper Section 3.2) or over the FULL cache with a
 * refresh that rebuilds the partial cache (Section 3.3).  Call names follow Algorithm 1 and the
 * section titles of the paper.
 *
 * Conventions that hold for every call unless stated otherwise
 *   - "device" pointers are CUDA device memory owned by the caller; the library never allocates,
 *     frees or keeps them.  "host" pointers are ordinary process memory.
 *   - Calls that launch work take a `stream` (a cudaStream_t passed as void*; NULL = the legacy
 *     default stream), enqueue on it and return without synchronising.
 *   - Return value: SPECPV_OK or an error found by host-side validation; nothing is launched on
 *     error.  Faults only the device can see (a page id outside the pool, a cache that would
 *     overflow, a bounded wait that gave up) are recorded in a status word at the head of the
 *     `workspace`; the offending work item is skipped and the status is read by
 *     specpv_poll_status().  No kernel traps or spins without a limit.
 *   - dtype 0 = float32, 1 = bfloat16 for Q, K, V, the caches, the summaries and the output
 *     (the output is float32 instead when cfg->out_f32 is set); accumulation is float32; scores
 *     and log-sum-exp are float32.
 *   - Every device pointer must be 16-byte aligned; pools should be 128-byte aligned.
 *
 * Tensor layouts (row-major, innermost last)
 *   K/V pool      [n_layers][n_pages][Hkv][bs][d]     a "page" holds bs tokens of all KV heads
 *   block_table   [batch][max_blocks] int32           logical block of a sequence -> page id
 *   seq_lens      [batch] int32                       tokens held by the cache for each sequence
 *   Q, O          [n_layers_in_call][batch][M_max][Hq][d]
 *   Knew, Vnew    [n_layers_in_call][batch][M_max][Hkv][d]   keys/values of the step's own tokens
 *   tree_mask     [batch][M_max][W] uint64, W = ceil(M_max/64); bit a of row j: token j sees token a
 *   q_lens        [batch] int32   rows actually used per sequence (<= M_max); NULL = M_max for all
 *                 M_max (chain + tree of a step) is at most 128: a larger value makes the verify calls
 *                 return SPECPV_ERR_CAPACITY
 *   LSE           [n_layers_in_call][batch][M_max][Hq] float32 (natural log)
 *   summaries     kmax, kmin [n_layers][batch][Hkv][max_blocks][d]   (indexed by LOGICAL block)
 *   scores        [n_layers_in_call][batch][Hkv][max_blocks] float32
 *   idx           [n_layers_in_call][batch][Hkv][budget_blocks] int32, count [batch] int32
 * A partial cache is an ordinary specpv_paged_kv with its own pools, table and lengths; sequence
 * b's partial segment is the first partial_lens[b] tokens reached through its table.
 */
#ifndef SPECPV_H
#define SPECPV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SPECPV_OK = 0,
    SPECPV_ERR_INVALID_ARG = 1,     /* null pointer, misaligned pointer, negative size */
    SPECPV_ERR_SHAPE = 2,           /* head counts / head_dim / block size outside what is built */
    SPECPV_ERR_BUDGET = 3,          /* budget_blocks < sink_blocks + local_blocks + 1 */
    SPECPV_ERR_CAPACITY = 4,        /* a cache, the workspace or M_max too small for the request */
    SPECPV_ERR_BAD_TREE = 5,        /* parents[] is not a tree in topological order */
    SPECPV_ERR_BAD_BLOCK_TABLE = 6, /* a page id outside [0, n_pages) (device-detected) */
    SPECPV_ERR_UNSUPPORTED = 7,     /* valid request the kernels do not cover */
    SPECPV_ERR_CUDA = 8,            /* a CUDA runtime call failed */
    SPECPV_ERR_TIMEOUT = 9          /* a bounded device-side wait gave up (device-detected) */
} specpv_status;

enum { SPECPV_DTYPE_F32 = 0, SPECPV_DTYPE_BF16 = 1 };
enum { SPECPV_REDUCE_MEAN = 0, SPECPV_REDUCE_MAX = 1, SPECPV_REDUCE_LAST = 2 };
enum { SPECPV_MODE_FULL = 0, SPECPV_MODE_PARTIAL = 1, SPECPV_MODE_REFRESH = 2 };

/* Geometry and the method's hyper-parameters (paper Appendix "Generation Settings": block 16,
 * sink 32 tokens, local 128 tokens, buffer 20 + one step's tokens, reduction = mean). */
typedef struct {
    int32_t n_layers;      /* layers held by the pools */
    int32_t n_q_heads;     /* Hq */
    int32_t n_kv_heads;    /* Hkv; Hq % Hkv == 0, G = Hq / Hkv */
    int32_t head_dim;      /* d: 64 or 128 */
    int32_t block_tokens;  /* bs: tokens per page (16, 32 or 64) */
    int32_t dtype;         /* SPECPV_DTYPE_* */
    int32_t sink_blocks;   /* always-kept leading blocks (Section 3.2, "sink tokens") */
    int32_t local_blocks;  /* always-kept trailing blocks (Section 3.2, "local tokens") */
    int32_t budget_blocks; /* sink + retrieval + local blocks of the partial cache */
    int32_t buffer_tokens; /* extra room after the budget for partially verified + candidate tokens */
    int32_t reduce;        /* SPECPV_REDUCE_*: the f of Eq. 3 */
    int32_t score_mode;    /* 0 = Eq. 2 as printed (max of the two full dot products); 1 = the channel-wise
                              form sum_c max(q_c Kmax_c, q_c Kmin_c) of the method Section 3.2 cites */
    float softmax_scale;   /* 0 => 1/sqrt(head_dim) */
    int32_t out_f32;       /* 1 => the attention output O is written as float32 whatever dtype is
                              (the accumulator before the final rounding); 0 => O has type dtype */
    int32_t select_shared; /* 1 => one block set per (layer, sequence): every KV head keeps the blocks ranked on the
                              mean of the heads' scores (the paper does not say whether heads select separately);
                              0 => each KV head selects on its own scores */
} specpv_config;

typedef struct {
    void *k_pool;               /* device, [n_layers][n_pages][Hkv][bs][d] */
    void *v_pool;               /* device, same shape */
    const int32_t *block_table; /* device, [batch][max_blocks] */
    const int32_t *seq_lens;    /* device, [batch] */
    int32_t batch;
    int32_t max_blocks;
    int32_t n_pages;
    int32_t max_seq_len; /* host-known upper bound of seq_lens[], used only to size grids */
} specpv_paged_kv;

/* Human-readable name of a status code (static string, never NULL). */
const char *specpv_status_string(specpv_status s);

/* Bytes of device workspace that any call below needs for the given limits.  The first
 * SPECPV_WORKSPACE_HEAD_BYTES hold the device status word and the arrival counters of KV ranges that
 * several CTAs share; the caller zeroes them once (cudaMemset) before first use and the library
 * leaves them zero after every call that completes (after SPECPV_ERR_TIMEOUT zero them again).  The
 * rest is scratch (split-KV partial results, host-call staging) with no state between calls. */
#define SPECPV_WORKSPACE_HEAD_BYTES (256u << 10)
size_t specpv_workspace_bytes(const specpv_config *cfg, int n_layers_per_call, int max_batch,
                              int max_seq_len, int M_max);

/* Number of kernels this library has launched in this process so far (all streams, monotonic). */
uint64_t specpv_kernel_launches(void);

/* Synchronises `stream`, returns the device-recorded status (SPECPV_OK if none) and clears it.
 * info[0..3] (host, nullable) receive kernel-specific details of the first fault. */
specpv_status specpv_poll_status(void *workspace, void *stream, int32_t *info);

/* Section 3.3 / Algorithm 1 "TreeDecode": ancestor-or-self mask of the step's tokens.
 * parents (host, [n_tree]): tree-relative parent of each node, parents[0] = -1, parents[i] < i.
 * n_chain: partially verified tokens placed in front of the tree in a refresh (0 otherwise); they
 * form a chain and the tree root hangs off the chain's last token.
 * mask (host, [n_chain + n_tree][row_words] uint64, row_words >= ceil(M/64)) is fully overwritten. */
specpv_status specpv_build_tree_mask(const int32_t *parents, int n_tree, int n_chain,
                                     uint64_t *mask, int row_words);

/* Section 3.3 third paragraph / Algorithm 1 "SelectMode": SPECPV_MODE_FULL while the context is
 * shorter than the budget; one REFRESH to initialise the partial cache; PARTIAL afterwards; REFRESH
 * again when partially verified + candidate tokens exceed the buffer.  Pure host function. */
int specpv_select_mode(int ctx_len, int budget_tokens, int n_partially_verified, int n_candidates,
                       int buffer_tokens, int partial_initialised);

/* Eq. 1: (re)compute Kmax/Kmin of the blocks that hold tokens >= tok_begin[b] (device [batch];
 * NULL = from token 0) for layers [layer0, layer0 + n_layers).  max_blocks_touched bounds how many
 * trailing blocks per sequence can change (grid size); pass kv->max_blocks for a full rebuild.
 * Only the valid tokens of a ragged last block enter the max/min. */
specpv_status specpv_update_block_summaries(const specpv_config *cfg, int layer0, int n_layers,
                                            const specpv_paged_kv *kv, const int32_t *tok_begin,
                                            int max_blocks_touched, void *kmax, void *kmin,
                                            void *workspace, size_t workspace_bytes, void *stream);

/* Eq. 2-3: scores[l][b][h][i] = f_j max(q_j . Kmax_i, q_j . Kmin_i) over the step's query rows of
 * KV head h's group (all G heads x q_lens[b] tokens; for SPECPV_REDUCE_LAST the G heads of row
 * last_query[b] (device [batch], NULL = row 0)).  With cfg->score_mode = 1 the maximum is taken per channel
 * before the sum (an upper bound of q . k over the block's keys).  Blocks >= ceil(seq_len/bs) are left
 * untouched. */
specpv_status specpv_score_blocks(const specpv_config *cfg, int layer0, int n_layers, const void *q,
                                  const int32_t *q_lens, int M_max, const int32_t *last_query,
                                  const void *kmax, const void *kmin, const specpv_paged_kv *kv,
                                  float *scores, void *workspace, size_t workspace_bytes, void *stream);

/* Section 3.2: the retained block set of every (layer, sequence, KV head): sink blocks, the
 * budget - sink - local best-scored blocks of [sink, nb - local), and the local blocks, written
 * ascending to idx; count[b] = min(nb, budget_blocks).  Ties go to the lower block index, NaN
 * ranks last; the result is a pure function of the float32 scores (bit-exact, deterministic).  With
 * cfg->select_shared the ranking uses the float32 mean over the KV heads (summed in head order) and all
 * heads of a layer receive the same list. */
specpv_status specpv_select_partial_kv(const specpv_config *cfg, int n_layers, const float *scores,
                                       const int32_t *seq_lens, int batch, int max_blocks,
                                       int32_t *idx, int32_t *count, void *workspace,
                                       size_t workspace_bytes, void *stream);

/* Section 3.3 ("refresh the partial KV cache"): copy the selected blocks of every layer and KV
 * head from the full cache into the partial cache in ascending token order and set
 * partial_lens[b] = (count[b]-1)*bs + valid tokens of the last block; the buffer starts empty. */
specpv_status specpv_refresh_partial(const specpv_config *cfg, const specpv_paged_kv *full,
                                     const int32_t *idx, const int32_t *count,
                                     const specpv_paged_kv *partial, int32_t *partial_lens,
                                     void *workspace, size_t workspace_bytes, void *stream);

/* Section 3.2 / Algorithm 1 "TreeDecode" with KV_in = KV_partial: tree-masked GQA attention of
 * the step's tokens over the partial segment (sink | retrieval | local | buffer) followed by the
 * step's own keys under the tree mask.  out (and lse if not NULL) are fully written for rows
 * < q_lens[b].
 * Two tensor-core kernels serve bfloat16 / head_dim 128: by default one CTA per KV range; with the
 * environment variable SPECPV_ATTN_KERNEL=pair (read at every call) shapes with more than 128 query
 * rows per KV head (M_max * Hq / Hkv) run on a kernel that gives a pair of SMs the two halves of
 * those rows.  The results agree within the tolerance of either; the default is the faster one when
 * steps follow one another (see the comment at attention_pair_wanted). */
specpv_status specpv_verify_partial(const specpv_config *cfg, int layer0, int n_layers, const void *q,
                                    const void *k_new, const void *v_new, const uint64_t *tree_mask,
                                    const int32_t *q_lens, int M_max, const specpv_paged_kv *partial,
                                    void *out, float *lse, void *workspace, size_t workspace_bytes,
                                    void *stream);

/* Section 3.3 / Algorithm 1 "TreeDecode" with KV_in = KV_full: the same attention over the whole
 * cache through the block table.  In a refresh the rows are the partially verified chain followed
 * by the tree (see specpv_build_tree_mask). */
specpv_status specpv_verify_full(const specpv_config *cfg, int layer0, int n_layers, const void *q,
                                 const void *k_new, const void *v_new, const uint64_t *tree_mask,
                                 const int32_t *q_lens, int M_max, const specpv_paged_kv *full,
                                 void *out, float *lse, void *workspace, size_t workspace_bytes,
                                 void *stream);

/* (No counterpart in the paper: an allocation-free variant of specpv_verify_partial.)
 *
 * Some callers cannot give this library a workspace because they cannot allocate device memory at
 * the point where they call it: an inference server that handed all of the GPU's memory to its own
 * KV-cache pool at start-up, a plug-in that runs inside such a server's decode loop where a
 * cudaMalloc would stall every stream of the device (or simply fail because nothing is left), or a
 * process whose allocator is owned by another component.  For them this call keeps its split-KV
 * scratch and its status word in a fixed array of SPECPV_STATIC_SCRATCH_BYTES that is part of the
 * library image: every GPU on which the library is used holds that array from the first use until
 * the process exits, whether or not this call is ever made again.  The call itself performs no
 * cudaMalloc / cudaFree and calls no allocating routine; q, k_new, v_new, tree_mask, the partial
 * cache, out and lse are still the caller's device buffers, with the meaning they have in
 * specpv_verify_partial.
 *
 * Limit: n_layers * batch * Hkv * ceil(M_max * G / 256) * 256 * (head_dim + 2) * 4 bytes (one
 * KV split's partial results) must fit twice into SPECPV_STATIC_SCRATCH_BYTES -
 * SPECPV_WORKSPACE_HEAD_BYTES; a larger
 * request returns SPECPV_ERR_CAPACITY and launches nothing.  Within the limit the scratch only
 * bounds how many KV splits are used, never the result.
 *
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.  Every call uses the same array: two calls
 * whose kernels can overlap on the GPU (different streams without an ordering between them) race
 * on it; calls on one stream, or ordered by events, are safe.  The array keeps the previous
 * call's partial results; its head (status word, arrival counters) starts at zero because the array
 * is zero-initialised with the library image, the counters are back at zero when a call completes,
 * and the status word is cleared on `stream` before launching.  device_status (device, 5 x int32, nullable) receives
 * a copy of the status word at the end of the call's work on `stream`: word 0 is the first
 * device-detected specpv_status of this call (0 = none), words 1..4 its details. */
#define SPECPV_STATIC_SCRATCH_BYTES (16u << 20)
specpv_status specpv_verify_partial_static(const specpv_config *cfg, int layer0, int n_layers,
                                           const void *q, const void *k_new, const void *v_new,
                                           const uint64_t *tree_mask, const int32_t *q_lens, int M_max,
                                           const specpv_paged_kv *partial, void *out, float *lse,
                                           int32_t *device_status, void *stream);

/* The same step with HOST step tensors (q, k_new, v_new, tree_mask, out, lse are host pointers,
 * ideally pinned): copies the inputs to staging space inside the workspace, runs the attention
 * (mode = SPECPV_MODE_PARTIAL or SPECPV_MODE_FULL selects only validation), copies out/lse back and
 * synchronises the stream before returning.  The KV cache stays device-resident state.  The layers go
 * through in up to eight groups so that one group's attention overlaps the next group's input copy and
 * the previous group's output copy; the two copy streams this needs are created on the first call on
 * each device and kept until the process exits. */
specpv_status specpv_verify_host(const specpv_config *cfg, int mode, int layer0, int n_layers,
                                 const void *q_host, const void *k_new_host, const void *v_new_host,
                                 const uint64_t *tree_mask_host, int M_max, const specpv_paged_kv *kv,
                                 void *out_host, float *lse_host, void *workspace,
                                 size_t workspace_bytes, void *stream);

/* Section 3.2 (buffer) / Section 3.3 (removing invalid tokens): append rows accepted[b][0..n) of
 * Knew/Vnew (device int32 [batch][A_max], n = n_accepted[b] device [batch]) to cache `dst` at token
 * positions seq_lens[b].., then seq_lens[b] += n (seq_lens is dst->seq_lens, written in place).
 * Layers may be committed in groups (layer0, n_layers), in ascending order: every group writes its
 * rows at the lengths as they stand, and the lengths advance with the group that contains the
 * model's last layer (layer0 + n_layers == cfg->n_layers), so a step's commit must end with that
 * group and include every layer exactly once.
 * Rejected candidates are simply never appended.  If kmax/kmin are not NULL the summaries of the
 * touched blocks are recomputed.  A sequence whose cache would overflow is skipped and
 * SPECPV_ERR_CAPACITY recorded in the status word. */
specpv_status specpv_commit_accepted(const specpv_config *cfg, int layer0, int n_layers,
                                     const void *k_new, const void *v_new, int M_max,
                                     const int32_t *accepted, const int32_t *n_accepted, int A_max,
                                     const specpv_paged_kv *dst, void *kmax, void *kmin,
                                     void *workspace, size_t workspace_bytes, void *stream);

/* ---- The linear maps either side of the verification attention -------------------------------
 * Algorithm 1 "TreeDecode" runs the target model's attention block on the step's tokens, and
 * Section 3.3 has the refresh pass compute the key-value states of the partially verified and the
 * candidate tokens.  The paper leaves the block's arithmetic to the target model; these calls
 * implement the LLaMA / Qwen form: q = x Wq^T, k = x Wk^T, v = x Wv^T with weights stored
 * [out feature][in feature], a rotary position embedding on q and k that pairs channel c < d/2
 * with channel c + d/2 (angle = position * theta^(-2c/d)), and o = attn Wo^T (+ residual).
 * Their outputs are exactly the q / k_new / v_new inputs of the verify calls, and the attention
 * output (cfg->out_f32 = 0) is the `attn` input of specpv_o_proj.
 *
 *   x, attn, residual, y   [n_layers_in_call][batch][M_max][features]   of cfg->dtype
 *   w_qkv                  [n_layers][(Hq + 2 Hkv) d][hidden]           q heads, then k heads, then v heads
 *   w_o                    [n_layers][hidden][Hq d]
 *   cos_sin                [batch][M_max][d/2][2] float32               (cos, sin) of every row's angles
 * hidden must be a multiple of 16.  bfloat16 with d = 128 and hidden, Hq d multiples of 64 (128 for
 * the output side of specpv_o_proj) runs on the tensor cores, everything else on a plain kernel.
 * Rows >= q_lens[b] are computed like any other row (from whatever x holds there); the caller
 * ignores them. */

/* Positions and angles of a step's rows: row j of sequence b sits at base_pos[b] + depth(j), where
 * depth(j) = (number of step tokens row j sees under the ancestor-or-self mask) - 1, so that the
 * partially verified chain of a refresh counts on from base_pos[b] and the tree from the chain's end.
 * base_pos (device [batch]) = tokens of the sequence in front of the step (full-cache length in a full
 * or refresh step, full-cache length + partially verified tokens in a partial step).  The angles are
 * formed in double precision and rounded once to float32.  One table serves every layer of the step. */
specpv_status specpv_rope_table(const specpv_config *cfg, const uint64_t *tree_mask, const int32_t *q_lens,
                                const int32_t *base_pos, int batch, int M_max, double rope_theta,
                                float *cos_sin, void *stream);

/* q, k_new (rotated) and v_new (not rotated) of the step's tokens for layers [layer0, layer0 + n_layers)
 * of w_qkv; x, q, k_new, v_new are indexed by layer-in-call.  Needs no more workspace than the verify
 * calls (specpv_workspace_bytes); a smaller workspace only costs speed. */
specpv_status specpv_qkv_rope(const specpv_config *cfg, int layer0, int n_layers, const void *x, int hidden,
                              const void *w_qkv, const float *cos_sin, int batch, int M_max, void *q,
                              void *k_new, void *v_new, void *workspace, size_t workspace_bytes, void *stream);

/* y = attn Wo^T (+ residual if not NULL) for the same rows; attn is the attention output
 * [..][Hq][d] read as [..][Hq d]. */
specpv_status specpv_o_proj(const specpv_config *cfg, int layer0, int n_layers, const void *attn,
                            const void *w_o, int hidden, const void *residual, int batch, int M_max, void *y,
                            void *workspace, size_t workspace_bytes, void *stream);

/* ---- Full KV cache in host memory ---------------------------------------------------------------
 * Section 3.3, last paragraph: when device memory is short only the FULL cache is offloaded to host
 * memory (the partial cache stays resident); a full verification keeps one layer's keys and values
 * on the device at a time and prefetches the next layer.
 *
 * k_host / v_host are page-locked host memory that the device can address (cudaHostAlloc or
 * cudaHostRegister with the mapped flag; under unified addressing the same pointer serves both
 * sides), laid out like a K/V pool.  k_stage / v_stage are two layer slots of device memory.
 * Every other call of this header that takes a specpv_paged_kv also accepts such host pointers as
 * k_pool / v_pool and then reads or writes the cache over the bus in place: that is how
 * specpv_commit_accepted appends the accepted rows to an offloaded cache and how
 * specpv_refresh_partial fetches only the selected blocks (a few percent of the cache) instead of
 * whole layers.  The summaries (Eq. 1) stay device-resident. */
typedef struct {
    const void *k_host;         /* host (device-addressable), [n_layers][n_pages][Hkv][bs][d] */
    const void *v_host;
    void *k_stage;              /* device, [2][n_pages][Hkv][bs][d] */
    void *v_stage;
    const int32_t *block_table; /* device, [batch][max_blocks] */
    const int32_t *seq_lens;    /* device, [batch] */
    int32_t batch;
    int32_t max_blocks;
    int32_t n_pages;
    int32_t max_seq_len;
} specpv_offloaded_kv;

/* specpv_verify_full over an offloaded cache: for each layer of [layer0, layer0 + n_layers) the layer's
 * K and V pools are copied host -> device into one of the two slots on `copy_stream` while the attention
 * of the previous layer runs from the other slot on `stream`.  On return everything is ordered on
 * `stream` (later work on `stream` sees out / lse; the slots may be reused by a later call on it).
 * copy_stream must not be a stream that waits on `stream`'s later work; pass a stream of its own
 * (the same stream is accepted and runs the copies and the attention one after the other).  The call
 * creates and destroys four CUDA events; it allocates no device memory. */
specpv_status specpv_verify_full_offloaded(const specpv_config *cfg, int layer0, int n_layers, const void *q,
                                           const void *k_new, const void *v_new, const uint64_t *tree_mask,
                                           const int32_t *q_lens, int M_max, const specpv_offloaded_kv *full,
                                           void *out, float *lse, void *workspace, size_t workspace_bytes,
                                           void *stream, void *copy_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECPV_H */
