// C-ABI entry points of the SpecPV library: host-side validation and kernel dispatch.
// The operations follow the paper's Section 3.2 (partial verification), Section 3.3 (full
// verification with refresh) and Algorithm 1; see include/specpv.h for the contract of each call.
#include <math.h>
#include <string.h>

#include "aux_kernels.cuh"
#include "common.cuh"
#include "proj.cuh"

#define SPECPV_EXPORT extern "C" __attribute__((visibility("default")))

#include <atomic>
#include <mutex>

namespace specpv {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

specpv_status validate_config(const specpv_config* cfg, Geometry* g) {
    if (!cfg) return SPECPV_ERR_INVALID_ARG;
    if (cfg->n_layers <= 0 || cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0) return SPECPV_ERR_SHAPE;
    if (cfg->n_q_heads % cfg->n_kv_heads != 0) return SPECPV_ERR_SHAPE;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return SPECPV_ERR_SHAPE;
    if (cfg->block_tokens != 16 && cfg->block_tokens != 32 && cfg->block_tokens != 64) return SPECPV_ERR_SHAPE;
    if (cfg->dtype != SPECPV_DTYPE_F32 && cfg->dtype != SPECPV_DTYPE_BF16) return SPECPV_ERR_SHAPE;
    if (cfg->sink_blocks < 0 || cfg->local_blocks < 1 || cfg->buffer_tokens < 0) return SPECPV_ERR_BUDGET;
    if (cfg->budget_blocks < cfg->sink_blocks + cfg->local_blocks + 1) return SPECPV_ERR_BUDGET;
    if (cfg->reduce < 0 || cfg->reduce > 2) return SPECPV_ERR_INVALID_ARG;
    if (cfg->score_mode != 0 && cfg->score_mode != 1) return SPECPV_ERR_UNSUPPORTED;
    if (cfg->out_f32 != 0 && cfg->out_f32 != 1) return SPECPV_ERR_INVALID_ARG;
    if (cfg->select_shared != 0 && cfg->select_shared != 1) return SPECPV_ERR_INVALID_ARG;
    if (!(cfg->softmax_scale >= 0.f) || isinf(cfg->softmax_scale)) return SPECPV_ERR_INVALID_ARG;
    g->n_layers = cfg->n_layers;
    g->Hq = cfg->n_q_heads;
    g->Hkv = cfg->n_kv_heads;
    g->G = g->Hq / g->Hkv;
    g->d = cfg->head_dim;
    g->bs = cfg->block_tokens;
    g->dtype = cfg->dtype;
    g->es = cfg->dtype == SPECPV_DTYPE_F32 ? 4 : 2;
    g->out_f32 = (cfg->out_f32 != 0 || cfg->dtype == SPECPV_DTYPE_F32) ? 1 : 0;
    g->out_es = g->out_f32 ? 4 : 2;
    g->sink_blocks = cfg->sink_blocks;
    g->local_blocks = cfg->local_blocks;
    g->budget_blocks = cfg->budget_blocks;
    g->buffer_tokens = cfg->buffer_tokens;
    g->reduce = cfg->reduce;
    g->score_mode = cfg->score_mode;
    g->select_shared = cfg->select_shared;
    g->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
    return SPECPV_OK;
}

specpv_status validate_kv(const Geometry& g, const specpv_paged_kv* kv) {
    (void)g;
    if (!kv || !kv->k_pool || !kv->v_pool || !kv->block_table || !kv->seq_lens) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(kv->k_pool) || !aligned16(kv->v_pool)) return SPECPV_ERR_INVALID_ARG;
    if (kv->batch <= 0 || kv->max_blocks <= 0 || kv->n_pages <= 0 || kv->max_seq_len < 0) return SPECPV_ERR_INVALID_ARG;
    if ((int64_t)kv->max_seq_len > (int64_t)kv->max_blocks * g.bs) return SPECPV_ERR_CAPACITY;
    return SPECPV_OK;
}

StagingPlan plan_staging(const Geometry& g, int n_layers_per_call, int batch, int M_max) {
    StagingPlan s{};
    const size_t rows = (size_t)n_layers_per_call * batch * M_max;
    size_t off = 0;
    s.q = off;      off += round_up(rows * g.Hq * g.d * g.es, 256);
    s.k_new = off;  off += round_up(rows * g.Hkv * g.d * g.es, 256);
    s.v_new = off;  off += round_up(rows * g.Hkv * g.d * g.es, 256);
    s.mask = off;   off += round_up((size_t)batch * M_max * ((M_max + 63) / 64) * sizeof(uint64_t), 256);
    s.out = off;    off += round_up(rows * g.Hq * g.d * g.out_es, 256);
    s.lse = off;    off += round_up(rows * g.Hq * sizeof(float), 256);
    s.total = off;
    return s;
}

WorkspacePlan plan_workspace(const Geometry& g, int n_layers_per_call, int max_batch, int M_max) {
    WorkspacePlan w{};
    const size_t base = (size_t)g.Hkv * n_layers_per_call * max_batch;
    const size_t R_pad = round_up((size_t)M_max * g.G, 256);
    w.counter_off = kStatusBytes;
    w.counter_bytes = kHeaderBytes - kStatusBytes;
    w.partial_off = kHeaderBytes;
    // room for kMaxSplitCtas + base split results of R_pad rows of (d + 2) floats
    w.partial_bytes = round_up((kMaxSplitCtas + base) * R_pad * (g.d + 2) * sizeof(float), 256);
    w.staging_off = w.partial_off + w.partial_bytes;
    w.staging_bytes = plan_staging(g, n_layers_per_call, max_batch, M_max).total;
    w.total = w.staging_off + w.staging_bytes;
    return w;
}

static specpv_status verify_common(const specpv_config* cfg, int layer0, int n_layers, const void* q,
                                   const void* k_new, const void* v_new, const uint64_t* tree_mask,
                                   const int32_t* q_lens, int M_max, const specpv_paged_kv* kv, void* out,
                                   float* lse, void* workspace, size_t workspace_bytes, void* stream,
                                   bool is_partial) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    st = validate_kv(g, kv);
    if (st != SPECPV_OK) return st;
    if (!q || !k_new || !v_new || !tree_mask || !out || !workspace) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out) || !aligned16(workspace))
        return SPECPV_ERR_INVALID_ARG;
    if (layer0 < 0 || n_layers <= 0 || layer0 + n_layers > g.n_layers) return SPECPV_ERR_INVALID_ARG;
    if (M_max <= 0) return SPECPV_ERR_INVALID_ARG;
    if (M_max > kMaxQTokens) return SPECPV_ERR_CAPACITY;
    if (is_partial) {
        // the partial cache must be able to hold the budget plus the buffer (Section 3.2)
        if ((int64_t)kv->max_blocks * g.bs < (int64_t)g.budget_blocks * g.bs + g.buffer_tokens) return SPECPV_ERR_CAPACITY;
    }
    WorkspacePlan w = plan_workspace(g, n_layers, kv->batch, M_max);
    if (workspace_bytes < w.partial_off + w.partial_bytes) return SPECPV_ERR_CAPACITY;

    AttnArgs a{};
    a.g = g;
    a.layer0 = layer0; a.n_layers = n_layers; a.batch = kv->batch; a.M_max = M_max;
    a.mask_words = (M_max + 63) / 64;
    a.q = q; a.k_new = k_new; a.v_new = v_new; a.tree_mask = tree_mask; a.q_lens = q_lens;
    a.k_pool = kv->k_pool; a.v_pool = kv->v_pool; a.block_table = kv->block_table; a.seq_lens = kv->seq_lens;
    a.max_blocks = kv->max_blocks; a.n_pages = kv->n_pages; a.max_seq_len = kv->max_seq_len;
    a.out = out; a.lse = lse; a.workspace = workspace;
    a.partial_off = w.partial_off;
    a.partial_bytes = workspace_bytes - w.partial_off < w.partial_bytes ? workspace_bytes - w.partial_off : w.partial_bytes;
    a.counter_off = w.counter_off;
    a.counter_bytes = w.counter_bytes;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (attention_tc_supported(a)) return launch_attention_tc(a, s);
    return launch_attention_simt(a, s);
}

// Two copy streams per device for specpv_verify_host, created on first use and kept for the life of the process.
struct HostCopyStreams {
    cudaStream_t in, out;
};
static HostCopyStreams* host_copy_streams() {
    static std::mutex mu;
    static HostCopyStreams per_device[64];
    static bool made[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!made[dev]) {
        if (cudaStreamCreateWithFlags(&per_device[dev].in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithFlags(&per_device[dev].out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        made[dev] = true;
    }
    return &per_device[dev];
}

}  // namespace specpv

using namespace specpv;

SPECPV_EXPORT const char* specpv_status_string(specpv_status s) {
    switch (s) {
        case SPECPV_OK: return "ok";
        case SPECPV_ERR_INVALID_ARG: return "invalid argument";
        case SPECPV_ERR_SHAPE: return "unsupported shape";
        case SPECPV_ERR_BUDGET: return "budget smaller than sink + local + 1 blocks";
        case SPECPV_ERR_CAPACITY: return "capacity exceeded";
        case SPECPV_ERR_BAD_TREE: return "parents[] is not a tree in topological order";
        case SPECPV_ERR_BAD_BLOCK_TABLE: return "page id outside the pool";
        case SPECPV_ERR_UNSUPPORTED: return "unsupported request";
        case SPECPV_ERR_CUDA: return "CUDA runtime error";
        case SPECPV_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

SPECPV_EXPORT uint64_t specpv_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

SPECPV_EXPORT size_t specpv_workspace_bytes(const specpv_config* cfg, int n_layers_per_call, int max_batch,
                                            int max_seq_len, int M_max) {
    Geometry g;
    (void)max_seq_len;
    if (validate_config(cfg, &g) != SPECPV_OK || n_layers_per_call <= 0 || max_batch <= 0 || M_max <= 0) return 0;
    return plan_workspace(g, n_layers_per_call, max_batch, M_max).total;
}

SPECPV_EXPORT specpv_status specpv_poll_status(void* workspace, void* stream, int32_t* info) {
    if (!workspace) return SPECPV_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    StatusWord sw;
    if (cudaMemcpyAsync(&sw, workspace, sizeof sw, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SPECPV_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return SPECPV_ERR_CUDA;
    if (sw.code != 0) {
        if (cudaMemsetAsync(workspace, 0, sizeof sw, s) != cudaSuccess) return SPECPV_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return SPECPV_ERR_CUDA;
    }
    if (info) memcpy(info, sw.info, sizeof sw.info);
    return (specpv_status)sw.code;
}

SPECPV_EXPORT specpv_status specpv_build_tree_mask(const int32_t* parents, int n_tree, int n_chain, uint64_t* mask,
                                                   int row_words) {
    if (!parents || !mask || n_tree <= 0 || n_chain < 0) return SPECPV_ERR_INVALID_ARG;
    const int M = n_tree + n_chain;
    if (row_words < (M + 63) / 64) return SPECPV_ERR_CAPACITY;
    if (parents[0] != -1) return SPECPV_ERR_BAD_TREE;
    for (int i = 1; i < n_tree; ++i)
        if (parents[i] < 0 || parents[i] >= i) return SPECPV_ERR_BAD_TREE;
    memset(mask, 0, (size_t)M * row_words * sizeof(uint64_t));
    // chain rows: the lower triangle.  Row r's words are built from row r-1's.
    for (int r = 0; r < n_chain; ++r) {
        uint64_t* row = mask + (size_t)r * row_words;
        if (r > 0) memcpy(row, row - row_words, row_words * sizeof(uint64_t));
        row[r >> 6] |= 1ull << (r & 63);
    }
    // tree rows: a node's visible set is its parent's plus itself (parents precede children)
    for (int i = 0; i < n_tree; ++i) {
        const int r = n_chain + i;
        uint64_t* row = mask + (size_t)r * row_words;
        const int pr = parents[i] < 0 ? n_chain - 1 : n_chain + parents[i];
        if (pr >= 0) memcpy(row, mask + (size_t)pr * row_words, row_words * sizeof(uint64_t));
        row[r >> 6] |= 1ull << (r & 63);
    }
    return SPECPV_OK;
}

SPECPV_EXPORT int specpv_select_mode(int ctx_len, int budget_tokens, int n_partially_verified, int n_candidates,
                                     int buffer_tokens, int partial_initialised) {
    if (ctx_len < budget_tokens) return SPECPV_MODE_FULL;
    if (!partial_initialised) return SPECPV_MODE_REFRESH;
    return n_partially_verified + n_candidates > buffer_tokens ? SPECPV_MODE_REFRESH : SPECPV_MODE_PARTIAL;
}

SPECPV_EXPORT specpv_status specpv_update_block_summaries(const specpv_config* cfg, int layer0, int n_layers,
                                                          const specpv_paged_kv* kv, const int32_t* tok_begin,
                                                          int max_blocks_touched, void* kmax, void* kmin,
                                                          void* workspace, size_t workspace_bytes, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    st = validate_kv(g, kv);
    if (st != SPECPV_OK) return st;
    if (!kmax || !kmin || !workspace || workspace_bytes < kStatusBytes) return SPECPV_ERR_INVALID_ARG;
    if (layer0 < 0 || n_layers <= 0 || layer0 + n_layers > g.n_layers || max_blocks_touched < 0) return SPECPV_ERR_INVALID_ARG;
    if (max_blocks_touched > kv->max_blocks) max_blocks_touched = kv->max_blocks;
    SummaryParams p{};
    p.k_pool = kv->k_pool; p.block_table = kv->block_table; p.seq_lens = kv->seq_lens; p.tok_begin = tok_begin;
    p.n_appended = nullptr; p.kmax = kmax; p.kmin = kmin; p.workspace = workspace;
    p.layer0 = layer0; p.batch = kv->batch; p.Hkv = g.Hkv; p.bs = g.bs; p.d = g.d; p.max_blocks = kv->max_blocks;
    p.n_pages = kv->n_pages; p.A_max = 0;
    return launch_summaries(p, n_layers, max_blocks_touched, g.dtype, reinterpret_cast<cudaStream_t>(stream));
}

SPECPV_EXPORT specpv_status specpv_score_blocks(const specpv_config* cfg, int layer0, int n_layers, const void* q,
                                                const int32_t* q_lens, int M_max, const int32_t* last_query,
                                                const void* kmax, const void* kmin, const specpv_paged_kv* kv,
                                                float* scores, void* workspace, size_t workspace_bytes, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    st = validate_kv(g, kv);
    if (st != SPECPV_OK) return st;
    if (!q || !kmax || !kmin || !scores || !workspace || workspace_bytes < kStatusBytes) return SPECPV_ERR_INVALID_ARG;
    if (layer0 < 0 || n_layers <= 0 || layer0 + n_layers > g.n_layers || M_max <= 0) return SPECPV_ERR_INVALID_ARG;
    ScoreParams p{};
    p.q = q; p.q_lens = q_lens; p.last_query = last_query; p.kmax = kmax; p.kmin = kmin; p.seq_lens = kv->seq_lens;
    p.scores = scores; p.layer0 = layer0; p.batch = kv->batch; p.M_max = M_max; p.Hq = g.Hq; p.Hkv = g.Hkv; p.G = g.G;
    p.bs = g.bs; p.max_blocks = kv->max_blocks; p.reduce = g.reduce;
    p.workspace = workspace;
    p.score_mode = g.score_mode;
    const int max_nb = (kv->max_seq_len + g.bs - 1) / g.bs;
    // both forms of Eq. 2 run on the tensor-core kernel (the channel-wise one as Kmax . q+ + Kmin . q-)
    if (scores_tc_supported(g.dtype, g.d, g.G, M_max) && aligned16(q) && aligned16(kmax) && aligned16(kmin))
        return launch_scores_tc(p, n_layers, g.n_layers, max_nb, reinterpret_cast<cudaStream_t>(stream));
    return launch_scores(p, n_layers, max_nb, g.dtype, g.d, reinterpret_cast<cudaStream_t>(stream));
}

SPECPV_EXPORT specpv_status specpv_select_partial_kv(const specpv_config* cfg, int n_layers, const float* scores,
                                                     const int32_t* seq_lens, int batch, int max_blocks, int32_t* idx,
                                                     int32_t* count, void* workspace, size_t workspace_bytes,
                                                     void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    if (!scores || !seq_lens || !idx || !count || !workspace || workspace_bytes < kStatusBytes) return SPECPV_ERR_INVALID_ARG;
    if (n_layers <= 0 || batch <= 0 || max_blocks <= 0) return SPECPV_ERR_INVALID_ARG;
    if (batch > 65535 || n_layers > 65535) return SPECPV_ERR_CAPACITY;
    SelectParams p{};
    p.scores = scores; p.seq_lens = seq_lens; p.idx = idx; p.count = count; p.batch = batch; p.Hkv = g.Hkv; p.bs = g.bs;
    p.max_blocks = max_blocks; p.sink_blocks = g.sink_blocks; p.local_blocks = g.local_blocks;
    p.budget_blocks = g.budget_blocks;
    p.share_heads = g.select_shared;
    return launch_select(p, n_layers, reinterpret_cast<cudaStream_t>(stream));
}

SPECPV_EXPORT specpv_status specpv_refresh_partial(const specpv_config* cfg, const specpv_paged_kv* full,
                                                   const int32_t* idx, const int32_t* count,
                                                   const specpv_paged_kv* partial, int32_t* partial_lens,
                                                   void* workspace, size_t workspace_bytes, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    st = validate_kv(g, full);
    if (st != SPECPV_OK) return st;
    if (!partial || !partial->k_pool || !partial->v_pool || !partial->block_table) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(partial->k_pool) || !aligned16(partial->v_pool)) return SPECPV_ERR_INVALID_ARG;
    if (!idx || !count || !partial_lens || !workspace || workspace_bytes < kStatusBytes) return SPECPV_ERR_INVALID_ARG;
    if (partial->batch != full->batch || partial->n_pages <= 0) return SPECPV_ERR_INVALID_ARG;
    if ((int64_t)partial->max_blocks * g.bs < (int64_t)g.budget_blocks * g.bs + g.buffer_tokens) return SPECPV_ERR_CAPACITY;
    GatherParams p{};
    p.full_k = full->k_pool; p.full_v = full->v_pool; p.full_table = full->block_table; p.seq_lens = full->seq_lens;
    p.idx = idx; p.count = count; p.part_k = partial->k_pool; p.part_v = partial->v_pool;
    p.part_table = partial->block_table; p.partial_lens = partial_lens; p.workspace = workspace;
    p.batch = full->batch; p.Hkv = g.Hkv; p.bs = g.bs; p.d = g.d; p.es = g.es; p.budget_blocks = g.budget_blocks;
    p.full_max_blocks = full->max_blocks; p.full_pages = full->n_pages; p.part_max_blocks = partial->max_blocks;
    p.part_pages = partial->n_pages;
    return launch_gather(p, g.n_layers, reinterpret_cast<cudaStream_t>(stream));
}

SPECPV_EXPORT specpv_status specpv_verify_partial(const specpv_config* cfg, int layer0, int n_layers, const void* q,
                                                  const void* k_new, const void* v_new, const uint64_t* tree_mask,
                                                  const int32_t* q_lens, int M_max, const specpv_paged_kv* partial,
                                                  void* out, float* lse, void* workspace, size_t workspace_bytes,
                                                  void* stream) {
    return verify_common(cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, partial, out, lse,
                         workspace, workspace_bytes, stream, true);
}

// ---- allocation-free variant of specpv_verify_partial -------------------------------------------
// The scratch lives in the library image.  In host code the array's name is only a handle for the
// runtime, not a device address: the address is looked up once per device and that is what the
// kernels get.
static __device__ __align__(256) unsigned char g_static_scratch[SPECPV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_addr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device (looked up on first use).
specpv_status static_scratch(void** addr) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPECPV_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return SPECPV_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return SPECPV_ERR_CUDA;
        g_static_addr[dev] = ptr;
    }
    *addr = g_static_addr[dev];
    return SPECPV_OK;
}
}  // namespace

SPECPV_EXPORT specpv_status specpv_verify_partial_static(const specpv_config* cfg, int layer0, int n_layers,
                                                         const void* q, const void* k_new, const void* v_new,
                                                         const uint64_t* tree_mask, const int32_t* q_lens, int M_max,
                                                         const specpv_paged_kv* partial, void* out, float* lse,
                                                         int32_t* device_status, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    st = validate_kv(g, partial);
    if (st != SPECPV_OK) return st;
    if (!q || !k_new || !v_new || !tree_mask || !out) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return SPECPV_ERR_INVALID_ARG;
    if (layer0 < 0 || n_layers <= 0 || layer0 + n_layers > g.n_layers || M_max <= 0) return SPECPV_ERR_INVALID_ARG;
    if (M_max > kMaxQTokens) return SPECPV_ERR_CAPACITY;
    if ((int64_t)partial->max_blocks * g.bs < (int64_t)g.budget_blocks * g.bs + g.buffer_tokens) return SPECPV_ERR_CAPACITY;
    // the fixed scratch must hold the partial results of at least two KV splits
    const size_t scratch = (size_t)SPECPV_STATIC_SCRATCH_BYTES - kHeaderBytes;
    const size_t per_split = (size_t)n_layers * partial->batch * g.Hkv * round_up((size_t)M_max * g.G, 256) *
                             (g.d + 2) * sizeof(float);
    if (per_split > scratch / 2) return SPECPV_ERR_CAPACITY;
    void* base = nullptr;
    st = static_scratch(&base);
    if (st != SPECPV_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // the status word is the only part of the array that has to start at zero
    if (cudaMemsetAsync(base, 0, kStatusBytes, s) != cudaSuccess) return SPECPV_ERR_CUDA;

    AttnArgs a{};
    a.g = g;
    a.layer0 = layer0; a.n_layers = n_layers; a.batch = partial->batch; a.M_max = M_max;
    a.mask_words = (M_max + 63) / 64;
    a.q = q; a.k_new = k_new; a.v_new = v_new; a.tree_mask = tree_mask; a.q_lens = q_lens;
    a.k_pool = partial->k_pool; a.v_pool = partial->v_pool; a.block_table = partial->block_table;
    a.seq_lens = partial->seq_lens;
    a.max_blocks = partial->max_blocks; a.n_pages = partial->n_pages; a.max_seq_len = partial->max_seq_len;
    a.out = out; a.lse = lse; a.workspace = base;
    a.counter_off = kStatusBytes;
    a.counter_bytes = kHeaderBytes - kStatusBytes;
    a.partial_off = kHeaderBytes;
    a.partial_bytes = scratch;
    st = attention_tc_supported(a) ? launch_attention_tc(a, s) : launch_attention_simt(a, s);
    if (st != SPECPV_OK) return st;
    if (device_status &&
        cudaMemcpyAsync(device_status, base, sizeof(StatusWord), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return SPECPV_ERR_CUDA;
    return SPECPV_OK;
}

SPECPV_EXPORT specpv_status specpv_verify_full(const specpv_config* cfg, int layer0, int n_layers, const void* q,
                                               const void* k_new, const void* v_new, const uint64_t* tree_mask,
                                               const int32_t* q_lens, int M_max, const specpv_paged_kv* full,
                                               void* out, float* lse, void* workspace, size_t workspace_bytes,
                                               void* stream) {
    return verify_common(cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, full, out, lse,
                         workspace, workspace_bytes, stream, false);
}

SPECPV_EXPORT specpv_status specpv_verify_host(const specpv_config* cfg, int mode, int layer0, int n_layers,
                                               const void* q_host, const void* k_new_host, const void* v_new_host,
                                               const uint64_t* tree_mask_host, int M_max, const specpv_paged_kv* kv,
                                               void* out_host, float* lse_host, void* workspace,
                                               size_t workspace_bytes, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    st = validate_kv(g, kv);
    if (st != SPECPV_OK) return st;
    if (mode != SPECPV_MODE_PARTIAL && mode != SPECPV_MODE_FULL) return SPECPV_ERR_INVALID_ARG;
    if (!q_host || !k_new_host || !v_new_host || !tree_mask_host || !out_host || !workspace) return SPECPV_ERR_INVALID_ARG;
    if (n_layers <= 0 || M_max <= 0 || M_max > kMaxQTokens) return SPECPV_ERR_INVALID_ARG;
    WorkspacePlan w = plan_workspace(g, n_layers, kv->batch, M_max);
    if (workspace_bytes < w.total) return SPECPV_ERR_CAPACITY;
    StagingPlan sp = plan_staging(g, n_layers, kv->batch, M_max);
    char* stage = reinterpret_cast<char*>(workspace) + w.staging_off;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t rows_l = (size_t)kv->batch * M_max;  // rows of one layer
    const size_t q_l = rows_l * g.Hq * g.d * g.es, kv_l = rows_l * g.Hkv * g.d * g.es;
    const size_t out_l = rows_l * g.Hq * g.d * g.out_es, lse_l = rows_l * g.Hq * sizeof(float);
    const size_t mask_bytes = (size_t)kv->batch * M_max * ((M_max + 63) / 64) * sizeof(uint64_t);

    // The layers go through in groups: while one group's attention runs on `stream`, the next group's inputs arrive
    // on a copy-in stream and the previous group's outputs leave on a copy-out stream (the host link carries both
    // directions at once).  The two copy streams are created once per device and kept.
    HostCopyStreams* cs = host_copy_streams();
    if (!cs) return SPECPV_ERR_CUDA;
    constexpr int kMaxGroups = 8;
    const int n_groups = n_layers < kMaxGroups ? n_layers : kMaxGroups;
    const int per_group = (n_layers + n_groups - 1) / n_groups;
    cudaEvent_t begin = nullptr, in_done[kMaxGroups] = {}, run_done[kMaxGroups] = {}, out_done = nullptr;
    bool ok = cudaEventCreateWithFlags(&begin, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&out_done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < n_groups && ok; ++i)
        ok = cudaEventCreateWithFlags(&in_done[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&run_done[i], cudaEventDisableTiming) == cudaSuccess;
    // the staging area may still be in use by earlier work on `stream`
    ok = ok && cudaEventRecord(begin, s) == cudaSuccess && cudaStreamWaitEvent(cs->in, begin, 0) == cudaSuccess &&
         cudaStreamWaitEvent(cs->out, begin, 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(stage + sp.mask, tree_mask_host, mask_bytes, cudaMemcpyHostToDevice, cs->in) == cudaSuccess;
    int n_used = 0;
    for (int i = 0; i < n_groups && ok && st == SPECPV_OK; ++i) {
        const int l0 = i * per_group, nl = n_layers - l0 < per_group ? n_layers - l0 : per_group;
        if (nl <= 0) break;
        n_used = i + 1;
        ok = cudaMemcpyAsync(stage + sp.q + l0 * q_l, static_cast<const char*>(q_host) + l0 * q_l, nl * q_l,
                             cudaMemcpyHostToDevice, cs->in) == cudaSuccess &&
             cudaMemcpyAsync(stage + sp.k_new + l0 * kv_l, static_cast<const char*>(k_new_host) + l0 * kv_l, nl * kv_l,
                             cudaMemcpyHostToDevice, cs->in) == cudaSuccess &&
             cudaMemcpyAsync(stage + sp.v_new + l0 * kv_l, static_cast<const char*>(v_new_host) + l0 * kv_l, nl * kv_l,
                             cudaMemcpyHostToDevice, cs->in) == cudaSuccess &&
             cudaEventRecord(in_done[i], cs->in) == cudaSuccess && cudaStreamWaitEvent(s, in_done[i], 0) == cudaSuccess;
        if (!ok) break;
        st = verify_common(cfg, layer0 + l0, nl, stage + sp.q + l0 * q_l, stage + sp.k_new + l0 * kv_l,
                           stage + sp.v_new + l0 * kv_l, reinterpret_cast<const uint64_t*>(stage + sp.mask), nullptr, M_max, kv,
                           stage + sp.out + l0 * out_l,
                           lse_host ? reinterpret_cast<float*>(stage + sp.lse + l0 * lse_l) : nullptr, workspace,
                           w.partial_off + w.partial_bytes, stream, mode == SPECPV_MODE_PARTIAL);
        if (st != SPECPV_OK) break;
        ok = cudaEventRecord(run_done[i], s) == cudaSuccess && cudaStreamWaitEvent(cs->out, run_done[i], 0) == cudaSuccess &&
             cudaMemcpyAsync(static_cast<char*>(out_host) + l0 * out_l, stage + sp.out + l0 * out_l, nl * out_l,
                             cudaMemcpyDeviceToHost, cs->out) == cudaSuccess;
        if (ok && lse_host)
            ok = cudaMemcpyAsync(reinterpret_cast<char*>(lse_host) + l0 * lse_l, stage + sp.lse + l0 * lse_l, nl * lse_l,
                                 cudaMemcpyDeviceToHost, cs->out) == cudaSuccess;
    }
    // everything is joined back onto `stream` before the call returns (also on the error paths: no copy may outlive it)
    const bool joined = cudaEventRecord(out_done, cs->out) == cudaSuccess && cudaStreamWaitEvent(s, out_done, 0) == cudaSuccess;
    const bool in_idle = cudaStreamSynchronize(cs->in) == cudaSuccess;
    const bool synced = cudaStreamSynchronize(s) == cudaSuccess && (joined || cudaStreamSynchronize(cs->out) == cudaSuccess);
    (void)n_used;
    if (begin) cudaEventDestroy(begin);
    if (out_done) cudaEventDestroy(out_done);
    for (int i = 0; i < kMaxGroups; ++i) {
        if (in_done[i]) cudaEventDestroy(in_done[i]);
        if (run_done[i]) cudaEventDestroy(run_done[i]);
    }
    if (st != SPECPV_OK) return st;
    return ok && in_idle && synced ? SPECPV_OK : SPECPV_ERR_CUDA;
}

SPECPV_EXPORT specpv_status specpv_commit_accepted(const specpv_config* cfg, int layer0, int n_layers,
                                                   const void* k_new, const void* v_new, int M_max,
                                                   const int32_t* accepted, const int32_t* n_accepted, int A_max,
                                                   const specpv_paged_kv* dst, void* kmax, void* kmin,
                                                   void* workspace, size_t workspace_bytes, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    st = validate_kv(g, dst);
    if (st != SPECPV_OK) return st;
    if (!k_new || !v_new || !accepted || !n_accepted || !workspace || workspace_bytes < kStatusBytes) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new)) return SPECPV_ERR_INVALID_ARG;
    if ((kmax == nullptr) != (kmin == nullptr)) return SPECPV_ERR_INVALID_ARG;
    // the lengths advance once, when the last layer of the model has been committed
    if (layer0 < 0 || n_layers <= 0 || layer0 + n_layers > g.n_layers || M_max <= 0 || A_max <= 0) return SPECPV_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    CommitParams p{};
    p.k_new = k_new; p.v_new = v_new; p.accepted = accepted; p.n_accepted = n_accepted; p.k_pool = dst->k_pool;
    p.v_pool = dst->v_pool; p.block_table = dst->block_table; p.seq_lens = dst->seq_lens; p.workspace = workspace;
    p.layer0 = layer0; p.batch = dst->batch; p.M_max = M_max; p.A_max = A_max; p.Hkv = g.Hkv; p.bs = g.bs; p.d = g.d;
    p.es = g.es; p.max_blocks = dst->max_blocks; p.n_pages = dst->n_pages;
    st = launch_commit(p, n_layers, nullptr, s);
    if (st != SPECPV_OK) return st;
    if (kmax) {
        SummaryParams sp{};
        sp.k_pool = dst->k_pool; sp.block_table = dst->block_table; sp.seq_lens = dst->seq_lens;
        sp.tok_begin = dst->seq_lens; sp.n_appended = n_accepted; sp.kmax = kmax; sp.kmin = kmin; sp.workspace = workspace;
        sp.layer0 = layer0; sp.batch = dst->batch; sp.Hkv = g.Hkv; sp.bs = g.bs; sp.d = g.d; sp.max_blocks = dst->max_blocks;
        sp.n_pages = dst->n_pages; sp.A_max = A_max;
        st = launch_summaries(sp, n_layers, (A_max + g.bs - 1) / g.bs + 1, g.dtype, s);
        if (st != SPECPV_OK) return st;
    }
    if (layer0 + n_layers == g.n_layers)
        return launch_commit_lens(const_cast<int32_t*>(dst->seq_lens), n_accepted, dst->batch, A_max,
                                  dst->max_blocks * g.bs, s);
    return SPECPV_OK;
}

// ---- the linear maps either side of the attention --------------------------------------------------------------
SPECPV_EXPORT specpv_status specpv_rope_table(const specpv_config* cfg, const uint64_t* tree_mask, const int32_t* q_lens,
                                              const int32_t* base_pos, int batch, int M_max, double rope_theta,
                                              float* cos_sin, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    if (!tree_mask || !base_pos || !cos_sin || !aligned16(cos_sin)) return SPECPV_ERR_INVALID_ARG;
    if (batch <= 0 || M_max <= 0 || !(rope_theta > 1.0) || isinf(rope_theta)) return SPECPV_ERR_INVALID_ARG;
    if (M_max > kMaxQTokens) return SPECPV_ERR_CAPACITY;
    return launch_rope_table(tree_mask, q_lens, base_pos, batch, M_max, g.d, rope_theta, cos_sin,
                             reinterpret_cast<cudaStream_t>(stream));
}

static specpv_status proj_dispatch(ProjArgs& a, const Geometry& g, int layer0, int n_layers, int batch, int M_max,
                                   void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || !aligned16(workspace) || workspace_bytes < kStatusBytes) return SPECPV_ERR_INVALID_ARG;
    if (layer0 < 0 || n_layers <= 0 || layer0 + n_layers > g.n_layers || batch <= 0 || M_max <= 0)
        return SPECPV_ERR_INVALID_ARG;
    if ((int64_t)batch * M_max > (int64_t)1 << 24) return SPECPV_ERR_CAPACITY;
    a.dtype = g.dtype;
    a.layer0 = layer0; a.n_layers_call = n_layers; a.n_layers_total = g.n_layers;
    a.tokens = batch * M_max;
    a.workspace = workspace;
    if (workspace_bytes < kHeaderBytes) return SPECPV_ERR_CAPACITY;
    a.scratch_off = kHeaderBytes;
    a.scratch_bytes = workspace_bytes - kHeaderBytes;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (proj_tc_supported(a)) return launch_proj_tc(a, s);
    return launch_proj_simt(a, s);
}

SPECPV_EXPORT specpv_status specpv_qkv_rope(const specpv_config* cfg, int layer0, int n_layers, const void* x, int hidden,
                                            const void* w_qkv, const float* cos_sin, int batch, int M_max, void* q,
                                            void* k_new, void* v_new, void* workspace, size_t workspace_bytes,
                                            void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    if (!x || !w_qkv || !cos_sin || !q || !k_new || !v_new) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_qkv) || !aligned16(cos_sin) || !aligned16(q) || !aligned16(k_new) || !aligned16(v_new))
        return SPECPV_ERR_INVALID_ARG;
    if (hidden <= 0 || hidden % 16 != 0) return SPECPV_ERR_SHAPE;
    ProjArgs a{};
    a.x = x; a.w = w_qkv; a.cos_sin = cos_sin; a.residual = nullptr;
    a.n_in = hidden; a.n_out = (g.Hq + 2 * g.Hkv) * g.d; a.tile = g.d;
    a.n_seg = 3;
    a.seg[0] = ProjSegment{q, 0, g.Hq * g.d, 1};
    a.seg[1] = ProjSegment{k_new, g.Hq, g.Hkv * g.d, 1};
    a.seg[2] = ProjSegment{v_new, g.Hq + g.Hkv, g.Hkv * g.d, 0};
    return proj_dispatch(a, g, layer0, n_layers, batch, M_max, workspace, workspace_bytes, stream);
}

SPECPV_EXPORT specpv_status specpv_o_proj(const specpv_config* cfg, int layer0, int n_layers, const void* attn,
                                          const void* w_o, int hidden, const void* residual, int batch, int M_max, void* y,
                                          void* workspace, size_t workspace_bytes, void* stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    if (!attn || !w_o || !y) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(attn) || !aligned16(w_o) || !aligned16(y) || (residual && !aligned16(residual)))
        return SPECPV_ERR_INVALID_ARG;
    if (hidden <= 0 || hidden % 16 != 0) return SPECPV_ERR_SHAPE;
    ProjArgs a{};
    a.x = attn; a.w = w_o; a.cos_sin = nullptr; a.residual = residual;
    a.n_in = g.Hq * g.d; a.n_out = hidden; a.tile = hidden % 128 == 0 ? 128 : 16;
    a.n_seg = 1;
    a.seg[0] = ProjSegment{y, 0, hidden, 0};
    return proj_dispatch(a, g, layer0, n_layers, batch, M_max, workspace, workspace_bytes, stream);
}
