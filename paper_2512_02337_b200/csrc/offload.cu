// Full verification over a KV cache that lives in host memory (paper Section 3.3, last paragraph): one
// layer's keys and values on the device at a time, the next layer's copy in flight on a second stream
// while the current layer's attention runs.  Host-side orchestration only; the attention kernels are the
// ones of the resident path, pointed at a two-layer staging pool.
#include "common.cuh"

#define SPECPV_EXPORT extern "C" __attribute__((visibility("default")))

using namespace specpv;

SPECPV_EXPORT specpv_status specpv_verify_full_offloaded(const specpv_config* cfg, int layer0, int n_layers, const void* q,
                                                         const void* k_new, const void* v_new, const uint64_t* tree_mask,
                                                         const int32_t* q_lens, int M_max, const specpv_offloaded_kv* full,
                                                         void* out, float* lse, void* workspace, size_t workspace_bytes,
                                                         void* stream, void* copy_stream) {
    Geometry g;
    specpv_status st = validate_config(cfg, &g);
    if (st != SPECPV_OK) return st;
    if (!full || !full->k_host || !full->v_host || !full->k_stage || !full->v_stage || !full->block_table || !full->seq_lens)
        return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(full->k_host) || !aligned16(full->v_host) || !aligned16(full->k_stage) || !aligned16(full->v_stage))
        return SPECPV_ERR_INVALID_ARG;
    if (full->batch <= 0 || full->max_blocks <= 0 || full->n_pages <= 0 || full->max_seq_len < 0) return SPECPV_ERR_INVALID_ARG;
    if ((int64_t)full->max_seq_len > (int64_t)full->max_blocks * g.bs) return SPECPV_ERR_CAPACITY;
    if (!q || !k_new || !v_new || !tree_mask || !out || !workspace) return SPECPV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out) || !aligned16(workspace))
        return SPECPV_ERR_INVALID_ARG;
    if (layer0 < 0 || n_layers <= 0 || layer0 + n_layers > g.n_layers || M_max <= 0) return SPECPV_ERR_INVALID_ARG;
    if (M_max > kMaxQTokens) return SPECPV_ERR_CAPACITY;
    WorkspacePlan w = plan_workspace(g, 1, full->batch, M_max);
    if (workspace_bytes < w.partial_off + w.partial_bytes) return SPECPV_ERR_CAPACITY;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaStream_t cs = reinterpret_cast<cudaStream_t>(copy_stream);
    const size_t layer_bytes = (size_t)full->n_pages * g.Hkv * g.bs * g.d * g.es;
    const size_t q_layer = (size_t)full->batch * M_max * g.Hq * g.d * g.es;
    const size_t kv_layer = (size_t)full->batch * M_max * g.Hkv * g.d * g.es;
    const size_t out_layer = (size_t)full->batch * M_max * g.Hq * g.d * g.out_es;
    const size_t lse_layer = (size_t)full->batch * M_max * g.Hq;

    cudaEvent_t ready[2] = {nullptr, nullptr}, done[2] = {nullptr, nullptr}, begin = nullptr;
    bool ok = cudaEventCreateWithFlags(&begin, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
        ok = cudaEventCreateWithFlags(&ready[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&done[i], cudaEventDisableTiming) == cudaSuccess;
    // earlier work on `stream` may still read the slots: the first copies wait for it
    ok = ok && cudaEventRecord(begin, s) == cudaSuccess && cudaStreamWaitEvent(cs, begin, 0) == cudaSuccess;

    Geometry g2 = g;
    g2.n_layers = 2;  // the staging pool holds two layer slots
    auto copy_layer = [&](int i) {  // layer layer0 + i -> slot i & 1
        const int slot = i & 1;
        const size_t src = (size_t)(layer0 + i) * layer_bytes, dst = (size_t)slot * layer_bytes;
        if (i >= 2 && cudaStreamWaitEvent(cs, done[slot], 0) != cudaSuccess) return false;  // the slot's last reader
        if (cudaMemcpyAsync(static_cast<char*>(full->k_stage) + dst, static_cast<const char*>(full->k_host) + src,
                            layer_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess)
            return false;
        if (cudaMemcpyAsync(static_cast<char*>(full->v_stage) + dst, static_cast<const char*>(full->v_host) + src,
                            layer_bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess)
            return false;
        return cudaEventRecord(ready[slot], cs) == cudaSuccess;
    };
    ok = ok && copy_layer(0);
    for (int i = 0; i < n_layers && ok && st == SPECPV_OK; ++i) {
        const int slot = i & 1;
        // the next layer's copy is queued before this layer's attention: it needs the other slot, which the
        // attention of layer i - 1 (already queued on `stream`) is the last to read
        if (i + 1 < n_layers) ok = copy_layer(i + 1);
        ok = ok && cudaStreamWaitEvent(s, ready[slot], 0) == cudaSuccess;
        if (!ok) break;
        AttnArgs a{};
        a.g = g2;
        a.layer0 = slot; a.n_layers = 1; a.batch = full->batch; a.M_max = M_max;
        a.mask_words = (M_max + 63) / 64;
        a.q = static_cast<const char*>(q) + i * q_layer;
        a.k_new = static_cast<const char*>(k_new) + i * kv_layer;
        a.v_new = static_cast<const char*>(v_new) + i * kv_layer;
        a.tree_mask = tree_mask; a.q_lens = q_lens;
        a.k_pool = full->k_stage; a.v_pool = full->v_stage; a.block_table = full->block_table; a.seq_lens = full->seq_lens;
        a.max_blocks = full->max_blocks; a.n_pages = full->n_pages; a.max_seq_len = full->max_seq_len;
        a.out = static_cast<char*>(out) + i * out_layer;
        a.lse = lse ? lse + i * lse_layer : nullptr;
        a.workspace = workspace;
        a.partial_off = w.partial_off;
        a.partial_bytes = workspace_bytes - w.partial_off < w.partial_bytes ? workspace_bytes - w.partial_off : w.partial_bytes;
        a.counter_off = w.counter_off;
        a.counter_bytes = w.counter_bytes;
        st = attention_tc_supported(a) ? launch_attention_tc(a, s) : launch_attention_simt(a, s);
        ok = cudaEventRecord(done[slot], s) == cudaSuccess;
    }
    // events may be destroyed while work that uses them is pending: their resources are released when it completes
    if (begin) cudaEventDestroy(begin);
    for (int i = 0; i < 2; ++i) {
        if (ready[i]) cudaEventDestroy(ready[i]);
        if (done[i]) cudaEventDestroy(done[i]);
    }
    if (st != SPECPV_OK) return st;
    return ok ? SPECPV_OK : SPECPV_ERR_CUDA;
}
