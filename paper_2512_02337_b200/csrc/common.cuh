// Shared declarations of the SpecPV CUDA library: validated geometry, the device status word,
// workspace carving and dtype helpers.  Nothing here is shared with the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/specpv.h"

namespace specpv {

// ---- device status word: workspace[0..255] ------------------------------------------------
// word 0: first recorded specpv_status (0 = none); words 1..4: details of that first fault.
struct StatusWord {
    int32_t code;
    int32_t info[4];
};

__device__ __forceinline__ void record_fault(void* workspace, int code, int i0, int i1, int i2, int i3) {
    StatusWord* sw = reinterpret_cast<StatusWord*>(workspace);
    if (atomicCAS(&sw->code, 0, code) == 0) {
        sw->info[0] = i0;
        sw->info[1] = i1;
        sw->info[2] = i2;
        sw->info[3] = i3;
    }
}

constexpr size_t kStatusBytes = 256;
// Head of every workspace: the status word, then arrival counters of KV ranges shared between CTAs (two per (layer,
// sequence, KV head, group of 256 rows) of a call; zero between launches).  All scratch starts behind it.
constexpr size_t kHeaderBytes = 256 * 1024;
constexpr int kMaxQTokens = 128;      // M_max supported by the attention kernels (two mask words)
constexpr int kMaxSplitCtas = 8 * 148;  // the workspace holds split-KV partial results of this many CTAs (+ one per head)

// process-wide count of kernel launches (reported by specpv_kernel_launches)
void count_launch(int n = 1);

// ---- geometry after validation ---------------------------------------------------------------
struct Geometry {
    int n_layers, Hq, Hkv, G, d, bs, dtype, es;  // es = element size in bytes
    int out_f32, out_es;                          // output element type / size
    int sink_blocks, local_blocks, budget_blocks, buffer_tokens, reduce, score_mode, select_shared;
    float scale;
};

specpv_status validate_config(const specpv_config* cfg, Geometry* g);
specpv_status validate_kv(const Geometry& g, const specpv_paged_kv* kv);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- workspace carving --------------------------------------------------------------------
struct WorkspacePlan {
    size_t counter_off, counter_bytes;  // arrival counters of KV ranges shared between CTAs (zero between launches)
    size_t partial_off, partial_bytes;  // split-KV partial results
    size_t staging_off, staging_bytes;  // device copies of host step tensors (specpv_verify_host)
    size_t total;
};
WorkspacePlan plan_workspace(const Geometry& g, int n_layers_per_call, int max_batch, int M_max);

// offsets inside the staging area
struct StagingPlan {
    size_t q, k_new, v_new, mask, out, lse, total;
};
StagingPlan plan_staging(const Geometry& g, int n_layers_per_call, int batch, int M_max);

// ---- dtype helpers ------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---- launchers implemented in the kernel files --------------------------------------------------
struct AttnArgs {
    Geometry g;
    int layer0, n_layers, batch, M_max, mask_words;
    const void* q;
    const void* k_new;
    const void* v_new;
    const uint64_t* tree_mask;
    const int32_t* q_lens;
    const void* k_pool;
    const void* v_pool;
    const int32_t* block_table;
    const int32_t* seq_lens;
    int max_blocks, n_pages, max_seq_len;
    void* out;
    float* lse;
    void* workspace;
    size_t partial_off, partial_bytes;
    size_t counter_off, counter_bytes;
};

specpv_status launch_attention_simt(const AttnArgs& a, cudaStream_t stream);
specpv_status launch_attention_tc(const AttnArgs& a, cudaStream_t stream);  // bf16, d = 128, bs = 64
bool attention_tc_supported(const AttnArgs& a);

}  // namespace specpv
