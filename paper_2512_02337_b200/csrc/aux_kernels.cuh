// Parameter blocks and launchers of the cache-management kernels (see aux_kernels.cu).
#pragma once
#include "common.cuh"

namespace specpv {

struct SummaryParams {
    const void* k_pool;
    const int32_t* block_table;
    const int32_t* seq_lens;
    const int32_t* tok_begin;   // nullable
    const int32_t* n_appended;  // nullable: tokens a commit in flight adds to seq_lens
    void* kmax;
    void* kmin;
    void* workspace;
    int layer0, batch, Hkv, bs, d, max_blocks, n_pages, A_max;
};

struct ScoreParams {
    const void* q;
    const int32_t* q_lens;
    const int32_t* last_query;
    const void* kmax;
    const void* kmin;
    const int32_t* seq_lens;
    float* scores;
    void* workspace;
    int layer0, batch, M_max, Hq, Hkv, G, bs, max_blocks, reduce;
    int score_mode;  // 0: max of the two full dot products (Eq. 2 as printed), 1: maximum per channel
};

struct SelectParams {
    const float* scores;
    const int32_t* seq_lens;
    int32_t* idx;
    int32_t* count;
    int batch, Hkv, bs, max_blocks, sink_blocks, local_blocks, budget_blocks;
    int share_heads;  // 1: every KV head of a layer keeps the blocks chosen on the mean of the heads' scores
};

struct GatherParams {
    const void* full_k;
    const void* full_v;
    const int32_t* full_table;
    const int32_t* seq_lens;
    const int32_t* idx;
    const int32_t* count;
    void* part_k;
    void* part_v;
    const int32_t* part_table;
    int32_t* partial_lens;
    void* workspace;
    int batch, Hkv, bs, d, es, budget_blocks, full_max_blocks, full_pages, part_max_blocks, part_pages;
};

struct CommitParams {
    const void* k_new;
    const void* v_new;
    const int32_t* accepted;
    const int32_t* n_accepted;
    void* k_pool;
    void* v_pool;
    const int32_t* block_table;
    const int32_t* seq_lens;
    void* workspace;
    int layer0, batch, M_max, A_max, Hkv, bs, d, es, max_blocks, n_pages;
};

specpv_status launch_summaries(const SummaryParams& p, int n_layers, int blocks_touched, int dtype, cudaStream_t stream);
specpv_status launch_scores(const ScoreParams& p, int n_layers, int max_nb, int dtype, int d, cudaStream_t stream);
bool scores_tc_supported(int dtype, int d, int G, int M_max);
specpv_status launch_scores_tc(const ScoreParams& p, int n_layers_call, int n_layers_total, int max_nb,
                               cudaStream_t stream);
specpv_status launch_select(const SelectParams& p, int n_layers, cudaStream_t stream);
specpv_status launch_gather(const GatherParams& p, int n_layers, cudaStream_t stream);
specpv_status launch_commit(const CommitParams& p, int n_layers, int32_t* seq_lens, cudaStream_t stream);
specpv_status launch_commit_lens(int32_t* seq_lens, const int32_t* n_accepted, int batch, int A_max,
                                 int capacity_tokens, cudaStream_t stream);

}  // namespace specpv
