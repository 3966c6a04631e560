// Tree-masked GQA verification attention, float32 SIMT path (paper Section 3.2-3.3, Algorithm 1
// "TreeDecode").  Covers every geometry (float32 or bfloat16 storage, any group size, any block
// size) with float32 arithmetic and accurate expf; it is the path for float32 caches and the
// on-device second opinion for the tensor-core kernel.
//
// Work split: grid = (KV splits, KV heads, layers x sequences).  A CTA walks its token range in
// 32-token tiles staged in shared memory; warp w owns 4 query rows per pass (lane <-> token for the
// logits, lane <-> channel for the PV product) and keeps the running (max, sum, accumulator) of an
// online softmax.  The last split also attends the step's own tokens under the tree mask.  With
// more than one split the unnormalised partial results go to the workspace and merge_splits_kernel
// combines them with a log-sum-exp merge.
#include <math.h>

#include "common.cuh"

namespace specpv {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTile = 32;         // tokens per tile (one per lane)
constexpr int kRowsPerWarp = 4;   // query rows a warp carries per pass
constexpr int kRowsPerPass = kWarps * kRowsPerWarp;

struct SimtParams {
    const void* q;
    const void* k_new;
    const void* v_new;
    const uint64_t* tree_mask;
    const int32_t* q_lens;
    const void* k_pool;
    const void* v_pool;
    const int32_t* block_table;
    const int32_t* seq_lens;
    void* out;
    float* lse;
    float* part_o;   // [lb][Hkv][splits][R_max][D]
    float* part_ml;  // [lb][Hkv][splits][R_max][2]
    void* workspace;
    int layer0, batch, M_max, mask_words, Hq, Hkv, G, bs, max_blocks, n_pages;
    int n_splits, chunk;
    float scale;
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T, typename TO, int D>
__global__ void __launch_bounds__(kThreads) attn_simt_kernel(SimtParams p) {
    constexpr int CPL = D / 32;  // channels per lane
    extern __shared__ float smem[];
    float* Ks = smem;                       // [kTile][D + 1]
    float* Vs = Ks + kTile * (D + 1);       // [kTile][D]
    float* Qs = Vs + kTile * D;             // [kRowsPerPass][D]
    __shared__ int s_tile_valid;

    const int split = blockIdx.x, h = blockIdx.y, lb = blockIdx.z;
    const int b = lb % p.batch, l = lb / p.batch;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int seq_len = p.seq_lens[b];
    int M = p.q_lens ? p.q_lens[b] : p.M_max;
    M = min(max(M, 0), p.M_max);
    const int R = M * p.G;
    const int R_max = p.M_max * p.G;

    const bool last_split = split == p.n_splits - 1;
    const int ctx_begin = min(split * p.chunk, seq_len);
    const int ctx_end = last_split ? seq_len : min((split + 1) * p.chunk, seq_len);
    const int n_ctx_tiles = (ctx_end - ctx_begin + kTile - 1) / kTile;
    const int n_new_tiles = last_split ? (M + kTile - 1) / kTile : 0;

    const T* q = reinterpret_cast<const T*>(p.q) + (size_t)lb * p.M_max * p.Hq * D;
    const T* k_new = reinterpret_cast<const T*>(p.k_new) + (size_t)lb * p.M_max * p.Hkv * D;
    const T* v_new = reinterpret_cast<const T*>(p.v_new) + (size_t)lb * p.M_max * p.Hkv * D;
    const size_t layer_stride = (size_t)p.n_pages * p.Hkv * p.bs * D;
    const T* k_pool = reinterpret_cast<const T*>(p.k_pool) + (size_t)(p.layer0 + l) * layer_stride;
    const T* v_pool = reinterpret_cast<const T*>(p.v_pool) + (size_t)(p.layer0 + l) * layer_stride;
    const int32_t* table = p.block_table + (size_t)b * p.max_blocks;
    const uint64_t* mask = p.tree_mask + (size_t)b * p.M_max * p.mask_words;

    for (int pass_row0 = 0; pass_row0 < R; pass_row0 += kRowsPerPass) {
        __syncthreads();
        // stage this pass's query rows (row r = token j * G + head g of the group)
        for (int e = tid; e < kRowsPerPass * D; e += kThreads) {
            int r = pass_row0 + e / D, c = e % D;
            float v = 0.f;
            if (r < R) {
                int j = r / p.G, g = r % p.G;
                v = to_float(q[((size_t)j * p.Hq + h * p.G + g) * D + c]);
            }
            Qs[e] = v;
        }
        float m_run[kRowsPerWarp], l_run[kRowsPerWarp], acc[kRowsPerWarp][CPL];
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            m_run[i] = -INFINITY;
            l_run[i] = 0.f;
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[i][c] = 0.f;
        }

        for (int tile = 0; tile < n_ctx_tiles + n_new_tiles; ++tile) {
            const bool is_new = tile >= n_ctx_tiles;
            const int tok0 = is_new ? (tile - n_ctx_tiles) * kTile : ctx_begin + tile * kTile;
            const int tok_end = is_new ? M : ctx_end;
            __syncthreads();
            if (tid == 0) s_tile_valid = 1;
            __syncthreads();
            // stage K and V of the tile as float32
            for (int e = tid; e < kTile * D; e += kThreads) {
                int tt = e / D, c = e % D;
                int t = tok0 + tt;
                float kv = 0.f, vv = 0.f;
                if (t < tok_end) {
                    if (is_new) {
                        size_t off = ((size_t)t * p.Hkv + h) * D + c;
                        kv = to_float(k_new[off]);
                        vv = to_float(v_new[off]);
                    } else {
                        int page = table[t / p.bs];
                        if (page < 0 || page >= p.n_pages) {
                            if (c == 0) record_fault(p.workspace, SPECPV_ERR_BAD_BLOCK_TABLE, b, t / p.bs, page, l);
                            s_tile_valid = 0;
                        } else {
                            size_t off = (((size_t)page * p.Hkv + h) * p.bs + t % p.bs) * D + c;
                            kv = to_float(k_pool[off]);
                            vv = to_float(v_pool[off]);
                        }
                    }
                }
                Ks[tt * (D + 1) + c] = kv;
                Vs[tt * D + c] = vv;
            }
            __syncthreads();
            const bool tile_ok = s_tile_valid != 0;  // a tile reached through a bad page id is skipped
            const int t_lane = tok0 + lane;
            // logits of this lane's token against the warp's rows
            float s[kRowsPerWarp];
#pragma unroll
            for (int i = 0; i < kRowsPerWarp; ++i) s[i] = 0.f;
            const float* krow = Ks + lane * (D + 1);
            const float* qrow = Qs + warp * kRowsPerWarp * D;
#pragma unroll 8
            for (int c = 0; c < D; ++c) {
                float kc = krow[c];
#pragma unroll
                for (int i = 0; i < kRowsPerWarp; ++i) s[i] = fmaf(qrow[i * D + c], kc, s[i]);
            }
#pragma unroll
            for (int i = 0; i < kRowsPerWarp; ++i) {
                const int r = pass_row0 + warp * kRowsPerWarp + i;
                bool visible = tile_ok && t_lane < tok_end && r < R;
                if (visible && is_new) {
                    int j = r / p.G;
                    visible = (mask[(size_t)j * p.mask_words + t_lane / 64] >> (t_lane % 64)) & 1ull;
                }
                float logit = visible ? s[i] * p.scale : -INFINITY;
                float m_new = fmaxf(m_run[i], warp_max(logit));
                float m_safe = m_new == -INFINITY ? 0.f : m_new;
                float pr = expf(logit - m_safe);       // exp(-inf) = 0 for masked keys
                float corr = expf(m_run[i] - m_safe);  // 0 while nothing has been seen
                l_run[i] = l_run[i] * corr + warp_sum(pr);
                m_run[i] = m_new;
#pragma unroll
                for (int c = 0; c < CPL; ++c) acc[i][c] *= corr;
                s[i] = pr;
            }
            // PV: lane <-> channel
#pragma unroll 4
            for (int tt = 0; tt < kTile; ++tt) {
                float vv[CPL];
#pragma unroll
                for (int c = 0; c < CPL; ++c) vv[c] = Vs[tt * D + lane + 32 * c];
#pragma unroll
                for (int i = 0; i < kRowsPerWarp; ++i) {
                    float pr = __shfl_sync(0xffffffffu, s[i], tt);
#pragma unroll
                    for (int c = 0; c < CPL; ++c) acc[i][c] = fmaf(pr, vv[c], acc[i][c]);
                }
            }
        }

        // write this pass's rows
#pragma unroll
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const int r = pass_row0 + warp * kRowsPerWarp + i;
            if (r >= R) continue;
            if (p.n_splits == 1) {
                const int j = r / p.G, g = r % p.G;
                const size_t row = ((size_t)lb * p.M_max + j) * p.Hq + h * p.G + g;
                TO* o = reinterpret_cast<TO*>(p.out) + row * D;
                float inv = 1.f / l_run[i];
#pragma unroll
                for (int c = 0; c < CPL; ++c) o[lane + 32 * c] = from_float<TO>(acc[i][c] * inv);
                if (p.lse && lane == 0) p.lse[row] = m_run[i] + logf(l_run[i]);
            } else {
                const size_t prow = (((size_t)lb * p.Hkv + h) * p.n_splits + split) * R_max + r;
#pragma unroll
                for (int c = 0; c < CPL; ++c) p.part_o[prow * D + lane + 32 * c] = acc[i][c];
                if (lane == 0) {
                    p.part_ml[prow * 2] = m_run[i];
                    p.part_ml[prow * 2 + 1] = l_run[i];
                }
            }
        }
    }
}

// Log-sum-exp merge of the per-split partial results: grid = (R_max rows, KV heads, layers x seqs),
// one thread per channel.
template <typename TO, int D>
__global__ void __launch_bounds__(D) merge_splits_kernel(SimtParams p) {
    const int r = blockIdx.x, h = blockIdx.y, lb = blockIdx.z, c = threadIdx.x;
    const int b = lb % p.batch;
    int M = p.q_lens ? p.q_lens[b] : p.M_max;
    M = min(max(M, 0), p.M_max);
    if (r >= M * p.G) return;
    const int R_max = p.M_max * p.G;
    const size_t base = ((size_t)lb * p.Hkv + h) * p.n_splits;
    float m_all = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s) m_all = fmaxf(m_all, p.part_ml[((base + s) * R_max + r) * 2]);
    float l_all = 0.f, o = 0.f;
    for (int s = 0; s < p.n_splits; ++s) {
        const size_t prow = (base + s) * R_max + r;
        float m_s = p.part_ml[prow * 2];
        if (m_s == -INFINITY) continue;  // an empty split
        float w = expf(m_s - m_all);
        l_all = fmaf(p.part_ml[prow * 2 + 1], w, l_all);
        o = fmaf(p.part_o[prow * D + c], w, o);
    }
    const int j = r / p.G, g = r % p.G;
    const size_t row = ((size_t)lb * p.M_max + j) * p.Hq + h * p.G + g;
    reinterpret_cast<TO*>(p.out)[row * D + c] = from_float<TO>(o / l_all);
    if (p.lse && c == 0) p.lse[row] = m_all + logf(l_all);
}

template <typename T, typename TO, int D>
specpv_status launch_typed(const AttnArgs& a, SimtParams& p, cudaStream_t stream) {
    const size_t smem = (size_t)(kTile * (D + 1) + kTile * D + kRowsPerPass * D) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(attn_simt_kernel<T, TO, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return SPECPV_ERR_CUDA;
    dim3 grid(p.n_splits, a.g.Hkv, a.n_layers * a.batch);
    attn_simt_kernel<T, TO, D><<<grid, kThreads, smem, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    if (p.n_splits > 1) {
        dim3 mgrid(a.M_max * a.g.G, a.g.Hkv, a.n_layers * a.batch);
        merge_splits_kernel<TO, D><<<mgrid, D, 0, stream>>>(p);
        if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
        count_launch();
    }
    return SPECPV_OK;
}

}  // namespace

specpv_status launch_attention_simt(const AttnArgs& a, cudaStream_t stream) {
    SimtParams p{};
    p.q = a.q; p.k_new = a.k_new; p.v_new = a.v_new; p.tree_mask = a.tree_mask; p.q_lens = a.q_lens;
    p.k_pool = a.k_pool; p.v_pool = a.v_pool; p.block_table = a.block_table; p.seq_lens = a.seq_lens;
    p.out = a.out; p.lse = a.lse; p.workspace = a.workspace;
    p.layer0 = a.layer0; p.batch = a.batch; p.M_max = a.M_max; p.mask_words = a.mask_words;
    p.Hq = a.g.Hq; p.Hkv = a.g.Hkv; p.G = a.g.G; p.bs = a.g.bs; p.max_blocks = a.max_blocks; p.n_pages = a.n_pages;
    p.scale = a.g.scale;

    // split the KV range so that the launch has about two CTAs per SM, as far as the workspace allows
    constexpr int kTargetCtas = 2 * 148;
    const int base = a.g.Hkv * a.n_layers * a.batch;
    const int R_max = a.M_max * a.g.G;
    int n_splits = (kTargetCtas + base - 1) / base;
    const int max_by_len = (a.max_seq_len + 255) / 256;
    if (n_splits > max_by_len) n_splits = max_by_len;
    const size_t per_split = (size_t)base * R_max * (a.g.d + 2) * sizeof(float);
    if (n_splits > 1 && per_split * n_splits > a.partial_bytes) n_splits = (int)(a.partial_bytes / per_split);
    if (n_splits < 1) n_splits = 1;
    p.n_splits = n_splits;
    int chunk = (a.max_seq_len + n_splits - 1) / n_splits;
    p.chunk = (chunk + kTile - 1) / kTile * kTile;
    if (p.chunk < kTile) p.chunk = kTile;
    char* ws = reinterpret_cast<char*>(a.workspace) + a.partial_off;
    p.part_o = reinterpret_cast<float*>(ws);
    p.part_ml = reinterpret_cast<float*>(ws + (size_t)base * n_splits * R_max * a.g.d * sizeof(float));

    if (a.g.dtype == SPECPV_DTYPE_F32) {
        if (a.g.d == 64) return launch_typed<float, float, 64>(a, p, stream);
        if (a.g.d == 128) return launch_typed<float, float, 128>(a, p, stream);
    } else if (a.g.out_f32) {
        if (a.g.d == 64) return launch_typed<__nv_bfloat16, float, 64>(a, p, stream);
        if (a.g.d == 128) return launch_typed<__nv_bfloat16, float, 128>(a, p, stream);
    } else {
        if (a.g.d == 64) return launch_typed<__nv_bfloat16, __nv_bfloat16, 64>(a, p, stream);
        if (a.g.d == 128) return launch_typed<__nv_bfloat16, __nv_bfloat16, 128>(a, p, stream);
    }
    return SPECPV_ERR_SHAPE;
}

}  // namespace specpv
