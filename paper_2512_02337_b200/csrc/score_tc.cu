// Block scores on the tensor cores (paper Eq. 2-3): s_i = f_r max(q_r . Kmax_i, q_r . Kmin_i) for
// bfloat16 summaries with head_dim 128, and the channel-wise form s_i = f_r sum_c max(q_rc Kmax_ic, q_rc Kmin_ic).
// Because Kmax >= Kmin in every channel, the channel-wise maximum takes Kmax where q is positive and Kmin where it
// is negative, so that form is the single contraction  Kmax . q+  +  Kmin . q-  with q+ = max(q, 0), q- = min(q, 0)
// (both exact in bfloat16): the CTA splits Q by sign in shared memory and accumulates both products into one
// accumulator.
//
// Per (layer, sequence, KV head) the two products are dense contractions
//     Dmax[128 blocks x R] = Kmax_tile[128 x 128] * Q^T[128 x R],   Dmin likewise with Kmin,
// issued as tcgen05.mma with both operands in shared memory (128-byte swizzle, loaded by TMA) and
// float32 accumulators in tensor memory (Dmax in columns [0, 256), Dmin in [256, 512)).  A CTA owns a
// run of 128-block tiles of one head; thread i of the 128 epilogue threads owns block i of the tile
// (tensor-memory lane i), takes max(Dmax, Dmin) per query row and reduces over the rows (mean, max,
// or the rows of the "last" query).  The summaries of the next tile are in flight while a tile is
// reduced.  Every wait is bounded.
#include "aux_kernels.cuh"
#include "tc_common.cuh"

namespace specpv {

namespace {

using namespace tc;

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

constexpr int kScoreThreads = 192;       // warp 0: TMA + MMA issue, warp 1: idle, warps 2-5: epilogue (lane quarters 2,3,0,1)
constexpr int kTileBlocks = 128;
constexpr int kSumTileBytes = 32768;     // [2 d-halves][128 blocks][64 d] bf16
constexpr int kScoreStages = 2;
constexpr int kScoreQBytes = 65536;      // [2 d-halves][256 rows][64 d] bf16
constexpr int kScoreSmem = 1024 + kScoreQBytes + kScoreStages * 2 * kSumTileBytes;

struct ScoreTcParams {
    CUtensorMap tm_q;     // (d, Hq, tokens)  box (64, G, 128/G)
    CUtensorMap tm_kmax;  // (d, rows)        box (64, 128)
    CUtensorMap tm_kmin;
    const int32_t* q_lens;
    const int32_t* last_query;
    const int32_t* seq_lens;
    float* scores;
    void* workspace;
    int layer0, batch, M_max, Hkv, G, bs, max_blocks, reduce, tiles_per_cta, n_cols;
    int tok0, tok_n;  // this pass covers step tokens [tok0, tok0 + tok_n): 256 query rows at most (the accumulator's columns)
    int accumulate;   // a later pass: combine with the scores the earlier passes left
};

struct __align__(8) ScoreBarriers {
    uint64_t q_full;
    uint64_t sum_full[kScoreStages];
    uint64_t sum_empty[kScoreStages];
    uint64_t d_full;
    uint64_t d_empty;
    uint64_t q_split;  // channel-wise form: the epilogue warps have split Q by sign
    uint32_t tmem_base;
    int abort_flag;
};

// kCw: the channel-wise form (a compile-time switch, so that the printed form's code is exactly what it was).
template <bool kCw>
__global__ void __launch_bounds__(kScoreThreads, 1) scores_tc_kernel(const __grid_constant__ ScoreTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ ScoreBarriers bars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y, lb = blockIdx.z;
    const int b = lb % p.batch, l = lb / p.batch;
    const int seq_len = max(p.seq_lens[b], 0);
    const int nb = min((seq_len + p.bs - 1) / p.bs, p.max_blocks);
    const int tile_begin = blockIdx.x * p.tiles_per_cta;
    const int tile_end = min(tile_begin + p.tiles_per_cta, (nb + kTileBlocks - 1) / kTileBlocks);
    if (tile_begin >= tile_end) return;
    const int n_tiles = tile_end - tile_begin;
    int M = p.q_lens ? p.q_lens[b] : p.M_max;
    M = min(max(M, 0), p.M_max);
    // query rows r = token * G + head of this pass's tokens, one accumulator column each
    int col_begin = 0, col_end = min(max(M - p.tok0, 0), p.tok_n) * p.G;
    int denom = M * p.G;  // rows the mean runs over (all passes together)
    if (p.reduce == SPECPV_REDUCE_LAST) {
        int last = p.last_query ? p.last_query[b] : 0;
        last = min(max(last, 0), max(M - 1, 0));
        if (M <= 0 || last < p.tok0 || last >= p.tok0 + p.tok_n) return;  // another pass holds that row
        col_begin = (last - p.tok0) * p.G;
        col_end = col_begin + p.G;
        denom = p.G;
    }
    if (col_end <= col_begin) return;
    const bool combine = p.accumulate && p.reduce != SPECPV_REDUCE_LAST;

    const uint32_t q_smem = smem_u32(smem);
    // channel-wise form: q- takes the place of the second summary stage, the summaries go through a single stage
    constexpr int stages = kCw ? 1 : kScoreStages;
    const uint32_t qneg_smem = q_smem + kScoreQBytes;
    const uint32_t sum_smem = q_smem + (kCw ? 2 : 1) * kScoreQBytes;
    volatile int* abort_flag = &bars.abort_flag;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.q_full), 1);
        for (int s = 0; s < kScoreStages; ++s) {
            mbar_init(smem_u32(&bars.sum_full[s]), 1);
            mbar_init(smem_u32(&bars.sum_empty[s]), 1);
        }
        mbar_init(smem_u32(&bars.d_full), 1);
        mbar_init(smem_u32(&bars.d_empty), 4);  // one arrival per epilogue warp
        mbar_init(smem_u32(&bars.q_split), 4);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&bars.tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;
    const int tok_per_tile = 128 / p.G;
    const uint32_t idesc = make_idesc((uint32_t)p.n_cols, false);

    if (warp == 0) {
        // ---- producer + MMA issue: the whole warp runs the loop (a lone lane of a diverged warp runs
        // slowly), lane 0 issues ----------------------------------------------------------------------
        const uint32_t qbar = smem_u32(&bars.q_full);
        const int n_q_tiles = p.n_cols > 128 ? 2 : 1;
        const int row0 = (((p.layer0 + l) * p.batch + b) * p.Hkv + h) * p.max_blocks;
        auto load_tile = [&](int i) {  // lane 0 only
            const int slot = i % stages;
            const uint32_t full = smem_u32(&bars.sum_full[slot]);
            mbar_expect_tx(full, 2 * kSumTileBytes);
            const uint32_t dst = sum_smem + slot * 2 * kSumTileBytes;
            const int row = row0 + (tile_begin + i) * kTileBlocks;
            for (int half = 0; half < 2; ++half) {
                tma_load_2d(dst + half * 16384, &p.tm_kmax, half * 64, row, full);
                tma_load_2d(dst + kSumTileBytes + half * 16384, &p.tm_kmin, half * 64, row, full);
            }
        };
        if (lane == 0) {
            mbar_expect_tx(qbar, (uint32_t)(n_q_tiles * 32768));
            for (int t = 0; t < n_q_tiles; ++t)
                for (int half = 0; half < 2; ++half)
                    tma_load_3d(q_smem + half * 32768 + t * 16384, &p.tm_q, half * 64, h * p.G,
                                lb * p.M_max + p.tok0 + t * tok_per_tile, qbar);
            load_tile(0);
        }
        __syncwarp();
        // descriptors: constant upper word (8-row group stride 1024 B, version, 128-byte swizzle); lower word =
        // 16-byte address, leading offset 16 B
        const uint32_t desc_hi = (uint32_t)((1024u >> 4) | (1u << 14) | (2u << 29));
        const uint32_t q_lo = ((q_smem >> 4) & 0x3FFFu) | (1u << 16);
        const uint32_t sum_lo = ((sum_smem >> 4) & 0x3FFFu) | (1u << 16);
        const uint32_t qneg_lo = ((qneg_smem >> 4) & 0x3FFFu) | (1u << 16);
        bool ok = mbar_wait(qbar, 0, abort_flag, p.workspace, 20);
        if (kCw) ok &= mbar_wait(smem_u32(&bars.q_split), 0, abort_flag, p.workspace, 25);
        for (int i = 0; i < n_tiles; ++i) {
            if (stages > 1 && i + 1 < n_tiles) {  // the next tile goes into the other stage while this one is used
                const int use = i + 1;
                if (use >= stages)
                    ok &= mbar_wait(smem_u32(&bars.sum_empty[use % stages]), ((use / stages) - 1) & 1,
                                    abort_flag, p.workspace, 21);
                if (lane == 0 && ok) load_tile(use);
                __syncwarp();
            }
            const int slot = i % stages;
            ok &= mbar_wait(smem_u32(&bars.sum_full[slot]), (i / stages) & 1, abort_flag, p.workspace, 22);
            if (i > 0) ok &= mbar_wait(smem_u32(&bars.d_empty), (i - 1) & 1, abort_flag, p.workspace, 23);
            if (!ok) break;  // a wait gave up: nothing more is copied or issued
            tc_fence_after();
            if (lane == 0) {
                const uint32_t a_max = sum_lo + (uint32_t)slot * (2 * kSumTileBytes >> 4), a_min = a_max + (kSumTileBytes >> 4);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t a_off = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    const uint32_t b_off = (uint32_t)((kk >> 2) * 32768 + (kk & 3) * 32) >> 4;
                    const uint64_t bdesc = ((uint64_t)desc_hi << 32) | (q_lo + b_off);
                    mma_ss(tmem, ((uint64_t)desc_hi << 32) | (a_max + a_off), bdesc, idesc, kk > 0);
                    // channel-wise: Kmin . q- joins Kmax . q+ in the same accumulator
                    if (kCw)
                        mma_ss(tmem, ((uint64_t)desc_hi << 32) | (a_min + a_off), ((uint64_t)desc_hi << 32) | (qneg_lo + b_off),
                               idesc, 1);
                    else
                        mma_ss(tmem + 256, ((uint64_t)desc_hi << 32) | (a_min + a_off), bdesc, idesc, kk > 0);
                }
                tc_commit(smem_u32(&bars.d_full));
                tc_commit(smem_u32(&bars.sum_empty[slot]));
            }
            __syncwarp();
            if (stages == 1 && i + 1 < n_tiles) {
                // a single stage: the next tile can only follow the contractions just issued (their completion is
                // release number i of the stage); it still overlaps this tile's reduction
                ok &= mbar_wait(smem_u32(&bars.sum_empty[0]), i & 1, abort_flag, p.workspace, 21);
                if (lane == 0 && ok) load_tile(i + 1);
                __syncwarp();
            }
        }
        (void)ok;
    } else if (warp >= 2) {
        // ---- epilogue: thread <-> block of the tile -----------------------------------------------
        const int q = warp & 3;  // tensor-memory lane quarter of this warp
        const int blk_in_tile = q * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        bool ok = true;
        if (kCw) {
            // split Q by sign in place: q+ stays where Q landed, q- goes to the buffer behind it (same swizzled layout,
            // the split is element-wise).  A bfloat16 is negative when its top bit is set.
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.q_full), 0, abort_flag, p.workspace, 26));
            uint4* qp = reinterpret_cast<uint4*>(smem);
            uint4* qn = reinterpret_cast<uint4*>(smem + kScoreQBytes);
            for (int v = threadIdx.x - 64; v < kScoreQBytes / 16; v += 128) {
                const uint4 w = qp[v];
                const uint32_t in[4] = {w.x, w.y, w.z, w.w};
                uint32_t pos[4], neg[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t m = ((in[e] >> 15) & 0x00010001u) * 0xFFFFu;  // all ones in the negative halves
                    neg[e] = in[e] & m;
                    pos[e] = in[e] & ~m;
                }
                qp[v] = make_uint4(pos[0], pos[1], pos[2], pos[3]);
                qn[v] = make_uint4(neg[0], neg[1], neg[2], neg[3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the tensor pipe reads these through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.q_split));
        }
        for (int i = 0; i < n_tiles && ok; ++i) {
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.d_full), i & 1, abort_flag, p.workspace, 24));
            if (!ok) break;
            tc_fence_after();
            // four independent partial reductions: a single chain through one register would leave this
            // warp, alone on its scheduler, waiting out the latency of every instruction
            const bool is_max = p.reduce == SPECPV_REDUCE_MAX;
            float r4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) r4[e] = is_max ? -INFINITY : 0.f;
            for (int c0 = (col_begin / 64) * 64; c0 < col_end; c0 += 64) {
                uint32_t vmax[64], vmin[64];
                TMEM_LD32(tmem + lane_addr + c0, vmax);
                TMEM_LD32(tmem + lane_addr + c0 + 32, (vmax + 32));
                if (!kCw) {
                    TMEM_LD32(tmem + lane_addr + 256 + c0, vmin);
                    TMEM_LD32(tmem + lane_addr + 256 + c0 + 32, (vmin + 32));
                }
                tmem_wait_ld();
                if (kCw) {  // one accumulator already holds the score: max(x, x) = x below
#pragma unroll
                    for (int k = 0; k < 64; ++k) vmin[k] = vmax[k];
                }
                const bool whole = c0 >= col_begin && c0 + 64 <= col_end;  // warp-uniform
                if (whole && !is_max) {
#pragma unroll
                    for (int k = 0; k < 64; ++k)
                        r4[k & 3] += fmaxf(__uint_as_float(vmax[k]), __uint_as_float(vmin[k]));
                } else if (whole) {
#pragma unroll
                    for (int k = 0; k < 64; ++k)
                        r4[k & 3] = fmax3(r4[k & 3], __uint_as_float(vmax[k]), __uint_as_float(vmin[k]));
                } else {
#pragma unroll
                    for (int k = 0; k < 64; ++k) {
                        const int c = c0 + k;
                        const float sc = fmaxf(__uint_as_float(vmax[k]), __uint_as_float(vmin[k]));
                        if (c >= col_begin && c < col_end) r4[k & 3] = is_max ? fmaxf(r4[k & 3], sc) : r4[k & 3] + sc;
                    }
                }
            }
            float red = is_max ? fmaxf(fmaxf(r4[0], r4[1]), fmaxf(r4[2], r4[3])) : (r4[0] + r4[1]) + (r4[2] + r4[3]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.d_empty));
            const int blk = (tile_begin + i) * kTileBlocks + blk_in_tile;
            if (blk < nb) {
                float* dst = p.scores + ((size_t)lb * p.Hkv + h) * p.max_blocks + blk;
                if (p.reduce != SPECPV_REDUCE_MAX) red /= (float)denom;
                if (combine) red = is_max ? fmaxf(red, *dst) : red + *dst;
                *dst = red;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // after a give-up nothing new was issued; the few copies and contractions in flight end within microseconds
        if (*abort_flag) __nanosleep(1000000);
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

}  // namespace

bool scores_tc_supported(int dtype, int d, int G, int M_max) {
    return dtype == SPECPV_DTYPE_BF16 && d == 128 && G <= 128 && (128 % G) == 0 && M_max * G <= 4 * 256 &&
           tc::get_encode_fn() != nullptr;
}

specpv_status launch_scores_tc(const ScoreParams& sp, int n_layers_call, int n_layers_total, int max_nb,
                               cudaStream_t stream) {
    if (!tc::set_smem_limit_once(reinterpret_cast<const void*>(scores_tc_kernel<false>), kScoreSmem) ||
        !tc::set_smem_limit_once(reinterpret_cast<const void*>(scores_tc_kernel<true>), kScoreSmem))
        return SPECPV_ERR_CUDA;
    if (max_nb <= 0 || n_layers_call <= 0) return SPECPV_OK;
    ScoreTcParams p{};
    const uint64_t step_tokens = (uint64_t)n_layers_call * sp.batch * sp.M_max;
    {
        uint64_t dims[3] = {128, (uint64_t)sp.Hq, step_tokens};
        uint64_t strides[2] = {256, (uint64_t)sp.Hq * 256};
        uint32_t box[3] = {64, (uint32_t)sp.G, (uint32_t)(128 / sp.G)};
        if (!tc::encode_map(&p.tm_q, sp.q, 3, dims, strides, box)) return SPECPV_ERR_CUDA;
    }
    {
        uint64_t dims[2] = {128, (uint64_t)n_layers_total * sp.batch * sp.Hkv * sp.max_blocks};
        if (dims[1] >= 0x7FFFFF00ull) return SPECPV_ERR_UNSUPPORTED;
        uint64_t strides[1] = {256};
        uint32_t box[2] = {64, 128};
        if (!tc::encode_map(&p.tm_kmax, sp.kmax, 2, dims, strides, box)) return SPECPV_ERR_CUDA;
        if (!tc::encode_map(&p.tm_kmin, sp.kmin, 2, dims, strides, box)) return SPECPV_ERR_CUDA;
    }
    p.q_lens = sp.q_lens; p.last_query = sp.last_query; p.seq_lens = sp.seq_lens; p.scores = sp.scores;
    p.workspace = sp.workspace;
    p.layer0 = sp.layer0; p.batch = sp.batch; p.M_max = sp.M_max; p.Hkv = sp.Hkv; p.G = sp.G; p.bs = sp.bs;
    p.max_blocks = sp.max_blocks; p.reduce = sp.reduce;
    const int n_tiles = (max_nb + kTileBlocks - 1) / kTileBlocks;
    const int heads = sp.Hkv * n_layers_call * sp.batch;
    // enough CTAs to fill the machine, but at least a few tiles each so that Q is amortised
    int ctas_x = (2 * 148 + heads - 1) / heads;
    if (ctas_x > n_tiles) ctas_x = n_tiles;
    if (ctas_x < 1) ctas_x = 1;
    p.tiles_per_cta = (n_tiles + ctas_x - 1) / ctas_x;
    ctas_x = (n_tiles + p.tiles_per_cta - 1) / p.tiles_per_cta;
    dim3 grid(ctas_x, sp.Hkv, n_layers_call * sp.batch);
    // The accumulator holds 256 query rows; a step with more (the chain and the tree of a refresh) goes through in
    // passes over the step's tokens, each later pass combining with what is there (sum of per-pass means, or max).
    const int tok_per_pass = 256 / sp.G;
    for (int tok0 = 0; tok0 < sp.M_max; tok0 += tok_per_pass) {
        p.tok0 = tok0;
        p.tok_n = sp.M_max - tok0 < tok_per_pass ? sp.M_max - tok0 : tok_per_pass;
        p.accumulate = tok0 > 0;
        p.n_cols = p.tok_n * sp.G <= 128 ? 128 : 256;  // accumulator columns, padded to whole 128-row Q tiles
        if (sp.score_mode == 1)
            scores_tc_kernel<true><<<grid, kScoreThreads, kScoreSmem, stream>>>(p);
        else
            scores_tc_kernel<false><<<grid, kScoreThreads, kScoreSmem, stream>>>(p);
        if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
        count_launch();
    }
    return SPECPV_OK;
}

}  // namespace specpv
