// The linear maps either side of the verification attention (Algorithm 1 "TreeDecode"; Section 3.3:
// the refresh pass computes key-value states of the partially verified and the candidate tokens):
//     [q | k | v] = x Wqkv^T  with a rotary position embedding on q and k,      y = attn Wo^T (+ residual).
//
// A step has few rows (a draft tree of some tens of tokens), so both maps stream their weights once and
// are bound by HBM.  The weights are therefore the M operand of the tensor-core contraction,
//     D[128 out features x tokens] += W_tile[128 x 64] * X_tile[tokens x 64]^T     (tcgen05.mma, kind::f16),
// both operands K-major in shared memory (128-byte swizzle, loaded by TMA through a ring of stages), the
// float32 accumulator in tensor memory.  A CTA owns one 128-feature tile (one head of the QKV map) and a
// range of the input features; with several ranges per tile (few tiles, one layer) the partial sums go to
// the workspace and a second kernel adds them in a fixed order.  The epilogue turns the accumulator
// through shared memory so that a thread holds channels (2j, 2j+1) and their rotary partners
// (64+2j, 64+2j+1) of one row, rotates, adds the residual and writes bfloat16.  Every wait is bounded.
#include "proj.cuh"
#include "tc_common.cuh"

namespace specpv {

namespace {

using namespace tc;

constexpr int kProjThreads = 192;          // warp 0: TMA producer, warp 1: MMA issue + tensor memory, warps 2-5: epilogue
constexpr int kFeatTile = 128;             // output features per CTA
constexpr int kWTileBytes = kFeatTile * 128;  // 128 features x 64 input features, bfloat16
constexpr int kProjDataBytes = 192 * 1024;
constexpr int kProjSmem = 1024 + kProjDataBytes;
constexpr int kProjMaxStages = 8;
constexpr int kIssueGroup = 2;             // stages whose copies are issued together
constexpr int kMaxTokTile = 256;           // rows per CTA (accumulator columns)

struct ProjTcParams {
    CUtensorMap tm_w;  // (n_in, n_layers_total * n_out)  box (64, 128)
    CUtensorMap tm_x;  // (n_in, n_layers_call * tokens)  box (64, n_pad)
    const float* cos_sin;
    const __nv_bfloat16* residual;
    float* partials;
    void* workspace;
    ProjSegment seg[3];
    int n_seg, layer0, n_tiles, n_out, tokens, n_pad, ksteps, splits, stages, group;
};

struct __align__(8) ProjBarriers {
    uint64_t full[kProjMaxStages];
    uint64_t empty[kProjMaxStages];
    uint64_t d_full;
    uint32_t tmem_base;
    int abort_flag;
};

// Channels (2j, 2j+1) = lo and (64+2j, 64+2j+1) = hi of feature tile `tile`, row `tok` of layer-in-call `l`.
__device__ __forceinline__ void proj_finish(const ProjTcParams& p, int tile, int l, int tok, int j, float2 lo, float2 hi) {
    int s = 0;
    for (int i = 1; i < p.n_seg; ++i)
        if (tile >= p.seg[i].first_tile) s = i;
    const ProjSegment& sg = p.seg[s];
    if (sg.rope) {
        const float4 cs = __ldg(reinterpret_cast<const float4*>(p.cos_sin + ((size_t)tok * 64 + 2 * j) * 2));  // cos, sin, cos, sin
        const float2 rl = make_float2(lo.x * cs.x - hi.x * cs.y, lo.y * cs.z - hi.y * cs.w);
        const float2 rh = make_float2(hi.x * cs.x + lo.x * cs.y, hi.y * cs.z + lo.y * cs.w);
        lo = rl;
        hi = rh;
    }
    const size_t off = ((size_t)l * p.tokens + tok) * sg.row_stride + (size_t)(tile - sg.first_tile) * kFeatTile + 2 * j;
    if (p.residual && s == 0) {
        const uint32_t a = __ldg(reinterpret_cast<const uint32_t*>(p.residual + off));
        const uint32_t b = __ldg(reinterpret_cast<const uint32_t*>(p.residual + off + 64));
        lo.x += __uint_as_float(a << 16); lo.y += __uint_as_float(a & 0xFFFF0000u);
        hi.x += __uint_as_float(b << 16); hi.y += __uint_as_float(b & 0xFFFF0000u);
    }
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(sg.base) + off;
    *reinterpret_cast<uint32_t*>(dst) = pack_bf16(lo.x, lo.y);
    *reinterpret_cast<uint32_t*>(dst + 64) = pack_bf16(hi.x, hi.y);
}

__device__ __forceinline__ size_t partial_base(const ProjTcParams& p, int l, int chunk, int n_chunks, int tile, int split) {
    const size_t unit = ((size_t)l * n_chunks + chunk) * p.n_tiles + tile;
    return (unit * p.splits + split) * (size_t)p.n_pad * kFeatTile;
}

__global__ void __launch_bounds__(kProjThreads, 2) proj_tc_kernel(const __grid_constant__ ProjTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ ProjBarriers bars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x / p.splits, split = blockIdx.x % p.splits;
    const int chunk = blockIdx.y, l = blockIdx.z;
    const int tok0 = chunk * kMaxTokTile;
    const int valid = min(p.n_pad, p.tokens - tok0);
    const int kb = (int)((long long)split * p.ksteps / p.splits);
    const int ke = (int)((long long)(split + 1) * p.ksteps / p.splits);
    const int n_k = ke - kb;
    const uint32_t data = smem_u32(smem);
    const uint32_t stage_bytes = (uint32_t)(kWTileBytes + p.n_pad * 128);
    volatile int* abort_flag = &bars.abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        mbar_init(smem_u32(&bars.d_full), 1);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&bars.tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;

    if (warp == 0) {
        // ---- producer: the whole warp walks the ring, lane 0 issues the copies ----------------------------
        const int w_row = (p.layer0 + l) * p.n_out + tile * kFeatTile;
        const int x_row = l * p.tokens + tok0;
        bool ok = true;
        // The copies of p.group consecutive stages are issued together: a weight row is 128 contiguous bytes
        // per stage, and DRAM serves the same row's neighbouring chunks far better when they are asked for at
        // nearly the same time than one stage apart.
        for (int i0 = 0; i0 < n_k; i0 += p.group) {
            const int i1 = min(i0 + p.group, n_k);
            for (int i = i0; i < i1; ++i)
                if (i >= p.stages)
                    ok &= mbar_wait(smem_u32(&bars.empty[i % p.stages]), ((i / p.stages) - 1) & 1, abort_flag, p.workspace, 30);
            if (!ok) break;  // a wait gave up: nothing more is copied
            if (lane == 0) {
                for (int i = i0; i < i1; ++i) {
                    const int slot = i % p.stages;
                    const uint32_t full = smem_u32(&bars.full[slot]);
                    const uint32_t dst = data + slot * stage_bytes;
                    mbar_expect_tx(full, stage_bytes);
                    tma_load_2d(dst, &p.tm_w, (kb + i) * 64, w_row, full);
                    tma_load_2d(dst + kWTileBytes, &p.tm_x, (kb + i) * 64, x_row, full);
                }
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ---- MMA issue --------------------------------------------------------------------------------------
        const uint32_t idesc = make_idesc((uint32_t)p.n_pad, false);
        const uint32_t desc_hi = (uint32_t)((1024u >> 4) | (1u << 14) | (2u << 29));
        bool ok = true;
        for (int i = 0; i < n_k; ++i) {
            const int slot = i % p.stages;
            ok &= mbar_wait(smem_u32(&bars.full[slot]), (i / p.stages) & 1, abort_flag, p.workspace, 31);
            if (!ok) break;  // a wait gave up: nothing more is issued
            tc_fence_after();
            if (lane == 0) {
                const uint32_t a_lo = (((data + slot * stage_bytes) >> 4) & 0x3FFFu) | (1u << 16);
                const uint32_t b_lo = (((data + slot * stage_bytes + kWTileBytes) >> 4) & 0x3FFFu) | (1u << 16);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss(tmem, ((uint64_t)desc_hi << 32) | (a_lo + kk * 2), ((uint64_t)desc_hi << 32) | (b_lo + kk * 2),
                           idesc, (i | kk) != 0);
                tc_commit(smem_u32(&bars.empty[slot]));
                if (i == n_k - 1) tc_commit(smem_u32(&bars.d_full));
            }
            __syncwarp();
        }
    } else {
        // ---- epilogue: thread <-> output feature (tensor-memory lane), then thread <-> (row, channel pairs) ---
        const int q = warp & 3;
        const int f = q * 32 + lane;
        const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.d_full), 0, abort_flag, p.workspace, 32));
        tc_fence_after();
        float* stage = reinterpret_cast<float*>(smem);  // [n_pad][128]; every copy into the ring has been consumed
        if (ok) {
            for (int c0 = 0; c0 < p.n_pad; c0 += 32) {
                uint32_t v[32];
                TMEM_LD32(tmem + ((uint32_t)(q * 32) << 16) + c0, v);
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 32; ++k) stage[(c0 + k) * kFeatTile + f] = __uint_as_float(v[k]);
            }
        }
        tc_fence_before();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ok) {
            const int et = threadIdx.x - 64, j = et & 31;
            float* part = p.splits > 1 ? p.partials + partial_base(p, l, chunk, gridDim.y, tile, split) : nullptr;
#pragma unroll 4
            for (int t = et >> 5; t < valid; t += 4) {
                const float2 lo = *reinterpret_cast<const float2*>(stage + t * kFeatTile + 2 * j);
                const float2 hi = *reinterpret_cast<const float2*>(stage + t * kFeatTile + 64 + 2 * j);
                if (part) {
                    *reinterpret_cast<float2*>(part + (size_t)t * kFeatTile + 2 * j) = lo;
                    *reinterpret_cast<float2*>(part + (size_t)t * kFeatTile + 64 + 2 * j) = hi;
                } else {
                    proj_finish(p, tile, l, tok0 + t, j, lo, hi);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // after a give-up nothing new was issued; the few copies and contractions in flight end within microseconds
        if (*abort_flag) __nanosleep(1000000);
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
    }
}

// Adds the partial sums of a tile's input-feature ranges in range order and finishes the rows: a CTA takes four rows
// of one tile, a thread one row's channels (2j, 2j+1, 64+2j, 64+2j+1), so that all its loads are in flight together.
__global__ void __launch_bounds__(128) proj_reduce_kernel(const __grid_constant__ ProjTcParams p, int n_chunks) {
    const int tile = blockIdx.x, l = blockIdx.z / n_chunks, chunk = blockIdx.z % n_chunks;
    const int tok0 = chunk * kMaxTokTile;
    const int valid = min(p.n_pad, p.tokens - tok0);
    const int j = threadIdx.x & 31, t = blockIdx.y * 4 + (threadIdx.x >> 5);
    if (t >= valid) return;
    const float* part = p.partials + partial_base(p, l, chunk, n_chunks, tile, 0) + (size_t)t * kFeatTile + 2 * j;
    const size_t split_stride = (size_t)p.n_pad * kFeatTile;
    float2 a[8], b[8];
#pragma unroll
    for (int s = 0; s < 8; ++s)
        if (s < p.splits) {
            a[s] = __ldg(reinterpret_cast<const float2*>(part + s * split_stride));
            b[s] = __ldg(reinterpret_cast<const float2*>(part + s * split_stride + 64));
        }
    float2 lo = make_float2(0.f, 0.f), hi = lo;
#pragma unroll
    for (int s = 0; s < 8; ++s)
        if (s < p.splits) {
            lo.x += a[s].x; lo.y += a[s].y; hi.x += b[s].x; hi.y += b[s].y;
        }
    proj_finish(p, tile, l, tok0 + t, j, lo, hi);
}

// ---- plain kernel: any dtype / head size ---------------------------------------------------------------------
struct ProjSimtParams {
    const void* x;
    const void* w;
    const float* cos_sin;
    const void* residual;
    ProjSegment seg[3];
    int n_seg, layer0, n_out, n_in, tokens, tile;
};

template <typename T>
__global__ void __launch_bounds__(128) proj_simt_kernel(const __grid_constant__ ProjSimtParams p) {
    extern __shared__ float vals[];  // one output tile of one row
    const int tok = blockIdx.x, tile = blockIdx.y, l = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T* xr = reinterpret_cast<const T*>(p.x) + ((size_t)l * p.tokens + tok) * p.n_in;
    const T* wt = reinterpret_cast<const T*>(p.w) + ((size_t)(p.layer0 + l) * p.n_out + (size_t)tile * p.tile) * p.n_in;
    for (int f = warp; f < p.tile; f += 4) {
        const T* wr = wt + (size_t)f * p.n_in;
        float acc = 0.f;
        for (int c = lane; c < p.n_in; c += 32) acc = fmaf(to_float<T>(xr[c]), to_float<T>(wr[c]), acc);
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) vals[f] = acc;
    }
    __syncthreads();
    int s = 0;
    for (int i = 1; i < p.n_seg; ++i)
        if (tile >= p.seg[i].first_tile) s = i;
    const ProjSegment& sg = p.seg[s];
    const int half = p.tile / 2;
    const size_t off = ((size_t)l * p.tokens + tok) * sg.row_stride + (size_t)(tile - sg.first_tile) * p.tile;
    T* dst = reinterpret_cast<T*>(sg.base) + off;
    const T* res = (p.residual && s == 0) ? reinterpret_cast<const T*>(p.residual) + off : nullptr;
    for (int c = threadIdx.x; c < half; c += blockDim.x) {
        float lo = vals[c], hi = vals[c + half];
        if (sg.rope) {
            const float2 cs = *reinterpret_cast<const float2*>(p.cos_sin + ((size_t)tok * half + c) * 2);
            const float rl = lo * cs.x - hi * cs.y, rh = hi * cs.x + lo * cs.y;
            lo = rl;
            hi = rh;
        }
        if (res) {
            lo += to_float<T>(res[c]);
            hi += to_float<T>(res[c + half]);
        }
        dst[c] = from_float<T>(lo);
        dst[c + half] = from_float<T>(hi);
    }
}

// ---- positions and rotary angles of a step's rows ------------------------------------------------------------
__global__ void rope_table_kernel(const uint64_t* __restrict__ tree_mask, const int32_t* __restrict__ q_lens,
                                  const int32_t* __restrict__ base_pos, int M_max, int d, double theta,
                                  float* __restrict__ cos_sin) {
    const int row = blockIdx.x, b = row / M_max, j = row % M_max;
    const int W = (M_max + 63) / 64, half = d / 2;
    int M = q_lens ? q_lens[b] : M_max;
    M = min(max(M, 0), M_max);
    int seen = 0;
    if (j < M)
        for (int w = 0; w < W; ++w) seen += __popcll(tree_mask[(size_t)row * W + w]);
    const double pos = (double)base_pos[b] + (double)max(seen - 1, 0);
    for (int c = threadIdx.x; c < half; c += blockDim.x) {
        const double angle = pos * pow(theta, -2.0 * (double)c / (double)d);
        double sn, cs;
        sincos(angle, &sn, &cs);
        reinterpret_cast<float2*>(cos_sin)[(size_t)row * half + c] = make_float2((float)cs, (float)sn);
    }
}

}  // namespace

bool proj_tc_supported(const ProjArgs& a) {
    return a.dtype == SPECPV_DTYPE_BF16 && a.tile == kFeatTile && a.n_in % 64 == 0 && a.n_in >= 64 &&
           a.n_out % kFeatTile == 0 && (uint64_t)a.n_layers_total * a.n_out < 0x7FFFFF00ull &&
           (uint64_t)a.n_layers_call * a.tokens < 0x7FFFFF00ull && tc::get_encode_fn() != nullptr;
}

specpv_status launch_proj_tc(const ProjArgs& a, cudaStream_t stream) {
    if (!tc::set_smem_limit_once(reinterpret_cast<const void*>(proj_tc_kernel), kProjSmem)) return SPECPV_ERR_CUDA;
    if (a.tokens <= 0 || a.n_layers_call <= 0) return SPECPV_OK;
    ProjTcParams p{};
    p.n_pad = a.tokens >= kMaxTokTile ? kMaxTokTile : (a.tokens + 31) / 32 * 32;
    const int n_chunks = (a.tokens + kMaxTokTile - 1) / kMaxTokTile;
    {
        uint64_t dims[2] = {(uint64_t)a.n_in, (uint64_t)a.n_layers_total * a.n_out};
        uint64_t strides[1] = {(uint64_t)a.n_in * 2};
        uint32_t box[2] = {64, (uint32_t)kFeatTile};
        if (!tc::encode_map(&p.tm_w, a.w, 2, dims, strides, box)) return SPECPV_ERR_CUDA;
    }
    {
        uint64_t dims[2] = {(uint64_t)a.n_in, (uint64_t)a.n_layers_call * a.tokens};
        uint64_t strides[1] = {(uint64_t)a.n_in * 2};
        uint32_t box[2] = {64, (uint32_t)p.n_pad};
        if (!tc::encode_map(&p.tm_x, a.x, 2, dims, strides, box)) return SPECPV_ERR_CUDA;
    }
    p.cos_sin = a.cos_sin;
    p.residual = reinterpret_cast<const __nv_bfloat16*>(a.residual);
    p.workspace = a.workspace;
    p.n_seg = a.n_seg;
    for (int i = 0; i < a.n_seg; ++i) p.seg[i] = a.seg[i];
    p.layer0 = a.layer0; p.n_tiles = a.n_out / kFeatTile; p.n_out = a.n_out; p.tokens = a.tokens;
    p.ksteps = a.n_in / 64;
    const int stage_bytes = kWTileBytes + p.n_pad * 128;
    // up to 128 rows the ring and the epilogue's staging tile fit in half the shared memory, and two CTAs per SM
    // cover each other's start and epilogue
    const bool small_ring = p.n_pad <= 128;
    const int ring_bytes = small_ring ? kProjDataBytes / 2 : kProjDataBytes;
    p.stages = ring_bytes / stage_bytes;
    if (p.stages > kProjMaxStages) p.stages = kProjMaxStages;
    p.group = kIssueGroup <= p.stages / 2 ? kIssueGroup : (p.stages / 2 > 0 ? p.stages / 2 : 1);
    // enough CTAs to fill every SM's slots: split the input features while the tiles alone cannot
    const long long units = (long long)a.n_layers_call * n_chunks * p.n_tiles;
    const int slots = small_ring ? 2 * 148 : 148;
    int splits = 1;
    if (units < 120) {
        splits = (int)(slots / units);
        if (splits > 8) splits = 8;
        if (splits > p.ksteps) splits = p.ksteps;
        const size_t per_split = (size_t)units * p.n_pad * kFeatTile * sizeof(float);
        while (splits > 1 && per_split * splits > a.scratch_bytes) --splits;
    }
    p.splits = splits;
    p.partials = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(a.workspace) + a.scratch_off);
    dim3 grid(p.n_tiles * splits, n_chunks, a.n_layers_call);
    proj_tc_kernel<<<grid, kProjThreads, 1024 + ring_bytes, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    if (splits > 1) {
        proj_reduce_kernel<<<dim3(p.n_tiles, (p.n_pad + 3) / 4, a.n_layers_call * n_chunks), 128, 0, stream>>>(p, n_chunks);
        if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
        count_launch();
    }
    return SPECPV_OK;
}

specpv_status launch_proj_simt(const ProjArgs& a, cudaStream_t stream) {
    if (a.tokens <= 0 || a.n_layers_call <= 0) return SPECPV_OK;
    ProjSimtParams p{};
    p.x = a.x; p.w = a.w; p.cos_sin = a.cos_sin; p.residual = a.residual;
    p.n_seg = a.n_seg;
    for (int i = 0; i < a.n_seg; ++i) p.seg[i] = a.seg[i];
    p.layer0 = a.layer0; p.n_out = a.n_out; p.n_in = a.n_in; p.tokens = a.tokens; p.tile = a.tile;
    dim3 grid(a.tokens, a.n_out / a.tile, a.n_layers_call);
    const size_t smem = (size_t)a.tile * sizeof(float);
    if (a.dtype == SPECPV_DTYPE_F32)
        proj_simt_kernel<float><<<grid, 128, smem, stream>>>(p);
    else
        proj_simt_kernel<__nv_bfloat16><<<grid, 128, smem, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    return SPECPV_OK;
}

specpv_status launch_rope_table(const uint64_t* tree_mask, const int32_t* q_lens, const int32_t* base_pos, int batch,
                                int M_max, int d, double theta, float* cos_sin, cudaStream_t stream) {
    rope_table_kernel<<<batch * M_max, 64, 0, stream>>>(tree_mask, q_lens, base_pos, M_max, d, theta, cos_sin);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    return SPECPV_OK;
}

}  // namespace specpv
