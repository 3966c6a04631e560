// Tensor-core verification attention on CTA pairs (B200, sm_100a): bfloat16, head_dim 128, pages of 16, 32 or 64
// tokens, more than 128 query rows per KV head.  Tree-masked GQA attention of the step's tokens over a paged cache
// (paper Section 3.2-3.3, Algorithm 1 "TreeDecode"), for both the partial and the full cache.
//
// A cluster of two CTAs owns one (layer, sequence, KV head, KV split, group of 256 rows).  Each CTA holds one
// 128-row tile of the group (row = step token * G + query head) and HALF of every 128-token K/V tile: the 64 tokens
// of K it contributes to S = Q K^T and the 64 channels of V it contributes to O += P V.  The contractions are
// pair-wide tcgen05.mma (cta_group::2, M = 256), issued by one thread of the even CTA, which read both CTAs'
// shared memory, so a K/V byte is fetched from HBM once and read from shared memory once per pair.
//
// S lives in one of THREE tensor-memory buffers (tile mod 3) and P(j) overwrites the first half of S(j)'s own
// buffer, so the softmax warps never wait for a buffer: the buffer of tile j is theirs from the completion of
// QK(j) until they hand P(j) over; QK(j+3) reuses it once PV(j) has completed.
// Issuing one tcgen05.mma costs its thread 55-60 cycles whatever the shape, against 64 cycles of execution for
// 128x128x16 per SM, and the tensor pipe queues next to nothing ahead: one issuing thread that also waits and
// commits cannot keep the pipe busy (measured: 84-98 cycles per instruction, 65 with two issuing warps).  So the
// two streams have a warp each, ordered against one another by commit barriers only.
//   warp 0      TMA producer (both CTAs): its Q tile per stretch, then per tile its halves of K (ring of 5) and of V
//               (ring of 5, three tiles behind) through the block table (128-byte swizzle); completion is counted on
//               the even CTA's barriers
//   warp 1      PV issuer (even CTA): O += P(j) V_j once the 16 softmax warps have stored P(j); commit = V slot free,
//               O holds PV(j)
//   warp 3      QK issuer (even CTA): S(t) = Q K_t^T once PV(t-3) has completed; commits: S ready, K slot free
//   warp 2      zeroes the rows of its V half past the valid tokens (ragged last tile, the step's own tokens)
//   warps 4-11  softmax (both CTAs): a warp owns 16 rows, four threads per row (tcgen05.ld 16x256b), so the row
//               maximum and the overflow check stay inside the warp; online softmax in the log2 domain with a
//               reference maximum that is only moved when it must be
// Tensor memory (512 columns per CTA): S0/P0 | S1/P1 | S2/P2 | O (128 columns each).
// With several KV splits the unnormalised (O, m, l) go to the workspace and the merge kernel combines them by
// log-sum-exp.  Every wait is bounded; a wait that gives up records SPECPV_ERR_TIMEOUT, stops its loop, raises
// the abort flag of both CTAs, and the pair still drains its copies and frees its tensor memory.
#include <limits.h>
#include <stdlib.h>
#include <string.h>

#include "attn_tc.cuh"

namespace specpv {

namespace {

using namespace tc;

constexpr int kPairThreads = 384;   // 12 warps
constexpr int kRing = 5;            // K tiles and V tiles in flight per CTA (a ring each)
constexpr int kHalf = 16384;        // a K slot [2 d-halves x 64 tokens x 64 d] or a V slot [128 tokens x 64 channels]
constexpr int kQTile = 32768;       // [2 d-halves][128 rows][64 d]
constexpr int kPairSmem = 1024 + 2 * kQTile + 2 * kRing * kHalf;
constexpr uint32_t kColO = 384;     // tensor-memory columns: S/P buffer b at b * 128, O behind them
constexpr int kLag = 3;             // PV runs this many tiles behind QK (= number of S/P buffers)
constexpr uint64_t kWaitNs = 2000000000ull;

// Instruction descriptors, kind::f16: D = f32, A = B = bf16, M = 256 over the pair, N = 128.
constexpr uint32_t idesc_pair(bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((128u >> 3) << 17) | ((256u >> 4) << 24);
}
constexpr uint32_t kIdescQK2 = idesc_pair(false);
constexpr uint32_t kIdescPV2 = idesc_pair(true);  // B (= V) is MN-major

struct __align__(8) PairBars {
    uint64_t q_full[2];          // even CTA: both CTAs' Q tiles of a stretch have landed (transaction bytes)
    uint64_t q_empty[2];         // both: the last QK of the stretch that used this Q buffer has completed
    uint64_t k_full[kRing];      // even CTA: both CTAs' halves of a K tile have landed
    uint64_t k_empty[kRing];     // both: QK of the tile in this slot has completed
    uint64_t v_full[kRing];      // even CTA: both halves of a V tile are in place (bytes + one "V ready" per CTA)
    uint64_t v_empty[kRing];     // both: PV of the tile in this slot has completed (slot free, O holds that PV)
    uint64_t vfix_full[kRing];   // own: this CTA's V half of a tile that needs zeroed rows has landed
    uint64_t s_full[kLag];       // both: S(j) is complete
    uint64_t p_full[kLag];       // even CTA: all 16 softmax warps have stored P(j)
    uint64_t o_full;             // both: the last PV of a stretch has completed
    uint64_t o_free;             // even CTA: all 16 softmax warps have read O of the finished stretch
    uint64_t drain;              // even CTA: completion of whatever was issued before an abort
    uint64_t rows_done;          // own: the eight softmax warps have written their rows of a shared unit / seen the ticket
    uint32_t tmem_base;
    int abort_flag;
    int ticket;                  // own: this CTA's arrival number on a shared unit (read by its softmax warps)
};

// One stretch of KV tiles of one unit = (layer, sequence, KV head, row group) processed by a pair.
struct Seg {
    int lb, b, l, h, rg;
    int M, seq_len, tok0;
    int tile_begin;   // first tile of the stretch within the unit (context tiles, then the tile of the step's own tokens)
    int n_ctx;        // context tiles in the stretch
    int n_tiles;      // n_ctx + 1 if the stretch ends with the tile of the step's own tokens
    int first_fix;    // first tile (stretch-local) whose V rows past the valid tokens must be zeroed; n_tiles if none
    bool direct;      // the stretch covers the whole unit: results are final
    int slot;         // otherwise: where its partial results go (two slots per pair)
    int counter;      // ... the unit's arrival counter (one per CTA rank) ...
    int p_first, n_seg;          // ... and the pairs that share the unit: p_first .. p_first + n_seg - 1
    long long unit_x0;           // global index of the unit's first tile
};

// The work of a launch is the sequence of all tiles of all units, unit after unit (layer-major, then sequence, KV
// head, row group); a pair takes an equal contiguous share of that sequence, so it meets at most two units that it
// shares with neighbouring pairs (their partial results are merged by whichever CTA finishes a shared unit last).
// SegIter walks a pair's share unit by unit.  Lengths live on the device, so every role computes the split itself.
struct SegIter {
    long long x = 0, x_end = 0, tiles_per_layer = 0, quota = 1;
    bool first = true, ready = false;
    __device__ static int row_groups(const TcParams& p, int M) { return (M * p.G + 255) / 256; }
    __device__ static int seq_M(const TcParams& p, int b) {
        const int M = p.q_lens ? p.q_lens[b] : p.M_max;
        return min(max(M, 0), p.M_max);
    }
    __device__ void init(const TcParams& p) {
        ready = true;
        if (p.pairs_per_unit > 0) {  // the one stretch of this pair is worked out in next()
            x = 0; x_end = 1; quota = 1;
            return;
        }
        tiles_per_layer = 0;
        for (int b = 0; b < p.batch; ++b) {
            const int tiles = (max(p.seq_lens[b], 0) + kTileTokens - 1) / kTileTokens + 1;
            tiles_per_layer += (long long)tiles * p.Hkv * row_groups(p, seq_M(p, b));
        }
        const long long total = tiles_per_layer * p.n_layers_call;
        const long long n_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
        quota = max((total + n_pairs - 1) / n_pairs, 1ll);
        x = min(pair * quota, total);
        x_end = min(x + quota, total);
    }
    __device__ bool next(const TcParams& p, Seg& s) {
        if (!ready) init(p);
        if (x >= x_end) return false;
        if (p.pairs_per_unit > 0) {
            // With fewer units than pairs every unit gets k pairs of its own, each an equal part of the unit's tiles: no
            // pair meets two units (which would cost it a second Q tile, first tile and epilogue).
            x = x_end;
            const int k = p.pairs_per_unit, pair = (int)(blockIdx.x >> 1), unit = pair / k, part = pair % k;
            s.rg = unit % p.n_row_groups;
            s.h = (unit / p.n_row_groups) % p.Hkv;
            s.lb = unit / (p.n_row_groups * p.Hkv);
            s.b = s.lb % p.batch; s.l = s.lb / p.batch;
            s.seq_len = max(p.seq_lens[s.b], 0);
            s.M = seq_M(p, s.b);
            s.tok0 = s.rg * (256 / p.G);
            if (s.tok0 >= s.M) return false;  // no step tokens in this row group
            const int n_ctx_unit = (s.seq_len + kTileTokens - 1) / kTileTokens, tiles = n_ctx_unit + 1;
            const int per = (tiles + k - 1) / k, off = part * per;
            if (off >= tiles) return false;
            const int n = min(per, tiles - off);
            s.tile_begin = off;
            s.n_tiles = n;
            s.n_ctx = max(min(off + n, n_ctx_unit) - off, 0);
            const bool ragged = (s.seq_len % kTileTokens) != 0;
            const int fix_unit = ragged ? n_ctx_unit - 1 : (s.M < kTileTokens ? n_ctx_unit : tiles);
            s.first_fix = min(max(fix_unit - off, 0), n);
            s.n_seg = (tiles + per - 1) / per;
            s.direct = s.n_seg == 1;
            s.slot = pair * 2;
            s.p_first = unit * k;
            s.unit_x0 = s.p_first;  // with quota = 1: every partial result sits in its pair's first slot
            s.counter = unit * 2;
            return true;
        }
        s.l = (int)(x / tiles_per_layer);
        long long r = x % tiles_per_layer;
        int b = 0, tiles = 1, rgs = 1, M = 0, seq_len = 0;
        for (;; ++b) {  // the sequence this tile belongs to
            seq_len = max(p.seq_lens[b], 0);
            M = seq_M(p, b);
            tiles = (seq_len + kTileTokens - 1) / kTileTokens + 1;
            rgs = row_groups(p, M);
            const long long nb = (long long)tiles * p.Hkv * rgs;
            if (r < nb || b == p.batch - 1) break;
            r -= nb;
        }
        const int unit_in_b = (int)(r / tiles), off = (int)(r % tiles);
        s.b = b; s.lb = s.l * p.batch + b; s.h = unit_in_b / rgs; s.rg = unit_in_b % rgs;
        s.M = M; s.seq_len = seq_len; s.tok0 = s.rg * (256 / p.G);
        const int n_ctx_unit = tiles - 1;
        const int n = (int)min((long long)(tiles - off), x_end - x);
        s.tile_begin = off;
        s.n_tiles = n;
        s.n_ctx = max(min(off + n, n_ctx_unit) - off, 0);
        const bool ragged = (seq_len % kTileTokens) != 0;
        const int fix_unit = ragged ? n_ctx_unit - 1 : (M < kTileTokens ? n_ctx_unit : tiles);  // unit-local
        s.first_fix = min(max(fix_unit - off, 0), n);
        s.direct = off == 0 && n == tiles;
        s.slot = (int)(blockIdx.x >> 1) * 2 + (first ? 0 : 1);
        s.unit_x0 = x - off;
        s.p_first = (int)(s.unit_x0 / quota);
        s.n_seg = (int)((s.unit_x0 + tiles - 1) / quota) - s.p_first + 1;
        s.counter = ((s.lb * p.Hkv + s.h) * p.n_row_groups + s.rg) * 2;
        first = false;
        x += n;
        return true;
    }
};

// 2^x for a pair of finite x (clamped to [-126, 127]) on the FMA and integer pipes (the special-function unit, 16 exponentials per
// cycle and SM, is the softmax's scarcest resource): x = n + f with n = round(x) taken from the low mantissa bits of
// x + 1.5 * 2^23, f in [-0.5, 0.5], 2^f by a cubic with maximum relative error 7.5e-5 (the weight is rounded to
// bfloat16, relative error 3.9e-3, right after), n added to the exponent field.
__device__ __forceinline__ float2 exp2_fma_pair(float2 x) {
    const float kMagic = 12582912.f;  // 1.5 * 2^23
    x.x = fminf(fmaxf(x.x, -126.f), 127.f);  // 2^127 and the like trip the caller's overflow check, as +inf would
    x.y = fminf(fmaxf(x.y, -126.f), 127.f);
    const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
    const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
    const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
    float2 r = __ffma2_rn(make_float2(0.055171459913253784f, 0.055171459913253784f), f, make_float2(0.2426108568906784f, 0.2426108568906784f));
    r = __ffma2_rn(r, f, make_float2(0.6932609677314758f, 0.6932609677314758f));
    r = __ffma2_rn(r, f, make_float2(0.9999281167984009f, 0.9999281167984009f));
    r.x = __int_as_float(__float_as_int(r.x) + (__float_as_int(t.x) << 23));
    r.y = __int_as_float(__float_as_int(r.y) + (__float_as_int(t.y) << 23));
    return r;
}
// which of the 16 column groups of a row pair take their exponentials on the FMA pipe (fast path only)
constexpr uint32_t kFmaExpGroups = 0x1111u;  // groups 0, 4, 8, 12: a quarter (measured: 1577 cycles per tile with none, 1392 with 4, 1446 with 5)

// Log-sum-exp merge of the partial results of a unit shared between pairs, for the 128 rows of one CTA rank, by the
// eight softmax warps of the CTA that finished the unit last (w8 = 0..7).  Warp w8 owns rows 16 w8 .. 16 w8 + 15, in two
// passes of eight; a lane owns four channels of each, so a warp-wide load covers one whole row (512 contiguous bytes:
// with a row half per thread instead, the same merge took 40 us for nine pairs).  Everything comes from L2 at 1.5-2 us
// per dependent round trip, so the partial rows of four pairs x eight rows are requested together.  Lane r < 8 keeps
// row r's running maximum and sum.
__device__ __forceinline__ void merge_shared_unit(const TcParams& p, const Seg& s, long long quota, int rank, int w8, int lane) {
    auto slot_of = [&](int q) { return (s.p_first + q) * 2 + ((q == 0 && (long long)s.p_first * quota < s.unit_x0) ? 1 : 0); };
    for (int pass = 0; pass < 2; ++pass) {
        const int row0 = rank * 128 + w8 * 16 + pass * 8;  // first row (within the row group) of this pass
        if (s.tok0 + row0 / p.G >= s.M) return;              // rows ascend with the token: no row in use from here on
        float m_all = -INFINITY, l_all = 0.f;                // state of row row0 + lane (lanes 0..7)
        float4 o[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) o[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int q0 = 0; q0 < s.n_seg; q0 += 4) {
            float2 ml[4];
            float4 po[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const size_t prow0 = (size_t)slot_of(min(q0 + u, s.n_seg - 1)) * 256 + row0;
                ml[u] = make_float2(-INFINITY, 0.f);
                if (lane < 8 && q0 + u < s.n_seg) ml[u] = __ldcg(reinterpret_cast<const float2*>(p.part_ml) + prow0 + lane);
                const float4* src = reinterpret_cast<const float4*>(p.part_o + prow0 * kD) + lane;
#pragma unroll
                for (int r = 0; r < 8; ++r) po[u][r] = __ldcg(src + r * (kD / 4));
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                // this lane's row: new maximum, factor for what has been gathered so far, weight of this pair
                const float m_new = fmaxf(m_all, ml[u].x);
                const float f_mine = (m_all == -INFINITY || m_new == -INFINITY) ? 0.f : __expf(m_all - m_new);
                const float w_mine = ml[u].x == -INFINITY ? 0.f : __expf(ml[u].x - m_new);
                m_all = m_new;
                l_all = fmaf(l_all, f_mine, ml[u].y * w_mine);
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    const float f = __shfl_sync(0xffffffffu, f_mine, r), w = __shfl_sync(0xffffffffu, w_mine, r);
                    o[r].x = fmaf(o[r].x, f, w == 0.f ? 0.f : po[u][r].x * w); o[r].y = fmaf(o[r].y, f, w == 0.f ? 0.f : po[u][r].y * w);
                    o[r].z = fmaf(o[r].z, f, w == 0.f ? 0.f : po[u][r].z * w); o[r].w = fmaf(o[r].w, f, w == 0.f ? 0.f : po[u][r].w * w);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int grow = row0 + r;
            const int tok = s.tok0 + grow / p.G;
            const float l_r = __shfl_sync(0xffffffffu, l_all, r), m_r = __shfl_sync(0xffffffffu, m_all, r);
            if (tok >= s.M) continue;  // warp-uniform
            const size_t out_row = ((size_t)s.lb * p.M_max + tok) * p.Hq + s.h * p.G + grow % p.G;
            const float inv = 1.f / l_r;
            const float4 v = make_float4(o[r].x * inv, o[r].y * inv, o[r].z * inv, o[r].w * inv);
            if (p.out_f32) {
                reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + out_row * kD)[lane] = v;
            } else {
                uint2 w2;
                w2.x = pack_bf16(v.x, v.y);
                w2.y = pack_bf16(v.z, v.w);
                reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + out_row * kD)[lane] = w2;
            }
            if (p.lse && lane == 0) p.lse[out_row] = m_r + logf(l_r);
        }
    }
}

// Bounded wait for the pair kernel: a wait that gives up records the fault and raises the abort flag of both CTAs.
__device__ __forceinline__ bool pair_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t peer_abort,
                                               void* workspace, int where, uint64_t limit_ns) {
    const uint64_t t0 = global_ns();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((it & 255u) == 255u && global_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            st_cluster_u32(peer_abort, 1u);
            record_fault(workspace, SPECPV_ERR_TIMEOUT, where, (int)blockIdx.x, (int)blockIdx.y, (int)blockIdx.z);
            return false;
        }
    }
}
__device__ __forceinline__ bool pair_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t peer_abort,
                                          void* workspace, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    return pair_wait_slow(bar, parity, abort_flag, peer_abort, workspace, where, kWaitNs);
}

// =================================================================================================
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1) attn_pair_kernel(const __grid_constant__ TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the 128-byte swizzle atoms (the same offset in both CTAs)
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ PairBars bars;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0: the CTA that issues the contractions and counts the completions
    const int tok_per_tile = 128 / p.G;       // step tokens per 128-row tile

    // A pair without work leaves at once (uniform for both CTAs).
    {
        SegIter it;
        Seg s;
        if (!it.next(p, s)) return;
    }

    const uint32_t q_smem = smem_u32(smem);
    const uint32_t k_smem = q_smem + 2 * kQTile, v_smem = k_smem + kRing * kHalf;
    volatile int* abort_flag = &bars.abort_flag;
    const uint32_t peer_abort = mapa(smem_u32(&bars.abort_flag), rank ^ 1u);

    // ---- set-up ------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bars.q_full[i]), 1);
            mbar_init(smem_u32(&bars.q_empty[i]), 1);
        }
        for (int i = 0; i < kLag; ++i) {
            mbar_init(smem_u32(&bars.s_full[i]), 1);
            mbar_init(smem_u32(&bars.p_full[i]), 16);  // one arrival per softmax warp of the pair
        }
        for (int s = 0; s < kRing; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 3);  // the byte count's arrival + one "V half ready" per CTA
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
            mbar_init(smem_u32(&bars.vfix_full[s]), 1);
        }
        mbar_init(smem_u32(&bars.o_full), 1);
        mbar_init(smem_u32(&bars.o_free), 16);
        mbar_init(smem_u32(&bars.drain), 1);
        mbar_init(smem_u32(&bars.rows_done), 8);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {  // one warp of each CTA: the allocation is made in both CTAs' tensor memory at once
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&bars.tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the other CTA's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;

    // barriers of the even CTA, as seen from this CTA
    const uint32_t lead_q_full0 = mapa(smem_u32(&bars.q_full[0]), 0);
    const uint32_t lead_k_full0 = mapa(smem_u32(&bars.k_full[0]), 0);
    const uint32_t lead_v_full0 = mapa(smem_u32(&bars.v_full[0]), 0);
    const uint32_t lead_p_full0 = mapa(smem_u32(&bars.p_full[0]), 0);
    const uint32_t lead_o_free = mapa(smem_u32(&bars.o_free), 0);

    // Register budget: the control warpgroup (warps 0-3) gives registers to the two softmax warpgroups.
    // Block-table access of the two producer warps: the entry of the next tile is loaded while the current one is
    // issued and only looked at when its tile comes up, so the load's latency never stalls the warp.
    constexpr int kNoPage = INT_MIN;  // the block lies past the sequence: the copy engine fills zeros
    const int ppt = kTileTokens / p.bs;  // pages per tile
    auto page_load = [&](const Seg& s, int blk) {
        return ((long long)blk * p.bs < s.seq_len && blk < p.max_blocks) ? __ldg(p.block_table + (size_t)s.b * p.max_blocks + blk) : kNoPage;
    };
    // pool row of a page (an out-of-range row makes the copy engine fill zeros); a bad entry is recorded and read as zeros
    auto page_row = [&](const Seg& s, int blk, int page, bool report) {
        if (page == kNoPage) return (int)p.pool_rows;
        if (page < 0 || page >= p.n_pages) {
            if (report) record_fault(p.workspace, SPECPV_ERR_BAD_BLOCK_TABLE, s.b, blk, page, s.l);
            return (int)p.pool_rows;
        }
        return (((p.layer0 + s.l) * p.n_pages + page) * p.Hkv + s.h) * p.bs;  // < 2^31: checked on the host
    };

    // Register budget: the control warpgroup (warps 0-3) gives registers to the two softmax warpgroups.
    if (warp == 0) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // =========================== K producer (both CTAs) ======================================
        // Per stretch its Q tile, then per tile this CTA's 64 tokens of K into the K ring.  The whole warp runs the
        // loop; lane 0 does the barrier bookkeeping; lane 2 pg + half copies the 64-channel half `half` of page pg.
        const bool k_lane = lane < ppt;
        const int k_pg = lane >> 1, k_half = lane & 1;
        SegIter it;
        Seg s;
        uint32_t t = 0;
        bool ok = true;
        for (int sidx = 0; ok && it.next(p, s); ++sidx) {
            const int qb = sidx & 1;
            if (sidx >= 2) ok = pair_wait(smem_u32(&bars.q_empty[qb]), ((sidx >> 1) - 1) & 1, abort_flag, peer_abort, p.workspace, 1);
            if (!ok) break;
            if (lane == 0) {
                if (rank == 0) mbar_expect_tx(smem_u32(&bars.q_full[qb]), 2 * kQTile);
                for (int half = 0; half < 2; ++half)
                    tma_load_3d_pair(q_smem + qb * kQTile + half * 16384, &p.tm_q, half * 64, s.h * p.G,
                                     s.lb * p.M_max + s.tok0 + (int)rank * tok_per_tile, lead_q_full0 + qb * 8);
            }
            __syncwarp();
            int blk = s.tile_begin * ppt + (int)rank * (ppt >> 1) + k_pg;  // this lane's block of the current tile
            int page_next = (k_lane && s.n_ctx > 0) ? page_load(s, blk) : kNoPage;
            for (int j = 0; j < s.n_tiles; ++j, ++t, blk += ppt) {
                const uint32_t ks = t % kRing;
                const int page = page_next;
                if (k_lane && j + 1 < s.n_ctx) page_next = page_load(s, blk + ppt);
                if (t >= (uint32_t)kRing) ok = pair_wait(smem_u32(&bars.k_empty[ks]), ((t / kRing) - 1) & 1, abort_flag, peer_abort, p.workspace, 2);
                if (!ok) break;
                const uint32_t dst = k_smem + ks * kHalf, full = lead_k_full0 + ks * 8;
                if (lane == 0 && rank == 0) mbar_expect_tx(smem_u32(&bars.k_full[ks]), 2 * kHalf);
                __syncwarp();
                if (j >= s.n_ctx) {  // the step's own tokens
                    if (lane < 2) tma_load_3d_pair(dst + lane * 8192, &p.tm_knew, lane * 64, s.h, s.lb * p.M_max + (int)rank * 64, full);
                } else if (k_lane) {
                    tma_load_2d_pair(dst + k_half * 8192 + k_pg * p.bs * 128, &p.tm_kpool, k_half * 64, page_row(s, blk, page, k_half == 0), full);
                }
            }
        }
    } else if (warp == 1) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // =========================== PV issuer (even CTA) ========================================
        // O += P(j) V_j for every tile j, in order.  The whole warp runs the loop, lane 0 issues.  The tile counter
        // runs across stretches; only O is handed over between them.
        if (rank == 0) {
            const uint32_t desc_hi = (uint32_t)((1024u >> 4) | (1u << 14) | (2u << 29));
            const uint32_t v_lo0 = ((v_smem >> 4) & 0x3FFFu) | ((16u >> 4) << 16);
            SegIter it;
            Seg s;
            uint32_t g = 0;
            bool ok = true;
            for (int sidx = 0; ok && it.next(p, s); ++sidx) {
                for (int j = 0; j < s.n_tiles; ++j, ++g) {
                    const uint32_t vs = g % kRing, buf = g % kLag;
                    ok = pair_wait(smem_u32(&bars.v_full[vs]), (g / kRing) & 1, abort_flag, peer_abort, p.workspace, 4);
                    if (ok && j == 0 && sidx > 0) ok = pair_wait(smem_u32(&bars.o_free), (sidx - 1) & 1, abort_flag, peer_abort, p.workspace, 6);
                    if (ok) ok = pair_wait(smem_u32(&bars.p_full[buf]), (g / kLag) & 1, abort_flag, peer_abort, p.workspace, 7);
                    if (!ok) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t b_lo = launder(v_lo0 + vs * (kHalf >> 4));
                        const uint32_t a = tmem + buf * 128, d = tmem + kColO;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)  // 16 tokens per instruction: two 8-row groups of 1024 bytes
                            mma2_ts_lohi(d, a + kk * 8, b_lo + (uint32_t)kk * (2048u >> 4), desc_hi, kIdescPV2, (j > 0 || kk > 0) ? 1u : 0u);
                        tc_commit_pair(smem_u32(&bars.v_empty[vs]));
                        if (j == s.n_tiles - 1) tc_commit_pair(smem_u32(&bars.o_full));
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp == 2) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // =========================== V producer (both CTAs) ======================================
        // Per tile this CTA's 64 channels of V (all 128 tokens) into the V ring; lane pg copies page pg.  Rows of a V tile
        // past its valid tokens may hold anything (stale pages, rows of other sequences' steps): for a ragged last
        // context tile and for the tile of the step's own tokens the copies complete on this CTA's own barrier, the
        // warp zeroes those rows in its half (so that 0 * garbage cannot give NaN) and only then reports the half ready.
        const bool v_lane = lane < ppt;
        SegIter it;
        Seg s;
        uint32_t g = 0, fix_parity = 0;  // bit `slot`: parity of the next use of that slot's zeroing barrier
        bool ok = true;
        while (ok && it.next(p, s)) {
            int blk = s.tile_begin * ppt + lane;
            int page_next = (v_lane && s.n_ctx > 0) ? page_load(s, blk) : kNoPage;
            for (int j = 0; j < s.n_tiles; ++j, ++g, blk += ppt) {
                const uint32_t vs = g % kRing;
                const int page = page_next;
                if (v_lane && j + 1 < s.n_ctx) page_next = page_load(s, blk + ppt);
                if (g >= (uint32_t)kRing) ok = pair_wait(smem_u32(&bars.v_empty[vs]), ((g / kRing) - 1) & 1, abort_flag, peer_abort, p.workspace, 16);
                if (!ok) break;
                const bool fix = j >= s.first_fix;
                const uint32_t dst = v_smem + vs * kHalf, full = lead_v_full0 + vs * 8, vfix = smem_u32(&bars.vfix_full[vs]);
                if (lane == 0) {
                    if (fix) mbar_expect_tx(vfix, kHalf);
                    if (rank == 0) {
                        if (fix) mbar_arrive(smem_u32(&bars.v_full[vs]));  // the bytes are counted on the zeroing barriers
                        else mbar_expect_tx(smem_u32(&bars.v_full[vs]), 2 * kHalf);
                    }
                }
                __syncwarp();
                const uint32_t vbar = fix ? vfix : full;
                if (j >= s.n_ctx) {  // the step's own tokens
                    if (lane < 2) tma_load_3d_pair(dst + lane * 8192, &p.tm_vnew, (int)rank * 64, s.h, s.lb * p.M_max + lane * 64, vbar);
                } else if (v_lane) {
                    tma_load_2d_pair(dst + lane * p.bs * 128, &p.tm_vpool, (int)rank * 64, page_row(s, blk, page, rank == 0), vbar);
                }
                __syncwarp();
                if (fix) {
                    ok = pair_wait(vfix, (fix_parity >> vs) & 1u, abort_flag, peer_abort, p.workspace, 8);
                    if (!ok) break;
                    fix_parity ^= 1u << vs;
                    const int n_valid = max(j >= s.n_ctx ? s.M : min(kTileTokens, s.seq_len - (s.tile_begin + j) * kTileTokens), 0);
                    uint8_t* v = smem + 2 * kQTile + (size_t)kRing * kHalf + (size_t)vs * kHalf;
                    for (int i = lane; i < (kTileTokens - n_valid) * 8; i += 32)
                        *reinterpret_cast<uint4*>(v + (size_t)(n_valid + (i >> 3)) * 128 + (i & 7) * 16) = make_uint4(0, 0, 0, 0);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
                if (lane == 0) mbar_arrive_cluster(full);  // this CTA's V half is ready
            }
        }
    } else if (warp == 3) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        // =========================== QK issuer (even CTA) ========================================
        // S(t) = Q K_t^T into buffer t mod 3, which still holds P(t-3): not before PV(t-3) has completed (the two
        // issuing warps are ordered by that commit barrier only).  QK runs up to three tiles ahead of the softmax.
        if (rank == 0) {
            const uint32_t desc_hi = (uint32_t)((1024u >> 4) | (1u << 14) | (2u << 29));
            const uint32_t q_lo0 = ((q_smem >> 4) & 0x3FFFu) | ((16u >> 4) << 16);
            const uint32_t k_lo0 = ((k_smem >> 4) & 0x3FFFu) | ((16u >> 4) << 16);
            SegIter it;
            Seg s;
            uint32_t t = 0;
            bool ok = true;
            for (int sidx = 0; ok && it.next(p, s); ++sidx) {
                for (int j = 0; j < s.n_tiles; ++j, ++t) {
                    const uint32_t ks = t % kRing, buf = t % kLag;
                    if (j == 0) ok = pair_wait(smem_u32(&bars.q_full[sidx & 1]), (sidx >> 1) & 1, abort_flag, peer_abort, p.workspace, 3);
                    if (ok) ok = pair_wait(smem_u32(&bars.k_full[ks]), (t / kRing) & 1, abort_flag, peer_abort, p.workspace, 13);
                    if (ok && t >= (uint32_t)kLag)
                        ok = pair_wait(smem_u32(&bars.v_empty[(t - kLag) % kRing]), ((t - kLag) / kRing) & 1, abort_flag, peer_abort, p.workspace, 14);
                    if (!ok) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t a_lo = launder(q_lo0 + (uint32_t)(sidx & 1) * (kQTile >> 4));
                        const uint32_t b_lo = launder(k_lo0 + ks * (kHalf >> 4));
                        const uint32_t d = tmem + buf * 128;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {  // 16 channels of d per instruction
                            const uint32_t a_off = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                            const uint32_t b_off = (uint32_t)((kk >> 2) * 8192 + (kk & 3) * 32) >> 4;
                            mma2_ss_lohi(d, a_lo + a_off, b_lo + b_off, desc_hi, kIdescQK2, kk > 0 ? 1u : 0u);
                        }
                        tc_commit_pair(smem_u32(&bars.s_full[buf]));
                        tc_commit_pair(smem_u32(&bars.k_empty[ks]));
                        if (j == s.n_tiles - 1) tc_commit_pair(smem_u32(&bars.q_empty[sidx & 1]));
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        // =========================== softmax / correction / epilogue ==============================
        const int q = warp & 3;                    // tensor-memory lane quarter this warp may access
        const int hf = (warp - 4) >> 2;            // lower or upper 16 lanes of the quarter
        const int lrow = q * 32 + hf * 16;
        const int ra = lrow + (lane >> 2), rb = ra + 8;   // this thread's two rows within the CTA's tile
        const int cq = (lane & 3) * 2;             // its two adjacent columns in every group of eight
        const uint32_t lane_addr = (uint32_t)lrow << 16;
        const uint32_t o_addr = tmem + lane_addr + kColO;
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
        SegIter it;
        Seg s;
        uint32_t g = 0, rows_phase = 0;
        bool ok = true;
        for (int sidx = 0; ok && it.next(p, s); ++sidx) {
            const int row_a = (int)rank * 128 + ra, row_b = (int)rank * 128 + rb;  // rows within the row group
            const int tok_a = s.tok0 + row_a / p.G, tok_b = s.tok0 + row_b / p.G;
            const bool valid_a = tok_a < s.M, valid_b = tok_b < s.M;
            uint64_t mlo_a = 0, mhi_a = 0, mlo_b = 0, mhi_b = 0;
            if (valid_a) {
                const uint64_t* mrow = p.tree_mask + ((size_t)s.b * p.M_max + tok_a) * p.mask_words;
                mlo_a = mrow[0];
                if (p.mask_words > 1) mhi_a = mrow[1];
            }
            if (valid_b) {
                const uint64_t* mrow = p.tree_mask + ((size_t)s.b * p.M_max + tok_b) * p.mask_words;
                mlo_b = mrow[0];
                if (p.mask_words > 1) mhi_b = mrow[1];
            }
            float m_a = -INFINITY, m_b = -INFINITY;  // reference maxima (log2 domain), the same in the four threads of a row
            float l_a = 0.f, l_b = 0.f;              // this thread's share of the row sums
            for (int j = 0; j < s.n_tiles && ok; ++j, ++g) {
                const bool is_new = j >= s.n_ctx;
                const int n_valid = is_new ? s.M : min(kTileTokens, s.seq_len - (s.tile_begin + j) * kTileTokens);
                const bool masked = is_new || n_valid < kTileTokens;
                const uint32_t buf = g % kLag;
                const uint32_t s_addr = tmem + lane_addr + buf * 128;
                ok = __all_sync(0xffffffffu, pair_wait(smem_u32(&bars.s_full[buf]), (g / kLag) & 1, abort_flag, peer_abort, p.workspace, 9));
                if (!ok) break;
                tc_fence_after();
                uint32_t v[64];  // v[4n + k]: row a (k < 2) or b, column 8n + cq + (k & 1)
                TMEM_LD_16x256_X8(s_addr, v);
                TMEM_LD_16x256_X8(s_addr + 64, (v + 32));
                tmem_wait_ld();
                // P = 2^(s*scale - m) as bf16 pairs: word 2n + k/2 of P (row a or b, columns 8n + cq, + 1) goes to
                // v[2n + k/2], whose own value was consumed earlier.  The row sums are taken over the ROUNDED weights
                // the tensor core will use, so that O / l is an exact weighted average of V rows.
                auto exp_rows = [&](float ma, float mb, float& sum_a, float& sum_b, const uint32_t fma_groups) {
                    const float2 na = make_float2(-ma, -ma), nb = make_float2(-mb, -mb);
                    float2 acc_a[2], acc_b[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) acc_a[e] = acc_b[e] = make_float2(0.f, 0.f);
#pragma unroll
                    for (int n = 0; n < 16; ++n) {
                        const float2 xa = __ffma2_rn(make_float2(__uint_as_float(v[4 * n]), __uint_as_float(v[4 * n + 1])), sc2, na);
                        const float2 xb = __ffma2_rn(make_float2(__uint_as_float(v[4 * n + 2]), __uint_as_float(v[4 * n + 3])), sc2, nb);
                        uint32_t wa, wb;
                        if ((fma_groups >> n) & 1u) {
                            const float2 ea = exp2_fma_pair(xa), eb = exp2_fma_pair(xb);
                            wa = pack_bf16(ea.x, ea.y);
                            wb = pack_bf16(eb.x, eb.y);
                        } else {
                            wa = pack_bf16(ex2(xa.x), ex2(xa.y));
                            wb = pack_bf16(ex2(xb.x), ex2(xb.y));
                        }
                        v[2 * n] = wa;
                        v[2 * n + 1] = wb;
                        add_bf16_pair(acc_a[n & 1], wa);
                        add_bf16_pair(acc_b[n & 1], wb);
                    }
                    sum_a = (acc_a[0].x + acc_a[1].x) + (acc_a[0].y + acc_a[1].y);
                    sum_b = (acc_b[0].x + acc_b[1].x) + (acc_b[0].y + acc_b[1].y);
                };
                // Fast path (every full context tile after the first of a stretch): keep the reference maxima and skip
                // the row maximum.  Weights may then exceed 1; float32 sums and bf16 weights keep their relative precision
                // whatever the exponent, so only overflow has to be ruled out: if a row's share of the sum leaves the safe
                // range (or a row has no reference yet), the warp takes the tile again from tensor memory (S(j) stays
                // intact until every warp has arrived on the P barrier) on the general path.
                float add_a = 0.f, add_b = 0.f;
                bool general = j == 0 || masked;
                if (!general) {
                    exp_rows(m_a, m_b, add_a, add_b, kFmaExpGroups);
                    const bool bad = (valid_a && (!(add_a < kSafeRowSum) || m_a == -INFINITY)) ||
                                     (valid_b && (!(add_b < kSafeRowSum) || m_b == -INFINITY));
                    if (__any_sync(0xffffffffu, bad)) {
                        general = true;
                        TMEM_LD_16x256_X8(s_addr, v);
                        TMEM_LD_16x256_X8(s_addr + 64, (v + 32));
                        tmem_wait_ld();
                    }
                }
                if (general) {
                    if (masked) {  // ragged or tree-masked tile: invisible columns become -inf
                        uint64_t va_lo = ~0ull, va_hi = ~0ull, vb_lo = ~0ull, vb_hi = ~0ull;
                        if (is_new) { va_lo = mlo_a; va_hi = mhi_a; vb_lo = mlo_b; vb_hi = mhi_b; }
                        uint64_t keep_lo = ~0ull, keep_hi = ~0ull;
                        if (n_valid < 64) {
                            keep_lo = (n_valid <= 0) ? 0ull : (~0ull >> (64 - n_valid));
                            keep_hi = 0;
                        } else if (n_valid < 128) {
                            keep_hi = (n_valid == 64) ? 0ull : (~0ull >> (128 - n_valid));
                        }
                        va_lo = (va_lo & keep_lo) >> cq; va_hi = (va_hi & keep_hi) >> cq;
                        vb_lo = (vb_lo & keep_lo) >> cq; vb_hi = (vb_hi & keep_hi) >> cq;
#pragma unroll
                        for (int n = 0; n < 16; ++n) {
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint64_t word = (k < 2) ? (n < 8 ? va_lo : va_hi) : (n < 8 ? vb_lo : vb_hi);
                                if (!((word >> ((n & 7) * 8 + (k & 1))) & 1ull)) v[4 * n + k] = 0xff800000u;
                            }
                        }
                    }
                    float xa0 = __uint_as_float(v[0]), xa1 = __uint_as_float(v[1]);
                    float xb0 = __uint_as_float(v[2]), xb1 = __uint_as_float(v[3]);
#pragma unroll
                    for (int n = 1; n < 16; n += 2) {  // three-input max: two new values per instruction
                        xa0 = fmax3(xa0, __uint_as_float(v[4 * n]), __uint_as_float(v[4 * n + 1]));
                        xb0 = fmax3(xb0, __uint_as_float(v[4 * n + 2]), __uint_as_float(v[4 * n + 3]));
                        if (n + 1 < 16) {
                            xa1 = fmax3(xa1, __uint_as_float(v[4 * n + 4]), __uint_as_float(v[4 * n + 5]));
                            xb1 = fmax3(xb1, __uint_as_float(v[4 * n + 6]), __uint_as_float(v[4 * n + 7]));
                        }
                    }
                    float mx_a = fmaxf(xa0, xa1), mx_b = fmaxf(xb0, xb1);
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
                    // The reference is a whole number of octaves (ceil(-inf) = -inf): weights 2^(x - m) taken against
                    // references that differ by an integer differ by an exact power of two, so their bfloat16 roundings,
                    // and with them the result, do not depend on where the KV range was cut between pairs.
                    const float mt_a = ceilf(mx_a * p.scale_log2), mt_b = ceilf(mx_b * p.scale_log2);
                    // lazy rescale: keep the old reference unless the new maximum is more than 2^8 larger.  The decision
                    // is per row, the tensor-memory traffic is warp-wide (factor 1 where nothing changes).
                    bool need_a = false, need_b = false;
                    if (j == 0) {
                        m_a = mt_a;
                        m_b = mt_b;
                    } else {
                        need_a = mt_a > m_a + kRescaleThreshold || (m_a == -INFINITY && mt_a > -INFINITY);
                        need_b = mt_b > m_b + kRescaleThreshold || (m_b == -INFINITY && mt_b > -INFINITY);
                    }
                    if (__any_sync(0xffffffffu, need_a || need_b)) {
                        const float fa = !need_a ? 1.f : (m_a == -INFINITY ? 0.f : ex2(m_a - mt_a));
                        const float fb = !need_b ? 1.f : (m_b == -INFINITY ? 0.f : ex2(m_b - mt_b));
                        // O must hold PV(j-1) before it is rescaled: the commit behind that PV frees its V slot (the barrier
                        // cannot run a phase ahead: that takes PV(j+4), which needs the P this warp has not stored yet)
                        ok = __all_sync(0xffffffffu, pair_wait(smem_u32(&bars.v_empty[(g - 1) % kRing]), ((g - 1) / kRing) & 1,
                                                               abort_flag, peer_abort, p.workspace, 10));
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            uint32_t o[32];
                            TMEM_LD_16x256_X8(o_addr + c * 64, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * ((i & 2) ? fb : fa));
                            TMEM_ST_16x256_X8(o_addr + c * 64, o);
                        }
                        if (need_a) { l_a *= fa; m_a = mt_a; }
                        if (need_b) { l_b *= fb; m_b = mt_b; }
                    }
                    exp_rows(m_a == -INFINITY ? 0.f : m_a, m_b == -INFINITY ? 0.f : m_b, add_a, add_b, 0u);
                }
                l_a += add_a;
                l_b += add_b;
                // P(j) goes over the first half of S(j)'s own buffer (nothing else touches it before PV(j))
                TMEM_ST_16x128_X16(s_addr, v);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(lead_p_full0 + buf * 8);
            }
            if (!ok) break;
            // ---- epilogue of the stretch: wait for the last PV, hand O back, normalise, write out ------------
            ok = __all_sync(0xffffffffu, pair_wait(smem_u32(&bars.o_full), sidx & 1, abort_flag, peer_abort, p.workspace, 12));
            if (!ok) break;
            tc_fence_after();
            uint32_t o[64];
            TMEM_LD_16x256_X8(o_addr, o);
            TMEM_LD_16x256_X8(o_addr + 64, (o + 32));
            tmem_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(lead_o_free);
            // the four threads of a row add their shares of the row sum
            l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
            l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
            l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
            l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const bool valid = r ? valid_b : valid_a;
                if (!valid) continue;
                const int row = r ? row_b : row_a, tok = r ? tok_b : tok_a;
                const float l_run = r ? l_b : l_a, m_run = r ? m_b : m_a;
                const size_t out_row = ((size_t)s.lb * p.M_max + tok) * p.Hq + s.h * p.G + row % p.G;
                const size_t prow = (size_t)s.slot * 256 + row;
                const float inv = s.direct ? 1.f / l_run : 1.f;
#pragma unroll
                for (int n = 0; n < 16; ++n) {
                    const int ch = 8 * n + cq;
                    const float x = __uint_as_float(o[4 * n + 2 * r]) * inv, y = __uint_as_float(o[4 * n + 2 * r + 1]) * inv;
                    if (!s.direct) {
                        *reinterpret_cast<float2*>(p.part_o + prow * kD + ch) = make_float2(x, y);
                    } else if (p.out_f32) {
                        *reinterpret_cast<float2*>(reinterpret_cast<float*>(p.out) + out_row * kD + ch) = make_float2(x, y);
                    } else {
                        *reinterpret_cast<uint32_t*>(reinterpret_cast<__nv_bfloat16*>(p.out) + out_row * kD + ch) = pack_bf16(x, y);
                    }
                }
                if ((lane & 3) == 0) {
                    if (s.direct) {
                        if (p.lse) p.lse[out_row] = m_run * kLn2 + logf(l_run);
                    } else {
                        p.part_ml[prow * 2] = m_run * kLn2;  // natural-log units for the merge
                        p.part_ml[prow * 2 + 1] = l_run;
                    }
                }
            }
            if (!s.direct) {
                // ---- a unit shared with other pairs: the CTA that arrives last (per CTA rank: each rank owns its 128
                // rows) merges every pair's partial results by log-sum-exp.  Arrival counters live in the zeroed head of
                // the workspace and are put back to zero by the merging CTA.
                // (the eight warps meet on a shared-memory barrier with a bounded wait, not on bar.sync: after a wait that
                // gave up somewhere a warp may never get here)
                __threadfence();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.rows_done));
                if (warp == 4) {  // every warp of this CTA has written its rows: take a ticket
                    ok = pair_wait(smem_u32(&bars.rows_done), rows_phase & 1, abort_flag, peer_abort, p.workspace, 17);
                    if (ok && lane == 0) bars.ticket = atomicAdd(p.counters + s.counter + (int)rank, 1);
                    __syncwarp();
                } else {
                    ok = pair_wait(smem_u32(&bars.rows_done), rows_phase & 1, abort_flag, peer_abort, p.workspace, 17);
                }
                if (!ok) break;
                ++rows_phase;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.rows_done));  // second round: the ticket is in shared memory
                ok = pair_wait(smem_u32(&bars.rows_done), rows_phase & 1, abort_flag, peer_abort, p.workspace, 18);
                if (!ok) break;
                ++rows_phase;
                if (*reinterpret_cast<volatile int*>(&bars.ticket) == s.n_seg - 1) {
                    __threadfence();
                    merge_shared_unit(p, s, it.quota, (int)rank, warp - 4, lane);
                    if (warp == 4 && lane == 0) p.counters[s.counter + (int)rank] = 0;
                }
            }
        }
    }

    // ---- teardown ----------------------------------------------------------------------------
    // After an abort nothing new is issued; copies already in flight land within microseconds, contractions already
    // issued are waited for (bounded) before the tensor memory goes back.
    __syncwarp();
    if (*abort_flag) {
        __nanosleep(1000000);
        if (warp == 1 && rank == 0) {
            if (lane == 0) tc_commit_pair(smem_u32(&bars.drain));
            __syncwarp();
            const uint64_t t0 = global_ns();
            while (!mbar_try_wait(smem_u32(&bars.drain), 0) && global_ns() - t0 < 100000000ull) {}
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA leaves while the other may still touch its shared memory or barriers
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

}  // namespace

// The pair kernel serves the shapes of the single-CTA kernel whenever a KV head has more than one 128-row tile, but
// only on request (environment variable SPECPV_ATTN_KERNEL=pair, read at every call).  It needs about 7 % fewer
// cycles per tile than the single-CTA kernel and wins short bursts, but both kernels run into the board's power
// limit when verification steps follow one another, and there the pair kernel's operand exchange between the two SMs
// costs it clock: measured inside the benchmark step it is 8-10 % slower (4.56 against 4.12-4.23 ms for 32 layers at
// 128K), and its set-up and merge tail make it slower on single-layer calls (33 against 21 us for a 4096-token cache).
bool attention_pair_wanted(const AttnArgs& a) {
    if (a.M_max * a.g.G <= 128) return false;
    const char* v = getenv("SPECPV_ATTN_KERNEL");
    return v != nullptr && strcmp(v, "pair") == 0;
}

specpv_status launch_attention_pair(TcParams& p, const AttnArgs& a, cudaStream_t stream) {
    if (!set_smem_limit_once(reinterpret_cast<const void*>(attn_pair_kernel), kPairSmem)) return SPECPV_ERR_CUDA;
    const int Hkv = a.g.Hkv;
    // one pair per two SMs the device can hold at once; a persistent grid, the work split evenly inside the kernel
    static int pairs_cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPECPV_ERR_CUDA;
    int n_pairs = (dev >= 0 && dev < 64) ? pairs_cached[dev] : 0;
    if (n_pairs <= 0) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(2, 1, 1);
        cfg.blockDim = dim3(kPairThreads, 1, 1);
        cfg.dynamicSmemBytes = kPairSmem;
        if (cudaOccupancyMaxActiveClusters(&n_pairs, attn_pair_kernel, &cfg) != cudaSuccess || n_pairs <= 0) {
            (void)cudaGetLastError();
            n_pairs = 74;
        }
        if (dev >= 0 && dev < 64) pairs_cached[dev] = n_pairs;
    }
    const long long units = (long long)Hkv * a.n_layers * a.batch * p.n_row_groups;
    const long long max_tiles = (a.max_seq_len + kTileTokens - 1) / kTileTokens + 1;  // context tiles + the step's own tokens
    // How many pairs: all the device holds when there are at least as many units; with fewer units, k pairs per unit,
    // k chosen by a small cost model (microseconds): a pair's tiles one after the other, then the merge of the unit's k
    // partial results by the CTA that arrives last, one dependent round trip to L2 per partial result.
    long long use = n_pairs;
    p.pairs_per_unit = 0;
    if (units < n_pairs) {
        p.pairs_per_unit = 1;
        const double t_tile = 1.0, t_seg = 1.4;
        double best = 1e30;
        for (long long k = 1; k * units <= n_pairs && k <= max_tiles; ++k) {
            const double cost = (double)((max_tiles + k - 1) / k) * t_tile + (k > 1 ? k * t_seg : 0.0);
            if (cost < best) {
                best = cost;
                use = k * units;
                p.pairs_per_unit = (int)k;
            }
        }
    }
    // partial results: two slots of 256 rows per pair; arrival counters: two per unit
    const size_t slot_bytes = (size_t)256 * (kD + 2) * sizeof(float);
    if ((size_t)use * 2 * slot_bytes > a.partial_bytes) use = (long long)(a.partial_bytes / (2 * slot_bytes));  // fewer pairs: slower, same result
    if (use < 1 || (size_t)units * 2 * sizeof(int32_t) > a.counter_bytes) return SPECPV_ERR_CAPACITY;
    if (p.pairs_per_unit > 0) {  // keep k pairs per unit within what the scratch allows
        p.pairs_per_unit = (int)(use / units);
        use = p.pairs_per_unit * units;
    }
    char* ws = reinterpret_cast<char*>(a.workspace) + a.partial_off;
    p.part_o = reinterpret_cast<float*>(ws);
    p.part_ml = reinterpret_cast<float*>(ws + (size_t)use * 2 * 256 * kD * sizeof(float));
    p.counters = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(a.workspace) + a.counter_off);
    p.n_layers_call = a.n_layers;
    p.n_splits = 1;

    attn_pair_kernel<<<dim3((unsigned)(2 * use), 1, 1), kPairThreads, kPairSmem, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    return SPECPV_OK;
}

}  // namespace specpv
