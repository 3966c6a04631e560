// Block scores on the tensor cores (paper Eq. 2-3): s_i = f_r max(q_r . Kmax_i, q_r . Kmin_i) for
// bfloat16 summaries with head_dim 128, and the channel-wise form s_i = f_r sum_c max(q_rc Kmax_ic, q_rc Kmin_ic).
// Because Kmax >= Kmin in every channel, the channel-wise maximum takes Kmax where q is positive and Kmin where it
// is negative, so that form is the single contraction  Kmax . q+  +  Kmin . q-  with q+ = max(q, 0), q- = min(q, 0)
// (both exact in bfloat16): the CTA splits Q by sign in shared memory and accumulates both products into one
// accumulator.
//
// Per (layer, sequence, KV head) the two products are dense contractions
//     Dmax[128 blocks x R] = Kmax_tile[128 x 128] * Q^T[128 x R],   Dmin likewise with Kmin,
// issued as tcgen05.mma with both operands in shared memory (128-byte swizzle, loaded by TMA) and float32
// accumulators in tensor memory.
//
// The kernel is persistent: one CTA per SM takes an equal contiguous share of all 128-block tiles of the launch
// (layer-major, then sequence, KV head, tile), so a CTA sets up once and reloads Q only where its share crosses
// into another head.  Tensor memory holds two accumulator regions of 256 columns (one per query row): Dmax in the
// first, Dmin in the second.  Each product has its own issuing warp and its own stream of ring slots, so the barrier
// work of one overlaps the contractions of the other, and a region is free again as soon as the epilogue has READ it:
// Dmax is read into registers while the Dmin contractions run; Dmin is read in two round trips, only the maximum is
// taken, and its region is released before the reduction over the rows; the next tile's contractions run meanwhile.
// (The channel-wise form has one accumulator per tile: its tiles alternate between the two regions, issued by one warp.)
//   warp 0      TMA producer: Q of a head, then per tile its Kmax rows and its Kmin rows through a ring of 32 KB slots
//   warps 1, 2  MMA issue: Dmax / Dmin (warp 1 also allocates the tensor memory)
//   warps 4-11  epilogue: thread <-> block of the tile (tensor-memory lane) and one half of the query rows; reduces
//               over its rows (mean, max, or the rows of the "last" query); the two halves meet in shared memory, the
//               lower half picking the upper half's result up one tile later
// Every wait is bounded; after a wait that gave up the loops end and nothing more is copied or issued.
#include "aux_kernels.cuh"
#include "tc_common.cuh"

namespace specpv {

namespace {

using namespace tc;

constexpr int kScoreThreads = 384;       // 12 warps; the four control warps hand registers to the eight epilogue warps
constexpr int kScoreCtas = 148;          // one per SM
constexpr int kTileBlocks = 128;
constexpr int kSumTileBytes = 32768;     // a ring slot: the Kmax or the Kmin rows of a tile, [2 d-halves][128 blocks][64 d] bf16
constexpr int kScoreStages = 5;          // ring slots (the channel-wise form gives two of them to q-)
constexpr int kScoreQBytes = 65536;      // [2 d-halves][256 rows][64 d] bf16
constexpr int kScoreSmem = 1024 + kScoreQBytes + kScoreStages * kSumTileBytes;

struct ScoreTcParams {
    CUtensorMap tm_q;     // (d, Hq, tokens)  box (64, G, 128/G)
    CUtensorMap tm_kmax;  // (d, rows)        box (64, 128)
    CUtensorMap tm_kmin;
    const int32_t* q_lens;
    const int32_t* last_query;
    const int32_t* seq_lens;
    float* scores;
    void* workspace;
    int layer0, batch, M_max, Hkv, G, bs, max_blocks, reduce, n_cols;
    int tiles_max;    // tiles per head of the longest sequence: the launch's work is n_heads * tiles_max tile positions
    int n_heads;      // layers of the call * sequences * KV heads
    int tok0, tok_n;  // this pass covers step tokens [tok0, tok0 + tok_n): 256 query rows at most (the accumulator's columns)
    int accumulate;   // a later pass: combine with the scores the earlier passes left
};

struct __align__(8) ScoreBarriers {
    uint64_t q_full;                   // Q of a head has landed
    uint64_t q_empty;                  // the last contraction that reads this Q has completed
    uint64_t q_split;                  // channel-wise form: the eight epilogue warps have split Q by sign
    uint64_t sum_full[kScoreStages];
    uint64_t sum_empty[kScoreStages];
    uint64_t r_full[2];                // per accumulator region: the contractions of a tile are complete
    uint64_t r_empty[2];               // ... and the eight epilogue warps have read the region
    uint64_t x_full[3];                // the warps of the upper half of the query rows have left their partial results (tile mod 3)
    uint32_t tmem_base;
    int abort_flag;
};

// A stretch of tiles of one head that a CTA works on.
struct ScoreSeg {
    int lb, b, l, h;
    int t0, t1;                      // tiles [t0, t1) of the head
    int nb;                          // blocks of the sequence
    int col_begin, col_end, denom;   // query rows (accumulator columns) that count, and what the mean divides by
};

// Walks a CTA's share [x, x_end) of the launch's tile positions head by head.  Lengths live on the device, so every
// role works the stretches out for itself; all of them see the same sequence.
struct ScoreIter {
    long long x, x_end;
    __device__ void init(const ScoreTcParams& p) {
        const long long total = (long long)p.n_heads * p.tiles_max;
        x = total * blockIdx.x / gridDim.x;
        x_end = total * (blockIdx.x + 1) / gridDim.x;
    }
    __device__ bool next(const ScoreTcParams& p, ScoreSeg& s) {
        while (x < x_end) {
            const long long head = x / p.tiles_max;
            const long long stop = min(x_end, (head + 1) * p.tiles_max);
            s.t0 = (int)(x - head * p.tiles_max);
            x = stop;
            s.h = (int)(head % p.Hkv);
            s.lb = (int)(head / p.Hkv);
            s.b = s.lb % p.batch;
            s.l = s.lb / p.batch;
            const int seq_len = max(p.seq_lens[s.b], 0);
            s.nb = min((seq_len + p.bs - 1) / p.bs, p.max_blocks);
            s.t1 = min((int)(stop - head * p.tiles_max), (s.nb + kTileBlocks - 1) / kTileBlocks);
            int M = p.q_lens ? p.q_lens[s.b] : p.M_max;
            M = min(max(M, 0), p.M_max);
            // query rows r = token * G + head of this pass's tokens, one accumulator column each
            s.col_begin = 0;
            s.col_end = min(max(M - p.tok0, 0), p.tok_n) * p.G;
            s.denom = M * p.G;  // rows the mean runs over (all passes together)
            if (p.reduce == SPECPV_REDUCE_LAST) {
                int last = p.last_query ? p.last_query[s.b] : 0;
                last = min(max(last, 0), max(M - 1, 0));
                if (M <= 0 || last < p.tok0 || last >= p.tok0 + p.tok_n) continue;  // another pass holds that row
                s.col_begin = (last - p.tok0) * p.G;
                s.col_end = s.col_begin + p.G;
                s.denom = p.G;
            }
            if (s.col_end > s.col_begin && s.t1 > s.t0) return true;
        }
        return false;
    }
};

// dynamic + static shared memory of the kernel below must fit the 227 KB a CTA may have
static_assert(kScoreSmem + sizeof(ScoreBarriers) + 3 * kTileBlocks * sizeof(float) + 64 <= 227 * 1024, "shared memory of scores_tc_kernel");

// kCw: the channel-wise form (a compile-time switch).
template <bool kCw>
__global__ void __launch_bounds__(kScoreThreads, 1) scores_tc_kernel(const __grid_constant__ ScoreTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ ScoreBarriers bars;
    __shared__ float xch[3][kTileBlocks];  // partial results of the upper half of the query rows, by tile mod 3
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const uint32_t q_smem = smem_u32(smem);
    // channel-wise form: q- takes the place of two ring slots
    constexpr int stages = kCw ? kScoreStages - 2 : kScoreStages;
    const uint32_t qneg_smem = q_smem + kScoreQBytes;
    const uint32_t sum_smem = q_smem + (kCw ? 2 : 1) * kScoreQBytes;
    volatile int* abort_flag = &bars.abort_flag;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.q_full), 1);
        mbar_init(smem_u32(&bars.q_empty), 2);  // both issuing warps
        mbar_init(smem_u32(&bars.q_split), 8);  // one arrival per epilogue warp
        for (int s = 0; s < kScoreStages; ++s) {
            mbar_init(smem_u32(&bars.sum_full[s]), 1);
            mbar_init(smem_u32(&bars.sum_empty[s]), 1);
        }
        for (int r = 0; r < 2; ++r) {
            mbar_init(smem_u32(&bars.r_full[r]), 1);
            mbar_init(smem_u32(&bars.r_empty[r]), 8);
        }
        for (int x = 0; x < 3; ++x) mbar_init(smem_u32(&bars.x_full[x]), 4);
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

    // Register budget: 384 threads start with 168 registers each; the control warps keep 48, which is what lets the
    // epilogue warps grow to 224 (128 x 120 released, 256 x 56 taken).
    if (warp == 0) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        // ---- producer: the whole warp runs the loop (a lone lane of a diverged warp runs slowly), lane 0 copies ----
        const int n_q_tiles = p.n_cols > 128 ? 2 : 1;
        ScoreIter it;
        it.init(p);
        ScoreSeg s;
        uint32_t g = 0;  // tiles so far, across stretches
        bool ok = true;
        for (int sidx = 0; ok && it.next(p, s); ++sidx) {
            // Q may only be replaced once the contractions of the previous stretch have read it
            if (sidx > 0) ok &= mbar_wait(smem_u32(&bars.q_empty), (sidx - 1) & 1, abort_flag, p.workspace, 27);
            if (lane == 0 && ok) {
                const uint32_t qbar = smem_u32(&bars.q_full);
                mbar_expect_tx(qbar, (uint32_t)(n_q_tiles * 32768));
                for (int t = 0; t < n_q_tiles; ++t)
                    for (int half = 0; half < 2; ++half)
                        tma_load_3d(q_smem + half * 32768 + t * 16384, &p.tm_q, half * 64, s.h * p.G,
                                    s.lb * p.M_max + p.tok0 + t * tok_per_tile, qbar);
            }
            __syncwarp();
            const int row0 = (((p.layer0 + s.l) * p.batch + s.b) * p.Hkv + s.h) * p.max_blocks;
            for (int t = s.t0; t < s.t1 && ok; ++t, ++g) {
                for (uint32_t which = 0; which < 2; ++which) {  // the Kmax rows of the tile, then its Kmin rows
                    const uint32_t u = 2 * g + which, slot = u % stages;
                    if (u >= (uint32_t)stages)
                        ok &= mbar_wait(smem_u32(&bars.sum_empty[slot]), ((u / stages) - 1) & 1, abort_flag, p.workspace, 21);
                    if (lane == 0 && ok) {
                        const uint32_t full = smem_u32(&bars.sum_full[slot]);
                        mbar_expect_tx(full, kSumTileBytes);
                        const uint32_t dst = sum_smem + slot * kSumTileBytes;
                        const int row = row0 + t * kTileBlocks;
                        for (int half = 0; half < 2; ++half)
                            tma_load_2d(dst + half * 16384, which ? &p.tm_kmin : &p.tm_kmax, half * 64, row, full);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp == 1 || warp == 2) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        // ---- MMA issue: warp 1 issues Kmax . Q into region 0, warp 2 Kmin . Q into region 1.  The whole warp runs the
        // loop, lane 0 issues.  A thread that issues also waits and commits, and the tensor pipe queues next to
        // nothing ahead, so the barrier work of one warp overlaps the contractions of the other.
        // A warp meets every other use of a ring slot (five slots, uses alternate between Kmax and Kmin), so it
        // waits on the same parity each time; that is sound because the use in between has completed by then: a warp
        // can issue tile g - 1 only after the epilogue has reached tile g - 2, hence after the other warp's
        // contractions of tile g - 3, whose slot use is the one in between.
        // Channel-wise form: one accumulator per tile, so warp 1 issues every tile, alternating between the regions
        // (a warp that took every other tile would skip ring-slot phases without that guarantee); warp 2 only
        // takes part in releasing Q.
        // descriptors: constant upper word (8-row group stride 1024 B, version, 128-byte swizzle); lower word =
        // 16-byte address, leading offset 16 B
        const uint32_t w = (uint32_t)(warp - 1);
        const uint32_t desc_hi = (uint32_t)((1024u >> 4) | (1u << 14) | (2u << 29));
        const uint32_t q_lo = ((q_smem >> 4) & 0x3FFFu) | (1u << 16);
        const uint32_t sum_lo = ((sum_smem >> 4) & 0x3FFFu) | (1u << 16);
        const uint32_t qneg_lo = ((qneg_smem >> 4) & 0x3FFFu) | (1u << 16);
        const uint32_t idesc = make_idesc((uint32_t)p.n_cols, false);

        ScoreIter it;
        it.init(p);
        ScoreSeg s;
        uint32_t g = 0;  // tiles so far, across stretches
        bool ok = true;
        for (int sidx = 0; ok && it.next(p, s); ++sidx) {
            ok &= mbar_wait(smem_u32(&bars.q_full), sidx & 1, abort_flag, p.workspace, 20);
            if (kCw) ok &= mbar_wait(smem_u32(&bars.q_split), sidx & 1, abort_flag, p.workspace, 25);
            for (int t = s.t0; t < s.t1; ++t, ++g) {
                if (!kCw || w == 0) {
                    const uint32_t r = kCw ? (g & 1u) : w;    // accumulator region of this tile
                    const uint32_t use = kCw ? (g >> 1) : g;  // earlier uses of that region
                    const uint32_t d = tmem + r * 256u;
                    const uint32_t rfull = smem_u32(&bars.r_full[r]), rempty = smem_u32(&bars.r_empty[r]);
                    const uint32_t u0 = kCw ? 2 * g : 2 * g + w, s0 = u0 % stages;
                    const uint32_t u1 = 2 * g + 1, s1 = u1 % stages;  // channel-wise only: the tile's Kmin rows
                    ok &= mbar_wait(smem_u32(&bars.sum_full[s0]), (u0 / stages) & 1, abort_flag, p.workspace, 22);
                    if (kCw) ok &= mbar_wait(smem_u32(&bars.sum_full[s1]), (u1 / stages) & 1, abort_flag, p.workspace, 22);
                    if (use > 0) ok &= mbar_wait(rempty, (use - 1) & 1, abort_flag, p.workspace, 23);
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t a0 = sum_lo + s0 * (kSumTileBytes >> 4), a1 = sum_lo + s1 * (kSumTileBytes >> 4);
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t a_off = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                            const uint32_t b_off = (uint32_t)((kk >> 2) * 32768 + (kk & 3) * 32) >> 4;
                            mma_ss(d, ((uint64_t)desc_hi << 32) | (a0 + a_off), ((uint64_t)desc_hi << 32) | (q_lo + b_off), idesc, kk > 0);
                            // channel-wise: Kmin . q- joins Kmax . q+ in the same accumulator
                            if (kCw)
                                mma_ss(d, ((uint64_t)desc_hi << 32) | (a1 + a_off), ((uint64_t)desc_hi << 32) | (qneg_lo + b_off), idesc, 1);
                        }
                        tc_commit(rfull);
                        tc_commit(smem_u32(&bars.sum_empty[s0]));
                        if (kCw) tc_commit(smem_u32(&bars.sum_empty[s1]));
                    }
                }
                // Q is released by both warps: each commit covers the contractions its own thread has issued
                if (t == s.t1 - 1 && lane == 0) tc_commit(smem_u32(&bars.q_empty));
                __syncwarp();
                if (!ok) break;  // a wait gave up: nothing is issued past this tile
            }
        }
    } else if (warp == 3) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        // ---- epilogue: thread <-> (block of the tile, half of the query rows) ------------------------------------
        const int q = warp & 3;           // tensor-memory lane quarter of this warp
        const int ch = (warp - 4) >> 2;   // its half of the query rows: accumulator columns [ch * 128, ch * 128 + 128)
        const int blk_in_tile = q * 32 + lane;
        const uint32_t my_cols = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(ch * 128);
        const bool is_max = p.reduce == SPECPV_REDUCE_MAX;
        const bool combine = p.accumulate && p.reduce != SPECPV_REDUCE_LAST;
        ScoreIter it;
        it.init(p);
        ScoreSeg s;
        uint32_t g = 0;
        bool ok = true;
        // lower half: the tile whose exchange with the upper half is still to come
        bool have_prev = false;
        float prev_red = 0.f, prev_denom = 1.f;
        uint32_t xs = 0, xp = 0, prev_xs = 0, prev_xp = 0;  // exchange slot (tile mod 3) and its parity, now and of the pending tile
        float* prev_dst = nullptr;
        auto finish_prev = [&]() -> bool {
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.x_full[prev_xs]), prev_xp, abort_flag, p.workspace, 28)))
                return false;
            float red = xch[prev_xs][blk_in_tile];
            red = is_max ? fmaxf(prev_red, red) : prev_red + red;
            if (prev_dst) {
                if (p.reduce != SPECPV_REDUCE_MAX) red /= prev_denom;
                if (combine) red = is_max ? fmaxf(red, *prev_dst) : red + *prev_dst;
                *prev_dst = red;
            }
            have_prev = false;
            return true;
        };
        for (int sidx = 0; ok && it.next(p, s); ++sidx) {
            if (kCw) {
                // split Q by sign in place: q+ stays where Q landed, q- goes to the buffer behind it (same swizzled layout,
                // the split is element-wise).  A bfloat16 is negative when its top bit is set.
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.q_full), sidx & 1, abort_flag, p.workspace, 26));
                if (!ok) break;
                uint4* qp = reinterpret_cast<uint4*>(smem);
                uint4* qn = reinterpret_cast<uint4*>(smem + kScoreQBytes);
                for (int v = threadIdx.x - 128; v < kScoreQBytes / 16; v += 256) {
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
            // the rows of this thread's half that count: columns [lo, hi) of its 128
            const int lo = max(s.col_begin - ch * 128, 0), hi = min(s.col_end - ch * 128, 128);
            for (int t = s.t0; t < s.t1 && ok; ++t, ++g) {
                // four independent partial reductions: a single chain through one register would leave the warp
                // waiting out the latency of every instruction
                float r4[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) r4[e] = is_max ? -INFINITY : 0.f;
                // one 32-column chunk of scores sc[k] = column c0 + k of this thread's half
                auto reduce_chunk = [&](int c0, const float* sc) {
                    if (c0 + 32 <= lo || c0 >= hi) return;  // warp-uniform
                    if (c0 >= lo && c0 + 32 <= hi) {
                        if (!is_max) {
#pragma unroll
                            for (int k = 0; k < 32; ++k) r4[k & 3] += sc[k];
                        } else {
#pragma unroll
                            for (int k = 0; k < 32; ++k) r4[k & 3] = fmaxf(r4[k & 3], sc[k]);
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            if (c0 + k >= lo && c0 + k < hi) r4[k & 3] = is_max ? fmaxf(r4[k & 3], sc[k]) : r4[k & 3] + sc[k];
                    }
                };
                if (!kCw) {
                    // Dmax of this half into registers, and its region is free for the next tile at once
                    uint32_t hold[128];
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.r_full[0]), g & 1, abort_flag, p.workspace, 24));
                    if (!ok) break;
                    tc_fence_after();
                    if (lo < hi) {
                        TMEM_LD32(my_cols, hold);
                        TMEM_LD32(my_cols + 32, (hold + 32));
                        TMEM_LD32(my_cols + 64, (hold + 64));
                        TMEM_LD32(my_cols + 96, (hold + 96));
                        tmem_wait_ld();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.r_empty[0]));
                    // while the Dmin contractions of this tile run: the lower half finishes the previous tile
                    if (ch == 0 && have_prev) {
                        ok = finish_prev();
                        if (!ok) break;
                    }
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.r_full[1]), g & 1, abort_flag, p.workspace, 24));
                    if (!ok) break;
                    tc_fence_after();
                    // Dmin in two round trips of 64 columns (a round trip to tensor memory costs about 300 cycles while the
                    // tensor pipe is writing the other region, whatever it carries); only the maximum is taken before the
                    // region is released, the reduction over the rows follows from registers
                    if (lo < hi) {
#pragma unroll
                        for (int c2 = 0; c2 < 2; ++c2) {
                            if (c2 * 64 + 64 <= lo || c2 * 64 >= hi) continue;  // warp-uniform
                            uint32_t v[64];
                            TMEM_LD32(my_cols + 256 + c2 * 64, v);
                            TMEM_LD32(my_cols + 256 + c2 * 64 + 32, (v + 32));
                            tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 64; ++k)
                                hold[c2 * 64 + k] = __float_as_uint(fmaxf(__uint_as_float(hold[c2 * 64 + k]), __uint_as_float(v[k])));
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.r_empty[1]));
                    if (lo < hi) {
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) reduce_chunk(c4 * 32, reinterpret_cast<const float*>(hold + c4 * 32));
                    }
                } else {
                    // one accumulator holds the score; the tiles alternate between the regions
                    const uint32_t r = g & 1u;
                    if (ch == 0 && have_prev) {
                        ok = finish_prev();
                        if (!ok) break;
                    }
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.r_full[r]), (g >> 1) & 1, abort_flag, p.workspace, 24));
                    if (!ok) break;
                    tc_fence_after();
                    // the whole half in one round trip to tensor memory, the region released before the reduction
                    uint32_t v[128];
                    if (lo < hi) {
                        TMEM_LD32(my_cols + r * 256u, v);
                        TMEM_LD32(my_cols + r * 256u + 32, (v + 32));
                        TMEM_LD32(my_cols + r * 256u + 64, (v + 64));
                        TMEM_LD32(my_cols + r * 256u + 96, (v + 96));
                        tmem_wait_ld();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.r_empty[r]));
                    if (lo < hi) {
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) reduce_chunk(c4 * 32, reinterpret_cast<const float*>(v + c4 * 32));
                    }
                }
                const float red = is_max ? fmaxf(fmaxf(r4[0], r4[1]), fmaxf(r4[2], r4[3])) : (r4[0] + r4[1]) + (r4[2] + r4[3]);
                // The two halves of the query rows meet in shared memory, in one of three slots (tile mod 3).  The upper half
                // leaves its partial result; the lower half keeps its own and picks the other up one tile later, so that it
                // never waits for the upper half inside a tile.  The slot of tile g is rewritten at tile g + 3, whose
                // contractions cannot start before every warp has released a region of tile g + 2 (Dmax) or g + 1
                // (channel-wise form), which the lower half does after its exchange of tile g.
                if (ch == 1) {
                    xch[xs][blk_in_tile] = red;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.x_full[xs]));
                } else {
                    const int blk = t * kTileBlocks + blk_in_tile;
                    prev_red = red;
                    prev_xs = xs;
                    prev_xp = xp;
                    prev_denom = (float)s.denom;
                    prev_dst = blk < s.nb ? p.scores + ((size_t)s.lb * p.Hkv + s.h) * p.max_blocks + blk : nullptr;
                    have_prev = true;
                }
                if (++xs == 3) { xs = 0; xp ^= 1; }
            }
        }
        if (ok && ch == 0 && have_prev) ok = finish_prev();
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
    // one CTA per SM, each with an equal share of all tile positions; fewer CTAs when there are fewer tiles than SMs
    p.tiles_max = (max_nb + kTileBlocks - 1) / kTileBlocks;
    p.n_heads = sp.Hkv * n_layers_call * sp.batch;
    const long long total = (long long)p.n_heads * p.tiles_max;
    dim3 grid((unsigned)(total < kScoreCtas ? total : kScoreCtas), 1, 1);
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
