// Tensor-core verification attention for B200 (sm_100a): bfloat16, head_dim 128, pages of 16, 32 or 64 tokens.
// Tree-masked GQA attention of the step's tokens over a paged cache (paper Section 3.2-3.3,
// Algorithm 1 "TreeDecode"), used for both the partial and the full cache.
//
// One CTA owns one (layer, sequence, KV head, KV split, row group).  All G query heads of the KV
// head times up to 2*(128/G) step tokens are packed into two 128-row tiles, so QK^T and PV are
// dense 128x128x128 contractions:
//   warp 0      TMA producer: Q once, then K and V tiles of 128 tokens (2, 4 or 8 pages, one copy per page
//               and 64-channel half, each issued by its own lane) through the block table into a ring of
//               32 KB shared-memory slots (128-byte swizzle)
//   warp 1      MMA issuer: tcgen05.mma  S_t = Q_t K^T  (both operands in shared memory) and
//               O_t += P_t V (P read from tensor memory, V MN-major from shared memory)
//   warps 4-7   softmax of row tile 0, warps 8-11 of row tile 1: one thread per row reads S from
//               tensor memory, keeps the running max / sum of an online softmax in the log2
//               domain, writes P (bfloat16) over S, rescales O only when the max grew by > 2^8,
//               and finally normalises O and writes it out
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 columns each, P_t aliases S_t.
// With several KV splits the unnormalised (O, m, l) go to the workspace and merge_kernel combines
// them by log-sum-exp.  Every wait is bounded; a wait that gives up records SPECPV_ERR_TIMEOUT.
#include "attn_tc.cuh"

namespace specpv {

namespace {

constexpr int kThreadsTc = 384;          // 12 warps
constexpr int kSlotBytes = 32768;        // one K or V tile: [2 d-halves][128 tokens][64 d] bf16
constexpr int kStages = 5;
constexpr int kQBytes = 2 * 32768;       // two row tiles
constexpr int kSmemBytes = 1024 + kQBytes + kStages * kSlotBytes;

using namespace tc;

// Instruction descriptor, kind::f16: D = f32, A = B = bf16, M = 128, N = 128.
constexpr uint32_t kIdescQK = make_idesc(128, false);
constexpr uint32_t kIdescPV = make_idesc(128, true);  // B (= V) is MN-major

struct __align__(8) Barriers {
    uint64_t q_full;
    uint64_t kv_full[kStages];  // a K or V tile has landed in its slot
    uint64_t kv_empty[kStages]; // every contraction that reads the slot has completed (one barrier per slot: a barrier
                                // shared by all slots could run two phases ahead of the producer, which a parity
                                // wait cannot tell from none)
    uint64_t s_full[2];         // phase j: S_t(j) = Q_t K_j^T is complete
    uint64_t p_full[2];         // phase j: the four softmax warps of row tile t have stored P_t(j)
    uint64_t o_done[2];         // the last PV of row tile t has completed
    uint64_t v_need;            // MMA issuer -> warp 2: this V tile has landed and needs its tail rows zeroed
    uint64_t v_fixed;           // warp 2 -> MMA issuer: done
    uint64_t drain;             // completion of the contractions issued before a wait gave up
    uint32_t tmem_base;
    int abort_flag;
};

// =================================================================================================
__global__ void __launch_bounds__(kThreadsTc, 1) attn_tc_kernel(const __grid_constant__ TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the 128-byte swizzle atoms
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Barriers bars;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = blockIdx.x % p.n_splits, rg = blockIdx.x / p.n_splits;
    const int h = blockIdx.y, lb = blockIdx.z;
    const int b = lb % p.batch, l = lb / p.batch;

    const int seq_len = max(p.seq_lens[b], 0);
    int M = p.q_lens ? p.q_lens[b] : p.M_max;
    M = min(max(M, 0), p.M_max);
    const int tok_per_tile = 128 / p.G;               // step tokens per 128-row tile
    const int tok0 = rg * 2 * tok_per_tile;           // first step token of this row group
    if (tok0 >= M) return;                            // nothing to do (uniform for the CTA)
    const int n_q_tiles = (M - tok0 > tok_per_tile) ? 2 : 1;

    // KV range of this split: whole 128-token tiles, split evenly over the sequence's tiles
    const int total_tiles = (seq_len + kTileTokens - 1) / kTileTokens;
    const int tiles_per_split = (total_tiles + p.n_splits - 1) / p.n_splits;
    const int tile_begin = min(split * tiles_per_split, total_tiles);
    const int tile_end = min(tile_begin + tiles_per_split, total_tiles);
    const bool last_split = split == p.n_splits - 1;
    const int n_ctx_tiles = tile_end - tile_begin;
    const int n_tiles = n_ctx_tiles + (last_split ? 1 : 0);  // the last split also attends the step's own tokens
    // first tile whose V rows need zeroing past the valid tokens: a ragged last context tile, else the
    // tile of the step's own tokens (fewer than 128), else none
    const bool ragged_ctx = n_ctx_tiles > 0 && tile_end == total_tiles && (seq_len % kTileTokens) != 0;
    const int first_fix = ragged_ctx ? n_ctx_tiles - 1 : ((last_split && M < kTileTokens) ? n_ctx_tiles : n_tiles);

    const uint32_t q_smem = smem_u32(smem);
    const uint32_t kv_smem = q_smem + kQBytes;
    volatile int* abort_flag = &bars.abort_flag;

    if (n_tiles == 0) {
        // an empty split: publish (m = -inf, l = 0) so that the merge ignores it
        for (int r = threadIdx.x; r < 256; r += kThreadsTc) {
            const int row = rg * 256 + r;
            if (row < p.R_pad) {
                const size_t prow = (((size_t)lb * p.Hkv + h) * p.n_splits + split) * p.R_pad + row;
                p.part_ml[prow * 2] = -INFINITY;
                p.part_ml[prow * 2 + 1] = 0.f;
            }
        }
        return;
    }

    // ---- set-up ------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.q_full), 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars.kv_full[s]), 1);
            mbar_init(smem_u32(&bars.kv_empty[s]), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bars.s_full[t]), 1);
            mbar_init(smem_u32(&bars.p_full[t]), 4);  // one arrival per softmax warp
            mbar_init(smem_u32(&bars.o_done[t]), 1);
        }
        mbar_init(smem_u32(&bars.v_need), 1);
        mbar_init(smem_u32(&bars.v_fixed), 1);
        mbar_init(smem_u32(&bars.drain), 1);
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
    // tensor-memory columns: S_t at t*128, O_t at 256 + t*128; P_t aliases S_t (64 columns of bf16 pairs)

    // Register budget: the control warpgroup (warps 0-3) gives registers to the two softmax warpgroups.
    if (warp == 0) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        // =========================== TMA producer ================================================
        // The whole warp runs the loop (a lone lane of a diverged warp runs slowly); lane 0 issues the copies.
        const uint32_t qbar = smem_u32(&bars.q_full);
        if (lane == 0) {
            mbar_expect_tx(qbar, (uint32_t)(n_q_tiles * 32768));
            for (int t = 0; t < n_q_tiles; ++t)
                for (int half = 0; half < 2; ++half)
                    tma_load_3d(q_smem + t * 32768 + half * 16384, &p.tm_q, half * 64, h * p.G,
                                lb * p.M_max + tok0 + t * tok_per_tile, qbar);
        }
        __syncwarp();
        const int32_t* table = p.block_table + (size_t)b * p.max_blocks;
        const long long layer_row0 = (long long)(p.layer0 + l) * p.n_pages;
        bool ok = true;
        // Pool row coordinate of a context tile's pages (128 / page size of them).  Lane 2 pg + half looks page pg
        // up and later issues the copy of that page's 64-channel half, so that a tile's copies leave in one pass of
        // the warp; the table is read one tile ahead so that its latency hides behind the wait for a free slot.
        const int ppt = kTileTokens / p.bs;
        const int my_pg = lane >> 1, my_half = lane & 1;
        auto page_row = [&](int j) {
            int row = (int)p.pool_rows;  // out of range: the copy engine fills zeros
            const int blk = (tile_begin + j) * ppt + my_pg;
            if (my_pg < ppt && j < n_ctx_tiles && (long long)blk * p.bs < seq_len && blk < p.max_blocks) {
                const int page = table[blk];
                if (page < 0 || page >= p.n_pages) {
                    if (my_half == 0) record_fault(p.workspace, SPECPV_ERR_BAD_BLOCK_TABLE, b, blk, page, l);
                } else {
                    row = (int)(((layer_row0 + page) * p.Hkv + h) * p.bs);
                }
            }
            return row;
        };
        int row_next = page_row(0);
        uint32_t slot = 0, par = 1;  // ring position of the next use; parity of the release that frees its slot
        for (int j = 0; j < n_tiles; ++j) {
            const bool is_new = j >= n_ctx_tiles;
            const int row_mine = row_next;
            row_next = page_row(j + 1);
            for (int kv = 0; kv < 2; ++kv) {  // 0: K tile, 1: V tile
                const uint32_t full = smem_u32(&bars.kv_full[slot]), empty = smem_u32(&bars.kv_empty[slot]);
                if (2 * j + kv >= kStages) ok = mbar_wait(empty, par, abort_flag, p.workspace, 1);
                if (!ok) break;  // a wait gave up: nothing more is copied
                const uint32_t dst = kv_smem + slot * kSlotBytes + my_half * 16384;
                if (lane == 0) mbar_expect_tx(full, kSlotBytes);
                if (is_new) {  // the step's own tokens: two boxes of 64 rows per half
                    if (lane < 4)
                        tma_load_3d(dst + my_pg * 8192, kv ? &p.tm_vnew : &p.tm_knew, my_half * 64, h, lb * p.M_max + my_pg * 64,
                                    full);
                } else if (my_pg < ppt) {
                    tma_load_2d(dst + my_pg * p.bs * 128, kv ? &p.tm_vpool : &p.tm_kpool, my_half * 64, row_mine, full);
                }
                __syncwarp();
                if (++slot == kStages) { slot = 0; par ^= 1; }
            }
            if (!ok) break;
        }
    } else if (warp == 1) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        // =========================== MMA issuer ==================================================
        // One warp issues every contraction (issuing from two warps serialises the tensor pipe).  Issue
        // order (ping-pong of the two row tiles): QK(0,0) QK(0,1) | PV(0,0) QK(1,0) PV(0,1) QK(1,1) | ...
        // Barrier instructions do not overlap with queued MMAs (each costs the pipe 30-100 idle cycles),
        // so the loop keeps them to four waits per KV tile, without votes, and four commits behind MMAs.  The whole
        // warp runs the loop, lane 0 issues.
        bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.q_full), 0, abort_flag, p.workspace, 2));
        // Shared-memory descriptors: the upper word (stride between 8-row groups, version, swizzle) is
        // constant; the lower word is the 16-byte address plus the leading-dimension offset.
        const uint32_t desc_hi = (uint32_t)((1024u >> 4) | (1u << 14) | (2u << 29));
        const uint32_t q_lo = ((q_smem >> 4) & 0x3FFFu) | ((16u >> 4) << 16);
        const uint32_t k_lo0 = ((kv_smem >> 4) & 0x3FFFu) | ((16u >> 4) << 16);
        const uint32_t v_lo0 = ((kv_smem >> 4) & 0x3FFFu) | ((16384u >> 4) << 16);
        const uint32_t full0 = smem_u32(&bars.kv_full[0]), empty0 = smem_u32(&bars.kv_empty[0]);
        const uint32_t sfull0 = smem_u32(&bars.s_full[0]), pfull0 = smem_u32(&bars.p_full[0]);
        // ring position of K tile j (use 2j) and of V tile j-1 (use 2j-1): slot and phase parity
        uint32_t k_slot = 0, k_par = 0, v_slot = 1, v_par = 0;
        for (int j = 0; j <= n_tiles; ++j) {
            const int jp = j - 1;
            // A wait that gives up raises the abort flag, which makes the later waits of this tile return at once; the
            // loop ends after this tile, so at most one tile's contractions are issued past the failed wait.  (One exit
            // per tile: an exit after every wait costs the issuing thread 7 % of the kernel.)
            if (j < n_tiles) ok &= mbar_wait(full0 + k_slot * 8, k_par, abort_flag, p.workspace, 3);
            if (j > 0) {
                ok &= mbar_wait(full0 + v_slot * 8, v_par, abort_flag, p.workspace, 4);
                // a ragged or tree tile: warp 2 zeroes the rows of V past the valid tokens first
                if (jp >= first_fix) {
                    if (lane == 0) mbar_arrive(smem_u32(&bars.v_need));
                    ok &= mbar_wait(smem_u32(&bars.v_fixed), (jp - first_fix) & 1, abort_flag, p.workspace, 9);
                }
            }
            const uint32_t kb_lo = launder(k_lo0 + k_slot * (kSlotBytes >> 4));
            const uint32_t vb_lo = launder(v_lo0 + v_slot * (kSlotBytes >> 4));
            for (int t = 0; t < n_q_tiles; ++t) {
                if (j > 0) {
                    ok &= mbar_wait(pfull0 + t * 8, jp & 1, abort_flag, p.workspace, 5);
                    tc_fence_after();
                }
                if (lane == 0) {
                    if (j > 0) {  // O_t += P_t V_{j-1}
                        const uint32_t a = tmem + t * 128, d = tmem + 256 + t * 128;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)  // 16 tokens per instruction: two 8-row K groups of 1024 bytes
                            mma_ts_lohi(d, a + kk * 8, vb_lo + (uint32_t)kk * (2048u >> 4), desc_hi, kIdescPV,
                                        (jp > 0 || kk > 0) ? 1u : 0u);
                        if (t == n_q_tiles - 1) tc_commit(empty0 + v_slot * 8);
                        if (j == n_tiles) tc_commit(smem_u32(&bars.o_done[t]));
                    }
                    if (j < n_tiles) {  // S_t = Q_t K_j^T
                        const uint32_t a_lo = launder(q_lo + (uint32_t)t * (32768u >> 4));
                        const uint32_t d = tmem + t * 128;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {  // 16 channels of d per instruction
                            const uint32_t off = (uint32_t)((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                            mma_ss_lohi(d, a_lo + off, kb_lo + off, desc_hi, kIdescQK, kk > 0 ? 1u : 0u);
                        }
                        tc_commit(sfull0 + t * 8);
                        if (t == n_q_tiles - 1) tc_commit(empty0 + k_slot * 8);
                    }
                }
                __syncwarp();
            }
            if (!ok) break;
            if (j < n_tiles) { k_slot += 2; if (k_slot >= kStages) { k_slot -= kStages; k_par ^= 1; } }
            if (j > 0) { v_slot += 2; if (v_slot >= kStages) { v_slot -= kStages; v_par ^= 1; } }
        }
        if (!ok && lane == 0) {
            // after a give-up: wait (bounded) until the contractions that WERE issued have completed, so that the
            // tensor memory is not freed under them
            tc_commit(smem_u32(&bars.drain));
            const uint64_t t0 = global_ns();
            while (!mbar_try_wait(smem_u32(&bars.drain), 0) && global_ns() - t0 < 100000000ull) {}
        }
        __syncwarp();
    } else if (warp == 2) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        // =========================== V fixer =====================================================
        // Rows of a V tile past its valid tokens may hold anything (stale shared memory, rows of other
        // sequences' steps): zero them so that 0 * garbage cannot produce NaN.  Only the last context
        // tile (when ragged) and the tile of the step's own tokens can need it.
        for (int jp = first_fix; jp < n_tiles; ++jp) {
            const int use = 2 * jp + 1;
            // the request arrives once the tile has landed (a wait on the slot's own barrier this far
            // ahead of the pipeline could match an earlier phase of the same parity)
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.v_need), (jp - first_fix) & 1, abort_flag, p.workspace, 10)))
                break;
            const int n_valid = jp >= n_ctx_tiles ? M : min(kTileTokens, seq_len - (tile_begin + jp) * kTileTokens);
            uint8_t* v = smem + kQBytes + (size_t)(use % kStages) * kSlotBytes;
            const int n_rows = kTileTokens - n_valid;
            for (int i = lane; i < n_rows * 2 * 8; i += 32) {
                const int chunk = i & 7, half = (i >> 3) & 1, r = n_valid + (i >> 4);
                *reinterpret_cast<uint4*>(v + half * 16384 + r * 128 + chunk * 16) = make_uint4(0, 0, 0, 0);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.v_fixed));
        }
    } else if (warp == 3) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        // =========================== softmax / correction / epilogue ==============================
        const int t = (warp - 4) >> 2;           // row tile of this warpgroup
        const int q = warp & 3;                  // TMEM lane quarter this warp may access
        const int row_in_tile = q * 32 + lane;
        if (t < n_q_tiles) {
            const int row = t * 128 + row_in_tile;                 // row within the row group
            const int tok = tok0 + row / p.G;                      // step token of this row
            const int g = row % p.G;
            const bool row_valid = tok < M;
            const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
            const uint32_t s_addr = tmem + lane_addr + t * 128;
            const uint32_t o_addr = tmem + lane_addr + 256 + t * 128;
            uint64_t mask_lo = 0, mask_hi = 0;
            if (row_valid) {
                const uint64_t* mrow = p.tree_mask + ((size_t)b * p.M_max + tok) * p.mask_words;
                mask_lo = mrow[0];
                if (p.mask_words > 1) mask_hi = mrow[1];
            }
            float m_run = -INFINITY, l_run = 0.f;
            bool ok = true;
            const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
            for (int j = 0; j < n_tiles && ok; ++j) {
                const bool is_new = j >= n_ctx_tiles;
                const int n_valid = is_new ? M : min(kTileTokens, seq_len - (tile_begin + j) * kTileTokens);
                const bool masked = is_new || n_valid < kTileTokens;
                uint64_t vis_lo = ~0ull, vis_hi = ~0ull;  // visibility of the tile's 128 columns for this row
                if (masked) {
                    if (is_new) {
                        vis_lo = mask_lo;
                        vis_hi = mask_hi;
                    }
                    if (n_valid < 64) {
                        vis_lo &= (n_valid <= 0) ? 0ull : (~0ull >> (64 - n_valid));
                        vis_hi = 0;
                    } else if (n_valid < 128) {
                        vis_hi &= (n_valid == 64) ? 0ull : (~0ull >> (128 - n_valid));
                    }
                }
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.s_full[t]), j & 1, abort_flag, p.workspace, 6));
                if (!ok) break;
                tc_fence_after();
                // the whole row of S (128 columns) goes to registers in one round trip
                uint32_t v[128];
                TMEM_LD32(s_addr, v);
                TMEM_LD32(s_addr + 32, (v + 32));
                TMEM_LD32(s_addr + 64, (v + 64));
                TMEM_LD32(s_addr + 96, (v + 96));
                tmem_wait_ld();
                // P = 2^(s*scale - m) as bf16 pairs, packed in place: word i of P (columns 2i, 2i+1) overwrites
                // v[i], whose own value was consumed by an earlier pair, so no second register array is needed.
                // The row sum is taken over the ROUNDED weights the tensor core will use, so that O / l is an
                // exact weighted average of V rows (the rounding error of a dominant weight cancels instead of
                // scaling the output).
                auto exp_row = [&](float m_use) {
                    const float2 nm2 = make_float2(-m_use, -m_use);
                    float2 sum2[4];  // independent partial sums: one chain of 64 dependent adds would outlast the exponentials
#pragma unroll
                    for (int e = 0; e < 4; ++e) sum2[e] = make_float2(0.f, 0.f);
#pragma unroll
                    for (int i = 0; i < 64; ++i) {
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])),
                                                    sc2, nm2);
                        const uint32_t w = pack_bf16(ex2(x.x), ex2(x.y));
                        v[i] = w;
                        add_bf16_pair(sum2[i & 3], w);
                    }
                    const float2 s01 = __fadd2_rn(sum2[0], sum2[1]), s23 = __fadd2_rn(sum2[2], sum2[3]);
                    return (s01.x + s23.x) + (s01.y + s23.y);
                };
                // Fast path (every full context tile after the first): keep the reference m_run of the row as it
                // is and skip the row maximum.  Weights may then exceed 1; float32 sums and bf16 weights keep
                // their relative precision whatever the exponent, so only overflow has to be ruled out: if a
                // row sum leaves the safe range (or a row has no reference yet), the warp takes the tile again
                // from tensor memory on the general path, which brings m_run up to date.
                float l_add = 0.f;
                bool general = j == 0 || masked;
                if (!general) {
                    l_add = exp_row(m_run);
                    const bool bad = !(l_add < kSafeRowSum) || m_run == -INFINITY;
                    if (__any_sync(0xffffffffu, bad)) {
                        general = true;  // S_t is still intact: P has not been stored yet
                        TMEM_LD32(s_addr, v);
                        TMEM_LD32(s_addr + 32, (v + 32));
                        TMEM_LD32(s_addr + 64, (v + 64));
                        TMEM_LD32(s_addr + 96, (v + 96));
                        tmem_wait_ld();
                    }
                }
                if (general) {
                    if (masked) {  // ragged or tree-masked tile: invisible columns become -inf (at most two tiles per CTA)
#pragma unroll
                        for (int i = 0; i < 128; ++i) {
                            const uint64_t word = i < 64 ? vis_lo : vis_hi;
                            if (!((word >> (i & 63)) & 1ull)) v[i] = 0xff800000u;
                        }
                    }
                    float mx0 = __uint_as_float(v[0]), mx1 = __uint_as_float(v[1]), mx2 = __uint_as_float(v[2]),
                          mx3 = __uint_as_float(v[3]);
#pragma unroll
                    for (int i = 4; i < 124; i += 8) {  // three-input max: two new values per instruction
                        mx0 = fmax3(mx0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                        mx1 = fmax3(mx1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
                        mx2 = fmax3(mx2, __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
                        mx3 = fmax3(mx3, __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
                    }
                    mx0 = fmax3(mx0, __uint_as_float(v[124]), __uint_as_float(v[125]));
                    mx1 = fmax3(mx1, __uint_as_float(v[126]), __uint_as_float(v[127]));
                    const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                    const float m_tile = mx * p.scale_log2;
                    // lazy rescale: keep the old reference max unless the new one is more than 2^8 larger.
                    // The decision is per row, the tensor-memory traffic is warp-wide: if any row of the
                    // warp rescales, all 32 rows pass through it (with a factor of 1 where nothing changes).
                    bool need = false;
                    if (j == 0) {
                        m_run = m_tile;
                    } else {
                        need = m_tile > m_run + kRescaleThreshold || (m_run == -INFINITY && m_tile > -INFINITY);
                    }
                    if (__any_sync(0xffffffffu, need)) {
                        const float factor = !need ? 1.f : (m_run == -INFINITY ? 0.f : ex2(m_run - m_tile));
                        // O_t already holds every earlier PV: the tensor pipe runs in order, and S_t(j), issued
                        // after PV(j-1,t), is complete
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t o[32];
                            TMEM_LD32(o_addr + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                            TMEM_ST32(o_addr + c * 32, o);
                        }
                        if (need) {
                            l_run *= factor;
                            m_run = m_tile;
                        }
                    }
                    l_add = exp_row((m_run == -INFINITY) ? 0.f : m_run);
                }
                TMEM_ST32(s_addr, v);
                TMEM_ST32(s_addr + 32, (v + 32));
                l_run += l_add;
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.p_full[t]));
            }
            // ---- epilogue: wait for the last PV, normalise, write out ---------------------------
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.o_done[t]), 0, abort_flag, p.workspace, 8));
            if (ok) {
                tc_fence_after();
                const bool direct = p.n_splits == 1;
                const float inv = direct ? 1.f / l_run : 1.f;
                const size_t out_row = ((size_t)lb * p.M_max + tok) * p.Hq + h * p.G + g;
                const size_t prow = (((size_t)lb * p.Hkv + h) * p.n_splits + split) * p.R_pad + rg * 256 + row;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t v[32];
                    TMEM_LD32(o_addr + c * 32, v);
                    tmem_wait_ld();
                    if (!row_valid) continue;
                    if (!direct) {
                        // a thread's row is 512 contiguous bytes: 32-byte stores fill whole sectors, half as many
                        // memory transactions as 16-byte ones for this one-row-per-lane pattern
                        float* dst = p.part_o + prow * kD + c * 32;
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 8 * i),
                                         "r"(v[8 * i]), "r"(v[8 * i + 1]), "r"(v[8 * i + 2]), "r"(v[8 * i + 3]), "r"(v[8 * i + 4]),
                                         "r"(v[8 * i + 5]), "r"(v[8 * i + 6]), "r"(v[8 * i + 7])
                                         : "memory");
                    } else if (p.out_f32) {
                        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + out_row * kD + c * 32);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst[i] = make_float4(__uint_as_float(v[4 * i]) * inv, __uint_as_float(v[4 * i + 1]) * inv,
                                                 __uint_as_float(v[4 * i + 2]) * inv, __uint_as_float(v[4 * i + 3]) * inv);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + out_row * kD + c * 32);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 w;
                            w.x = pack_bf16(__uint_as_float(v[8 * i]) * inv, __uint_as_float(v[8 * i + 1]) * inv);
                            w.y = pack_bf16(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv);
                            w.z = pack_bf16(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv);
                            w.w = pack_bf16(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv);
                            dst[i] = w;
                        }
                    }
                }
                if (row_valid) {
                    if (direct) {
                        if (p.lse) p.lse[out_row] = m_run * kLn2 + logf(l_run);
                    } else {
                        p.part_ml[prow * 2] = m_run * kLn2;  // natural-log units for the merge
                        p.part_ml[prow * 2 + 1] = l_run;
                    }
                }
            }
        }
    }

    // ---- teardown ----------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // after a give-up no new copy was issued; the few in flight (at most a ring of them) land within microseconds
        if (*abort_flag) __nanosleep(1000000);
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

// Log-sum-exp merge of the KV splits: one warp per output row (a thread owns four channels), eight rows per
// CTA; grid = (row groups, Hkv, layers x seqs).
constexpr int kMergeRows = 8;
__global__ void __launch_bounds__(32 * kMergeRows) merge_tc_kernel(TcParams p) {
    const int r = blockIdx.x * kMergeRows + (threadIdx.x >> 5), h = blockIdx.y, lb = blockIdx.z, lane = threadIdx.x & 31;
    const int b = lb % p.batch;
    int M = p.q_lens ? p.q_lens[b] : p.M_max;
    M = min(max(M, 0), p.M_max);
    if (r >= M * p.G) return;
    const size_t base = ((size_t)lb * p.Hkv + h) * p.n_splits;
    const float2* ml = reinterpret_cast<const float2*>(p.part_ml);
    float m_all = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s) m_all = fmaxf(m_all, ml[(base + s) * p.R_pad + r].x);
    float l_all = 0.f;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    // four splits at a time, their loads in flight together (added in split order, so the result does not depend on
    // the batching); an empty split's partial O was never written and is not read
    for (int s0 = 0; s0 < p.n_splits; s0 += 4) {
        float2 m_l[4];
        float4 po[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t prow = (base + min(s0 + u, p.n_splits - 1)) * p.R_pad + r;
            m_l[u] = ml[prow];
            if (s0 + u >= p.n_splits) m_l[u].x = -INFINITY;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t prow = (base + min(s0 + u, p.n_splits - 1)) * p.R_pad + r;
            po[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (m_l[u].x != -INFINITY) po[u] = __ldg(reinterpret_cast<const float4*>(p.part_o + prow * kD) + lane);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (m_l[u].x == -INFINITY) continue;
            const float w = __expf(m_l[u].x - m_all);
            l_all = fmaf(m_l[u].y, w, l_all);
            o.x = fmaf(po[u].x, w, o.x);
            o.y = fmaf(po[u].y, w, o.y);
            o.z = fmaf(po[u].z, w, o.z);
            o.w = fmaf(po[u].w, w, o.w);
        }
    }
    const int j = r / p.G, g = r % p.G;
    const size_t row = ((size_t)lb * p.M_max + j) * p.Hq + h * p.G + g;
    const float inv = 1.f / l_all;
    o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
    if (p.out_f32) {
        reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + row * kD)[lane] = o;
    } else {
        uint2 w2;
        w2.x = pack_bf16(o.x, o.y);
        w2.y = pack_bf16(o.z, o.w);
        reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + row * kD)[lane] = w2;
    }
    if (p.lse && lane == 0) p.lse[row] = m_all + logf(l_all);
}

}  // namespace

bool attention_tc_supported(const AttnArgs& a) {
    if (a.g.dtype != SPECPV_DTYPE_BF16 || a.g.d != 128 || (a.g.bs != 64 && a.g.bs != 32 && a.g.bs != 16)) return false;
    if (a.g.G > 128 || (128 % a.g.G) != 0) return false;
    if (a.M_max > kMaxQTokens) return false;
    // row coordinates of the pool tensor map must fit in a positive int32
    const unsigned long long rows = (unsigned long long)a.g.n_layers * a.n_pages * a.g.Hkv * (unsigned long long)a.g.bs;
    if (rows >= 0x7FFFFF00ull) return false;
    return get_encode_fn() != nullptr;
}

specpv_status launch_merge_tc(const TcParams& p, int R_max, int n_lb, cudaStream_t stream) {
    dim3 mgrid((R_max + kMergeRows - 1) / kMergeRows, p.Hkv, n_lb);
    merge_tc_kernel<<<mgrid, 32 * kMergeRows, 0, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    return SPECPV_OK;
}

specpv_status launch_attention_tc(const AttnArgs& a, cudaStream_t stream) {
    TcParams p{};
    const int G = a.g.G, Hq = a.g.Hq, Hkv = a.g.Hkv;
    const uint64_t step_tokens = (uint64_t)a.n_layers * a.batch * a.M_max;
    {
        uint64_t dims[3] = {128, (uint64_t)Hq, step_tokens};
        uint64_t strides[2] = {256, (uint64_t)Hq * 256};
        uint32_t box[3] = {64, (uint32_t)G, (uint32_t)(128 / G)};
        if (!encode_map(&p.tm_q, a.q, 3, dims, strides, box)) return SPECPV_ERR_CUDA;
    }
    {
        uint64_t dims[3] = {128, (uint64_t)Hkv, step_tokens};
        uint64_t strides[2] = {256, (uint64_t)Hkv * 256};
        uint32_t box[3] = {64, 1, 64};
        if (!encode_map(&p.tm_knew, a.k_new, 3, dims, strides, box)) return SPECPV_ERR_CUDA;
        if (!encode_map(&p.tm_vnew, a.v_new, 3, dims, strides, box)) return SPECPV_ERR_CUDA;
    }
    const uint64_t pool_rows = (uint64_t)a.g.n_layers * a.n_pages * Hkv * (uint64_t)a.g.bs;
    {
        uint64_t dims[2] = {128, pool_rows};
        uint64_t strides[1] = {256};
        uint32_t box[2] = {64, (uint32_t)a.g.bs};
        if (!encode_map(&p.tm_kpool, a.k_pool, 2, dims, strides, box)) return SPECPV_ERR_CUDA;
        if (!encode_map(&p.tm_vpool, a.v_pool, 2, dims, strides, box)) return SPECPV_ERR_CUDA;
    }
    p.tree_mask = a.tree_mask; p.q_lens = a.q_lens; p.block_table = a.block_table; p.seq_lens = a.seq_lens;
    p.out = a.out; p.lse = a.lse; p.workspace = a.workspace;
    p.layer0 = a.layer0; p.batch = a.batch; p.M_max = a.M_max; p.mask_words = a.mask_words;
    p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.max_blocks = a.max_blocks; p.n_pages = a.n_pages;
    p.out_f32 = a.g.out_f32;
    p.bs = a.g.bs;
    p.pool_rows = (uint32_t)pool_rows;
    p.scale_log2 = a.g.scale * kLog2e;

    const int R_max = a.M_max * G;
    p.n_row_groups = (R_max + 255) / 256;
    p.R_pad = p.n_row_groups * 256;
    if (attention_pair_wanted(a)) return launch_attention_pair(p, a, stream);

    if (!set_smem_limit_once(reinterpret_cast<const void*>(attn_tc_kernel), kSmemBytes)) return SPECPV_ERR_CUDA;
    // KV splits: fill the 148 SMs (one CTA each) in whole waves as evenly as the workspace allows
    const int base = Hkv * a.n_layers * a.batch * p.n_row_groups;
    const int max_tiles = (a.max_seq_len + kTileTokens - 1) / kTileTokens;
    const size_t per_split = (size_t)Hkv * a.n_layers * a.batch * p.R_pad * (kD + 2) * sizeof(float);
    // Choose the split count with a small cost model (microseconds): whole waves of one CTA per SM,
    // each CTA paying a fixed set-up/drain cost plus its tiles; splitting adds the partial-result
    // round trip through the workspace and the merge launch.
    int best = 1;
    double best_cost = 1e30;
    const double t_tile = 1.3, t_cta = 6.0, t_partial = 3.0, t_merge_launch = 6.0;
    const double avg_tiles = max_tiles + 1.0;  // context tiles + the tile of the step's own tokens
    for (int s = 1; s <= 64; ++s) {
        if (s > 1 && (s > max_tiles / 2 || per_split * s > a.partial_bytes)) break;  // at least two tiles per CTA
        const long long ctas = (long long)base * s;
        const double waves = (double)((ctas + 147) / 148);
        double cost = waves * (t_cta + t_tile * (avg_tiles / s + (s > 1 ? 0.5 : 0.0)));
        if (s > 1) cost += waves * t_partial + t_merge_launch + (double)per_split * s * 2.0 / 4.0e6;  // bytes / (4 TB/s) in us
        if (cost < best_cost * 0.97) {
            best_cost = cost;
            best = s;
        }
    }
    p.n_splits = best;
    char* ws = reinterpret_cast<char*>(a.workspace) + a.partial_off;
    p.part_o = reinterpret_cast<float*>(ws);
    p.part_ml = reinterpret_cast<float*>(ws + (size_t)Hkv * a.n_layers * a.batch * p.n_splits * p.R_pad * kD * sizeof(float));

    dim3 grid(p.n_splits * p.n_row_groups, Hkv, a.n_layers * a.batch);
    attn_tc_kernel<<<grid, kThreadsTc, kSmemBytes, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA;
    count_launch();
    if (p.n_splits > 1) return launch_merge_tc(p, R_max, a.n_layers * a.batch, stream);
    return SPECPV_OK;
}

}  // namespace specpv
