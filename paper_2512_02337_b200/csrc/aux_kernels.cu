// Cache-management kernels of the SpecPV verification path (paper Section 3.2-3.3):
// block key summaries (Eq. 1), block scores (Eq. 2-3), the retained-block selection, the gather
// that rebuilds the partial cache, and the commit of accepted tokens.
#include <math.h>

#include "common.cuh"
#include "aux_kernels.cuh"

namespace specpv {

namespace {

// ---------------------------------------------------------------------------------------------
// Eq. 1: Kmax/Kmin per block.  grid = (blocks touched, Hkv, layers x seqs).  A thread owns one 16-byte
// chunk of channels (kChunk of them) and every kTokLanes-th token of the block, with all its loads in
// flight at once; the token lanes are then combined through shared memory.  max/min are exact, so the
// order of the reduction does not matter.
// ---------------------------------------------------------------------------------------------
constexpr int kSumThreads = 128;
template <typename T>
__global__ void __launch_bounds__(kSumThreads) summaries_kernel(SummaryParams p) {
    constexpr int kChunk = 16 / (int)sizeof(T);  // channels per 16-byte load
    __shared__ float s_max[kSumThreads * kChunk], s_min[kSumThreads * kChunk];
    const int h = blockIdx.y, lb = blockIdx.z, tid = threadIdx.x;
    const int b = lb % p.batch, l = lb / p.batch;
    int seq_len = p.seq_lens[b];
    if (p.n_appended) {  // summaries of a commit in flight: the lengths are not advanced yet
        const int n = min(max(p.n_appended[b], 0), p.A_max);
        if ((size_t)seq_len + n <= (size_t)p.max_blocks * p.bs) seq_len += n;
    }
    const int begin = p.tok_begin ? p.tok_begin[b] : 0;
    const int i = max(begin, 0) / p.bs + blockIdx.x;
    if ((size_t)i * p.bs >= (size_t)seq_len || i >= p.max_blocks) return;
    const int n_valid = min(p.bs, seq_len - i * p.bs);
    const int page = p.block_table[(size_t)b * p.max_blocks + i];
    if (page < 0 || page >= p.n_pages) {
        if (tid == 0) record_fault(p.workspace, SPECPV_ERR_BAD_BLOCK_TABLE, b, i, page, l);
        return;
    }
    const T* k = reinterpret_cast<const T*>(p.k_pool) +
                 (((size_t)(p.layer0 + l) * p.n_pages + page) * p.Hkv + h) * p.bs * p.d;
    const int chunks = p.d / kChunk;            // 16-byte chunks per token row (8, 16 or 32)
    const int tok_lanes = kSumThreads / chunks;  // tokens read side by side
    const int chunk = tid % chunks, tl = tid / chunks;
    float mx[kChunk], mn[kChunk];
#pragma unroll
    for (int e = 0; e < kChunk; ++e) { mx[e] = -INFINITY; mn[e] = INFINITY; }
    constexpr int kMaxIter = 16;  // bs <= 64 and tok_lanes >= 4
    uint4 buf[kMaxIter];
    int n_it = 0;
#pragma unroll
    for (int it = 0; it < kMaxIter; ++it) {
        const int t = tl + it * tok_lanes;
        if (t < n_valid) {
            buf[it] = *reinterpret_cast<const uint4*>(k + (size_t)t * p.d + chunk * kChunk);
            n_it = it + 1;
        }
    }
#pragma unroll
    for (int it = 0; it < kMaxIter; ++it) {
        if (it < n_it) {
            const T* e8 = reinterpret_cast<const T*>(&buf[it]);
#pragma unroll
            for (int e = 0; e < kChunk; ++e) {
                const float v = to_float(e8[e]);
                mx[e] = fmaxf(mx[e], v);
                mn[e] = fminf(mn[e], v);
            }
        }
    }
#pragma unroll
    for (int e = 0; e < kChunk; ++e) {
        s_max[(tl * chunks + chunk) * kChunk + e] = mx[e];
        s_min[(tl * chunks + chunk) * kChunk + e] = mn[e];
    }
    __syncthreads();
    // thread c < d finishes channel c over the token lanes
    for (int c = tid; c < p.d; c += kSumThreads) {
        float a = -INFINITY, z = INFINITY;
        for (int q = 0; q < tok_lanes; ++q) {
            a = fmaxf(a, s_max[q * p.d + c]);
            z = fminf(z, s_min[q * p.d + c]);
        }
        const size_t o = ((((size_t)(p.layer0 + l) * p.batch + b) * p.Hkv + h) * p.max_blocks + i) * p.d + c;
        reinterpret_cast<T*>(p.kmax)[o] = from_float<T>(a);
        reinterpret_cast<T*>(p.kmin)[o] = from_float<T>(z);
    }
}

// ---------------------------------------------------------------------------------------------
// Eq. 2-3 (SIMT form): lane <-> block, the CTA's 32*warps blocks' summaries staged in shared
// memory as float32, the group's query rows read as broadcasts.  grid = (block groups, Hkv,
// layers x seqs).
// ---------------------------------------------------------------------------------------------
constexpr int kScoreWarps = 4;
constexpr int kScoreBlocksPerCta = 32 * kScoreWarps;
constexpr int kScoreRowTile = 4;

template <typename T, int D>
__global__ void __launch_bounds__(32 * kScoreWarps) scores_simt_kernel(ScoreParams p) {
    extern __shared__ float smem[];
    float* Smax = smem;                                   // [blocks][D + 1]
    float* Smin = Smax + kScoreBlocksPerCta * (D + 1);    // [blocks][D + 1]
    float* Qs = Smin + kScoreBlocksPerCta * (D + 1);      // [kScoreRowTile][D]
    const int h = blockIdx.y, lb = blockIdx.z, tid = threadIdx.x;
    const int b = lb % p.batch, l = lb / p.batch;
    const int seq_len = p.seq_lens[b];
    const int nb = (seq_len + p.bs - 1) / p.bs;
    const int blk0 = blockIdx.x * kScoreBlocksPerCta;
    if (blk0 >= nb) return;
    int M = p.q_lens ? p.q_lens[b] : p.M_max;
    M = min(max(M, 0), p.M_max);
    int row_begin = 0, row_end = M * p.G;  // rows r = j * G + g
    if (p.reduce == SPECPV_REDUCE_LAST) {
        int last = p.last_query ? p.last_query[b] : 0;
        last = min(max(last, 0), max(M - 1, 0));
        row_begin = last * p.G;
        row_end = row_begin + p.G;
    }
    const size_t sum_base = ((((size_t)(p.layer0 + l) * p.batch + b) * p.Hkv + h) * p.max_blocks) * D;
    const T* kmax = reinterpret_cast<const T*>(p.kmax) + sum_base;
    const T* kmin = reinterpret_cast<const T*>(p.kmin) + sum_base;
    for (int e = tid; e < kScoreBlocksPerCta * D; e += blockDim.x) {
        int bi = e / D, c = e % D;
        int i = blk0 + bi;
        float vmax = 0.f, vmin = 0.f;
        if (i < nb) {
            vmax = to_float(kmax[(size_t)i * D + c]);
            vmin = to_float(kmin[(size_t)i * D + c]);
        }
        Smax[bi * (D + 1) + c] = vmax;
        Smin[bi * (D + 1) + c] = vmin;
    }
    const T* q = reinterpret_cast<const T*>(p.q) + (size_t)lb * p.M_max * p.Hq * D;
    const float* my_max = Smax + tid * (D + 1);
    const float* my_min = Smin + tid * (D + 1);
    float red = p.reduce == SPECPV_REDUCE_MAX ? -INFINITY : 0.f;
    for (int r0 = row_begin; r0 < row_end; r0 += kScoreRowTile) {
        __syncthreads();
        for (int e = tid; e < kScoreRowTile * D; e += blockDim.x) {
            int r = r0 + e / D, c = e % D;
            float v = 0.f;
            if (r < row_end) {
                int j = r / p.G, g = r % p.G;
                v = to_float(q[((size_t)j * p.Hq + h * p.G + g) * D + c]);
            }
            Qs[e] = v;
        }
        __syncthreads();
        float dmax[kScoreRowTile], dmin[kScoreRowTile];
#pragma unroll
        for (int i = 0; i < kScoreRowTile; ++i) dmax[i] = dmin[i] = 0.f;
        if (p.score_mode == 0) {
#pragma unroll 4
            for (int c = 0; c < D; ++c) {
                float a = my_max[c], bb = my_min[c];
#pragma unroll
                for (int i = 0; i < kScoreRowTile; ++i) {
                    float qc = Qs[i * D + c];
                    dmax[i] = fmaf(qc, a, dmax[i]);
                    dmin[i] = fmaf(qc, bb, dmin[i]);
                }
            }
        } else {
            // channel-wise form: a channel with q_c >= 0 takes Kmax_c, one with q_c < 0 takes Kmin_c
            // (Kmax_c >= Kmin_c), so the score is one dot product with a per-channel choice of operand
#pragma unroll 4
            for (int c = 0; c < D; ++c) {
                float a = my_max[c], bb = my_min[c];
#pragma unroll
                for (int i = 0; i < kScoreRowTile; ++i) {
                    float qc = Qs[i * D + c];
                    dmax[i] = fmaf(qc, qc < 0.f ? bb : a, dmax[i]);
                }
            }
#pragma unroll
            for (int i = 0; i < kScoreRowTile; ++i) dmin[i] = dmax[i];
        }
#pragma unroll
        for (int i = 0; i < kScoreRowTile; ++i) {
            if (r0 + i >= row_end) continue;
            float s = fmaxf(dmax[i], dmin[i]);
            red = p.reduce == SPECPV_REDUCE_MAX ? fmaxf(red, s) : red + s;
        }
    }
    const int i = blk0 + tid;
    if (i < nb) {
        if (p.reduce != SPECPV_REDUCE_MAX) red /= (float)(row_end - row_begin);
        p.scores[(((size_t)lb * p.Hkv + h) * p.max_blocks) + i] = red;
    }
}

// ---------------------------------------------------------------------------------------------
// Selection: one CTA per (layer, sequence, KV head).  The candidates' (score, index) pairs become
// unique 64-bit keys whose unsigned order is "score descending, then index ascending, NaN last";
// an 8-pass most-significant-digit radix select finds the k-th largest key exactly, and a
// block-wide ordered compaction writes sink | kept candidates | local in ascending order.
// ---------------------------------------------------------------------------------------------
constexpr int kSelectThreads = 256;

__device__ __forceinline__ uint64_t select_key(float score, int index) {
    uint32_t bits = __float_as_uint(score);
    uint32_t ord;
    if (score != score) ord = 0u;                         // NaN ranks below every number
    else if (score == 0.f) ord = 0x80000000u;             // -0 and +0 tie
    else ord = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
    return ((uint64_t)ord << 32) | (uint64_t)(0xFFFFFFFFu - (uint32_t)index);
}

__global__ void __launch_bounds__(kSelectThreads) select_kernel(SelectParams p) {
    __shared__ unsigned int hist[256];
    __shared__ uint64_t s_prefix;
    __shared__ int s_remaining;
    __shared__ int s_warp_counts[kSelectThreads / 32];
    __shared__ int s_running;
    __shared__ int s_round_counts[16 * (kSelectThreads / 32)];  // kept candidates per (round, warp)
    const int h = blockIdx.x, b = blockIdx.y, l = blockIdx.z, tid = threadIdx.x;
    const int seq_len = p.seq_lens[b];
    const int nb = min((seq_len + p.bs - 1) / p.bs, p.max_blocks);
    const float* scores = p.scores + (((size_t)l * p.batch + b) * p.Hkv + h) * p.max_blocks;
    // head-shared selection ranks the blocks on the mean of the layer's KV heads' scores, summed in float32 in
    // head order (the ranking is a pure function of these bits, the same in every head's CTA)
    const float* scores_h0 = p.scores + (((size_t)l * p.batch + b) * p.Hkv) * p.max_blocks;
    const float inv_heads = 1.0f / (float)p.Hkv;
    auto score_at = [&](int i) {
        if (!p.share_heads) return scores[i];
        float acc = 0.f;
        for (int hh = 0; hh < p.Hkv; ++hh) acc += scores_h0[(size_t)hh * p.max_blocks + i];
        return acc * inv_heads;
    };
    int32_t* idx = p.idx + (((size_t)l * p.batch + b) * p.Hkv + h) * p.budget_blocks;
    const int count = min(nb, p.budget_blocks);
    if (l == 0 && h == 0 && tid == 0) p.count[b] = count;
    if (nb <= p.budget_blocks) {
        for (int i = tid; i < p.budget_blocks; i += kSelectThreads) idx[i] = i < nb ? i : -1;
        return;
    }
    const int lo = p.sink_blocks, hi = nb - p.local_blocks;
    const int k = p.budget_blocks - p.sink_blocks - p.local_blocks;

    if (tid == 0) {
        s_prefix = 0;
        s_remaining = k;
    }
    // a thread's candidates lo + tid, lo + tid + 256, ...: the first kKeysPerThread keys stay in registers for
    // all eight passes (enough for 4096 candidate blocks), any further ones are recomputed from the scores
    constexpr int kKeysPerThread = 16;
    uint64_t keys[kKeysPerThread];
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        const int i = lo + tid + e * kSelectThreads;
        keys[e] = i < hi ? select_key(score_at(i), i) : 0ull;  // key 0 cannot occur: the index part of a real key is > 0
    }
    const int tail0 = lo + tid + kKeysPerThread * kSelectThreads;
    uint64_t known_mask = 0;
    const int lane = tid & 31, warp = tid >> 5;
    for (int pass = 7; pass >= 0; --pass) {
        hist[tid] = 0;  // kSelectThreads == 256 bins
        __syncthreads();
        const uint64_t prefix = s_prefix;
        const int remaining = s_remaining;
#pragma unroll
        for (int e = 0; e < kKeysPerThread; ++e) {
            const uint64_t key = keys[e];
            if (key != 0ull && (key & known_mask) == prefix) atomicAdd(&hist[(unsigned)(key >> (8 * pass)) & 255u], 1u);
        }
        for (int i = tail0; i < hi; i += kSelectThreads) {
            const uint64_t key = select_key(score_at(i), i);
            if ((key & known_mask) == prefix) atomicAdd(&hist[(unsigned)(key >> (8 * pass)) & 255u], 1u);
        }
        __syncthreads();
        // thread <-> bin: the digit of the k-th largest key is the bin whose suffix count (this bin and all higher
        // ones) first reaches `remaining`; found in parallel from a block-wide suffix sum
        const unsigned c = hist[tid];
        unsigned v = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned up = __shfl_down_sync(0xffffffffu, v, o);
            if (lane + o < 32) v += up;
        }
        if (lane == 0) s_warp_counts[warp] = (int)v;  // count of this warp's 32 bins
        __syncthreads();
        unsigned above = 0;
        for (int w2 = warp + 1; w2 < kSelectThreads / 32; ++w2) above += (unsigned)s_warp_counts[w2];
        const unsigned suffix = v + above, higher = suffix - c;
        if (suffix >= (unsigned)remaining && higher < (unsigned)remaining) {  // true for exactly one bin
            s_remaining = remaining - (int)higher;
            s_prefix = prefix | ((uint64_t)tid << (8 * pass));
        }
        known_mask |= 0xFFull << (8 * pass);
        __syncthreads();
    }
    const uint64_t threshold = s_prefix;  // the k-th largest key; keys are unique

    for (int i = tid; i < p.sink_blocks; i += kSelectThreads) idx[i] = i;
    for (int i = tid; i < p.local_blocks; i += kSelectThreads) idx[p.sink_blocks + k + i] = hi + i;
    // Ordered compaction of the kept candidates (ascending block index = round e, then thread).  Register part:
    // one ballot per round, the (round, warp) counts scanned once by warp 0.
    constexpr int kWarps = kSelectThreads / 32;
    unsigned ballots[kKeysPerThread];
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        const bool keep = keys[e] != 0ull && keys[e] >= threshold;
        ballots[e] = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) s_round_counts[e * kWarps + warp] = __popc(ballots[e]);
    }
    __syncthreads();
    if (warp == 0) {  // exclusive scan of the 128 counts: four per lane, then across lanes
        int c4[4], sum = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            c4[u] = s_round_counts[lane * 4 + u];
            sum += c4[u];
        }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        int run = incl - sum;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            s_round_counts[lane * 4 + u] = run;
            run += c4[u];
        }
        if (lane == 31) s_running = incl;  // kept so far
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        if ((ballots[e] >> lane) & 1u) {
            const int offset = s_round_counts[e * kWarps + warp] + __popc(ballots[e] & ((1u << lane) - 1u));
            if (offset < k) idx[p.sink_blocks + offset] = lo + tid + e * kSelectThreads;
        }
    }
    // candidates beyond the register part (more than 4096 of them): round by round
    for (int base = lo + kKeysPerThread * kSelectThreads; base < hi; base += kSelectThreads) {
        const int i = base + tid;
        const bool keep = i < hi && select_key(score_at(i), i) >= threshold;
        const unsigned ballot = __ballot_sync(0xffffffffu, keep);
        __syncthreads();  // s_running of the previous round has been read by everyone
        if (lane == 0) s_warp_counts[warp] = __popc(ballot);
        __syncthreads();
        int offset = s_running;
        for (int w = 0; w < warp; ++w) offset += s_warp_counts[w];
        offset += __popc(ballot & ((1u << lane) - 1u));
        if (keep && offset < k) idx[p.sink_blocks + offset] = i;
        __syncthreads();
        if (tid == 0) {
            int total = 0;
            for (int w = 0; w < kWarps; ++w) total += s_warp_counts[w];
            s_running += total;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Gather: grid = (budget blocks, Hkv, layers x seqs); a CTA copies the valid tokens of one selected
// block's K and V (16-byte vectors) into the partial cache.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) gather_kernel(GatherParams p) {
    const int s = blockIdx.x, h = blockIdx.y, lb = blockIdx.z;
    const int b = lb % p.batch, l = lb / p.batch;
    const int count = p.count[b];
    const int seq_len = p.seq_lens[b];
    const int nb = (seq_len + p.bs - 1) / p.bs;
    if (s == 0 && h == 0 && l == 0 && threadIdx.x == 0) {
        int plen = 0;
        // the last selected block is the sequence's last block (local window or, for short
        // contexts, simply every block): it keeps only its valid tokens
        if (count > 0) plen = (count - 1) * p.bs + (seq_len - (nb - 1) * p.bs);
        p.partial_lens[b] = plen;
    }
    if (s >= count) return;
    const int blk = p.idx[(((size_t)l * p.batch + b) * p.Hkv + h) * p.budget_blocks + s];
    if (blk < 0 || blk >= nb || blk >= p.full_max_blocks || s >= p.part_max_blocks) {
        if (threadIdx.x == 0) record_fault(p.workspace, SPECPV_ERR_INVALID_ARG, b, s, blk, l);
        return;
    }
    const int src_page = p.full_table[(size_t)b * p.full_max_blocks + blk];
    const int dst_page = p.part_table[(size_t)b * p.part_max_blocks + s];
    if (src_page < 0 || src_page >= p.full_pages || dst_page < 0 || dst_page >= p.part_pages) {
        if (threadIdx.x == 0) record_fault(p.workspace, SPECPV_ERR_BAD_BLOCK_TABLE, b, blk, src_page, dst_page);
        return;
    }
    const int n_valid = blk == nb - 1 ? seq_len - blk * p.bs : p.bs;
    const size_t row_bytes = (size_t)p.d * p.es;
    const size_t n_vec = (size_t)n_valid * row_bytes / 16;
    const size_t src_off = (((size_t)l * p.full_pages + src_page) * p.Hkv + h) * p.bs * row_bytes;
    const size_t dst_off = (((size_t)l * p.part_pages + dst_page) * p.Hkv + h) * p.bs * row_bytes;
    const uint4* ks = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(p.full_k) + src_off);
    const uint4* vs = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(p.full_v) + src_off);
    uint4* kd = reinterpret_cast<uint4*>(reinterpret_cast<char*>(p.part_k) + dst_off);
    uint4* vd = reinterpret_cast<uint4*>(reinterpret_cast<char*>(p.part_v) + dst_off);
    // four 16-byte loads of K and of V in flight per thread before the stores
    size_t i = threadIdx.x;
    for (; i + 3 * blockDim.x < n_vec; i += 4 * blockDim.x) {
        uint4 a[4], b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            a[u] = __ldg(ks + i + u * blockDim.x);
            b[u] = __ldg(vs + i + u * blockDim.x);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            kd[i + u * blockDim.x] = a[u];
            vd[i + u * blockDim.x] = b[u];
        }
    }
    for (; i < n_vec; i += blockDim.x) {
        kd[i] = ks[i];
        vd[i] = vs[i];
    }
}

// ---------------------------------------------------------------------------------------------
// Commit: grid = (A_max, Hkv, layers x seqs); a CTA appends one accepted token's K and V row.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32) commit_rows_kernel(CommitParams p) {
    const int a = blockIdx.x, h = blockIdx.y, lb = blockIdx.z;
    const int b = lb % p.batch, l = lb / p.batch;
    const int n = min(max(p.n_accepted[b], 0), p.A_max);
    if (a >= n) return;
    const int seq_len = p.seq_lens[b];
    if ((size_t)seq_len + n > (size_t)p.max_blocks * p.bs) {
        if (threadIdx.x == 0 && a == 0 && h == 0) record_fault(p.workspace, SPECPV_ERR_CAPACITY, b, seq_len, n, l);
        return;
    }
    const int row = p.accepted[(size_t)b * p.A_max + a];
    if (row < 0 || row >= p.M_max) {
        if (threadIdx.x == 0) record_fault(p.workspace, SPECPV_ERR_INVALID_ARG, b, a, row, l);
        return;
    }
    const int t = seq_len + a;
    const int page = p.block_table[(size_t)b * p.max_blocks + t / p.bs];
    if (page < 0 || page >= p.n_pages) {
        if (threadIdx.x == 0) record_fault(p.workspace, SPECPV_ERR_BAD_BLOCK_TABLE, b, t / p.bs, page, l);
        return;
    }
    const size_t row_bytes = (size_t)p.d * p.es;
    const size_t src = (((size_t)lb * p.M_max + row) * p.Hkv + h) * row_bytes;
    const size_t dst = ((((size_t)(p.layer0 + l) * p.n_pages + page) * p.Hkv + h) * p.bs + t % p.bs) * row_bytes;
    const uint4* ks = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(p.k_new) + src);
    const uint4* vs = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(p.v_new) + src);
    uint4* kd = reinterpret_cast<uint4*>(reinterpret_cast<char*>(p.k_pool) + dst);
    uint4* vd = reinterpret_cast<uint4*>(reinterpret_cast<char*>(p.v_pool) + dst);
    for (int i = threadIdx.x; i < (int)(row_bytes / 16); i += 32) {
        kd[i] = ks[i];
        vd[i] = vs[i];
    }
}

__global__ void commit_lens_kernel(int32_t* seq_lens, const int32_t* n_accepted, int batch, int A_max,
                                   int capacity_tokens) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int n = min(max(n_accepted[b], 0), A_max);
    if ((size_t)seq_lens[b] + n <= (size_t)capacity_tokens) seq_lens[b] += n;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
#define SPECPV_CHECK_LAUNCH()                                     \
    do {                                                          \
        if (cudaGetLastError() != cudaSuccess) return SPECPV_ERR_CUDA; \
        count_launch();                                           \
    } while (0)

specpv_status launch_summaries(const SummaryParams& p, int n_layers, int blocks_touched, int dtype,
                               cudaStream_t stream) {
    if (blocks_touched <= 0 || n_layers <= 0) return SPECPV_OK;
    dim3 grid(blocks_touched, p.Hkv, n_layers * p.batch);
    if (dtype == SPECPV_DTYPE_F32) summaries_kernel<float><<<grid, kSumThreads, 0, stream>>>(p);
    else summaries_kernel<__nv_bfloat16><<<grid, kSumThreads, 0, stream>>>(p);
    SPECPV_CHECK_LAUNCH();
    return SPECPV_OK;
}

template <typename T, int D>
static specpv_status launch_scores_typed(const ScoreParams& p, int n_layers, int max_nb, cudaStream_t stream) {
    const size_t smem = (size_t)(2 * kScoreBlocksPerCta * (D + 1) + kScoreRowTile * D) * sizeof(float);
    if (cudaFuncSetAttribute(scores_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SPECPV_ERR_CUDA;
    dim3 grid((max_nb + kScoreBlocksPerCta - 1) / kScoreBlocksPerCta, p.Hkv, n_layers * p.batch);
    scores_simt_kernel<T, D><<<grid, 32 * kScoreWarps, smem, stream>>>(p);
    SPECPV_CHECK_LAUNCH();
    return SPECPV_OK;
}

specpv_status launch_scores(const ScoreParams& p, int n_layers, int max_nb, int dtype, int d, cudaStream_t stream) {
    if (max_nb <= 0 || n_layers <= 0) return SPECPV_OK;
    if (dtype == SPECPV_DTYPE_F32) {
        if (d == 64) return launch_scores_typed<float, 64>(p, n_layers, max_nb, stream);
        if (d == 128) return launch_scores_typed<float, 128>(p, n_layers, max_nb, stream);
    } else {
        if (d == 64) return launch_scores_typed<__nv_bfloat16, 64>(p, n_layers, max_nb, stream);
        if (d == 128) return launch_scores_typed<__nv_bfloat16, 128>(p, n_layers, max_nb, stream);
    }
    return SPECPV_ERR_SHAPE;
}

specpv_status launch_select(const SelectParams& p, int n_layers, cudaStream_t stream) {
    if (n_layers <= 0 || p.batch <= 0) return SPECPV_OK;
    dim3 grid(p.Hkv, p.batch, n_layers);
    select_kernel<<<grid, kSelectThreads, 0, stream>>>(p);
    SPECPV_CHECK_LAUNCH();
    return SPECPV_OK;
}

specpv_status launch_gather(const GatherParams& p, int n_layers, cudaStream_t stream) {
    dim3 grid(p.budget_blocks, p.Hkv, n_layers * p.batch);
    gather_kernel<<<grid, 128, 0, stream>>>(p);
    SPECPV_CHECK_LAUNCH();
    return SPECPV_OK;
}

specpv_status launch_commit(const CommitParams& p, int n_layers, int32_t* seq_lens, cudaStream_t stream) {
    if (p.A_max > 0 && n_layers > 0) {
        dim3 grid(p.A_max, p.Hkv, n_layers * p.batch);
        commit_rows_kernel<<<grid, 32, 0, stream>>>(p);
        SPECPV_CHECK_LAUNCH();
    }
    (void)seq_lens;
    return SPECPV_OK;
}

specpv_status launch_commit_lens(int32_t* seq_lens, const int32_t* n_accepted, int batch, int A_max,
                                 int capacity_tokens, cudaStream_t stream) {
    commit_lens_kernel<<<(batch + 63) / 64, 64, 0, stream>>>(seq_lens, n_accepted, batch, A_max, capacity_tokens);
    SPECPV_CHECK_LAUNCH();
    return SPECPV_OK;
}

}  // namespace specpv
