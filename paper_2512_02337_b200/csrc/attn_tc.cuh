// Declarations shared by the tensor-core attention kernels (one CTA per head split in attn_tc.cu, a CTA
// pair per head split in attn_pair.cu): the kernel parameter block, small PTX helpers and the launchers.
#pragma once
#include "tc_common.cuh"

namespace specpv {

constexpr int kTileTokens = 128;         // KV tokens per tile (128 / page size pages)
constexpr int kD = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr float kSafeRowSum = 1.1529215e18f;  // 2^60: a tile's row sum below this cannot overflow the float32 sums

struct TcParams {
    CUtensorMap tm_q;      // (d, Hq, tokens)          box (64, G, 128/G)
    CUtensorMap tm_knew;   // (d, Hkv, tokens)         box (64, 1, 64)
    CUtensorMap tm_vnew;
    CUtensorMap tm_kpool;  // (d, rows)                box (64, page size)
    CUtensorMap tm_vpool;
    const uint64_t* tree_mask;
    const int32_t* q_lens;
    const int32_t* block_table;
    const int32_t* seq_lens;
    void* out;
    float* lse;
    float* part_o;   // [lb][Hkv][splits][R_pad][128]  (pair kernel: [pair][2][256][128])
    float* part_ml;  // [lb][Hkv][splits][R_pad][2]    (pair kernel: [pair][2][256][2])
    int32_t* counters;  // pair kernel: arrival counters of shared units, [unit][CTA rank], zero between launches
    void* workspace;
    int n_layers_call;
    int pairs_per_unit;  // pair kernel: > 0 = every unit has this many pairs of its own; 0 = pairs take equal shares of all tiles
    int layer0, batch, M_max, mask_words, Hq, Hkv, G, max_blocks, n_pages;
    int n_splits, n_row_groups, R_pad, out_f32;
    int bs;          // tokens per page (16, 32 or 64)
    uint32_t pool_rows;  // rows of the pool tensor map (an out-of-range row coordinate reads zeros)
    float scale_log2;
};

// tcgen05.mma with the shared-memory descriptors given as (low word, common high word); `acc` = 0
// overwrites D, anything else accumulates.
__device__ __forceinline__ void mma_ss_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                            uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void mma_ts_lohi(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                            uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc)
        : "memory");
}
// keeps the compiler from hoisting per-instruction descriptor words out of the tile loop
__device__ __forceinline__ uint32_t launder(uint32_t x) {
    asm volatile("" : "+r"(x));
    return x;
}
// acc.x += low bf16 of w, acc.y += high bf16 of w: the mixed-precision add takes the 16-bit halves as they
// are, so the packed word needs no shift / mask to be widened first (the sums are the same bit for bit)
__device__ __forceinline__ void add_bf16_pair(float2& acc, uint32_t w) {
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\t"
        "add.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}"
        : "+f"(acc.x), "+f"(acc.y)
        : "r"(w));
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}


// launchers: the split merge (attn_tc.cu) and the CTA-pair attention kernel (attn_pair.cu)
specpv_status launch_merge_tc(const TcParams& p, int R_max, int n_lb, cudaStream_t stream);
bool attention_pair_wanted(const AttnArgs& a);
specpv_status launch_attention_pair(TcParams& p, const AttnArgs& a, cudaStream_t stream);

}  // namespace specpv
