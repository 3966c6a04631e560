// Parameter blocks and launchers of the linear maps either side of the attention (see proj_tc.cu).
#pragma once
#include "common.cuh"

namespace specpv {

// A run of 128-feature output tiles that lands in one tensor: feature tile t (first_tile <= t < next
// segment's first_tile) of row `tok` of layer-in-call l goes to
//   base + (l * tokens + tok) * row_stride + (t - first_tile) * tile features.
struct ProjSegment {
    void* base;
    int first_tile;
    int row_stride;  // elements between consecutive rows
    int rope;        // rotate the tile's features (a tile is one head)
};

struct ProjArgs {
    const void* x;           // [n_layers_call][tokens][n_in]
    const void* w;           // [n_layers_total][n_out][n_in]
    const float* cos_sin;    // [tokens][tile/2][2], only read by segments with rope
    const void* residual;    // nullable, laid out like segment 0's tensor
    int dtype;               // SPECPV_DTYPE_*
    int layer0, n_layers_call, n_layers_total;
    int tokens;              // rows per layer (batch * M_max)
    int n_in, n_out;
    int tile;                // features per output tile = head_dim for the QKV map
    int n_seg;
    ProjSegment seg[3];
    void* workspace;
    size_t scratch_off, scratch_bytes;  // split-K partial sums
};

bool proj_tc_supported(const ProjArgs& a);
specpv_status launch_proj_tc(const ProjArgs& a, cudaStream_t stream);
specpv_status launch_proj_simt(const ProjArgs& a, cudaStream_t stream);
specpv_status launch_rope_table(const uint64_t* tree_mask, const int32_t* q_lens, const int32_t* base_pos, int batch,
                                int M_max, int d, double theta, float* cos_sin, cudaStream_t stream);

}  // namespace specpv
