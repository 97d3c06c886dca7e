// Stride-1 convolution on a flat pixel grid with the activation tile resident in shared memory:
// the second and third convolutions of the policy network (Appendix F.1 / F.2).
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include "common.cuh"

namespace hts {

struct ConvResParams {
    int tap_shift[9];       // row shift of each filter tap on the flat input grid (dy*W_in + dx)
    int tile_rows;          // rows of one activation tile: 128 + largest shift, rounded up to 8
    int n_env;              // valid environments
    int total_rows;         // n_env * P_in
    int P_in, W_in;         // input grid: pixels per environment, width
    int H_out, W_out, P_out;
    const float* bias;      // [64]
    const float* inv_scale; // device scalar undoing the weight scaling
    __half* out;            // rows [env*P_out + y*W_out + x][64]
    int* status;
};

// rows of the activation tile for a largest tap shift
inline int conv_res_tile_rows(int max_shift) { return (128 + max_shift + 7) / 8 * 8; }

// Shared memory the kernel needs for (taps, planes per tap) and a tile of `tile_rows` rows: resident filter plus the
// ring of activation tiles.  A geometry fits if this stays within 227 KB.
inline int conv_res_smem_bytes(int taps, int cpt, int tile_rows)
{
    const int nst = cpt == 2 ? 4 : 6;
    return 1024 + taps * cpt * 64 * 128 + nst * cpt * tile_rows * 128;
}

// TAPS x CPT = filter taps x 64-channel planes per tap: (4,2) for conv2 on the space-to-depth
// grid, (9,1) for conv3.  act_map: box [tile_rows x 64]; weight_map: box [64 x 64].
template <int TAPS, int CPT>
hts_status conv_res_launch(const CUtensorMap& act_map, const CUtensorMap& weight_map, const ConvResParams& p,
                           cudaStream_t s);

}  // namespace hts
