// conv2 / conv3 of the policy network (Appendix F.1 / F.2) with the A operand in tensor memory: stride-1
// convolutions on an fp16 pixel grid, marching down the grid rows (the formulation of conv1_tc.cu without the
// byte conversion).
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include "common.cuh"

namespace hts {

struct ConvMarchPlan {
    int TY, TX, CIN;        // filter taps down / across, input channels per grid pixel (64 or 128)
    int Hin, Win;           // input grid per environment
    int Hout, Wout;         // output grid (Hin - TY + 1, Win - TX + 1)
    int tile_cols;          // new grid columns per tile: 4 x (32 - (TX - 1))
    int env_max;            // environments a tile can touch
    int stage_bytes;        // one staged grid row: env_max x Win pixels x CIN fp16
    int stages;
    int smem_bytes;
};

// TY x TX taps on CIN channels: (2, 2, 128) is conv2 on the space-to-depth(2) grid of conv1's output,
// (3, 3, 64) is conv3.  false if the geometry does not fit (grid wider than a tile, not enough shared memory).
bool conv_march_plan(int TY, int TX, int CIN, int Hin, int Win, ConvMarchPlan* plan);

struct ConvMarchArgs {
    int n;                  // environments
    const float* bias;      // [64]
    const float* inv_scale; // device scalar undoing the weight scaling
    __half* out;            // rows [env * Hout * Wout + y * Wout + x][64]
    int* status;
};

// in_map: the input activations as [env][pixel][CIN] with box [64 (x CIN/64)] x Win pixels x env_max environments,
// 128-byte swizzle; weight_map: packed filter [TY * TX * 64 rows][CIN], box [TX * 64 rows][64].
hts_status conv_march_launch(const ConvMarchPlan& pl, const CUtensorMap& in_map, const CUtensorMap& weight_map,
                             const ConvMarchArgs& a, cudaStream_t s);

}  // namespace hts
