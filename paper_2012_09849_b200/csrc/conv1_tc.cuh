// First convolution of the policy network (8x8 stride 4, C -> 32; Appendix F.1 / F.2) as a fused
// tcgen05 kernel: uint8 frames -> shared memory -> fp16 space-to-depth tile -> tensor cores.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include "common.cuh"

namespace hts {

struct Conv1Plan {
    int C, H, W;            // observation
    int Hs, Ws, Cs;         // space-to-depth(4) grid and channels (16*C)
    int H1, W1;             // conv1 output extent (Hs-1, Ws-1)
    int cpt;                // 64-channel planes per tap (Cs/64)
    int R, bands;           // output rows per band, bands per environment
    int tile_rows;          // rows allocated per plane of the fp16 tile
    int u8_stage_bytes;     // one staged band of uint8 input
    int plane_bufs, u8_stages; // fp16 planes in the ring (3 or 4) and staged bands (2..4)
    int smem_bytes;         // dynamic shared memory of the kernel
    int H1s, W1s, P1s;      // space-to-depth(2) grid of the output (input layout of conv2)
    int ts;                 // 1: the tensor-memory variant applies (four-channel frames)
    int ts_chan_bytes, ts_stage_bytes, ts_stages, ts_smem_bytes;   // its staged input buffers and shared memory
};

// false if the geometry does not fit the kernel (C not a multiple of 4, W too wide, ...)
bool conv1_plan(const Geometry& g, Conv1Plan* plan);

// w1 [32,C,8,8] bf16 -> packed [32][4*Cs] fp16 scaled by *scale:
//   column (dy*2+dx)*Cs + c*16 + uy*4 + ux  holds  w1[o][c][4dy+uy][4dx+ux]
hts_status conv1_pack_weights(const Conv1Plan& pl, const __nv_bfloat16* w1, __half* packed, const float* scale,
                              cudaStream_t s);

// out: fp16 rows [env*P1s + (y/2)*W1s + x/2][128], column ((y%2)*2 + x%2)*32 + o
// ix: dense frames (row e = frame e of obs) or frames gathered by slot from a pool (see Indexing)
hts_status conv1_launch(const Conv1Plan& pl, const CUtensorMap& weight_map, const uint8_t* obs, const Indexing& ix, int n,
                        const float* bias, const float* inv_scale, __half* out, int* status, cudaStream_t s);

}  // namespace hts
