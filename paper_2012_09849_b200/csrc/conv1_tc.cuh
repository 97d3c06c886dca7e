// First convolution of the policy network (8x8 stride 4, C -> 32; Appendix F.1 / F.2) as a fused
// tcgen05 kernel: uint8 frames -> shared memory -> fp16 rows in tensor memory -> tensor cores.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include "common.cuh"

namespace hts {

struct Conv1Plan {
    int C, H, W;            // observation
    int CG;                 // groups of four channels (C / 4): 64 K values = 32 tensor-memory columns each
    int Hs, Ws;             // space-to-depth(4) grid
    int H1, W1;             // conv1 output extent (Hs-1, Ws-1)
    int H1s, W1s, P1s;      // space-to-depth(2) grid of the output (input layout of conv2)
    int env_max;            // environments one tile of 125 grid columns can touch
    int group_rows;         // grid rows per staged group (one TMA box per environment)
    int env_bytes;          // bytes of one environment's box: C x group_rows x 4 W
    int env_pitch;          // its pitch in the staged group (boxes start on 128-byte boundaries)
    int stage_bytes;        // one staged group: env_max boxes
    int stages;             // staged groups in the ring
    int ring;               // operand rows resident in tensor memory
    int accs;               // accumulators in tensor memory (64 columns each)
    int smem_bytes;         // dynamic shared memory of the kernel
};

// Tensor maps over the caller's frame buffers, keyed by (address, frames): encoding one costs about a
// microsecond of host time and actor loops hand in the same few buffers again and again.
struct Conv1MapCache {
    static constexpr int kEntries = 16;
    const void* ptr[kEntries] = {};
    int frames[kEntries] = {};
    CUtensorMap map[kEntries];
    int next = 0;
};

// false if the geometry does not fit the kernel (C not 4, 8 or 16; H or W not a multiple of 4; too wide)
bool conv1_plan(const Geometry& g, Conv1Plan* plan);

// w1 [32,C,8,8] bf16 -> packed [128][16*C] fp16 scaled by *scale:
//   row dy*64 + dx*32 + o, column c*16 + uy*4 + ux  holds  w1[o][c][4dy+uy][4dx+ux]
hts_status conv1_pack_weights(const Conv1Plan& pl, const __nv_bfloat16* w1, __half* packed, const float* scale,
                              cudaStream_t s);

// out: fp16 rows [env*P1s + (y/2)*W1s + x/2][128], column ((y%2)*2 + x%2)*32 + o
// ix: dense frames (row e = frame e of obs) or frames gathered by slot from a pool (see Indexing)
hts_status conv1_launch(const Conv1Plan& pl, const CUtensorMap& weight_map, Conv1MapCache& maps, const uint8_t* obs,
                        const Indexing& ix, int n, const float* bias, const float* inv_scale, __half* out, int* status,
                        cudaStream_t s);

}  // namespace hts
