// Layout of the prepared-codebook block shared by prepare.cu and the kernels
// that read it.
#pragma once

#include "common.cuh"

namespace rvq {

constexpr uint32_t kPreparedMagic = 0x52565133u;
constexpr int kSlotCodewords = 128;                       // codewords per operand slot
constexpr int kSlotCells = 10;                            // hi (4), lo (4), norm (1), zero (1) cells of 8 halves
constexpr int kSlotBytes = kSlotCells * kSlotCodewords * 16;   // 20480
constexpr size_t kPreparedParamsOffset = 256;             // StageParams[16]
constexpr size_t kPreparedMaximaOffset = 512;             // StageMaxima[16]
constexpr size_t kPreparedImageOffset = 768;              // operand image, [R][slots][kSlotBytes]

struct PreparedHeader {
    uint32_t magic, R, K, gd, slots;
};

struct StageParams {
    float scale;    // 2^k applied to residuals and codewords of this stage
    float a, b;     // |score error| <= a * ||Z|| + b
    float unsafe;   // non-zero: the scaled codebook left the half-precision range
};

struct StageMaxima {
    uint32_t emax, eerr, nmax, elomax;   // float bit patterns (non-negative), filled with atomicMax
};

__host__ __device__ inline int slots_per_stage(int K) { return (K + kSlotCodewords - 1) / kSlotCodewords; }

}  // namespace rvq
