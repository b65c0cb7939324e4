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
constexpr size_t kPreparedPartialsOffset = 768;           // StagePartial[16 stages][kPrepareParts], scratch of the prepare step
constexpr int kPrepareParts = 16;
constexpr size_t kPreparedImageOffset = 768 + 16 * 16 * 16;   // operand image, [R][slots][kSlotBytes]

struct PreparedHeader {
    uint32_t magic, R, K, gd, slots;
    uint32_t decode_offset;   // byte offset of the decoder section, 0 if absent
};

// Decoder section (group_dim 32, R <= 8, K <= kDecodeMaxK): per stage an affine
// map value = lo_r + q * scale_r * base with q a 16-bit level, scale_r an integer in
// 1..255 and base common to all stages, so that the sum over the stages is
// sum lo_r + base * (sum q_r scale_r) with the second sum exact in 32-bit integers
// (at most 8 * 65535 * 255); then channel slices of the codebooks as levels:
// table[slice][code][stage 0..7][CH channels] uint16.  A slice is CH = 8
// channels wide (four slices) while K <= kDecodeWideK and 4 channels (eight
// slices) above, so that one slice of all codes fits the shared memory of a CTA.
struct DecodeParams {
    float step[8];     // value of one level, scale_r * base, per stage; 0 for absent stages
    float bias;        // sum over stages of the stage minimum lo_r
    float err;         // bound on |sum of table values - sum of float32 values| per channel
    float base;
    float pad[5];
    uint32_t scale[8]; // integer scale of a stage's levels (0 for absent stages)
    // Second set of tables ("summed levels"): the stages of one parity (even r, odd r) share a unit
    // fine enough that the levels of all four of them add up to at most 65535, so a decoder adds
    // table words as they are (two 16-bit fields per 32-bit word, no carry between them) and scales
    // once per parity.  Coarser than the tables above by a factor of about four.
    float pstep[2];      // value of one summed level, pscale * pbase, for even / odd stages; 0 if unused
    float perr;          // bound on |sum of summed-table values - sum of float32 values| per channel
    float pbase;         // common base of the two parities' units
    uint32_t pscale[2];  // integer scales (1..255) of the two parities
};
constexpr int kDecodeWideK = 1536;                        // 128 bytes per code per slice in shared memory
constexpr int kDecodeMaxK = 3072;                         // 64 bytes per code per slice
__host__ __device__ inline int decode_slice_channels(int K) { return K <= kDecodeWideK ? 8 : 4; }
__host__ __device__ inline size_t decode_table_bytes(int K) { return (size_t)K * 512; }   // 32 channels x 8 stages x 2 bytes
// the prepared block holds two such tables: levels scaled per stage, then levels summed per stage parity
constexpr int kDecodeExactWideK = 1792;                   // float32 tables: 128 bytes per code per 4-channel slice
constexpr int kDecodeExactK = 3584;                       // ... 64 bytes per code per 2-channel slice
// Which decoder serves a shape (group_dim 32, a power-of-two number of groups up to 32, depth <= 8; everything
// else gathers from global memory):
//   - float32 table slices (exact sums, any output type) fit shared memory up to kDecodeExactK codes
//     (4 channels per slice up to kDecodeExactWideK, 2 beyond);
//   - 16-bit level tables (16-bit outputs only: their own rounding, 2^-9 or 2^-12 relative, dwarfs the
//     tables') fit up to kDecodeMaxK codes and are the faster ones while the deviations are moderate;
//   - where both fit (16-bit outputs, up to kDecodeMaxK codes) a sample of the deviations decides on the
//     device: four groups at depth 8 in one launch that holds all three kinds of table, other shapes as
//     two launches of which the one not called for returns at once.
__host__ __device__ inline bool decode_exact_tables(const Shape &s)
{
    return s.gd == 32 && s.G <= 32 && (s.G & (s.G - 1)) == 0 && s.R <= 8 && s.K <= kDecodeExactK;
}
__host__ __device__ inline int decode_exact_channels(int K) { return K <= kDecodeExactWideK ? 4 : 2; }
__host__ __device__ inline bool decode_levels_prepared(const Shape &s)    // the prepared block holds level tables
{
    return s.gd == 32 && s.G <= 32 && (s.G & (s.G - 1)) == 0 && s.R <= 8 && s.K <= kDecodeMaxK;
}
__host__ __device__ inline bool decode_levels_supported(const Shape &s)
{
    return decode_levels_prepared(s) && s.dtype != RVQ_F32;
}
__host__ __device__ inline bool decode_sliced_supported(const Shape &s)
{
    return decode_exact_tables(s) || decode_levels_supported(s);
}
__host__ __device__ inline size_t encode_image_bytes(const Shape &s)
{
    return s.gd == 32 ? (size_t)s.R * ((s.K + 127) / 128) * 20480 : 0;
}

struct StageParams {
    float scale;    // 2^k applied to residuals and codewords of this stage
    float a, b;     // |score error| <= a * ||Z|| + b
    float unsafe;   // non-zero: the scaled codebook left the half-precision range
};

struct StagePartial {
    double max_norm2;   // largest squared norm among this part's codewords
    float lo, hi;       // smallest and largest entry
};

struct StageMaxima {
    uint32_t emax, eerr, nmax, elomax;   // float bit patterns (non-negative), filled with atomicMax
};

__host__ __device__ inline int slots_per_stage(int K) { return (K + kSlotCodewords - 1) / kSlotCodewords; }

}  // namespace rvq
