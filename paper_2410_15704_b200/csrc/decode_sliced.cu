// Bandwidth decode for groups of 32 (a power-of-two number of them per head
// vector; written around dim 128 = 4 groups), depth <= 8 (Section 2.2, last
// sentence; Section 3.2).
//
// Every output element needs one codeword element per stage, so a head vector of
// 128 channels (256 output bytes) gathers 1024 table entries: the gather, not HBM, is the
// limit, and it has to come from shared memory without bank conflicts.
//   - A CTA keeps one channel slice (CH = 8 of the 32 codeword channels, 4 when
//     there are more than 1536 codes per stage) of all stages as 16-bit levels:
//     16 CH bytes per code = 8 stages x 2 CH bytes.  The 32 / CH slices of a row
//     tile are handled by as many CTAs; the codes they share come from L2.
//   - One thread produces the CH channels of one (group row, slice).  It reads
//     its codes as one 16-byte load (or cuts them out of the packed bit stream) and
//     visits the stages in an order rotated by its lane, so with CH = 8 the 8
//     lanes of a quarter warp always touch 8 different 16-byte bank groups
//     whatever the codes are (with CH = 4 two lanes of a half warp can meet).
//   - A table entry is a 16-bit level q of its stage's value range, whose unit is
//     an integer multiple (1..255) of a base common to all stages.  One 16-bit x
//     8-bit dot-product instruction per channel and stage accumulates q * scale
//     exactly in 32-bit integers; the sum is converted once, mapped back with the
//     base and the sum of the stage minima, multiplied by the stored deviation
//     and rounded once.
//   - The level tables are off by at most dp->err (half a level per stage) times
//     the deviation.  A row whose deviation makes that more than 0.9e-3 sums the
//     float32 codewords instead (stage order, from global memory), so the result
//     before the output rounding is always within 1e-3 of the exact sum.
//   - With strided groups the 4 lanes of a head vector exchange their results so
//     that every lane stores 16 contiguous bytes.
#include "prepared.cuh"

namespace rvq {

namespace {

constexpr int kDecThreads = 1024;

template <int DT> struct Out;
template <> struct Out<RVQ_BF16> {
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<uint32_t *>(&h);
    }
};
template <> struct Out<RVQ_F16> {
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __half2 h = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t *>(&h);
    }
};

// Codes r = 0 .. R-1 (R <= 8) of BITS bits each (BITS = 0: `bits`, known at run time only) from the 96-bit
// window u0:u1:u2, packed two per word into cw[4] (which comes in zeroed).
template <int BITS, bool FULL = false>      // FULL: R is 8
__device__ __forceinline__ void cut_codes(uint32_t u0, uint32_t u1, uint32_t u2, int R, uint32_t (&cw)[4], int bits = BITS)
{
    const int width = BITS ? BITS : bits;
    const uint32_t mask = (1u << width) - 1u;
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        if (FULL || r < R) {
            const int o = r * width, k = o >> 5;
            const uint32_t lo = k == 0 ? u0 : (k == 1 ? u1 : u2), hi = k == 0 ? u1 : (k == 1 ? u2 : 0u);
            cw[r >> 1] |= (__funnelshift_r(lo, hi, o & 31) & mask) << (16 * (r & 1));
        }
    }
}

struct RopeArgs {
    const int32_t *position;      // position of head vector v: position[v / per_position]
    int per_position;
    const float2 *table;          // (cos, sin) [positions][64]
    int positions;
    int shift;                    // log2(per_position) when that is a power of two, else -1
};

// Codeword element held at place i of slice `slice`.
template <int CH, int ROPE>
__device__ __forceinline__ int slice_element(int layout, int slice, int i)
{
    if (ROPE == 1 && layout == RVQ_GROUP_STRIDED)       // the first CH / 2 places and their partners 16 elements on
        return (CH / 2) * slice + (i % (CH / 2)) + 16 * (i / (CH / 2));
    return slice * CH + i;
}

// ROPE (float32 tables with 4-channel slices only): the rotary embedding is applied to the decoded
// head vector before it is rounded and stored (1: pairs are channels (k, k + 64), 2: (2k, 2k + 1)).
// Both channels of a pair are in one thread, or in two lanes of the head vector's four, for every
// combination but one: strided groups with half-split pairs, where the partner of element i of a
// group is element i + 16 of the same group.  There a slice is the elements {2 sl, 2 sl + 1,
// 2 sl + 16, 2 sl + 17} instead of four consecutive ones.
template <int DT, int CH, bool F32T, int ROPE = 0>
__device__ __forceinline__ void
decode_sliced_body(const Shape &s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t n,
                   const uint8_t *__restrict__ dsec, const float *__restrict__ cb, void *__restrict__ out,
                   int64_t stride, rvq_status *st, uint8_t *table, RopeArgs ra = RopeArgs())
{
    static_assert(ROPE == 0 || CH == 4 || CH == 2, "rotary decode uses 4- or 2-channel slices");
    static_assert(F32T || CH >= 4, "2-channel slices are for float32 tables");
    // table: [K][8 stages][kEntry bytes] in shared memory
    constexpr int NS = 32 / CH;                                  // slices
    if ((int)blockIdx.x >= ((int)gridDim.x / NS) * NS) return;   // (a grid sized for another slice count)
    constexpr uint32_t kEntry = (F32T ? 4 : 2) * CH, kLine = 8 * kEntry;   // bytes per (code, stage) and per code
    const DecodeParams *dp = reinterpret_cast<const DecodeParams *>(dsec);
    const int slice = blockIdx.x % NS, part = blockIdx.x / NS, parts = gridDim.x / NS;
    const int tid = threadIdx.x, lane = tid & 31, rot = lane & 7;
    if (F32T) {
        // entry (code j, stage r) = CH channels of codeword j of stage r; consecutive threads fill
        // consecutive entries (stage fastest), so the shared-memory stores do not collide
        for (int t = tid; t < s.K * 8; t += kDecThreads) {
            const int r = t & 7, j = t >> 3;
            float *dst = reinterpret_cast<float *>(table + (size_t)t * kEntry);
            const float *src = cb + ((size_t)r * s.K + j) * 32;
            float e[CH];
            if (r >= s.R) {
#pragma unroll
                for (int i = 0; i < CH; ++i) e[i] = 0.0f;
            } else if (CH == 4 && slice_element<CH, ROPE>(s.layout, slice, 0) == slice * CH &&
                       slice_element<CH, ROPE>(s.layout, slice, 1) == slice * CH + 1 &&
                       slice_element<CH, ROPE>(s.layout, slice, 2) == slice * CH + 2) {
                const float4 q = __ldg(reinterpret_cast<const float4 *>(src + slice * CH));
                e[0] = q.x; e[1] = q.y; e[CH - 2] = q.z; e[CH - 1] = q.w;
            } else if (CH == 2 && slice_element<CH, ROPE>(s.layout, slice, 0) == slice * CH &&
                       slice_element<CH, ROPE>(s.layout, slice, 1) == slice * CH + 1) {
                const float2 q = __ldg(reinterpret_cast<const float2 *>(src + slice * CH));
                e[0] = q.x; e[1] = q.y;
            } else {
#pragma unroll
                for (int i = 0; i < CH; ++i) e[i] = __ldg(src + slice_element<CH, ROPE>(s.layout, slice, i));
            }
            if (CH == 4) *reinterpret_cast<float4 *>(dst) = make_float4(e[0], e[1], e[CH - 2], e[CH - 1]);
            else if (CH == 2) *reinterpret_cast<float2 *>(dst) = make_float2(e[0], e[1]);
            else {
#pragma unroll
                for (int i = 0; i < CH; ++i) dst[i] = e[i];
            }
        }
    } else if (ROPE != 0) {
        // Level tables with the rotary slices: the prepared block keeps, per 4-element slice, entries of two
        // words (elements 4s, 4s+1 | 4s+2, 4s+3); this CTA's entry takes the word of its places 0-1 and the
        // word of its places 2-3, which for half-split pairs on strided groups come from two different slices.
        const uint32_t *lev = reinterpret_cast<const uint32_t *>(dsec + 256);
        const int ea = slice_element<CH, ROPE>(s.layout, slice, 0), eb = slice_element<CH, ROPE>(s.layout, slice, 2);
        for (int t = tid; t < s.K * 8; t += kDecThreads) {
            const int r = t & 7, j = t >> 3;
            const uint32_t wa = __ldg(lev + ((((size_t)(ea >> 2) * s.K + j) * 8 + r) * 2 + ((ea & 3) >> 1)));
            const uint32_t wb = __ldg(lev + ((((size_t)(eb >> 2) * s.K + j) * 8 + r) * 2 + ((eb & 3) >> 1)));
            *reinterpret_cast<uint2 *>(table + (size_t)t * kEntry) = make_uint2(wa, wb);
        }
    } else {
        const uint4 *src = reinterpret_cast<const uint4 *>(dsec + 256) + (size_t)slice * s.K * CH;
        uint4 *dst = reinterpret_cast<uint4 *>(table);
        for (int t = tid; t < s.K * CH; t += kDecThreads) dst[t] = __ldg(src + t);
    }
    // this thread visits stage (rot + k) & 7 at step k: its steps' scales and line offsets
    uint32_t scale[8];
    uint32_t unit[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { scale[k] = F32T ? 0u : dp->scale[(rot + k) & 7]; unit[k] = (uint32_t)((rot + k) & 7) * kEntry; }
    const float bias = F32T ? 0.0f : dp->bias, base = F32T ? 0.0f : dp->base;
    // deviations the tables may serve (a rotation mixes two table values: their errors add up to sqrt(2) times one)
    const float exact_above = F32T ? INFINITY : (dp->err > 0.0f ? (ROPE != 0 ? 0.6e-3f : 0.9e-3f) / dp->err : INFINITY);
    __syncthreads();

    // dim = 32 G with G a power of two; the stores of strided groups below are written for G = 4 (dim 128),
    // other G store element by element
    const int gs = __ffs(s.G) - 1;
    const int64_t rows = n << gs;
    uint32_t bad = 0;
    for (int64_t row = (int64_t)part * kDecThreads + tid; row - tid < rows; row += (int64_t)parts * kDecThreads) {
        // (the loop bound keeps whole warps together for the shuffles below)
        const bool live = row < rows;
        const int64_t v = live ? row >> gs : 0;
        const int g = (int)(row & (s.G - 1));
        // rotary decode: this row's cosines and sines, asked for first so that they arrive during the gather
        float2 rc[4];
        if (ROPE != 0) {
            // (the launcher sends larger problems elsewhere: a 64-bit division here is a subroutine call
            // that costs the whole loop its register allocation)
            const uint32_t token = ra.shift >= 0 ? (uint32_t)v >> ra.shift : (uint32_t)v / (uint32_t)ra.per_position;
            int pos = live ? __ldg(ra.position + token) : 0;
            pos = min(max(pos, 0), ra.positions - 1);
            const int hG = s.G >> 1;                                  // groups per half of the head vector
            const float2 *cs = ra.table + (size_t)pos * (16 * s.G);      // dim / 2 pairs per position
            if (CH == 2) {
                // one pair in the thread (half-split pairs on strided groups: pair 4 slice + g; adjacent pairs on
                // contiguous groups: pair 16 g + slice), or two places whose partners sit in another lane
                if (ROPE == 1 && s.layout == RVQ_GROUP_STRIDED) rc[0] = __ldg(cs + slice * s.G + g);
                else if (ROPE == 2 && s.layout != RVQ_GROUP_STRIDED) rc[0] = __ldg(cs + g * 16 + slice);
                else if (ROPE == 1) {                                  // pairs 32 (g mod G/2) + 2 slice + i
                    const float4 cc = __ldg(reinterpret_cast<const float4 *>(cs + (g & (hG - 1)) * 32 + slice * 2));
                    rc[0] = make_float2(cc.x, cc.y); rc[1] = make_float2(cc.z, cc.w);
                } else {                                               // pairs (G / 2) (2 slice + i) + g / 2
                    rc[0] = __ldg(cs + (slice * 2) * hG + (g >> 1)); rc[1] = __ldg(cs + (slice * 2 + 1) * hG + (g >> 1));
                }
            } else if (ROPE == 1 && s.layout == RVQ_GROUP_STRIDED) {   // pairs G (2 slice + i) + g
                rc[0] = __ldg(cs + (slice * 2) * s.G + g); rc[1] = __ldg(cs + (slice * 2 + 1) * s.G + g);
            } else if (ROPE == 2 && s.layout != RVQ_GROUP_STRIDED) {   // pairs 16 g + 2 slice + i
                const float4 cc = __ldg(reinterpret_cast<const float4 *>(cs + g * 16 + slice * 2));
                rc[0] = make_float2(cc.x, cc.y); rc[1] = make_float2(cc.z, cc.w);
            } else if (ROPE == 1) {                                    // pairs 32 (g mod G/2) + 4 slice + i
                const float4 *q = reinterpret_cast<const float4 *>(cs + (g & (hG - 1)) * 32 + slice * 4);
                const float4 lo = __ldg(q), hi = __ldg(q + 1);
                rc[0] = make_float2(lo.x, lo.y); rc[1] = make_float2(lo.z, lo.w);
                rc[2] = make_float2(hi.x, hi.y); rc[3] = make_float2(hi.z, hi.w);
            } else {                                                   // pairs 2 (4 slice + i) + g / 2
#pragma unroll
                for (int i = 0; i < 4; ++i) rc[i] = __ldg(cs + (slice * 4 + i) * hG + (g >> 1));
            }
        }
        // the 8 codes of this row as 4 words, stage r in half r
        uint32_t cw[4] = {0u, 0u, 0u, 0u};
        if (live) {
            if (s.bits == 16 && s.R == 8) {
                const uint4 c = __ldg(reinterpret_cast<const uint4 *>(codes) + row);
                cw[0] = c.x; cw[1] = c.y; cw[2] = c.z; cw[3] = c.w;
            } else if (s.R * s.bits <= 96) {
                // The row's R codes are R * bits <= 96 consecutive bits of the vector's stream, starting
                // at bit g * R * bits: fetch the (up to four) words that hold them, shift the window
                // down to bit 0, and cut the codes out of it.
                const int words = s.code_bytes >> 2;
                const uint32_t *wv = reinterpret_cast<const uint32_t *>(codes) + v * words;
                const int bit0 = g * s.R * s.bits, wi = bit0 >> 5, sh = bit0 & 31;
                const uint32_t q0 = __ldg(wv + wi);
                const uint32_t q1 = wi + 1 < words ? __ldg(wv + wi + 1) : 0u;
                const uint32_t q2 = wi + 2 < words ? __ldg(wv + wi + 2) : 0u;
                const uint32_t q3 = wi + 3 < words ? __ldg(wv + wi + 3) : 0u;
                const uint32_t u0 = __funnelshift_r(q0, q1, sh), u1 = __funnelshift_r(q1, q2, sh);
                const uint32_t u2 = __funnelshift_r(q2, q3, sh);
                switch (s.bits) {                  // the usual widths with their offsets known at compile time
                case 10: if (s.R == 8) cut_codes<10, true>(u0, u1, u2, 8, cw); else cut_codes<10>(u0, u1, u2, s.R, cw); break;
                case 11: if (s.R == 8) cut_codes<11, true>(u0, u1, u2, 8, cw); else cut_codes<11>(u0, u1, u2, s.R, cw); break;
                case 12: cut_codes<12>(u0, u1, u2, s.R, cw); break;
                default: cut_codes<0>(u0, u1, u2, s.R, cw, s.bits); break;
                }
            } else {
                const uint8_t *vec = reinterpret_cast<const uint8_t *>(codes) + v * s.code_bytes;
                for (int r = 0; r < s.R; ++r)
                    cw[r >> 1] |= read_code(vec, g * s.R + r, s.bits, s.code_bytes) << (16 * (r & 1));
            }
        }
        const uint32_t cn[4] = {cw[0], cw[1], cw[2], cw[3]};      // natural order, for the exact route
        // rotate the 8 halves left by `rot` so that step k finds its code at a fixed place
        {
            uint32_t a0 = cw[0], a1 = cw[1], a2 = cw[2], a3 = cw[3];
            if (rot & 4) { uint32_t t0 = a0, t1 = a1; a0 = a2; a1 = a3; a2 = t0; a3 = t1; }
            if (rot & 2) { uint32_t t0 = a0; a0 = a1; a1 = a2; a2 = a3; a3 = t0; }
            if (rot & 1) {
                const uint32_t b0 = __funnelshift_r(a0, a1, 16), b1 = __funnelshift_r(a1, a2, 16);
                const uint32_t b2 = __funnelshift_r(a2, a3, 16), b3 = __funnelshift_r(a3, a0, 16);
                a0 = b0; a1 = b1; a2 = b2; a3 = b3;
            }
            cw[0] = a0; cw[1] = a1; cw[2] = a2; cw[3] = a3;
        }
        // codes out of range (never produced by the encoder): counted, read as code 0
        {
            const uint32_t m = __vmaxu2(__vmaxu2(cw[0], cw[1]), __vmaxu2(cw[2], cw[3]));
            if (max(m & 0xFFFFu, m >> 16) >= (uint32_t)s.K) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t lo = cw[c] & 0xFFFFu, hi = cw[c] >> 16;
                    if (lo >= (uint32_t)s.K) { lo = 0; ++bad; }
                    if (hi >= (uint32_t)s.K) { hi = 0; ++bad; }
                    cw[c] = lo | (hi << 16);
                }
            }
        }
        const float sd = live ? __half2float(__ushort_as_half(std16[v])) : 0.0f;
        float o8[CH];
        if constexpr (F32T) {
            float acc[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i) acc[i] = 0.0f;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t j = (k & 1) ? (cw[k >> 1] >> 16) : (cw[k >> 1] & 0xFFFFu);
                if (CH == 4) {
                    const float4 t = *reinterpret_cast<const float4 *>(table + j * kLine + unit[k]);
                    acc[0] += t.x; acc[1] += t.y; acc[CH - 2] += t.z; acc[CH - 1] += t.w;
                } else {
                    const float2 t = *reinterpret_cast<const float2 *>(table + j * kLine + unit[k]);
                    acc[0] += t.x; acc[1] += t.y;
                }
            }
#pragma unroll
            for (int i = 0; i < CH; ++i) o8[i] = acc[i] * sd;
        } else {
            // integer sums of level * scale: one 16-bit x 8-bit dot-product instruction per channel and stage
            // (the scale sits in byte 0 for the low half of a table word, in byte 1 for the high half)
            uint32_t acc[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i) acc[i] = 0u;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t j = (k & 1) ? (cw[k >> 1] >> 16) : (cw[k >> 1] & 0xFFFFu);
                const uint32_t s_lo = scale[k], s_hi = scale[k] << 8;
                uint32_t e[CH / 2];
                if (CH == 8) {
                    const uint4 t = *reinterpret_cast<const uint4 *>(table + j * kLine + unit[k]);
                    e[0] = t.x; e[1] = t.y; e[CH / 2 - 2] = t.z; e[CH / 2 - 1] = t.w;
                } else {
                    const uint2 t = *reinterpret_cast<const uint2 *>(table + j * kLine + unit[k]);
                    e[0] = t.x; e[1] = t.y;
                }
#pragma unroll
                for (int i = 0; i < CH / 2; ++i) {
                    acc[2 * i] = __dp2a_lo(e[i], s_lo, acc[2 * i]);
                    acc[2 * i + 1] = __dp2a_lo(e[i], s_hi, acc[2 * i + 1]);
                }
            }
#pragma unroll
            for (int i = 0; i < CH; ++i) o8[i] = fmaf((float)acc[i], base, bias) * sd;
        }
        if constexpr (!F32T) if (fabsf(sd) > exact_above && fabsf(sd) < INFINITY) {
            // too coarse for this deviation: the float32 codewords themselves, summed in stage order
            float ex[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i) ex[i] = 0.0f;
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                if (r < s.R) {
                    uint32_t j = (r & 1) ? (cn[r >> 1] >> 16) : (cn[r >> 1] & 0xFFFFu);
                    if (j >= (uint32_t)s.K) j = 0;
                    if (ROPE != 0) {
                        const float *e = cb + ((size_t)r * s.K + j) * 32;
#pragma unroll
                        for (int i = 0; i < CH; ++i) ex[i] += __ldg(e + slice_element<CH, ROPE>(s.layout, slice, i));
                    } else {
                        const float4 *e = reinterpret_cast<const float4 *>(cb + ((size_t)r * s.K + j) * 32 + slice * CH);
#pragma unroll
                        for (int q = 0; q < CH / 4; ++q) {
                            const float4 t = __ldg(e + q);
                            ex[4 * q] += t.x; ex[4 * q + 1] += t.y; ex[4 * q + 2] += t.z; ex[4 * q + 3] += t.w;
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < CH; ++i) o8[i] = ex[i] * sd;
        }

        if (ROPE != 0) {
            const bool strided = s.layout == RVQ_GROUP_STRIDED;
            constexpr int H = CH / 2;
            if (ROPE == 1 && strided) {
                // places 0 .. H-1 are channels 4 e + g of the first half, places H .. CH-1 their partners 64 further on
#pragma unroll
                for (int i = 0; i < H; ++i) {
                    const float a = o8[i], b = o8[i + H];
                    o8[i] = a * rc[i].x - b * rc[i].y;
                    o8[i + H] = b * rc[i].x + a * rc[i].y;
                }
            } else if (ROPE == 2 && !strided) {
                // channels 32 g + CH slice + i: the pairs (0, 1) (and (2, 3)) are in this thread
#pragma unroll
                for (int i = 0; i < H; ++i) {
                    const float a = o8[2 * i], b = o8[2 * i + 1];
                    o8[2 * i] = a * rc[i].x - b * rc[i].y;
                    o8[2 * i + 1] = b * rc[i].x + a * rc[i].y;
                }
            } else {
                // the partner is the same place of another group: lane g ^ G/2 (half-split pairs, contiguous
                // groups: channels 32 g + e and 32 (g ^ G/2) + e) or lane g ^ 1 (adjacent pairs, strided groups:
                // channels G e + g and G e + (g ^ 1))
                const int other = ROPE == 1 ? (s.G >> 1) : 1;
                const bool first = (g & other) == 0;
#pragma unroll
                for (int i = 0; i < CH; ++i) {
                    const float b = __shfl_xor_sync(0xFFFFFFFFu, o8[i], other);
                    o8[i] = first ? o8[i] * rc[i].x - b * rc[i].y : o8[i] * rc[i].x + b * rc[i].y;
                }
            }
        }
        if (s.G != 4 && s.layout == RVQ_GROUP_STRIDED) {
            // channel of place i: element * G + g
            if (live) {
#pragma unroll
                for (int i = 0; i < CH; ++i)
                    store_from_float(out, v * stride + (int64_t)slice_element<CH, ROPE>(s.layout, slice, i) * s.G + g, DT, o8[i]);
            }
        } else if constexpr (CH == 2) {
            // two places per thread
            if (DT == RVQ_F32) {
                float *o = reinterpret_cast<float *>(out) + v * stride;
                if (s.layout == RVQ_GROUP_CONTIGUOUS) {
                    if (live) *reinterpret_cast<float2 *>(o + g * 32 + slice * 2) = make_float2(o8[0], o8[1]);
                } else if (live) {
                    o[4 * slice_element<CH, ROPE>(s.layout, slice, 0) + g] = o8[0];
                    o[4 * slice_element<CH, ROPE>(s.layout, slice, 1) + g] = o8[1];
                }
            } else {
                const uint32_t w0 = Out<DT == RVQ_F32 ? RVQ_BF16 : DT>::pack(o8[0], o8[1]);
                uint16_t *o16 = reinterpret_cast<uint16_t *>(out) + v * stride;
                if (s.layout == RVQ_GROUP_CONTIGUOUS) {
                    if (live) *reinterpret_cast<uint32_t *>(o16 + g * 32 + slice * 2) = w0;
                } else {
                    // Lane g holds places 0 and 1 of group g; the four lanes cover, per place, the four
                    // consecutive channels 4 element .. 4 element + 3.  Lane L stores two of them: place L / 2,
                    // groups 2 (L % 2) and 2 (L % 2) + 1, fetched from those two lanes.
                    const int base_lane = (tid & 31) & ~3, ga = 2 * (g & 1);
                    const uint32_t wa = __shfl_sync(0xFFFFFFFFu, w0, base_lane + ga);
                    const uint32_t wb = __shfl_sync(0xFFFFFFFFu, w0, base_lane + ga + 1);
                    const uint32_t both = __byte_perm(wa, wb, (g & 2) ? 0x7632 : 0x5410);
                    if (live)
                        *reinterpret_cast<uint32_t *>(o16 + 4 * slice_element<CH, ROPE>(s.layout, slice, g >> 1) + ga) = both;
                }
            }
        } else {
            if (DT == RVQ_F32) {
                if (s.layout == RVQ_GROUP_CONTIGUOUS) {
                    if (live) {
                        float4 *o = reinterpret_cast<float4 *>(reinterpret_cast<float *>(out) + v * stride + g * 32 + slice * CH);
    #pragma unroll
                        for (int i = 0; i < CH / 4; ++i)
                            o[i] = make_float4(o8[4 * i], o8[4 * i + 1], o8[4 * i + 2], o8[4 * i + 3]);
                    }
                } else if (live) {
                    float *o = reinterpret_cast<float *>(out) + v * stride + g;
    #pragma unroll
                    for (int i = 0; i < CH; ++i) o[4 * slice_element<CH, ROPE>(s.layout, slice, i)] = o8[i];   // channel 4 element + g
                }
            } else {
                uint32_t w[CH / 2];
    #pragma unroll
                for (int c = 0; c < CH / 2; ++c) w[c] = Out<DT == RVQ_F32 ? RVQ_BF16 : DT>::pack(o8[2 * c], o8[2 * c + 1]);
                uint16_t *o16 = reinterpret_cast<uint16_t *>(out) + v * stride;
                if (s.layout == RVQ_GROUP_CONTIGUOUS) {
                    if (live) {
                        if (CH == 8)
                            *reinterpret_cast<uint4 *>(o16 + g * 32 + slice * 8) = make_uint4(w[0], w[1], w[CH / 2 - 2], w[CH / 2 - 1]);
                        else
                            *reinterpret_cast<uint2 *>(o16 + g * 32 + slice * 4) = make_uint2(w[0], w[1]);
                    }
                } else if (CH == 8) {
                    // Lane g holds element pairs (2c, 2c+1) of group g, i.e. channels 32 slice + 8c + g and + 4.
                    // Lane c' of the 4-lane set wants pairs c' of all four groups: a 4x4 transpose of words.
                    // two butterfly steps: exchange odd/even words with lane g^1, then word pairs with lane g^2
                    uint32_t &w0 = w[0], &w1 = w[1], &w2 = w[CH / 2 - 2], &w3 = w[CH / 2 - 1];
                    {
                        const bool b1 = g & 1, b2 = g & 2;
                        const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, b1 ? w0 : w1, 1);
                        const uint32_t r1 = __shfl_xor_sync(0xFFFFFFFFu, b1 ? w2 : w3, 1);
                        if (b1) { w0 = r0; w2 = r1; } else { w1 = r0; w3 = r1; }
                        const uint32_t r2 = __shfl_xor_sync(0xFFFFFFFFu, b2 ? w0 : w2, 2);
                        const uint32_t r3 = __shfl_xor_sync(0xFFFFFFFFu, b2 ? w1 : w3, 2);
                        if (b2) { w0 = r2; w1 = r3; } else { w2 = r2; w3 = r3; }
                    }
                    // now w[q] = pair g of group q: (element 2g of group q, element 2g+1 of group q)
                    const uint32_t o0 = __byte_perm(w0, w1, 0x5410), o1 = __byte_perm(w2, w3, 0x5410);
                    const uint32_t o2 = __byte_perm(w0, w1, 0x7632), o3 = __byte_perm(w2, w3, 0x7632);
                    // channels 32 slice + 8 g + 0..7: element 2g of groups 0..3, then element 2g+1 of groups 0..3
                    if (live) *reinterpret_cast<uint4 *>(o16 + slice * 32 + g * 8) = make_uint4(o0, o1, o2, o3);
                } else {
                    // Lane g holds elements 4 slice + 0..3 of group g as w[0] = (e0, e1), w[1] = (e2, e3); the
                    // 16 channels 16 slice .. 16 slice + 15 are element-major, so lane L stores element L of
                    // the four groups.  Exchange words with lane g^2, then halves with lane g^1.
                    const bool b1 = g & 1, b2 = g & 2;
                    const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, b2 ? w[0] : w[1], 2);
                    // lanes 0, 1 now hold (e0, e1) of groups g and g + 2; lanes 2, 3 hold (e2, e3) of g - 2 and g
                    const uint32_t lo_g = b2 ? r0 : w[0], hi_g = b2 ? w[1] : r0;   // lower and upper group of the pair
                    // keep the half this lane stores (e_L), send the other one
                    const uint32_t keep = __byte_perm(lo_g, hi_g, b1 ? 0x7632 : 0x5410);
                    const uint32_t send = __byte_perm(lo_g, hi_g, b1 ? 0x5410 : 0x7632);
                    const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, send, 1);
                    // keep = element L of groups (g & 1) and (g & 1) + 2, got = element L of the other two
                    const uint32_t even = b1 ? got : keep, odd = b1 ? keep : got;   // groups (0, 2) and (1, 3)
                    if (live)
                        *reinterpret_cast<uint2 *>(o16 + 4 * slice_element<CH, ROPE>(s.layout, slice, g)) =
                            make_uint2(__byte_perm(even, odd, 0x5410), __byte_perm(even, odd, 0x7632));
                }
            }
    
        }
    }
    if (bad && st && slice == 0) atomicAdd(&st->bad_codes, bad);   // every slice sees the same codes
}

// The level-table decoder for the shapes the timings are quoted on: head vectors of four groups of 32
// (dim 128), depth 8, 16-bit outputs; codes as uint16 or as a packed stream of 10 to 12 bits.  Same
// tables, same arithmetic and same results as decode_sliced_body<DT, CH, false>; what differs is the
// instruction count (the loop is issue bound): 32-bit row numbers, table addresses cut out of the
// code words with one shift and one mask-or each, one scale register per stage for both halves of
// a table word (dp2a.lo reads bytes 0-1 of it, dp2a.hi bytes 2-3), layout and code width known at
// compile time, no per-row code range loop unless a code is out of range.
// SUMMED: the tables whose levels add up within 16 bits per stage parity (prepared.cuh): the table
// words of the even steps and of the odd steps are added as they are (which parity of stages a
// thread's even steps are depends on its lane), and scaled once per parity.
// ROPE (8-channel slices): the rotary embedding is applied to the float32 results before the one
// rounding (1: pairs are channels (k, k + 64), 2: (2k, 2k + 1)).  The partner of a channel is in the
// same thread (adjacent pairs on contiguous groups), in the lane of another group of the same head
// vector (half-split pairs on contiguous groups: lane g ^ 2; adjacent pairs on strided groups: lane
// g ^ 1), or -- half-split pairs on strided groups, where the partner of element i of a group is
// element i + 16 of the same group -- brought into the thread by making a slice the elements
// {4 sl .. 4 sl + 3} and {4 sl + 16 .. 4 sl + 19} instead of eight consecutive ones.
// Lanes g = 0..3 of a head vector hold the elements (e0, e1) and (e2, e3) of their group as two packed
// words; lane L gets back element L of the groups 0..3 (four consecutive channels of a strided row).
__device__ __forceinline__ uint2 transpose_group_elements(uint32_t w0, uint32_t w1, uint32_t g)
{
    const bool b1 = g & 1u, b2 = g & 2u;
    const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, b2 ? w0 : w1, 2);
    // lanes 0, 1 now hold (e0, e1) of groups g and g + 2; lanes 2, 3 hold (e2, e3) of g - 2 and g
    const uint32_t lo_g = b2 ? r0 : w0, hi_g = b2 ? w1 : r0;
    const uint32_t keep = __byte_perm(lo_g, hi_g, b1 ? 0x7632 : 0x5410);
    const uint32_t send = __byte_perm(lo_g, hi_g, b1 ? 0x5410 : 0x7632);
    const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, send, 1);
    const uint32_t even = b1 ? got : keep, odd = b1 ? keep : got;       // groups (0, 2) and (1, 3)
    return make_uint2(__byte_perm(even, odd, 0x5410), __byte_perm(even, odd, 0x7632));
}

// F32 (4 channels per slice): the table holds the float32 codeword channels themselves (16 bytes per
// code and stage, the geometry of the 8-channel level tables), filled from the codebooks by the CTA;
// exact float32 sums, no table error and no exact route.
template <int DT, int CH, int LAYOUT, int BITS, bool SUMMED, int ROPE = 0, bool F32 = false>
__device__ __forceinline__ void
decode_levels_fast(const Shape &s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t n,
                   const uint8_t *__restrict__ dsec, const float *__restrict__ cb, void *__restrict__ out,
                   int64_t stride, rvq_status *st, uint8_t *table, RopeArgs ra = RopeArgs())
{
    static_assert(ROPE == 0 || CH == 8 || F32, "the rotary variant uses 8-channel level slices or 4-channel float32 slices");
    static_assert(!F32 || (CH == 4 && !SUMMED), "float32 tables: 4-channel slices");
    // half-split pairs on strided groups: a slice is two runs of elements 16 apart (CH / 2 each), so that
    // both channels of a pair are in the thread
    constexpr bool SPLIT = ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED;
    constexpr int NS = 32 / CH;                                  // slices
    if ((int)blockIdx.x >= ((int)gridDim.x / NS) * NS) return;
    constexpr uint32_t kEntry = F32 ? 16 : 2 * CH;               // bytes per (code, stage); a code's line is 8 entries
    constexpr int kShift = (F32 || CH == 8) ? 7 : 6;             // log2 of the line's bytes
    const DecodeParams *dp = reinterpret_cast<const DecodeParams *>(dsec);
    const uint32_t slice = blockIdx.x % NS, part = blockIdx.x / NS, parts = gridDim.x / NS;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, rot = lane & 7u;
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(dsec + 256 + (SUMMED ? decode_table_bytes(s.K) : 0)) +
                           (size_t)slice * s.K * CH;
        uint4 *dst = reinterpret_cast<uint4 *>(table);
        if (F32) {
            // entry (code j, stage r) = elements 4 slice .. 4 slice + 3 of codeword j of stage r (rotary slices
            // of strided groups: 2 slice, 2 slice + 1 and the two 16 elements on)
            for (uint32_t t = tid; t < (uint32_t)s.K * 8; t += kDecThreads) {
                const uint32_t r = t & 7u, j = t >> 3;
                const float *src = cb + ((size_t)r * s.K + j) * 32;
                if (SPLIT) {
                    const uint2 a = __ldg(reinterpret_cast<const uint2 *>(src + 2 * slice));
                    const uint2 b = __ldg(reinterpret_cast<const uint2 *>(src + 2 * slice + 16));
                    dst[t] = make_uint4(a.x, a.y, b.x, b.y);
                } else {
                    dst[t] = __ldg(reinterpret_cast<const uint4 *>(src) + slice);
                }
            }
        } else if (SPLIT) {
            // entry (code, stage) = elements 4 slice .. + 3 (half of the entry of slice / 2 in the prepared
            // table) followed by their partners 16 elements on (the same half of the entry of slice / 2 + 2)
            const uint2 *half = reinterpret_cast<const uint2 *>(dsec + 256 + (SUMMED ? decode_table_bytes(s.K) : 0));
            const size_t per_slice = (size_t)s.K * 8;            // entries of one slice
            const uint2 *sa = half + ((size_t)(slice >> 1) * per_slice) * 2 + (slice & 1u);
            const uint2 *sb = half + ((size_t)((slice >> 1) + 2) * per_slice) * 2 + (slice & 1u);
            for (uint32_t t = tid; t < (uint32_t)s.K * 8; t += kDecThreads) {
                const uint2 a = __ldg(sa + 2 * (size_t)t), b = __ldg(sb + 2 * (size_t)t);
                dst[t] = make_uint4(a.x, a.y, b.x, b.y);
            }
        } else {
            for (uint32_t t = tid; t < (uint32_t)s.K * CH; t += kDecThreads) dst[t] = __ldg(src + t);
        }
    }
    // this thread visits stage (rot + k) & 7 at step k (the 8 lanes of a quarter warp then touch 8
    // different bank groups): the scale of that stage in bytes 0 and 3, and the byte offset of its entry
    uint32_t scale[SUMMED ? 2 : 8], unit[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        if (!SUMMED || k < 2) {
            const uint32_t sc = SUMMED ? dp->pscale[(rot + k) & 1u] : dp->scale[(rot + k) & 7u];
            scale[SUMMED ? (k & 1) : k] = sc | (sc << 24);
        }
        unit[k] = ((rot + k) & 7u) * kEntry;
    }
    const float bias = dp->bias, base = SUMMED ? dp->pbase : dp->base;
    const float terr = SUMMED ? dp->perr : dp->err;
    const float exact_above = terr > 0.0f ? (ROPE != 0 ? 0.6e-3f : 0.9e-3f) / terr : INFINITY;   // (a rotation adds two table errors)
    const uint32_t Ku = (uint32_t)s.K;
    __syncthreads();

    const uint32_t rows = (uint32_t)n << 2;                       // the launcher guarantees n * 4 < 2^31
    const uint32_t smem_table = (uint32_t)__cvta_generic_to_shared(table);
    uint32_t bad = 0;
    // The codes and the deviation of a row are fetched one iteration ahead, so that their latency is
    // spent while the previous row's table entries are gathered.
    auto fetch = [&](uint32_t row, uint32_t &c0, uint32_t &c1, uint32_t &c2, uint32_t &c3, uint16_t &sdb, int &posv) {
        c0 = c1 = c2 = c3 = 0u;
        sdb = 0;
        posv = 0;
        if (row >= rows) return;
        const uint32_t v = row >> 2, g = row & 3u;
        sdb = __ldg(std16 + v);
        if (ROPE != 0) posv = __ldg(ra.position + (ra.shift >= 0 ? v >> ra.shift : v / (uint32_t)ra.per_position));
        if (BITS == 16) {
            const uint4 c = __ldg(reinterpret_cast<const uint4 *>(codes) + row);
            c0 = c.x; c1 = c.y; c2 = c.z; c3 = c.w;
        } else {
            // the row's 8 codes are 8 * BITS <= 96 consecutive bits of the vector's stream of 32 * BITS
            // bits, starting at bit g * 8 * BITS: the words that hold them (cut below)
            constexpr int words = BITS;                                  // 32 * BITS / 32
            const uint32_t *wv = reinterpret_cast<const uint32_t *>(codes) + (size_t)v * words;
            const uint32_t wi = (g * (8u * BITS)) >> 5;
            c0 = __ldg(wv + wi); c1 = __ldg(wv + wi + 1);
            c2 = wi + 2 < (uint32_t)words ? __ldg(wv + wi + 2) : 0u;
            c3 = wi + 3 < (uint32_t)words ? __ldg(wv + wi + 3) : 0u;
        }
    };
    uint32_t p0, p1, p2, p3;
    uint16_t psd;
    int ppos;
    fetch(part * kDecThreads + tid, p0, p1, p2, p3, psd, ppos);
    for (uint32_t row = part * kDecThreads + tid; row - tid < rows; row += parts * kDecThreads) {
        // (the loop bound keeps whole warps together for the shuffles below)
        const bool live = row < rows;
        const uint32_t v = live ? row >> 2 : 0u, g = row & 3u;
        // the 8 codes of this row as 4 words, stage r in half r
        uint32_t c0 = p0, c1 = p1, c2 = p2, c3 = p3;
        const uint16_t sdb = psd;
        // rotary decode: the row of (cos, sin) pairs of this head vector's position; the 128-byte line
        // that holds this thread's pairs is asked into L1 now and read after the gather
        const float2 *cs = nullptr;
        if (ROPE != 0) {
            cs = ra.table + (size_t)min(max(ppos, 0), ra.positions - 1) * 64;
            // (pairs per slice: CH / 2 with both halves in the thread, CH otherwise)
            const float2 *mine = ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED ? cs + 2 * CH * slice
                                 : ROPE == 2 && LAYOUT == RVQ_GROUP_CONTIGUOUS ? cs + g * 16 + slice * (CH / 2)
                                 : ROPE == 1 ? cs + (g & 1u) * 32 + slice * CH : cs + 2 * CH * slice;
            asm volatile("prefetch.global.L1 [%0];" ::"l"(mine));
        }
        fetch(row + parts * kDecThreads, p0, p1, p2, p3, psd, ppos);
        if (BITS != 16) {
            // shift the window down to bit 0 and cut the codes out of it at offsets known at compile time
            const uint32_t sh = (g * (8u * BITS)) & 31u;
            const uint32_t u0 = __funnelshift_r(c0, c1, sh), u1 = __funnelshift_r(c1, c2, sh);
            const uint32_t u2 = __funnelshift_r(c2, c3, sh);
            uint32_t cw[4] = {0u, 0u, 0u, 0u};
            cut_codes<BITS, true>(u0, u1, u2, 8, cw);
            c0 = cw[0]; c1 = cw[1]; c2 = cw[2]; c3 = cw[3];
        }
        const uint32_t n0 = c0, n1 = c1, n2 = c2, n3 = c3;          // natural order, for the exact route
        // rotate the 8 halves left by `rot` so that step k finds its code at a fixed place
        if (rot & 4u) { const uint32_t t0 = c0, t1 = c1; c0 = c2; c1 = c3; c2 = t0; c3 = t1; }
        if (rot & 2u) { const uint32_t t0 = c0; c0 = c1; c1 = c2; c2 = c3; c3 = t0; }
        if (rot & 1u) {
            const uint32_t b0 = __funnelshift_r(c0, c1, 16), b1 = __funnelshift_r(c1, c2, 16);
            const uint32_t b2 = __funnelshift_r(c2, c3, 16), b3 = __funnelshift_r(c3, c0, 16);
            c0 = b0; c1 = b1; c2 = b2; c3 = b3;
        }
        // codes out of range (never produced by the encoder): counted, read as code 0
        {
            const uint32_t m = __vmaxu2(__vmaxu2(c0, c1), __vmaxu2(c2, c3));
            if (max(m & 0xFFFFu, m >> 16) >= Ku) {
                uint32_t *cc[4] = {&c0, &c1, &c2, &c3};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t lo = *cc[c] & 0xFFFFu, hi = *cc[c] >> 16;
                    if (lo >= Ku) { lo = 0; ++bad; }
                    if (hi >= Ku) { hi = 0; ++bad; }
                    *cc[c] = lo | (hi << 16);
                }
            }
        }
        const float sd = __half2float(__ushort_as_half(sdb));      // (0 beyond the last row)
        // integer sums of level * scale: one 16-bit x 8-bit dot-product instruction per channel and stage,
        // or (summed levels) plain additions of the table words and two such instructions per channel
        uint32_t acc[CH], even[CH / 2], odd[CH / 2];
        float facc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int i = 0; i < CH; ++i) acc[i] = 0u;
#pragma unroll
        for (int i = 0; i < CH / 2; ++i) { even[i] = 0u; odd[i] = 0u; }
        const uint32_t cwk[4] = {c0, c1, c2, c3};
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            // byte offset of the table line of this step's code: (code << kShift) | unit
            const uint32_t w = cwk[k >> 1];
            const uint32_t line = (k & 1) ? ((w >> (16 - kShift)) & (0xFFFFu << kShift)) : ((w << kShift) & (0xFFFFu << kShift));
            const uint32_t a = smem_table + (line | unit[k]);
            uint32_t e[CH / 2];
            if (F32) {
                float f0, f1, f2, f3;
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(f0), "=f"(f1), "=f"(f2), "=f"(f3) : "r"(a));
                facc[0] += f0; facc[1] += f1; facc[2] += f2; facc[3] += f3;
                continue;
            }
            if (CH == 8)
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(e[0]), "=r"(e[1]), "=r"(e[CH / 2 - 2]), "=r"(e[CH / 2 - 1]) : "r"(a));
            else
                asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(e[0]), "=r"(e[1]) : "r"(a));
#pragma unroll
            for (int i = 0; i < CH / 2; ++i) {
                if (SUMMED) {
                    if (k & 1) odd[i] += e[i]; else even[i] += e[i];
                } else {
                    asm("dp2a.lo.u32.u32 %0, %1, %2, %0;" : "+r"(acc[2 * i]) : "r"(e[i]), "r"(scale[k]));
                    asm("dp2a.hi.u32.u32 %0, %1, %2, %0;" : "+r"(acc[2 * i + 1]) : "r"(e[i]), "r"(scale[k]));
                }
            }
        }
        if (SUMMED) {
#pragma unroll
            for (int i = 0; i < CH / 2; ++i) {
                asm("dp2a.lo.u32.u32 %0, %1, %2, %0;" : "+r"(acc[2 * i]) : "r"(even[i]), "r"(scale[0]));
                asm("dp2a.lo.u32.u32 %0, %1, %2, %0;" : "+r"(acc[2 * i]) : "r"(odd[i]), "r"(scale[1]));
                asm("dp2a.hi.u32.u32 %0, %1, %2, %0;" : "+r"(acc[2 * i + 1]) : "r"(even[i]), "r"(scale[0]));
                asm("dp2a.hi.u32.u32 %0, %1, %2, %0;" : "+r"(acc[2 * i + 1]) : "r"(odd[i]), "r"(scale[1]));
            }
        }
        float o8[CH];
        {
            const float bs = base * sd, cs = bias * sd;
#pragma unroll
            for (int i = 0; i < CH; ++i) o8[i] = F32 ? facc[i & 3] * sd : fmaf((float)acc[i], bs, cs);
        }
        if (!F32 && fabsf(sd) > exact_above && fabsf(sd) < INFINITY) {
            // too coarse for this deviation: the float32 codewords themselves, summed in stage order
            float ex[CH];
#pragma unroll
            for (int i = 0; i < CH; ++i) ex[i] = 0.0f;
            const uint32_t cn[4] = {n0, n1, n2, n3};
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                uint32_t j = (r & 1) ? (cn[r >> 1] >> 16) : (cn[r >> 1] & 0xFFFFu);
                if (j >= Ku) j = 0;
                const float4 *e = reinterpret_cast<const float4 *>(cb + ((size_t)r * s.K + j) * 32 + (SPLIT ? slice * 4 : slice * CH));
#pragma unroll
                for (int q = 0; q < CH / 4; ++q) {
                    const float4 t = __ldg(e + (SPLIT ? 4 * q : q));
                    ex[4 * q] += t.x; ex[4 * q + 1] += t.y; ex[4 * q + 2] += t.z; ex[4 * q + 3] += t.w;
                }
            }
#pragma unroll
            for (int i = 0; i < CH; ++i) o8[i] = ex[i] * sd;
        }
        if (ROPE != 0 && F32) {
            // four channels per thread: the same four cases as below at half the width
            if (ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED) {
                // places (0, 2) and (1, 3): channels 4 (2 slice + i) + g = pair index, and 64 further on
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float2 c = __ldg(cs + (2 * slice + i) * 4 + g);
                    const float a = o8[i], b = o8[i + 2];
                    o8[i] = a * c.x - b * c.y;
                    o8[i + 2] = b * c.x + a * c.y;
                }
            } else if (ROPE == 2 && LAYOUT == RVQ_GROUP_CONTIGUOUS) {
                // channels 32 g + 4 slice + i: pairs 16 g + 2 slice + i / 2
                const float4 c = __ldg(reinterpret_cast<const float4 *>(cs + g * 16 + slice * 2));
                const float a0 = o8[0], b0 = o8[1], a1 = o8[2], b1 = o8[3];
                o8[0] = a0 * c.x - b0 * c.y; o8[1] = b0 * c.x + a0 * c.y;
                o8[2] = a1 * c.z - b1 * c.w; o8[3] = b1 * c.z + a1 * c.w;
            } else if (ROPE == 1) {
                // contiguous groups: the partner is the same place of group g ^ 2; pairs 32 (g & 1) + 4 slice + i
                const float4 *q = reinterpret_cast<const float4 *>(cs + (g & 1u) * 32 + slice * 4);
                const bool first = (g & 2u) == 0;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float4 c = __ldg(q + h);
                    const float p0 = __shfl_xor_sync(0xFFFFFFFFu, o8[2 * h], 2);
                    const float p1 = __shfl_xor_sync(0xFFFFFFFFu, o8[2 * h + 1], 2);
                    o8[2 * h] = first ? o8[2 * h] * c.x - p0 * c.y : o8[2 * h] * c.x + p0 * c.y;
                    o8[2 * h + 1] = first ? o8[2 * h + 1] * c.z - p1 * c.w : o8[2 * h + 1] * c.z + p1 * c.w;
                }
            } else {
                // strided groups, pairs (2k, 2k + 1): channels 4 e + g and 4 e + (g ^ 1), e = 4 slice + i; pair 2 e + g / 2
                const bool first = (g & 1u) == 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 c = __ldg(cs + 2 * (4 * slice + i) + (g >> 1));
                    const float p = __shfl_xor_sync(0xFFFFFFFFu, o8[i], 1);
                    o8[i] = first ? o8[i] * c.x - p * c.y : o8[i] * c.x + p * c.y;
                }
            }
        } else if (ROPE != 0) {
            // (cos, sin) of the pairs of this thread's channels
            if (ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED) {
                // places 0..3 are channels 4 (4 slice + i) + g = pair index; places 4..7 their partners 64 on
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 c = __ldg(cs + (4 * slice + i) * 4 + g);
                    const float a = o8[i], b = o8[i + 4];
                    o8[i] = a * c.x - b * c.y;
                    o8[i + 4] = b * c.x + a * c.y;
                }
            } else if (ROPE == 2 && LAYOUT == RVQ_GROUP_CONTIGUOUS) {
                // channels 32 g + 8 slice + i: pairs 16 g + 4 slice + i / 2, both halves in this thread
                const float4 *q = reinterpret_cast<const float4 *>(cs + g * 16 + slice * 4);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float4 c = __ldg(q + h);
                    const float a0 = o8[4 * h], b0 = o8[4 * h + 1], a1 = o8[4 * h + 2], b1 = o8[4 * h + 3];
                    o8[4 * h] = a0 * c.x - b0 * c.y;     o8[4 * h + 1] = b0 * c.x + a0 * c.y;
                    o8[4 * h + 2] = a1 * c.z - b1 * c.w; o8[4 * h + 3] = b1 * c.z + a1 * c.w;
                }
            } else if (ROPE == 1) {
                // contiguous groups, pairs (k, k + 64): the partner is the same place of group g ^ 2;
                // pairs 32 (g & 1) + 8 slice + i
                const float4 *q = reinterpret_cast<const float4 *>(cs + (g & 1u) * 32 + slice * 8);
                const bool first = (g & 2u) == 0;
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float4 c = __ldg(q + h);
                    const float p0 = __shfl_xor_sync(0xFFFFFFFFu, o8[2 * h], 2);
                    const float p1 = __shfl_xor_sync(0xFFFFFFFFu, o8[2 * h + 1], 2);
                    o8[2 * h] = first ? o8[2 * h] * c.x - p0 * c.y : o8[2 * h] * c.x + p0 * c.y;
                    o8[2 * h + 1] = first ? o8[2 * h + 1] * c.z - p1 * c.w : o8[2 * h + 1] * c.z + p1 * c.w;
                }
            } else {
                // strided groups, pairs (2k, 2k + 1): channels 4 e + g and 4 e + (g ^ 1), e = 8 slice + i;
                // pair 2 e + g / 2
                const bool first = (g & 1u) == 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float2 c = __ldg(cs + 2 * (8 * slice + i) + (g >> 1));
                    const float p = __shfl_xor_sync(0xFFFFFFFFu, o8[i], 1);
                    o8[i] = first ? o8[i] * c.x - p * c.y : o8[i] * c.x + p * c.y;
                }
            }
        }
        uint32_t w[CH / 2];
#pragma unroll
        for (int c = 0; c < CH / 2; ++c) w[c] = Out<DT>::pack(o8[2 * c], o8[2 * c + 1]);
        uint16_t *o16 = reinterpret_cast<uint16_t *>(out) + (size_t)v * stride;
        if (SPLIT && F32) {
            // the thread's places are elements 2 slice, 2 slice + 1 and their partners 16 on: lane L stores
            // the four groups of place L
            const uint2 t = transpose_group_elements(w[0], w[1], g);
            if (live) *reinterpret_cast<uint2 *>(o16 + 4 * (2 * slice + (g & 1u) + 16 * (g >> 1))) = t;
        } else if (SPLIT) {
            // lane L stores element 4 slice + L of the four groups, and its partner 16 elements on
            const uint2 lo = transpose_group_elements(w[0], w[1], g);
            const uint2 hi = transpose_group_elements(w[CH / 2 - 2], w[CH / 2 - 1], g);
            if (live) {
                *reinterpret_cast<uint2 *>(o16 + 4 * (4 * slice + g)) = lo;
                *reinterpret_cast<uint2 *>(o16 + 4 * (16 + 4 * slice + g)) = hi;
            }
        } else if (LAYOUT == RVQ_GROUP_CONTIGUOUS) {
            if (live) {
                if (CH == 8)
                    *reinterpret_cast<uint4 *>(o16 + g * 32 + slice * 8) = make_uint4(w[0], w[1], w[CH / 2 - 2], w[CH / 2 - 1]);
                else
                    *reinterpret_cast<uint2 *>(o16 + g * 32 + slice * 4) = make_uint2(w[0], w[1]);
            }
        } else if (CH == 8) {
            // Lane g holds element pairs (2c, 2c+1) of group g, i.e. channels 32 slice + 8c + g and + 4.
            // Lane c' of the 4-lane set wants pairs c' of all four groups: a 4x4 transpose of words in
            // two butterfly steps (odd/even words with lane g^1, then word pairs with lane g^2).
            uint32_t &w0 = w[0], &w1 = w[1], &w2 = w[CH / 2 - 2], &w3 = w[CH / 2 - 1];
            const bool b1 = g & 1u, b2 = g & 2u;
            const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, b1 ? w0 : w1, 1);
            const uint32_t r1 = __shfl_xor_sync(0xFFFFFFFFu, b1 ? w2 : w3, 1);
            if (b1) { w0 = r0; w2 = r1; } else { w1 = r0; w3 = r1; }
            const uint32_t r2 = __shfl_xor_sync(0xFFFFFFFFu, b2 ? w0 : w2, 2);
            const uint32_t r3 = __shfl_xor_sync(0xFFFFFFFFu, b2 ? w1 : w3, 2);
            if (b2) { w0 = r2; w1 = r3; } else { w2 = r2; w3 = r3; }
            // now w[q] = pair g of group q; channels 32 slice + 8 g + 0..7: element 2g of groups 0..3, then 2g+1
            const uint32_t o0 = __byte_perm(w0, w1, 0x5410), o1 = __byte_perm(w2, w3, 0x5410);
            const uint32_t o2 = __byte_perm(w0, w1, 0x7632), o3 = __byte_perm(w2, w3, 0x7632);
            if (live) *reinterpret_cast<uint4 *>(o16 + slice * 32 + g * 8) = make_uint4(o0, o1, o2, o3);
        } else {
            // Lane g holds elements 4 slice + 0..3 of group g as w[0] = (e0, e1), w[1] = (e2, e3); the 16
            // channels 16 slice .. 16 slice + 15 are element-major, so lane L stores element L of the four
            // groups.  Exchange words with lane g^2, then halves with lane g^1.
            const bool b1 = g & 1u, b2 = g & 2u;
            const uint32_t r0 = __shfl_xor_sync(0xFFFFFFFFu, b2 ? w[0] : w[1], 2);
            const uint32_t lo_g = b2 ? r0 : w[0], hi_g = b2 ? w[1] : r0;
            const uint32_t keep = __byte_perm(lo_g, hi_g, b1 ? 0x7632 : 0x5410);
            const uint32_t send = __byte_perm(lo_g, hi_g, b1 ? 0x5410 : 0x7632);
            const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, send, 1);
            const uint32_t even = b1 ? got : keep, odd = b1 ? keep : got;
            if (live)
                *reinterpret_cast<uint2 *>(o16 + 4 * (slice * 4 + g)) =
                    make_uint2(__byte_perm(even, odd, 0x5410), __byte_perm(even, odd, 0x7632));
        }
    }
    if (bad && st && slice == 0) atomicAdd(&st->bad_codes, bad);   // every slice sees the same codes
}

// True when more than one in 64 of a sample of up to 256 deviations is beyond the level tables' reach
// (such a row takes the exact route and holds its whole warp up).
// Uniform over the CTA (and over all CTAs of a launch: they read the same sample).
__device__ __forceinline__ bool sample_wants_float32(const uint16_t *__restrict__ std16, int64_t n,
                                                  const uint8_t *__restrict__ dsec, float reach)
{
    const DecodeParams *dp = reinterpret_cast<const DecodeParams *>(dsec);
    const float exact_above = dp->err > 0.0f ? reach / dp->err : INFINITY;
    const int64_t samples = n < 256 ? n : 256, every = n < 256 ? 1 : n >> 8;
    const bool beyond = threadIdx.x < samples &&
                        fabsf(__half2float(__ushort_as_half(std16[threadIdx.x * every]))) > exact_above;
    const int far = __syncthreads_count(beyond);
    return (int64_t)far * 64 > samples;
}

// PICK: with up to 1536 codes per stage and 16-bit outputs both kinds of table fit, and which one
// is faster depends on the deviations: level tables (8-channel slices) while most rows are within
// their reach, float32 tables (4-channel slices) when many rows would take the exact route.  Both
// kernels are launched; every CTA of both looks at the same sample of up to 256 deviations, so they
// agree, and the kernel that is not wanted (PICK 1: levels, PICK 2: float32) returns at once.
template <int DT, int CH, bool F32T, int PICK>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_sliced_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t n,
                     const uint8_t *__restrict__ dsec, const float *__restrict__ cb, void *__restrict__ out,
                     int64_t stride, rvq_status *st)
{
    extern __shared__ __align__(128) uint8_t table[];
    if (PICK != 0 && sample_wants_float32(std16, n, dsec, 0.9e-3f) != (PICK == 2)) return;
    decode_sliced_body<DT, CH, F32T>(s, codes, std16, n, dsec, cb, out, stride, st, table);
}

// 0: summed-level tables, 1: per-stage scaled levels, 2: float32 tables -- the first kind within whose reach
// all but one in 64 of a sample of up to 256 deviations lie.  Uniform over all CTAs of a launch.
__device__ __forceinline__ int sample_table_kind(const uint16_t *__restrict__ std16, int64_t n, const uint8_t *__restrict__ dsec,
                                                 float reach = 0.9e-3f)
{
    const DecodeParams *dp = reinterpret_cast<const DecodeParams *>(dsec);
    const float above_l = dp->err > 0.0f ? reach / dp->err : INFINITY;
    const float above_s = dp->perr > 0.0f ? reach / dp->perr : INFINITY;
    const int64_t samples = n < 256 ? n : 256, every = n < 256 ? 1 : n >> 8;
    const float sd = threadIdx.x < samples ? fabsf(__half2float(__ushort_as_half(std16[threadIdx.x * every]))) : 0.0f;
    const int far_s = __syncthreads_count(sd > above_s);
    const int far_l = __syncthreads_count(sd > above_l);
    // (a row beyond a table's reach takes the exact route, and its whole warp of eight head vectors waits
    // for it: a table is taken only while at most one sampled row in 64 is beyond it)
    if ((int64_t)far_s * 64 <= samples) return 0;
    return (int64_t)far_l * 64 <= samples ? 1 : 2;
}

// One launch for the quoted shapes (dim 128, depth 8, 16-bit outputs, up to 3072 codes): every CTA
// reads the same sample of deviations and takes the level tables (fast body) or, when the deviations
// are beyond their reach, the float32 tables; both carve their slices out of whatever grid they get.
template <int DT, int LCH, int FCH, int LAYOUT, int BITS>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_quoted_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t n,
                     const uint8_t *__restrict__ dsec, const float *__restrict__ cb, void *__restrict__ out,
                     int64_t stride, rvq_status *st)
{
    extern __shared__ __align__(128) uint8_t table[];
    const int kind = sample_table_kind(std16, n, dsec);
    if (kind == 2 && FCH == 4)
        decode_levels_fast<DT, 4, LAYOUT, BITS, false, 0, true>(s, codes, std16, n, dsec, cb, out, stride, st, table);
    else if (kind == 2)
        decode_sliced_body<DT, FCH, true>(s, codes, std16, n, dsec, cb, out, stride, st, table);
    else if (kind == 1)
        decode_levels_fast<DT, LCH, LAYOUT, BITS, false>(s, codes, std16, n, dsec, cb, out, stride, st, table);
    else
        decode_levels_fast<DT, LCH, LAYOUT, BITS, true>(s, codes, std16, n, dsec, cb, out, stride, st, table);
}

// The rotary decode of the quoted shapes (dim 128, depth 8, 16-bit outputs, up to 1536 codes, a prepared
// block): one launch that takes the level tables with 8-channel slices while the deviations allow it (a
// rotation adds two table errors, so their reach is 0.6e-3) and the float32 tables otherwise.
template <int DT, int LAYOUT, int BITS, int ROPE>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_rope_quoted_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t n,
                          const uint8_t *__restrict__ dsec, const float *__restrict__ cb, void *__restrict__ out,
                          int64_t stride, rvq_status *st, RopeArgs ra)
{
    extern __shared__ __align__(128) uint8_t table[];
    const int kind = sample_table_kind(std16, n, dsec, 0.6e-3f);
    if (kind == 2)
        decode_levels_fast<DT, 4, LAYOUT, BITS, false, ROPE, true>(s, codes, std16, n, dsec, cb, out, stride, st, table, ra);
    else if (kind == 1)
        decode_levels_fast<DT, 8, LAYOUT, BITS, false, ROPE>(s, codes, std16, n, dsec, cb, out, stride, st, table, ra);
    else
        decode_levels_fast<DT, 8, LAYOUT, BITS, true, ROPE>(s, codes, std16, n, dsec, cb, out, stride, st, table, ra);
}

// Decode with the rotary embedding, 4-channel slices (dim 128): float32 tables up to 1792 codes per stage,
// 16-bit level tables (16-bit outputs) up to 3072.
template <int DT, int ROPE, int CH, bool F32T, int PICK>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_rope_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t n,
                   const uint8_t *__restrict__ dsec, const float *__restrict__ cb, void *__restrict__ out,
                   int64_t stride, rvq_status *st, RopeArgs ra)
{
    extern __shared__ __align__(128) uint8_t table[];
    if (PICK != 0 && sample_wants_float32(std16, n, dsec, 0.6e-3f) != (PICK == 2)) return;
    decode_sliced_body<DT, CH, F32T, ROPE>(s, codes, std16, n, dsec, cb, out, stride, st, table, ra);
}

// Any other shape: a block decodes a few head vectors into shared memory (one thread per group row and
// four-element piece: float4 gathers of the float32 codebooks, float32 sums in stage order), then one thread
// per pair of channels rotates and stores.
__global__ void __launch_bounds__(256)
decode_rope_gather_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t n,
                          const float *__restrict__ cb, void *__restrict__ out, int64_t stride, rvq_status *st,
                          RopeArgs ra, int style, int vpb)
{
    extern __shared__ __align__(16) float xs[];                   // [vpb][dim]
    const int pieces = s.gd / 4, per_vec = s.G * pieces, half = s.dim / 2;
    for (int64_t v0 = (int64_t)blockIdx.x * vpb; v0 < n; v0 += (int64_t)gridDim.x * vpb) {
        for (int t = threadIdx.x; t < vpb * per_vec; t += 256) {
            const int vl = t / per_vec, rem = t - vl * per_vec, g = rem / pieces, q = rem - g * pieces;
            const int64_t v = v0 + vl;
            if (v >= n) continue;
            const uint8_t *vec = reinterpret_cast<const uint8_t *>(codes) + v * s.code_bytes;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int r = 0; r < s.R; ++r) {
                uint32_t j = read_code(vec, g * s.R + r, s.bits, s.code_bytes);
                if (j >= (uint32_t)s.K) { j = 0; if (st && q == 0) atomicAdd(&st->bad_codes, 1u); }
                const float4 e = __ldg(reinterpret_cast<const float4 *>(cb + ((size_t)r * s.K + j) * s.gd) + q);
                acc.x += e.x; acc.y += e.y; acc.z += e.z; acc.w += e.w;
            }
            const float sd = __half2float(__ushort_as_half(std16[v]));
            const float o[4] = {sd * acc.x, sd * acc.y, sd * acc.z, sd * acc.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) xs[vl * s.dim + channel_of(s.layout, s.G, s.gd, g, 4 * q + k)] = o[k];
        }
        __syncthreads();
        for (int t = threadIdx.x; t < vpb * half; t += 256) {
            const int vl = t / half, f = t - vl * half;
            const int64_t v = v0 + vl;
            if (v >= n) continue;
            const int c0 = style == 1 ? f : 2 * f, c1 = style == 1 ? f + half : 2 * f + 1;
            int pos = ra.position[v / ra.per_position];
            pos = min(max(pos, 0), ra.positions - 1);
            const float2 cs = __ldg(ra.table + (size_t)pos * half + f);
            const float a = xs[vl * s.dim + c0], b = xs[vl * s.dim + c1];
            store_from_float(out, v * stride + c0, s.dtype, a * cs.x - b * cs.y);
            store_from_float(out, v * stride + c1, s.dtype, b * cs.x + a * cs.y);
        }
        __syncthreads();
    }
}

// (cos, sin) of position * base^(-2k/dim), computed in double precision: the angles reach 1e5 radians.
__global__ void __launch_bounds__(256)
rope_table_kernel(int dim, double base, int positions, float2 *__restrict__ table)
{
    const int half = dim / 2;
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t >= (int64_t)positions * half) return;
    const int p = (int)(t / half), k = (int)(t - (int64_t)p * half);
    const double ang = (double)p * pow(base, -2.0 * (double)k / (double)dim);
    table[t] = make_float2((float)cos(ang), (float)sin(ang));
}

}  // namespace

int launch_rope_table(int dim, double base, int positions, float *table, cudaStream_t stream)
{
    const int64_t total = (int64_t)positions * (dim / 2);
    if (total == 0) return RVQ_OK;
    rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(dim, base, positions,
                                                                             reinterpret_cast<float2 *>(table));
    return check_launch();
}

int launch_decode_rope(const Shape &s, const void *codes, const uint16_t *std16, int64_t n, const float *cb,
                       const void *prepared, const int32_t *position, int per_position, const float *table,
                       int positions, int style, void *out, int64_t stride, rvq_status *st, cudaStream_t stream)
{
    if (n == 0) return RVQ_OK;
    int shift = -1;
    for (int b = 0; b < 31; ++b)
        if (per_position == (1 << b)) shift = b;
    RopeArgs ra{position, per_position, reinterpret_cast<const float2 *>(table), positions, shift};
    const bool f32t = decode_exact_tables(s) && s.G >= 2;         // (one group: the pairs are inside a row; gather kernel)
    const bool levels = prepared != nullptr && decode_levels_supported(s) && decode_slice_channels(s.K) == 4;
    if (!f32t || n > 0x7FFFFFFF) {
        const int per_vec = s.G * (s.gd / 4);
        int vpb = 256 / per_vec;
        if (vpb < 1) vpb = 1;
        int64_t blocks = (n + vpb - 1) / vpb;
        int dev_g = 0, sms_g = 0;
        if (cudaGetDevice(&dev_g) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms_g, cudaDevAttrMultiProcessorCount, dev_g) != cudaSuccess)
            return RVQ_ERR_DEVICE;
        if (blocks > (int64_t)sms_g * 16) blocks = (int64_t)sms_g * 16;
        const size_t smem = (size_t)vpb * s.dim * sizeof(float);
        decode_rope_gather_kernel<<<(unsigned)blocks, 256, smem, stream>>>(s, codes, std16, n, cb, out, stride, st, ra,
                                                                           style == 0 ? 1 : 2, vpb);
        return check_launch();
    }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return RVQ_ERR_DEVICE;
    const uint8_t *dsec = nullptr;
    if (levels)
        dsec = reinterpret_cast<const uint8_t *>(prepared) + (kPreparedImageOffset + encode_image_bytes(s) + 255) / 256 * 256;
    const int64_t tiles = (n * s.G + kDecThreads - 1) / kDecThreads;
    // the quoted shapes with a prepared block: one launch, tables chosen on the device
    if (prepared != nullptr && decode_levels_supported(s) && s.dim == 128 && s.G == 4 && s.R == 8 && s.K <= kDecodeWideK &&
        n * 4 < 0x7FFFFFFFLL && (s.bits == 16 || s.bits == 10 || s.bits == 11)) {
        const uint8_t *d = reinterpret_cast<const uint8_t *>(prepared) +
                           (kPreparedImageOffset + encode_image_bytes(s) + 255) / 256 * 256;
        auto quoted = [&](auto kernel) -> int {
            const size_t smem = (size_t)s.K * 128;               // 8 channels of levels or 4 of float32 per code
            const int grid = sms < 8 ? 8 : sms;
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
                return RVQ_ERR_LAUNCH;
            kernel<<<grid, kDecThreads, smem, stream>>>(s, codes, std16, n, d, cb, out, stride, st, ra);
            return check_launch();
        };
#define RVQ_RQ3(DT, LAY, ROPE)                                                                                       \
        (s.bits == 16 ? quoted(decode_rope_quoted_kernel<DT, LAY, 16, ROPE>)                                         \
         : s.bits == 10 ? quoted(decode_rope_quoted_kernel<DT, LAY, 10, ROPE>)                                       \
                        : quoted(decode_rope_quoted_kernel<DT, LAY, 11, ROPE>))
#define RVQ_RQ2(DT, LAY) (style == 0 ? RVQ_RQ3(DT, LAY, 1) : RVQ_RQ3(DT, LAY, 2))
#define RVQ_RQ1(DT) (s.layout == RVQ_GROUP_CONTIGUOUS ? RVQ_RQ2(DT, RVQ_GROUP_CONTIGUOUS) : RVQ_RQ2(DT, RVQ_GROUP_STRIDED))
        return s.dtype == RVQ_BF16 ? RVQ_RQ1(RVQ_BF16) : RVQ_RQ1(RVQ_F16);
#undef RVQ_RQ1
#undef RVQ_RQ2
#undef RVQ_RQ3
    }
    auto launch = [&](auto kernel, int ch, bool f32_tables) -> int {
        const int ns = 32 / ch;
        const size_t smem = (size_t)s.K * (f32_tables ? 32 : 16) * ch;
        int parts = sms / ns;
        if (parts > tiles) parts = (int)tiles;
        if (parts < 1) parts = 1;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return RVQ_ERR_LAUNCH;
        kernel<<<parts * ns, kDecThreads, smem, stream>>>(s, codes, std16, n, dsec, cb, out, stride, st, ra);
        return check_launch();
    };
    // style 0/1 -> ROPE 1/2; float32 tables with 4-channel slices up to 1792 codes, 2-channel ones beyond; where
    // level tables exist as well, both kernels are launched and the deviations decide on the device (PICK)
    const bool wide = decode_exact_channels(s.K) == 4;
#define RVQ_ROPE_F32(DT, PICK)                                                                                      \
    (style == 0 ? (wide ? launch(decode_rope_kernel<DT, 1, 4, true, PICK>, 4, true)                                \
                        : launch(decode_rope_kernel<DT, 1, 2, true, PICK>, 2, true))                               \
                : (wide ? launch(decode_rope_kernel<DT, 2, 4, true, PICK>, 4, true)                                \
                        : launch(decode_rope_kernel<DT, 2, 2, true, PICK>, 2, true)))
#define RVQ_ROPE_LEVELS(DT)                                                                                         \
    (style == 0 ? launch(decode_rope_kernel<DT, 1, 4, false, 1>, 4, false)                                         \
                : launch(decode_rope_kernel<DT, 2, 4, false, 1>, 4, false))
    int rc;
    if (levels) {
        if (s.dtype == RVQ_BF16) {
            if ((rc = RVQ_ROPE_LEVELS(RVQ_BF16)) != RVQ_OK) return rc;
            return RVQ_ROPE_F32(RVQ_BF16, 2);
        }
        if ((rc = RVQ_ROPE_LEVELS(RVQ_F16)) != RVQ_OK) return rc;
        return RVQ_ROPE_F32(RVQ_F16, 2);
    }
    switch (s.dtype) {
    case RVQ_F32: return RVQ_ROPE_F32(RVQ_F32, 0);
    case RVQ_BF16: return RVQ_ROPE_F32(RVQ_BF16, 0);
    default: return RVQ_ROPE_F32(RVQ_F16, 0);
    }
#undef RVQ_ROPE_F32
#undef RVQ_ROPE_LEVELS
}

int launch_decode_sliced(const Shape &s, const void *codes, const uint16_t *std16, int64_t n,
                         const float *cb, const void *prepared, void *out, int64_t stride, rvq_status *st,
                         cudaStream_t stream)
{
    if (n == 0) return RVQ_OK;
    const uint8_t *p = reinterpret_cast<const uint8_t *>(prepared);
    const size_t off = (kPreparedImageOffset + encode_image_bytes(s) + 255) / 256 * 256;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return RVQ_ERR_DEVICE;
    // which tables: see prepared.cuh
    const bool both = decode_levels_supported(s);                  // then the deviations decide on the device
    const int lch = decode_slice_channels(s.K), fch = decode_exact_channels(s.K);
    const int64_t tiles = (n * s.G + kDecThreads - 1) / kDecThreads;
    auto launch = [&](auto kernel, int ch, bool f32t) -> int {
        const int ns = 32 / ch;
        const size_t smem = (size_t)s.K * (f32t ? 32 : 16) * ch;
        int parts = sms / ns;
        if (parts > tiles) parts = (int)tiles;
        if (parts < 1) parts = 1;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return RVQ_ERR_LAUNCH;
        kernel<<<parts * ns, kDecThreads, smem, stream>>>(s, codes, std16, n, p + off, cb, out, stride, st);
        return check_launch();
    };
    // the quoted shapes: one launch, tables chosen on the device
    if (both && s.G == 4 && s.R == 8 && n * 4 < 0x7FFFFFFFLL && (s.bits == 16 || (s.bits >= 10 && s.bits <= 12)) &&
        !(lch == 4 && fch == 4)) {
        auto quoted = [&](auto kernel) -> int {
            const size_t smem = (size_t)s.K * 16 * lch > (size_t)s.K * 32 * fch ? (size_t)s.K * 16 * lch : (size_t)s.K * 32 * fch;
            int grid = sms < 8 ? 8 : sms;
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
                return RVQ_ERR_LAUNCH;
            kernel<<<grid, kDecThreads, smem, stream>>>(s, codes, std16, n, p + off, cb, out, stride, st);
            return check_launch();
        };
#define RVQ_Q4(DT, LCH, FCH, LAY)                                                                                   \
        (s.bits == 16 ? quoted(decode_quoted_kernel<DT, LCH, FCH, LAY, 16>)                                          \
         : s.bits == 10 ? quoted(decode_quoted_kernel<DT, LCH, FCH, LAY, 10>)                                        \
         : s.bits == 11 ? quoted(decode_quoted_kernel<DT, LCH, FCH, LAY, 11>)                                        \
                        : quoted(decode_quoted_kernel<DT, LCH, FCH, LAY, 12>))
#define RVQ_Q3(DT, LAY) (lch == 8 ? RVQ_Q4(DT, 8, 4, LAY) : RVQ_Q4(DT, 4, 2, LAY))
#define RVQ_Q2(DT) (s.layout == RVQ_GROUP_CONTIGUOUS ? RVQ_Q3(DT, RVQ_GROUP_CONTIGUOUS) : RVQ_Q3(DT, RVQ_GROUP_STRIDED))
        return s.dtype == RVQ_BF16 ? RVQ_Q2(RVQ_BF16) : RVQ_Q2(RVQ_F16);
#undef RVQ_Q2
#undef RVQ_Q3
#undef RVQ_Q4
    }
#define RVQ_DEC_F32(DT, PICK)                                                                                       \
    (fch == 4 ? launch(decode_sliced_kernel<DT, 4, true, PICK>, 4, true)                                           \
              : launch(decode_sliced_kernel<DT, 2, true, PICK>, 2, true))
#define RVQ_DEC_LEVELS(DT)                                                                                          \
    (lch == 8 ? launch(decode_sliced_kernel<DT, 8, false, 1>, 8, false)                                            \
              : launch(decode_sliced_kernel<DT, 4, false, 1>, 4, false))
    int rc;
    if (both) {
        if (s.dtype == RVQ_BF16) {
            if ((rc = RVQ_DEC_LEVELS(RVQ_BF16)) != RVQ_OK) return rc;
            return RVQ_DEC_F32(RVQ_BF16, 2);
        }
        if ((rc = RVQ_DEC_LEVELS(RVQ_F16)) != RVQ_OK) return rc;
        return RVQ_DEC_F32(RVQ_F16, 2);
    }
    switch (s.dtype) {
    case RVQ_F32: return RVQ_DEC_F32(RVQ_F32, 0);
    case RVQ_BF16: return RVQ_DEC_F32(RVQ_BF16, 0);
    default: return RVQ_DEC_F32(RVQ_F16, 0);
    }
#undef RVQ_DEC_F32
#undef RVQ_DEC_LEVELS
}

}  // namespace rvq
