// Prepared-codebook block: what the kernels read instead of the float32
// codebooks.  Written by rvq_prepare_codebooks, read-only afterwards.
//
// Encode section (group_dim 32 only).  Algorithm 1's argmin over
// ||z - e||^2 is taken over the scores ||e||^2 - 2 z.e, which are one dense
// contraction per stage.  Half-precision operands alone are too coarse when a
// few channels carry most of a vector's energy (the rounding error of the
// product then rivals the gap between the best codewords), so both operands
// are split into a half-precision head and a half-precision remainder and the
// contraction keeps the three leading products:
//     z.e  ~  z_hi.e_hi + z_hi.e_lo + z_lo.e_hi        (error ~ 2^-22 |z||e|).
// Per stage r the block holds
//   - a power-of-two scale 2^k chosen so that the largest scaled squared norm
//     is about 2^13 (keeps the operands out of the half-precision subnormals);
//   - the B operand image of tcgen05.mma: for every slot of 128 codewords ten
//     "cells" (8 halves = 16 bytes per codeword per cell, K-major, no swizzle):
//     cells 0-3 hold -2 e_hi, cells 4-7 hold -2 e_lo, cell 8 holds the scaled
//     squared norm split into three halves (hi, lo, lo2) then zeros, cell 9 is
//     zero.  The A operand carries (Z_hi, Z_lo, 1 1 1 0...), and seven K=16
//     steps pair the cells so that the accumulator is the score;
//   - two numbers (a, b) such that |score error| <= a * ||Z|| + b, from the
//     actual rounding errors of this codebook (see prepare_finish_kernel).
#include "prepared.cuh"

namespace rvq {

static size_t decode_section_offset(const Shape &s)
{
    return (kPreparedImageOffset + encode_image_bytes(s) + 255) / 256 * 256;
}

size_t prepared_bytes(const Shape &s)
{
    size_t b = decode_section_offset(s);
    if (decode_levels_prepared(s)) b += 256 + 2 * decode_table_bytes(s.K);
    return (b + 255) / 256 * 256;
}

// One thread per (channel octet, code, stage): 8 channels of levels, stored as one 16-byte
// entry of a wide slice or as the 8-byte entries of two narrow slices.
__global__ void __launch_bounds__(256)
decode_table_kernel(Shape s, const float *__restrict__ cb, const DecodeParams *__restrict__ dp,
                    const float *__restrict__ lo, uint4 *__restrict__ table)
{
    const int t = blockIdx.x * 256 + threadIdx.x, octet = blockIdx.y;
    const int j = t >> 3, r = t & 7;
    if (j >= s.K) return;
    const bool wide = decode_slice_channels(s.K) == 8;
    const bool used = r < s.R && dp->step[r] > 0.0f;
    float v[8];
    if (used) {
        const float4 *src = reinterpret_cast<const float4 *>(cb + ((size_t)r * s.K + j) * 32 + octet * 8);
        const float4 a = __ldg(src), b = __ldg(src + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
    uint32_t w[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t pair = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t level = 0;
            if (used) {
                const float q = rintf((v[2 * c + h] - lo[r]) / dp->step[r]);
                level = (uint32_t)fminf(fmaxf(q, 0.0f), 65535.0f);
            }
            pair |= level << (16 * h);
        }
        w[c] = pair;
    }
    // the same entry in units of its stage parity (summed levels)
    uint32_t pw[4];
    const float pst = r < 8 ? dp->pstep[r & 1] : 0.0f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t pair = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t level = 0;
            if (used && pst > 0.0f) {
                const float q = rintf((v[2 * c + h] - lo[r]) / pst);
                level = (uint32_t)fminf(fmaxf(q, 0.0f), 65535.0f);
            }
            pair |= level << (16 * h);
        }
        pw[c] = pair;
    }
    uint4 *ptable = table + decode_table_bytes(s.K) / sizeof(uint4);
    if (wide) {
        table[((size_t)octet * s.K + j) * 8 + r] = make_uint4(w[0], w[1], w[2], w[3]);
        ptable[((size_t)octet * s.K + j) * 8 + r] = make_uint4(pw[0], pw[1], pw[2], pw[3]);
    } else {
        uint2 *t2 = reinterpret_cast<uint2 *>(table), *p2 = reinterpret_cast<uint2 *>(ptable);
        t2[((size_t)(2 * octet) * s.K + j) * 8 + r] = make_uint2(w[0], w[1]);
        t2[((size_t)(2 * octet + 1) * s.K + j) * 8 + r] = make_uint2(w[2], w[3]);
        p2[((size_t)(2 * octet) * s.K + j) * 8 + r] = make_uint2(pw[0], pw[1]);
        p2[((size_t)(2 * octet + 1) * s.K + j) * 8 + r] = make_uint2(pw[2], pw[3]);
    }
}


// grid (kPrepareParts, R): largest squared norm and entry range of a share of one stage's codewords.
__global__ void __launch_bounds__(256)
prepare_reduce_kernel(Shape s, const float *__restrict__ cb, StagePartial *part)
{
    __shared__ double rn[256];
    __shared__ float rlo[256], rhi[256];
    const int r = blockIdx.y, tid = threadIdx.x;
    const int per = (s.K + kPrepareParts - 1) / kPrepareParts;
    const int j0 = blockIdx.x * per, j1 = min(s.K, j0 + per);
    double m = 0.0;
    float lo = INFINITY, hi = -INFINITY;
    for (int j = j0 + tid; j < j1; j += 256) {
        const float *e = cb + ((size_t)r * s.K + j) * s.gd;
        double acc = 0.0;
        for (int i = 0; i < s.gd; ++i) {
            const float v = e[i];
            acc += (double)v * (double)v;
            lo = fminf(lo, v); hi = fmaxf(hi, v);
        }
        m = fmax(m, acc);
    }
    rn[tid] = m; rlo[tid] = lo; rhi[tid] = hi;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (tid < w) {
            rn[tid] = fmax(rn[tid], rn[tid + w]);
            rlo[tid] = fminf(rlo[tid], rlo[tid + w]); rhi[tid] = fmaxf(rhi[tid], rhi[tid + w]);
        }
        __syncthreads();
    }
    if (tid == 0) {
        StagePartial &o = part[r * kPrepareParts + blockIdx.x];
        o.max_norm2 = rn[0]; o.lo = rlo[0]; o.hi = rhi[0];
    }
}

// One block, thread r per stage: scale exponent from the largest squared norm, the decoder's
// affine map from the entry range; clears the maxima the image kernel accumulates into.
__global__ void __launch_bounds__(32)
prepare_params_kernel(Shape s, const StagePartial *__restrict__ part, PreparedHeader *hdr, StageParams *sp,
                      StageMaxima *mx, DecodeParams *dp, float *dec_lo)
{
    __shared__ float s_lo[8], s_step[8];
    const int r = threadIdx.x;
    if (r < 8) { s_lo[r] = 0.0f; s_step[r] = 0.0f; }
    __syncwarp();
    if (r < s.R) {
        double maxn = 0.0;
        float lo = INFINITY, hi = -INFINITY;
        for (int q = 0; q < kPrepareParts; ++q) {
            const StagePartial &pp = part[r * kPrepareParts + q];
            maxn = fmax(maxn, pp.max_norm2); lo = fminf(lo, pp.lo); hi = fmaxf(hi, pp.hi);
        }
        int k = 12;
        if (maxn > 0.0 && isfinite(maxn)) {
            k = (int)floor(0.5 * log2(8192.0 / maxn));
            k = k > 12 ? 12 : (k < -12 ? -12 : k);
        }
        sp[r].scale = ldexpf(1.0f, k);
        sp[r].a = INFINITY;
        sp[r].b = INFINITY;
        sp[r].unsafe = (!isfinite(maxn) || ldexp(maxn, 2 * k) > 8200.0) ? 1.0f : 0.0f;
        mx[r].emax = 0u; mx[r].eerr = 0u; mx[r].nmax = 0u; mx[r].elomax = 0u;
        if (r < 8) { s_lo[r] = lo; s_step[r] = hi > lo ? (hi - lo) / 65535.0f : 0.0f; }     // finest unit the range allows
    }
    __syncwarp();
    if (r == 0) {
        hdr->magic = kPreparedMagic; hdr->R = s.R; hdr->K = s.K; hdr->gd = s.gd;
        hdr->slots = slots_per_stage(s.K);
        hdr->decode_offset = decode_levels_prepared(s)
            ? (uint32_t)((kPreparedImageOffset + encode_image_bytes(s) + 255) / 256 * 256) : 0u;
        if (dp) {
            // a common base and integer scales 1..255: the unit of a stage becomes scale * base >= its finest
            float umax = 0.0f;
            for (int q = 0; q < 8; ++q) umax = fmaxf(umax, s_step[q]);
            const float base = umax / 255.0f;
            float b = 0.0f, e = 0.0f;
            for (int q = 0; q < 8; ++q) {
                uint32_t sc = 0;
                if (s_step[q] > 0.0f) {
                    sc = (uint32_t)fminf(255.0f, ceilf(s_step[q] / base));
                    while (sc < 255u && (float)sc * base < s_step[q]) ++sc;       // (rounding of the division)
                }
                dp->scale[q] = sc;
                dp->step[q] = (float)sc * base; dec_lo[q] = s_lo[q];
                b += s_lo[q]; e += 0.5f * (float)sc * base * 1.0001f;             // half a level per stage
            }
            dp->bias = b; dp->err = e; dp->base = base;
            // summed levels: per parity the finest unit such that the four stages' top levels add up to
            // at most 65535 (each stage's top level is its range over the unit, rounded up: 8 spare levels),
            // expressed as an integer multiple (1..255) of a base of their own
            float punit[2] = {0.0f, 0.0f}, pe = 0.0f;
            int pstages[2] = {0, 0};
            for (int par = 0; par < 2; ++par) {
                float span = 0.0f;
                for (int q = par; q < 8; q += 2)
                    if (s_step[q] > 0.0f) { span += s_step[q] * 65535.0f; ++pstages[par]; }
                punit[par] = span / (65535.0f - 8.0f);
            }
            const float pbase = fmaxf(punit[0], punit[1]) * 1.000001f / 255.0f;
            for (int par = 0; par < 2; ++par) {
                uint32_t sc = 0;
                if (pstages[par] > 0 && pbase > 0.0f) {
                    sc = (uint32_t)fminf(255.0f, ceilf(punit[par] / pbase));
                    while (sc < 255u && (float)sc * pbase < punit[par]) ++sc;
                    if (!((float)sc * pbase >= punit[par])) pe = INFINITY;     // (rounding at 255: no summed tables)
                }
                dp->pscale[par] = sc;
                dp->pstep[par] = (float)sc * pbase;
                pe += 0.5f * (float)pstages[par] * (float)sc * pbase * 1.0001f;   // half a level per stage
            }
            dp->pbase = pbase;
            dp->perr = pe;
        }
    }
}

// One thread per (padded) codeword: operand image and the maxima the error
// bound needs.  grid = (slots * 128 / 128, R).
__global__ void __launch_bounds__(128)
prepare_image_kernel(Shape s, const float *__restrict__ cb, const StageParams *__restrict__ sp,
                     StageMaxima *mx, uint8_t *__restrict__ image)
{
    const int r = blockIdx.y;
    const int slot = blockIdx.x, jj = threadIdx.x;
    const int j = slot * kSlotCodewords + jj;            // padded codeword index
    const float scale = sp[r].scale;
    uint8_t *base = image + ((size_t)r * slots_per_stage(s.K) + slot) * kSlotBytes;
    __half cell[kSlotCells][8];
    for (int c = 0; c < kSlotCells; ++c)
        for (int i = 0; i < 8; ++i) cell[c][i] = __float2half_rn(0.0f);
    float emax = 0.f, eerr = 0.f, nmax = 0.f, elomax = 0.f;
    if (j < s.K) {
        const float *e = cb + ((size_t)r * s.K + j) * 32;
        double n2 = 0.0, l2 = 0.0, d2 = 0.0;
        for (int i = 0; i < 32; ++i) {
            const double es = (double)e[i] * (double)scale;     // exact: power-of-two scale
            const __half hi = __double2half(es);
            const double hv = (double)__half2float(hi);
            const __half lo = __double2half(es - hv);
            const double lv = (double)__half2float(lo);
            cell[i >> 3][i & 7] = __float2half_rn(-2.0f * __half2float(hi));          // exact doubling
            cell[4 + (i >> 3)][i & 7] = __float2half_rn(-2.0f * __half2float(lo));
            n2 += es * es; l2 += lv * lv; d2 += (es - hv - lv) * (es - hv - lv);
        }
        const __half n_hi = __double2half(n2);
        const double r1 = n2 - (double)__half2float(n_hi);
        const __half n_lo = __double2half(r1);
        const double r2 = r1 - (double)__half2float(n_lo);
        cell[8][0] = n_hi; cell[8][1] = n_lo; cell[8][2] = __double2half(r2);
        // round the maxima up so that the bound stays a bound in float32
        emax = __double2float_ru(sqrt(n2)); eerr = __double2float_ru(sqrt(d2));
        nmax = __double2float_ru(n2); elomax = __double2float_ru(sqrt(l2));
    } else {
        cell[8][0] = __float2half_rn(60000.0f);           // padding never wins
    }
    for (int c = 0; c < kSlotCells; ++c)
        *reinterpret_cast<uint4 *>(base + ((size_t)c * kSlotCodewords + jj) * 16) = *reinterpret_cast<const uint4 *>(cell[c]);
    // non-negative floats order like their bit patterns
    atomicMax(&mx[r].emax, __float_as_uint(emax));
    atomicMax(&mx[r].eerr, __float_as_uint(eerr));
    atomicMax(&mx[r].nmax, __float_as_uint(nmax));
    atomicMax(&mx[r].elomax, __float_as_uint(elomax));
}

// |approximate score - exact score| <= a * ||Z|| + b for every codeword of the
// stage, where Z is the scaled float32 residual, split as Z = Zh + Zl + rz and
// the scaled codeword as E = Eh + El + re:
//   Z.E - (Zh.Eh + Zh.El + Zl.Eh) = Zl.El + rz.E + (Zh + Zl).re
//   |.| <= ||Z|| (2^-11 elomax + 2^-22 emax + eerr) + sqrt(32) 2^-25 emax
//   (the last term: a subnormal Zl is off by at most 2^-25 per channel),
//   times 2 for the factor -2 of the score; plus the accumulation of 115 terms
//   in the tensor core, taken as 2^-19 of nmax + 2 ||Z|| emax, which bounds the
//   sum of the terms' magnitudes.  The hardware's accumulation is not
//   documented; measured on B200 against float64 on operands of this shape
//   (with and without x20 outlier channels) the chain's error stayed below
//   2^-20.6 of the sum of magnitudes, so 2^-19 leaves a factor of 3; the tests
//   compare tens of millions of choices with the all-float32 kernel's.
__global__ void prepare_finish_kernel(Shape s, StageParams *sp, const StageMaxima *mx)
{
    const int r = threadIdx.x;
    if (r >= s.R) return;
    const float emax = __uint_as_float(mx[r].emax), eerr = __uint_as_float(mx[r].eerr);
    const float nmax = __uint_as_float(mx[r].nmax), elomax = __uint_as_float(mx[r].elomax);
    if (sp[r].unsafe != 0.0f) return;                      // a, b stay infinite: every row is scanned exactly
    sp[r].a = 2.0f * (4.8828125e-4f * elomax + 2.384185791015625e-7f * emax + eerr) + 3.814697265625e-6f * emax;
    sp[r].b = 1.9073486328125e-6f * nmax + 4.76837158203125e-7f * emax;
}

int launch_prepare(const Shape &s, const float *cb, void *prepared, cudaStream_t stream)
{
    uint8_t *p = reinterpret_cast<uint8_t *>(prepared);
    PreparedHeader *hdr = reinterpret_cast<PreparedHeader *>(p);
    StageParams *sp = reinterpret_cast<StageParams *>(p + kPreparedParamsOffset);
    StageMaxima *mx = reinterpret_cast<StageMaxima *>(p + kPreparedMaximaOffset);
    StagePartial *part = reinterpret_cast<StagePartial *>(p + kPreparedPartialsOffset);
    const bool dec = decode_levels_prepared(s);
    const size_t off = decode_section_offset(s);
    DecodeParams *dp = dec ? reinterpret_cast<DecodeParams *>(p + off) : nullptr;
    float *lo = dec ? reinterpret_cast<float *>(p + off + 128) : nullptr;   // per-stage minima, second half of the parameter block
    prepare_reduce_kernel<<<dim3(kPrepareParts, s.R), 256, 0, stream>>>(s, cb, part);
    int rc = check_launch();
    if (rc != RVQ_OK) return rc;
    prepare_params_kernel<<<1, 32, 0, stream>>>(s, part, hdr, sp, mx, dp, lo);
    if ((rc = check_launch()) != RVQ_OK) return rc;
    if (s.gd == 32) {
        dim3 grid(slots_per_stage(s.K), s.R);
        prepare_image_kernel<<<grid, kSlotCodewords, 0, stream>>>(s, cb, sp, mx, p + kPreparedImageOffset);
        if ((rc = check_launch()) != RVQ_OK) return rc;
        prepare_finish_kernel<<<1, 32, 0, stream>>>(s, sp, mx);
        if ((rc = check_launch()) != RVQ_OK) return rc;
    }
    if (dec) {
        dim3 grid((s.K * 8 + 255) / 256, 4);
        decode_table_kernel<<<grid, 256, 0, stream>>>(s, cb, dp, lo, reinterpret_cast<uint4 *>(p + off + 256));
        if ((rc = check_launch()) != RVQ_OK) return rc;
    }
    return RVQ_OK;
}

}  // namespace rvq
