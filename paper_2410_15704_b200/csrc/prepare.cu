// Prepared-codebook block: what the kernels read instead of the float32
// codebooks.  Written by rvq_prepare_codebooks, read-only afterwards.
//
// Encode section (group_dim 32 only).  Algorithm 1's argmin over
// ||z - e||^2 is taken over the scores ||e||^2 - 2 z.e, which are one dense
// contraction per stage.  Per stage r the block holds
//   - a power-of-two scale 2^k chosen so that the largest scaled squared norm
//     is about 2^13 (keeps half-precision operands out of the subnormal range);
//   - the B operand image of tcgen05.mma: for every slot of 256 codewords six
//     "cells" (8 halves = 16 bytes per codeword per cell, K-major, no swizzle):
//     cells 0-3 hold -2 * fp16(2^k e), cell 4 holds the scaled squared norm
//     split into three halves (hi, lo, lo2) followed by zeros, cell 5 is zero.
//     The A operand carries (Z, 1, 1, 1, 0...) so the accumulator is the score;
//   - two numbers (a, b) such that |score error| <= a * ||Z|| + b, from the
//     actual rounding errors of this codebook (see prepare_finish_kernel).
#include "prepared.cuh"

namespace rvq {

size_t prepared_bytes(const Shape &s)
{
    size_t b = kPreparedImageOffset;
    if (s.gd == 32) b += (size_t)s.R * slots_per_stage(s.K) * kSlotBytes;
    return (b + 255) / 256 * 256;
}

// One block per stage: largest squared norm -> scale exponent; clears the maxima.
__global__ void __launch_bounds__(256)
prepare_scale_kernel(Shape s, const float *__restrict__ cb, PreparedHeader *hdr, StageParams *sp,
                     StageMaxima *mx)
{
    __shared__ double red[256];
    const int r = blockIdx.x, tid = threadIdx.x;
    double m = 0.0;
    for (int j = tid; j < s.K; j += 256) {
        const float *e = cb + ((size_t)r * s.K + j) * s.gd;
        double acc = 0.0;
        for (int i = 0; i < s.gd; ++i) acc += (double)e[i] * (double)e[i];
        m = fmax(m, acc);
    }
    red[tid] = m;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (tid < w) red[tid] = fmax(red[tid], red[tid + w]);
        __syncthreads();
    }
    if (tid == 0) {
        const double maxn = red[0];
        int k = 12;
        if (maxn > 0.0 && isfinite(maxn)) {
            k = (int)floor(0.5 * log2(8192.0 / maxn));
            k = k > 12 ? 12 : (k < -12 ? -12 : k);
        }
        sp[r].scale = ldexpf(1.0f, k);
        sp[r].a = INFINITY;
        sp[r].b = INFINITY;
        sp[r].unsafe = (!isfinite(maxn) || ldexp(maxn, 2 * k) > 8200.0) ? 1.0f : 0.0f;
        mx[r].emax = 0u; mx[r].eerr = 0u; mx[r].nmax = 0u;
        if (r == 0) {
            hdr->magic = kPreparedMagic; hdr->R = s.R; hdr->K = s.K; hdr->gd = s.gd;
            hdr->slots = slots_per_stage(s.K);
        }
    }
}

// One thread per (padded) codeword: operand image and the maxima the error
// bound needs.  grid = (slots * 256 / 256, R).
__global__ void __launch_bounds__(256)
prepare_image_kernel(Shape s, const float *__restrict__ cb, const StageParams *__restrict__ sp,
                     StageMaxima *mx, uint8_t *__restrict__ image)
{
    const int r = blockIdx.y;
    const int j = blockIdx.x * 256 + threadIdx.x;       // padded codeword index
    const int slot = j >> 8, jj = j & 255;
    const float scale = sp[r].scale;
    uint8_t *base = image + ((size_t)r * slots_per_stage(s.K) + slot) * kSlotBytes;
    __half cell[6][8];
    float emax = 0.f, eerr = 0.f, nmax = 0.f;
    if (j < s.K) {
        const float *e = cb + ((size_t)r * s.K + j) * 32;
        double n2 = 0.0, h2 = 0.0, d2 = 0.0;
        for (int i = 0; i < 32; ++i) {
            const double es = (double)e[i] * (double)scale;     // exact: power-of-two scale
            const __half h = __double2half(es);
            const double hv = (double)__half2float(h);
            cell[i >> 3][i & 7] = __float2half_rn(-2.0f * __half2float(h));
            n2 += es * es; h2 += hv * hv; d2 += (es - hv) * (es - hv);
        }
        const __half n_hi = __double2half(n2);
        const double r1 = n2 - (double)__half2float(n_hi);
        const __half n_lo = __double2half(r1);
        const double r2 = r1 - (double)__half2float(n_lo);
        const __half n_lo2 = __double2half(r2);
        cell[4][0] = n_hi; cell[4][1] = n_lo; cell[4][2] = n_lo2;
        // round the maxima up so that the bound stays a bound in float32
        emax = __double2float_ru(sqrt(h2)); eerr = __double2float_ru(sqrt(d2)); nmax = __double2float_ru(n2);
    } else {
        for (int i = 0; i < 32; ++i) cell[i >> 3][i & 7] = __float2half_rn(0.0f);
        cell[4][0] = __float2half_rn(60000.0f);           // padding never wins
        cell[4][1] = cell[4][2] = __float2half_rn(0.0f);
    }
    for (int i = 3; i < 8; ++i) cell[4][i] = __float2half_rn(0.0f);
    for (int i = 0; i < 8; ++i) cell[5][i] = __float2half_rn(0.0f);
    for (int c = 0; c < 6; ++c)
        *reinterpret_cast<uint4 *>(base + ((size_t)c * 256 + jj) * 16) = *reinterpret_cast<const uint4 *>(cell[c]);
    // non-negative floats order like their bit patterns
    atomicMax(&mx[r].emax, __float_as_uint(emax));
    atomicMax(&mx[r].eerr, __float_as_uint(eerr));
    atomicMax(&mx[r].nmax, __float_as_uint(nmax));
}

// |approximate score - exact score| <= a * ||Z|| + b for every codeword of the
// stage, where Z is the scaled float32 residual:
//   2 |sum (Z_i E_i - fp16(Z_i) fp16(E_i))| <= 2 ||Z|| (eerr + u emax) + 2 sqrt(32) 2^-25 emax
//   (u = 2^-11 half-precision rounding; the last term covers subnormal Z_i),
//   accumulation of 51 terms in the tensor core, each step within 2^-22 of the
//   running magnitude <= nmax + 2 ||Z|| emax:  2^-16 (nmax + 2 ||Z|| emax).
__global__ void prepare_finish_kernel(Shape s, StageParams *sp, const StageMaxima *mx)
{
    const int r = threadIdx.x;
    if (r >= s.R) return;
    const float emax = __uint_as_float(mx[r].emax), eerr = __uint_as_float(mx[r].eerr);
    const float nmax = __uint_as_float(mx[r].nmax);
    if (sp[r].unsafe != 0.0f) return;                      // a, b stay infinite: every row is scanned exactly
    const float u = 4.8828125e-4f;
    sp[r].a = 2.0f * (eerr + u * emax) + 3.0517578125e-5f * emax;
    sp[r].b = 1.52587890625e-5f * nmax + 4.76837158203125e-7f * emax;
}

int launch_prepare(const Shape &s, const float *cb, void *prepared, cudaStream_t stream)
{
    uint8_t *p = reinterpret_cast<uint8_t *>(prepared);
    PreparedHeader *hdr = reinterpret_cast<PreparedHeader *>(p);
    StageParams *sp = reinterpret_cast<StageParams *>(p + kPreparedParamsOffset);
    StageMaxima *mx = reinterpret_cast<StageMaxima *>(p + kPreparedMaximaOffset);
    prepare_scale_kernel<<<s.R, 256, 0, stream>>>(s, cb, hdr, sp, mx);
    int rc = check_launch();
    if (rc != RVQ_OK || s.gd != 32) return rc;
    dim3 grid(slots_per_stage(s.K), s.R);
    prepare_image_kernel<<<grid, 256, 0, stream>>>(s, cb, sp, mx, p + kPreparedImageOffset);
    if ((rc = check_launch()) != RVQ_OK) return rc;
    prepare_finish_kernel<<<1, 32, 0, stream>>>(s, sp, mx);
    return check_launch();
}

}  // namespace rvq
