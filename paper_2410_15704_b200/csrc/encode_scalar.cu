// Exact float32 encode on the CUDA cores: one thread per group row, squared
// distances in the direct form sum((z - e)^2), codebook chunks broadcast from
// shared memory.  Handles every supported shape; the tensor-core kernel takes
// over for the shapes it covers.  (Section 2.2, Algorithm 1.)
#include "common.cuh"

namespace rvq {

constexpr int kChunk = 128;   // codewords staged per shared-memory chunk

template <int GD>
__global__ void __launch_bounds__(128)
encode_scalar_kernel(Shape s, const void *__restrict__ x, int64_t n, int64_t stride,
                     const float *__restrict__ cb, void *__restrict__ codes,
                     uint16_t *__restrict__ std16, rvq_status *st, int vpb, float *energy)
{
    __shared__ float e_stage[16];                       // per-stage residual energy of this block's rows
    if (threadIdx.x < 16) e_stage[threadIdx.x] = 0.0f;
    extern __shared__ __align__(16) float smem[];
    float *xs = smem;                                   // [vpb][dim]
    float *cbs = xs + vpb * s.dim;                      // [kChunk][GD]
    float *part = cbs + kChunk * GD;                    // [blockDim]
    uint16_t *cs = reinterpret_cast<uint16_t *>(part + blockDim.x);   // [blockDim][R]

    const int tid = threadIdx.x;
    const int v_local = tid / s.G, g = tid - v_local * s.G;
    const int64_t v0 = (int64_t)blockIdx.x * vpb;
    const int64_t gv = v0 + v_local;

    load_tile(xs, x, v0, n, stride, vpb, s.dim, s.dtype);
    __syncthreads();

    float z[GD];
#pragma unroll
    for (int i = 0; i < GD; ++i) z[i] = xs[v_local * s.dim + channel_of(s.layout, s.G, GD, g, i)];
    const float dev = block_deviation<GD>(z, part, v_local, s.G, s.dim, s.ddof);
    const bool deg = deviation_is_degenerate(dev);
#pragma unroll
    for (int i = 0; i < GD; ++i) z[i] = deg ? 0.0f : z[i] / dev;

    for (int r = 0; r < s.R; ++r) {
        const float *cbr = cb + (size_t)r * s.K * GD;
        float best = INFINITY;
        int bj = 0;
        for (int j0 = 0; j0 < s.K; j0 += kChunk) {
            const int cnt = min(kChunk, s.K - j0);
            __syncthreads();
            for (int t = tid; t < cnt * GD / 4; t += blockDim.x)
                reinterpret_cast<float4 *>(cbs)[t] = reinterpret_cast<const float4 *>(cbr + (size_t)j0 * GD)[t];
            __syncthreads();
            for (int j = 0; j < cnt; ++j) {
                const float4 *e = reinterpret_cast<const float4 *>(cbs + j * GD);
                float acc = 0.0f;
#pragma unroll
                for (int q = 0; q < GD / 4; ++q) {
                    float4 ev = e[q];
                    float t0 = z[4 * q] - ev.x, t1 = z[4 * q + 1] - ev.y;
                    float t2 = z[4 * q + 2] - ev.z, t3 = z[4 * q + 3] - ev.w;
                    acc = fmaf(t0, t0, acc); acc = fmaf(t1, t1, acc);
                    acc = fmaf(t2, t2, acc); acc = fmaf(t3, t3, acc);
                }
                if (acc < best) { best = acc; bj = j0 + j; }      // strict: lowest index on ties
            }
        }
        if (deg) bj = 0;
        cs[tid * s.R + r] = (uint16_t)bj;
        const float4 *e = reinterpret_cast<const float4 *>(cbr + (size_t)bj * GD);
#pragma unroll
        for (int q = 0; q < GD / 4; ++q) {
            float4 ev = __ldg(e + q);
            z[4 * q] -= ev.x; z[4 * q + 1] -= ev.y; z[4 * q + 2] -= ev.z; z[4 * q + 3] -= ev.w;
        }
        if (energy && gv < n) {
            float e2 = 0.0f;
#pragma unroll
            for (int i = 0; i < GD; ++i) e2 = fmaf(z[i], z[i], e2);
            atomicAdd(&e_stage[r], e2);
        }
    }
    __syncthreads();
    if (energy && tid < s.R) atomicAdd(energy + tid, e_stage[tid]);

    // emit codes (Section 3.2 storage) and the half-precision deviation
    if (s.bits == 16) {
        if (gv < n) {
            uint16_t *o = reinterpret_cast<uint16_t *>(codes) + (gv * s.G + g) * s.R;
            for (int r = 0; r < s.R; ++r) o[r] = cs[tid * s.R + r];
        }
    } else {
        const int words = s.code_bytes / 4;
        for (int t = tid; t < vpb * words; t += blockDim.x) {
            int v = t / words, w = t - v * words;
            if (v0 + v >= n) continue;
            uint32_t word = 0;
            int k_lo = (32 * w) / s.bits, k_hi = min(s.per_vector - 1, (32 * w + 31) / s.bits);
            for (int k = k_lo; k <= k_hi; ++k) {
                uint32_t val = cs[v * s.per_vector + k];      // rows of a vector are adjacent: (v*G+g)*R+r
                int sh = k * s.bits - 32 * w;
                word |= sh >= 0 ? (val << sh) : (val >> (-sh));
            }
            reinterpret_cast<uint32_t *>(codes)[(v0 + v) * words + w] = word;
        }
    }
    if (g == 0 && gv < n) {
        __half h = __float2half_rn(dev);
        uint16_t hb = deg ? (uint16_t)0 : __half_as_ushort(h);
        std16[gv] = hb;
        if (st) {
            if (deg) atomicAdd(&st->degenerate_vectors, 1u);
            else if ((hb & 0x7FFFu) == 0 || (hb & 0x7FFFu) >= 0x7C00u) atomicAdd(&st->std_out_of_half, 1u);
        }
    }
}

template <int GD>
static int launch_gd(const Shape &s, const void *x, int64_t n, int64_t stride, const float *cb,
                     void *codes, uint16_t *std16, rvq_status *st, cudaStream_t stream, float *energy)
{
    const int vpb = 128 / s.G > 0 ? 128 / s.G : 1;
    const int threads = vpb * s.G;
    const size_t smem = sizeof(float) * ((size_t)vpb * s.dim + kChunk * GD + threads) +
                        sizeof(uint16_t) * (size_t)threads * s.R + 16;
    const int64_t blocks = (n + vpb - 1) / vpb;
    if (blocks > 0x7FFFFFFF) return RVQ_ERR_UNSUPPORTED;
    if (smem > 48 * 1024)
        cudaFuncSetAttribute(encode_scalar_kernel<GD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    encode_scalar_kernel<GD><<<(unsigned)blocks, threads, smem, stream>>>(s, x, n, stride, cb, codes, std16, st, vpb, energy);
    return check_launch();
}

int launch_encode_scalar(const Shape &s, const void *x, int64_t n, int64_t stride, const float *cb,
                         void *codes, uint16_t *std16, rvq_status *st, cudaStream_t stream, float *energy)
{
    if (n == 0) return RVQ_OK;
    switch (s.gd) {
    case 8: return launch_gd<8>(s, x, n, stride, cb, codes, std16, st, stream, energy);
    case 16: return launch_gd<16>(s, x, n, stride, cb, codes, std16, st, stream, energy);
    case 32: return launch_gd<32>(s, x, n, stride, cb, codes, std16, st, stream, energy);
    case 64: return launch_gd<64>(s, x, n, stride, cb, codes, std16, st, stream, energy);
    default: return RVQ_ERR_UNSUPPORTED;
    }
}

}  // namespace rvq
