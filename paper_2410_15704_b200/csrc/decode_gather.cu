// Generic decode: one thread per (head vector, group, 4-element piece), code
// rows gathered as float4 from the float32 codebooks (L1/L2 resident), summed in
// float32 in stage order, multiplied by the stored deviation and rounded once.
// Handles every supported shape.  (Section 2.2 last sentence, Section 3.2.)
#include "common.cuh"

namespace rvq {

__global__ void __launch_bounds__(256)
decode_gather_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16,
                     int64_t n, const float *__restrict__ cb, void *__restrict__ out, int64_t stride,
                     rvq_status *st)
{
    const int pieces = s.gd / 4;
    const int64_t total = n * s.G * pieces;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int q = (int)(t % pieces);
        const int64_t row = t / pieces;
        const int g = (int)(row % s.G);
        const int64_t v = row / s.G;
        const uint8_t *vec = reinterpret_cast<const uint8_t *>(codes) + v * s.code_bytes;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int r = 0; r < s.R; ++r) {
            uint32_t j = read_code(vec, g * s.R + r, s.bits, s.code_bytes);
            if (j >= (uint32_t)s.K) { j = 0; if (st && q == 0) atomicAdd(&st->bad_codes, 1u); }
            float4 e = __ldg(reinterpret_cast<const float4 *>(cb + ((size_t)r * s.K + j) * s.gd) + q);
            acc.x += e.x; acc.y += e.y; acc.z += e.z; acc.w += e.w;
        }
        const float sd = __half2float(__ushort_as_half(std16[v]));
        const float o[4] = {sd * acc.x, sd * acc.y, sd * acc.z, sd * acc.w};
#pragma unroll
        for (int k = 0; k < 4; ++k)
            store_from_float(out, v * stride + channel_of(s.layout, s.G, s.gd, g, 4 * q + k), s.dtype, o[k]);
    }
}

int launch_decode_gather(const Shape &s, const void *codes, const uint16_t *std16, int64_t n,
                         const float *cb, void *out, int64_t stride, rvq_status *st,
                         cudaStream_t stream)
{
    if (n == 0) return RVQ_OK;
    const int64_t total = n * s.G * (s.gd / 4);
    int64_t blocks = (total + 255) / 256;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return RVQ_ERR_DEVICE;
    if (blocks > (int64_t)sms * 64) blocks = (int64_t)sms * 64;
    decode_gather_kernel<<<(unsigned)blocks, 256, 0, stream>>>(s, codes, std16, n, cb, out, stride, st);
    return check_launch();
}

}  // namespace rvq
