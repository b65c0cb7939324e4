// EMA codebook update (Section 3; Section 2.1).  Two kernels: per-code counts
// and sums of the stage inputs, then the decayed, Laplace-smoothed
// normalisation.
#include "common.cuh"

namespace rvq {

static size_t round256(size_t b) { return (b + 255) / 256 * 256; }

// rvq_ema_stats scratch: integer counts, uint32 [R][K].
size_t ema_stats_scratch_bytes(const Shape &s) { return round256((size_t)s.R * s.K * sizeof(uint32_t)); }

// rvq_ema_update scratch: the above, then batch counts (float [R][K]) and
// batch sums (float [R][K][gd]).
size_t ema_workspace_bytes(const Shape &s)
{
    return ema_stats_scratch_bytes(s) + round256((size_t)s.R * s.K * sizeof(float)) +
           (size_t)s.R * s.K * s.gd * sizeof(float);
}

// One thread per group row: rebuild z_r stage by stage from x, the deviation
// and the codes, and add it to the bin of its stage-r code.
template <int GD>
__global__ void __launch_bounds__(128)
ema_stats_kernel(Shape s, const void *__restrict__ x, int64_t n, int64_t stride,
                 const void *__restrict__ codes, const float *__restrict__ cb,
                 uint32_t *__restrict__ cnt, float *__restrict__ sum, rvq_status *st, int vpb)
{
    extern __shared__ __align__(16) float smem[];
    float *xs = smem;
    float *part = xs + vpb * s.dim;
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
    if (gv >= n) return;
#pragma unroll
    for (int i = 0; i < GD; ++i) z[i] = deg ? 0.0f : z[i] / dev;

    const uint8_t *vec = reinterpret_cast<const uint8_t *>(codes) + gv * s.code_bytes;
    for (int r = 0; r < s.R; ++r) {
        uint32_t j = read_code(vec, g * s.R + r, s.bits, s.code_bytes);
        if (j >= (uint32_t)s.K) { j = 0; if (st) atomicAdd(&st->bad_codes, 1u); }
        const size_t bin = (size_t)r * s.K + j;
        atomicAdd(cnt + bin, 1u);
        float4 *m = reinterpret_cast<float4 *>(sum + bin * GD);
        const float4 *e = reinterpret_cast<const float4 *>(cb + bin * GD);
#pragma unroll
        for (int q = 0; q < GD / 4; ++q) {
            atomicAdd(m + q, make_float4(z[4 * q], z[4 * q + 1], z[4 * q + 2], z[4 * q + 3]));
            float4 ev = __ldg(e + q);
            z[4 * q] -= ev.x; z[4 * q + 1] -= ev.y; z[4 * q + 2] -= ev.z; z[4 * q + 3] -= ev.w;
        }
    }
}

__global__ void __launch_bounds__(256)
counts_to_float_kernel(const uint32_t *__restrict__ cnt, float *__restrict__ out, int total)
{
    int t = blockIdx.x * 256 + threadIdx.x;
    if (t < total) out[t] = (float)cnt[t];
}

// N <- decay N + (1-decay) n, element-wise.
__global__ void __launch_bounds__(256)
ema_count_kernel(const float *__restrict__ cnt, float *__restrict__ ema_count, int total, float decay)
{
    const int t = blockIdx.x * 256 + threadIdx.x;
    if (t < total) ema_count[t] = decay * ema_count[t] + (1.0f - decay) * cnt[t];
}

// grid (parts, R): every block sums the stage's updated counts (same order in
// every block, so all blocks of a stage get the same total), then updates its
// share of M <- decay M + (1-decay) m and C = M / ((N + eps) total / (total + K eps)).
__global__ void __launch_bounds__(256)
ema_apply_kernel(Shape s, const float *__restrict__ sum, float *__restrict__ cb,
                 const float *__restrict__ ema_count, float *__restrict__ ema_sum, float decay, float eps)
{
    __shared__ float red[256];
    const int r = blockIdx.y, tid = threadIdx.x;
    float local = 0.0f;
    for (int j = tid; j < s.K; j += 256) local += ema_count[(size_t)r * s.K + j];
    red[tid] = local;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (tid < w) red[tid] += red[tid + w];
        __syncthreads();
    }
    const float tot = red[0];
    const float scale = tot / (tot + (float)s.K * eps);
    const int per_stage = s.K * s.gd;
    for (int t = blockIdx.x * 256 + tid; t < per_stage; t += gridDim.x * 256) {
        const size_t p = (size_t)r * per_stage + t;
        const int j = t / s.gd;
        const float mm = decay * ema_sum[p] + (1.0f - decay) * sum[p];
        ema_sum[p] = mm;
        cb[p] = mm / ((ema_count[(size_t)r * s.K + j] + eps) * scale);
    }
}

template <int GD>
static int stats_gd(const Shape &s, const void *x, int64_t n, int64_t stride, const void *codes,
                    const float *cb, uint32_t *cnt, float *sum, rvq_status *st, cudaStream_t stream)
{
    const int vpb = 128 / s.G > 0 ? 128 / s.G : 1;
    const int threads = vpb * s.G;
    const size_t smem = sizeof(float) * ((size_t)vpb * s.dim + threads);
    const int64_t blocks = (n + vpb - 1) / vpb;
    if (blocks > 0x7FFFFFFF) return RVQ_ERR_UNSUPPORTED;
    ema_stats_kernel<GD><<<(unsigned)blocks, threads, smem, stream>>>(s, x, n, stride, codes, cb, cnt, sum, st, vpb);
    return check_launch();
}

int launch_ema_stats(const Shape &s, const void *x, int64_t n, int64_t stride, const void *codes,
                     const float *cb, float *batch_count, float *batch_sum, void *workspace,
                     rvq_status *st, cudaStream_t stream)
{
    uint32_t *cnt = reinterpret_cast<uint32_t *>(workspace);
    const int bins = s.R * s.K;
    if (cudaMemsetAsync(cnt, 0, (size_t)bins * sizeof(uint32_t), stream) != cudaSuccess ||
        cudaMemsetAsync(batch_sum, 0, (size_t)bins * s.gd * sizeof(float), stream) != cudaSuccess)
        return RVQ_ERR_LAUNCH;
    int rc = RVQ_OK;
    if (n > 0) {
        switch (s.gd) {
        case 8: rc = stats_gd<8>(s, x, n, stride, codes, cb, cnt, batch_sum, st, stream); break;
        case 16: rc = stats_gd<16>(s, x, n, stride, codes, cb, cnt, batch_sum, st, stream); break;
        case 32: rc = stats_gd<32>(s, x, n, stride, codes, cb, cnt, batch_sum, st, stream); break;
        case 64: rc = stats_gd<64>(s, x, n, stride, codes, cb, cnt, batch_sum, st, stream); break;
        default: rc = RVQ_ERR_UNSUPPORTED;
        }
    }
    if (rc != RVQ_OK) return rc;
    counts_to_float_kernel<<<(bins + 255) / 256, 256, 0, stream>>>(cnt, batch_count, bins);
    return check_launch();
}

int launch_counts_to_float(const uint32_t *cnt, float *out, int bins, cudaStream_t stream)
{
    counts_to_float_kernel<<<(bins + 255) / 256, 256, 0, stream>>>(cnt, out, bins);
    return check_launch();
}

int launch_ema_apply(const Shape &s, const float *batch_count, const float *batch_sum, float *cb,
                     float *ema_count, float *ema_sum, float decay, float eps, cudaStream_t stream)
{
    const int bins = s.R * s.K;
    ema_count_kernel<<<(bins + 255) / 256, 256, 0, stream>>>(batch_count, ema_count, bins, decay);
    int rc = check_launch();
    if (rc != RVQ_OK) return rc;
    int parts = (s.K * s.gd + 256 * 8 - 1) / (256 * 8);
    if (parts > 32) parts = 32;
    ema_apply_kernel<<<dim3(parts, s.R), 256, 0, stream>>>(s, batch_sum, cb, ema_count, ema_sum, decay, eps);
    return check_launch();
}

}  // namespace rvq

// ---------------------------------------------------------------------------
// rvq_ema_update_static: the same update with its scratch inside the library.
//
// The scratch of rvq_ema_update (integer counts, batch counts, batch sums) lives
// here in a fixed device array instead of a caller buffer, so a caller that has
// no way to obtain device memory of its own can still run the update.  The array
// is part of the library image: every GPU that loads the library carries it until
// the process exits, used or not.
namespace {

// Room for depth 8 x 2048 codes x 32 channels (the paper's default quantizer):
// 64 KiB of counts + 64 KiB of batch counts + 2 MiB of batch sums.
constexpr size_t kStaticScratchBytes = 65536 + 65536 + 2097152;
static __device__ __align__(256) unsigned char g_ema_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices];      // device address of g_ema_scratch per device ordinal (null: not looked up yet)

// The array's name is only a handle on the host; the address a kernel can use
// has to be asked for, once per device, with that device current.
int static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RVQ_ERR_DEVICE;
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_ema_scratch) != cudaSuccess || !ptr) return RVQ_ERR_DEVICE;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return RVQ_OK;
}

}  // namespace

extern "C" size_t rvq_ema_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" int rvq_ema_update_static(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                                     const void *codes, float *codebooks, float *ema_count, float *ema_sum,
                                     float *batch_count, float decay, float eps, rvq_status *status,
                                     void *stream)
{
    using namespace rvq;
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if (n < 0 || x_row_stride < s.dim || (n > 0 && (!x || !codes))) return RVQ_ERR_BADARG;
    if (!codebooks || !ema_count || !ema_sum) return RVQ_ERR_BADARG;
    if (!(decay >= 0.0f && decay <= 1.0f) || !(eps >= 0.0f)) return RVQ_ERR_BADARG;
    if (!aligned16(x) || (x_row_stride * s.elem_bytes) % 16 || !aligned16(codes) || !aligned16(codebooks) ||
        !aligned16(ema_sum))
        return RVQ_ERR_ALIGN;
    if (ema_workspace_bytes(s) > kStaticScratchBytes) return RVQ_ERR_STATIC_LIMIT;
    void *scratch = nullptr;
    if ((rc = static_scratch(&scratch)) != RVQ_OK) return rc;
    // same carving as rvq_ema_update: counts | batch counts | batch sums
    uint8_t *ws = reinterpret_cast<uint8_t *>(scratch);
    float *bc = reinterpret_cast<float *>(ws + ema_stats_scratch_bytes(s));
    float *bs = reinterpret_cast<float *>(ws + ema_stats_scratch_bytes(s) + round256((size_t)s.R * s.K * sizeof(float)));
    // launch_ema_stats zeroes the counts and the batch sums it accumulates into;
    // nothing else in the scratch is read before it is written
    rc = launch_ema_stats(s, x, n, x_row_stride, codes, codebooks, bc, bs, scratch, status, (cudaStream_t)stream);
    if (rc != RVQ_OK) return rc;
    if (batch_count &&
        cudaMemcpyAsync(batch_count, bc, (size_t)s.R * s.K * sizeof(float), cudaMemcpyDeviceToDevice,
                        (cudaStream_t)stream) != cudaSuccess)
        return RVQ_ERR_LAUNCH;
    return launch_ema_apply(s, bc, bs, codebooks, ema_count, ema_sum, decay, eps, (cudaStream_t)stream);
}

