// EMA codebook update (Section 3; Section 2.1).  Two kernels: per-code counts
// and sums of the stage inputs, then the decayed, Laplace-smoothed
// normalisation.
#include "common.cuh"

#include <atomic>

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

// Groups of 32 channels, at most 8 groups and 32 codes per head vector: one warp per head vector, lane = channel
// of the group.  A row's 32 floats then go to their bin as one coalesced 128-byte reduction (four
// sectors, one cache line) and the codeword that takes the residual to the next stage comes in as one
// 128-byte load, where a thread per row would scatter both over 32 lines per instruction (the L1's tag
// stage, not the atomics in L2, was what bound that form).  Counts go to a histogram [R][K] in shared
// memory, lanes that share a bin adding once (match.any), merged into the global counts once per CTA.
constexpr int kWarpStatsThreads = 256;

__global__ void __launch_bounds__(kWarpStatsThreads)
ema_stats_warp_kernel(Shape s, const void *__restrict__ x, int64_t n, int64_t stride,
                      const void *__restrict__ codes, const float *__restrict__ cb,
                      uint32_t *__restrict__ cnt, float *__restrict__ sum, rvq_status *st)
{
    extern __shared__ uint32_t hist[];                       // [R][K]
    const int bins = s.R * s.K;
    for (int t = threadIdx.x; t < bins; t += kWarpStatsThreads) hist[t] = 0u;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warps = (kWarpStatsThreads / 32) * gridDim.x;
    const int G = s.G, R = s.R, per = s.per_vector;            // per = G * R <= 32
    uint32_t bad = 0;
    for (int64_t v = (int64_t)blockIdx.x * (kWarpStatsThreads / 32) + warp; v < n; v += warps) {
        // element `lane` of every group: channel g*32+lane (contiguous groups) or lane*G+g (strided)
        float z[8];                                            // (G <= 8)
        float a = 0.0f;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            z[g] = g < G ? load_as_float(x, v * stride + channel_of(s.layout, G, 32, g, lane), s.dtype) : 0.0f;
            a += z[g];
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, off);
        const float mu = a / (float)s.dim;
        float b = 0.0f;
#pragma unroll
        for (int g = 0; g < 8; ++g) b += g < G ? (z[g] - mu) * (z[g] - mu) : 0.0f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) b += __shfl_xor_sync(0xFFFFFFFFu, b, off);
        const float dev = sqrtf(b / (float)(s.dim - s.ddof));
        const bool deg = deviation_is_degenerate(dev);
        // lane l holds code l of the vector (group l / R, stage l % R) and counts it
        uint32_t code = 0;
        if (lane < per) {
            code = read_code(reinterpret_cast<const uint8_t *>(codes) + v * s.code_bytes, lane, s.bits, s.code_bytes);
            if (code >= (uint32_t)s.K) { code = 0; ++bad; }
        }
        const int my_bin = lane < per ? (lane % R) * s.K + (int)code : -1 - lane;   // (idle lanes: bins of their own)
        const uint32_t same = __match_any_sync(0xFFFFFFFFu, my_bin);
        if (lane < per && lane == __ffs(same) - 1) atomicAdd(&hist[my_bin], (uint32_t)__popc(same));
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            if (g >= G) break;
            float zr = deg ? 0.0f : z[g] / dev;
            for (int r = 0; r < R; ++r) {
                const uint32_t j = __shfl_sync(0xFFFFFFFFu, code, g * R + r);
                const size_t at = ((size_t)r * s.K + j) * 32 + lane;
                const float e = __ldg(cb + at);
                atomicAdd(sum + at, zr);
                zr -= e;
            }
        }
    }
    __syncthreads();
    for (int t = threadIdx.x; t < bins; t += kWarpStatsThreads)
        if (hist[t]) atomicAdd(cnt + t, hist[t]);
    if (bad && st && lane < 32) atomicAdd(&st->bad_codes, bad);
}

// The same for head vectors of exactly four groups (dim 128): the warp takes the four rows of a vector
// at once, lane = (group, four-channel piece), so that every stage is one 16-byte reduction and one
// 16-byte load per lane (four cache lines per instruction) instead of eight instructions per row.
__global__ void __launch_bounds__(kWarpStatsThreads)
ema_stats_quad_kernel(Shape s, const void *__restrict__ x, int64_t n, int64_t stride,
                      const void *__restrict__ codes, const float *__restrict__ cb,
                      uint32_t *__restrict__ cnt, float *__restrict__ sum, rvq_status *st)
{
    extern __shared__ uint32_t hist[];                       // [R][K]
    const int bins = s.R * s.K;
    for (int t = threadIdx.x; t < bins; t += kWarpStatsThreads) hist[t] = 0u;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warps = (kWarpStatsThreads / 32) * gridDim.x;
    const int R = s.R, per = s.per_vector;                     // per = 4 * R <= 32
    const int g = lane >> 3, q = lane & 7;                     // this lane: elements 4q .. 4q+3 of group g
    uint32_t bad = 0;
    for (int64_t v = (int64_t)blockIdx.x * (kWarpStatsThreads / 32) + warp; v < n; v += warps) {
        float z[4];
        float a = 0.0f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            z[k] = load_as_float(x, v * stride + channel_of(s.layout, 4, 32, g, 4 * q + k), s.dtype);
            a += z[k];
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, off);
        const float mu = a / (float)s.dim;
        float b = 0.0f;
#pragma unroll
        for (int k = 0; k < 4; ++k) b += (z[k] - mu) * (z[k] - mu);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) b += __shfl_xor_sync(0xFFFFFFFFu, b, off);
        const float dev = sqrtf(b / (float)(s.dim - s.ddof));
        const bool deg = deviation_is_degenerate(dev);
#pragma unroll
        for (int k = 0; k < 4; ++k) z[k] = deg ? 0.0f : z[k] / dev;
        // lane l holds code l of the vector (group l / R, stage l % R) and counts it
        uint32_t code = 0;
        if (lane < per) {
            code = read_code(reinterpret_cast<const uint8_t *>(codes) + v * s.code_bytes, lane, s.bits, s.code_bytes);
            if (code >= (uint32_t)s.K) { code = 0; ++bad; }
        }
        const int my_bin = lane < per ? (lane % R) * s.K + (int)code : -1 - lane;   // (idle lanes: bins of their own)
        const uint32_t same = __match_any_sync(0xFFFFFFFFu, my_bin);
        if (lane < per && lane == __ffs(same) - 1) atomicAdd(&hist[my_bin], (uint32_t)__popc(same));
        // the codewords of all stages are asked for first (they depend on the codes only), then the
        // residual walks through the stages (R <= 8 here: four groups, at most 32 codes)
        size_t at[8];
        float4 e[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const uint32_t j = __shfl_sync(0xFFFFFFFFu, code, g * R + (r < R ? r : 0));
            at[r] = ((size_t)(r < R ? r : 0) * s.K + j) * 32 + 4 * q;
            e[r] = __ldg(reinterpret_cast<const float4 *>(cb + at[r]));
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            if (r < R) {
                atomicAdd(reinterpret_cast<float4 *>(sum + at[r]), make_float4(z[0], z[1], z[2], z[3]));
                z[0] -= e[r].x; z[1] -= e[r].y; z[2] -= e[r].z; z[3] -= e[r].w;
            }
        }
    }
    __syncthreads();
    for (int t = threadIdx.x; t < bins; t += kWarpStatsThreads)
        if (hist[t]) atomicAdd(cnt + t, hist[t]);
    if (bad && st) atomicAdd(&st->bad_codes, bad);
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
    if (n > 0 && s.gd == 32 && s.G <= 8 && s.per_vector <= 32 && (size_t)bins * sizeof(uint32_t) <= 160 * 1024) {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return RVQ_ERR_DEVICE;
        const size_t smem = (size_t)bins * sizeof(uint32_t);
        // as many CTAs per SM as the histograms leave room for (up to 8 of 256 threads)
        int per_sm = (int)((200 * 1024) / (smem + 1024));
        per_sm = per_sm < 1 ? 1 : (per_sm > 8 ? 8 : per_sm);
        int64_t want = (n + kWarpStatsThreads / 32 - 1) / (kWarpStatsThreads / 32);
        int grid = (int)(want < (int64_t)sms * per_sm ? want : (int64_t)sms * per_sm);
        auto kernel = s.G == 4 ? ema_stats_quad_kernel : ema_stats_warp_kernel;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return RVQ_ERR_LAUNCH;
        kernel<<<grid, kWarpStatsThreads, smem, stream>>>(s, x, n, stride, codes, cb, cnt, batch_sum, st);
        rc = check_launch();
    } else if (n > 0) {
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

// One thread per (bin, channel): the float32 count of the bin, and for the stages whose fused sums
// were taken after the subtraction of the codeword, the codeword's share back: sum += count * C.
__global__ void __launch_bounds__(256)
stats_finish_kernel(const uint32_t *__restrict__ cnt, const float *__restrict__ cb, float *__restrict__ sum,
                    float *__restrict__ out_count, int bins, int gd, int deferred_bins)
{
    const int t = blockIdx.x * 256 + threadIdx.x;
    if (t >= bins * gd) return;
    const int bin = t / gd, ch = t - bin * gd;
    const float c = (float)cnt[bin];
    if (ch == 0) out_count[bin] = c;
    if (bin < deferred_bins) sum[t] = fmaf(c, cb[t], sum[t]);
}

int launch_stats_finish(const Shape &s, const uint32_t *cnt, const float *cb, float *batch_sum, float *batch_count,
                        int deferred, cudaStream_t stream)
{
    const int bins = s.R * s.K, total = bins * s.gd;
    stats_finish_kernel<<<(total + 255) / 256, 256, 0, stream>>>(cnt, cb, batch_sum, batch_count, bins, s.gd, deferred * s.K);
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
// Device address of g_ema_scratch per device ordinal (null: not looked up yet).  Host threads may race to
// fill an entry: they all store the same value, and the atomic keeps the store and the loads whole.  The
// cache assumes the runtime's one primary context per device; after cudaDeviceReset the array lives at a
// new address, so a process that resets a device must not call this entry point on it again.
std::atomic<void *> g_scratch_addr[kMaxDevices];

// The array's name is only a handle on the host; the address a kernel can use
// has to be asked for, once per device, with that device current.
int static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RVQ_ERR_DEVICE;
    void *ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(&ptr, g_ema_scratch) != cudaSuccess || !ptr) return RVQ_ERR_DEVICE;
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
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

