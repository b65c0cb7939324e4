// Shared host/device helpers of the RVQ library: shape validation, element
// loads/stores for the three vector types, the channel map of Section 3.1 and
// the packed code stream of Section 3.2.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rvq.h"

namespace rvq {

struct Shape {
    int dim, gd, G, layout, R, K, bits, dtype, ddof;
    int per_vector;       // G * R codes per head vector
    int code_bytes;       // bytes of one head vector's codes
    int elem_bytes;       // bytes of one x element
    int raw;              // library-internal: the rows are stage inputs already (no deviation, no scaling)
};

// Fills `s` from a caller config; returns RVQ_OK or the error to hand back.
int make_shape(const rvq_config *cfg, Shape *s);

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

// Launchers (one per .cu file); all return RVQ_OK or RVQ_ERR_LAUNCH / _UNSUPPORTED.
int launch_encode_scalar(const Shape &s, const void *x, int64_t n, int64_t stride, const float *cb,
                         void *codes, uint16_t *std16, rvq_status *st, cudaStream_t stream,
                         float *energy = nullptr);
bool encode_tensor_supported(const Shape &s);
int launch_encode_tensor(const Shape &s, const void *x, int64_t n, int64_t stride, const float *cb,
                         const void *prepared, void *codes, uint16_t *std16, rvq_status *st,
                         cudaStream_t stream, uint32_t *stat_cnt = nullptr, float *stat_sum = nullptr,
                         float *energy = nullptr, uint32_t wait_limit = 0, int drop_last_chain = 0);
int launch_counts_to_float(const uint32_t *cnt, float *out, int bins, cudaStream_t stream);
int encode_tensor_deferred_stages(const Shape &s);
// counts to float32, and sum += count * codeword for the first `deferred` stages (see encode_tensor.cu)
int launch_stats_finish(const Shape &s, const uint32_t *cnt, const float *cb, float *batch_sum, float *batch_count,
                        int deferred, cudaStream_t stream);
int launch_decode_gather(const Shape &s, const void *codes, const uint16_t *std16, int64_t n,
                         const float *cb, void *out, int64_t stride, rvq_status *st,
                         cudaStream_t stream);
int launch_decode_sliced(const Shape &s, const void *codes, const uint16_t *std16, int64_t n,
                         const float *cb, const void *prepared, void *out, int64_t stride, rvq_status *st,
                         cudaStream_t stream);
int launch_rope_table(int dim, double base, int positions, float *table, cudaStream_t stream);
int launch_decode_rope(const Shape &s, const void *codes, const uint16_t *std16, int64_t n, const float *cb,
                       const void *prepared, const int32_t *position, int per_position, const float *table,
                       int positions, int style, void *out, int64_t stride, rvq_status *st, cudaStream_t stream);
int launch_ema_stats(const Shape &s, const void *x, int64_t n, int64_t stride, const void *codes,
                     const float *cb, float *batch_count, float *batch_sum, void *workspace,
                     rvq_status *st, cudaStream_t stream);
int launch_ema_apply(const Shape &s, const float *batch_count, const float *batch_sum, float *cb,
                     float *ema_count, float *ema_sum, float decay, float eps, cudaStream_t stream);
size_t ema_workspace_bytes(const Shape &s);     // all of rvq_ema_update's scratch
size_t ema_stats_scratch_bytes(const Shape &s); // the part rvq_ema_stats itself needs
size_t kmeans_workspace_bytes(const Shape &s, int64_t n);
int launch_kmeans(const Shape &s, const void *x, int64_t n, int64_t stride, const int64_t *seed_rows,
                  int iterations, float *codebooks, void *prepared, void *workspace, rvq_status *st,
                  cudaStream_t stream);
bool attention_supported(const Shape &sk, const Shape &sv, int kv_heads, int q_heads, int64_t tokens);
size_t attention_workspace_bytes(int64_t tokens, int q_heads);
int launch_attention_decode(const Shape &sk, const Shape &sv, const float *q, int q_heads, const void *codes_k,
                            const uint16_t *std_k, const void *codes_v, const uint16_t *std_v, int64_t tokens,
                            const float *cb_k, const float *cb_v, const int32_t *position, const float *cos_sin,
                            int positions, int pairing, float scale, float *out, void *workspace, rvq_status *st,
                            cudaStream_t stream);
size_t prepared_bytes(const Shape &s);
int launch_prepare(const Shape &s, const float *cb, void *prepared, cudaStream_t stream);

void count_launch();
inline int check_launch()
{
    count_launch();
    return cudaGetLastError() == cudaSuccess ? RVQ_OK : RVQ_ERR_LAUNCH;
}

#ifdef __CUDACC__

// Section 3.1: element i of group g is channel g*gd+i (contiguous groups) or
// channel i*G+g (channels G = d/d^ apart).
__device__ __forceinline__ int channel_of(int layout, int G, int gd, int g, int i)
{
    return layout == RVQ_GROUP_STRIDED ? i * G + g : g * gd + i;
}

__device__ __forceinline__ float load_as_float(const void *base, int64_t idx, int dtype)
{
    if (dtype == RVQ_F32) return reinterpret_cast<const float *>(base)[idx];
    if (dtype == RVQ_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(base)[idx]);
    return __half2float(reinterpret_cast<const __half *>(base)[idx]);
}

__device__ __forceinline__ void store_from_float(void *base, int64_t idx, int dtype, float v)
{
    if (dtype == RVQ_F32) reinterpret_cast<float *>(base)[idx] = v;
    else if (dtype == RVQ_BF16) reinterpret_cast<__nv_bfloat16 *>(base)[idx] = __float2bfloat16_rn(v);
    else reinterpret_cast<__half *>(base)[idx] = __float2half_rn(v);
}

// Code number k of one head vector whose codes start at `vec` (4-byte aligned).
__device__ __forceinline__ uint32_t read_code(const void *vec, int k, int bits, int code_bytes)
{
    if (bits == 16) return reinterpret_cast<const uint16_t *>(vec)[k];
    const uint32_t *w = reinterpret_cast<const uint32_t *>(vec);
    int off = k * bits, wi = off >> 5, sh = off & 31;
    uint32_t lo = w[wi];
    uint32_t hi = (sh + bits > 32 && (wi + 1) * 4 < code_bytes) ? w[wi + 1] : 0u;
    return __funnelshift_r(lo, hi, sh) & ((1u << bits) - 1u);
}

__device__ __forceinline__ bool deviation_is_degenerate(float s) { return !(s > 0.0f) || !isfinite(s); }

// Load a tile of `vpb` head vectors (first vector v0) into shared memory as
// float32 [vpb][dim]; rows past n are zero.
__device__ __forceinline__ void load_tile(float *xs, const void *x, int64_t v0, int64_t n,
                                          int64_t stride, int vpb, int dim, int dtype)
{
    for (int idx = threadIdx.x; idx < vpb * dim; idx += blockDim.x) {
        int v = idx / dim, c = idx - v * dim;
        int64_t gv = v0 + v;
        xs[idx] = gv < n ? load_as_float(x, gv * stride + c, dtype) : 0.0f;
    }
}

// Section 2.2: deviation of one head vector, float32, two passes (mean, then
// centred squares).  Every row thread (v_local, g) passes its group's channels
// in z[0..gd); `part` is shared scratch of blockDim.x floats.  All threads of
// the block must call this together.  Returns s for the caller's vector.
template <int GD>
__device__ __forceinline__ float block_deviation(const float (&z)[GD], float *part, int v_local,
                                                 int G, int dim, int ddof)
{
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < GD; ++i) a += z[i];
    part[threadIdx.x] = a;
    __syncthreads();
    float mu = 0.0f;
    for (int g = 0; g < G; ++g) mu += part[v_local * G + g];
    mu /= (float)dim;
    __syncthreads();
    float b = 0.0f;
#pragma unroll
    for (int i = 0; i < GD; ++i) b += (z[i] - mu) * (z[i] - mu);
    part[threadIdx.x] = b;
    __syncthreads();
    float ss = 0.0f;
    for (int g = 0; g < G; ++g) ss += part[v_local * G + g];
    __syncthreads();
    return sqrtf(ss / (float)(dim - ddof));
}

#endif  // __CUDACC__

}  // namespace rvq
