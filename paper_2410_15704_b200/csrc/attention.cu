// Attention of one new token over a compressed key/value cache (Section 1: the
// cache is what long-context decoding loads; Section 3: keys are stored before
// the rotary embedding; Section 2.2: a cached vector is the sum of its codewords
// times its deviation).  The decoded keys and values never reach global memory:
//   1. scores   s[t][h][j] = sum_c q[h J + j][c] * rot(k^[t][h])[c]        (att_scores_kernel)
//   2. maxima   m[h][j] = max_t scale * s[t][h][j]                          (att_max_kernel)
//   3. values   acc[h][j][c] = sum_t exp(scale s - m) v^[t][h][c], and the sum of the weights
//                                                                          (att_values_kernel)
//   4. out[h J + j][c] = acc / weights                                      (att_finish_kernel)
// Steps 1 and 3 are the table decoder's gather: a CTA keeps the float32 channels of one slice of
// four codeword elements for all codes and stages in shared memory (16 bytes per code and stage,
// stage order rotated by lane so that a quarter warp's reads never collide), a warp takes one
// token (its 32 lanes are the 8 kv heads x 4 groups, so a thread keeps one (head, group) for the
// whole launch and with it its query values and its output accumulators in registers), and the
// eight slices of a token are eight CTAs whose partial scores meet in global memory through
// float reductions.
#include "prepared.cuh"

namespace rvq {

namespace {

constexpr int kAttThreads = 1024;
constexpr int kAttSlices = 8;            // four codeword elements per slice
constexpr int kAttMaxK = 1792;           // 128 bytes per code: 224 KB of shared memory

// Codeword element at place i of slice sl.  Keys with half-split rotary pairs on strided groups
// keep two elements and their partners 16 elements on (channels 64 apart) in one slice.
template <int LAYOUT, int ROPE>
__device__ __forceinline__ int att_element(int sl, int i)
{
    if (ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED) return 2 * sl + (i & 1) + 16 * (i >> 1);
    return 4 * sl + i;
}
template <int LAYOUT>
__device__ __forceinline__ int att_channel(int g, int e)
{
    return LAYOUT == RVQ_GROUP_STRIDED ? 4 * e + g : 32 * g + e;
}

// table[code][stage] = the four float32 channels of this slice; absent stages are zero
template <int LAYOUT, int ROPE>
__device__ __forceinline__ void att_fill_table(const Shape &s, const float *__restrict__ cb, int sl, float4 *table)
{
    for (int t = threadIdx.x; t < s.K * 8; t += kAttThreads) {
        const int r = t & 7, j = t >> 3;
        float4 e = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (r < s.R) {
            const float *src = cb + ((size_t)r * s.K + j) * 32;
            if (ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED) {
                const float2 a = __ldg(reinterpret_cast<const float2 *>(src + 2 * sl));
                const float2 b = __ldg(reinterpret_cast<const float2 *>(src + 2 * sl + 16));
                e = make_float4(a.x, a.y, b.x, b.y);
            } else {
                e = __ldg(reinterpret_cast<const float4 *>(src + 4 * sl));
            }
        }
        table[t] = e;
    }
}

// The codes of group row `row` (= 4 * head vector + group) as four words, stage r in half r; the
// deviation of its head vector.
struct AttRow {
    uint32_t c0, c1, c2, c3;
    uint16_t sd;
};
// Position of a token: the caller's, or the token's index.
__device__ __forceinline__ int att_position(const int32_t *__restrict__ position, uint32_t token, uint32_t tokens)
{
    if (token >= tokens) return 0;
    return position ? __ldg(position + token) : (int)token;
}
__device__ __forceinline__ void att_fetch(const Shape &s, const void *__restrict__ codes,
                                          const uint16_t *__restrict__ std16, uint32_t token, uint32_t tokens, int lane,
                                          AttRow &a)
{
    a.c0 = a.c1 = a.c2 = a.c3 = 0u;
    a.sd = 0;
    if (token >= tokens) return;
    const uint32_t v = token * 8u + (uint32_t)(lane >> 2);    // (the launcher keeps tokens * 32 below 2^31)
    const int g = lane & 3;
    a.sd = __ldg(std16 + v);
    if (s.bits == 16 && s.R == 8) {
        const uint4 c = __ldg(reinterpret_cast<const uint4 *>(codes) + (v * 4u + (uint32_t)g));
        a.c0 = c.x; a.c1 = c.y; a.c2 = c.z; a.c3 = c.w;
    } else {
        const uint8_t *vec = reinterpret_cast<const uint8_t *>(codes) + (size_t)v * s.code_bytes;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int r = 0; r < 8; ++r)
            if (r < s.R) w[r >> 1] |= read_code(vec, g * s.R + r, s.bits, s.code_bytes) << (16 * (r & 1));
        a.c0 = w[0]; a.c1 = w[1]; a.c2 = w[2]; a.c3 = w[3];
    }
}

// Sum over the stages of the four channels of this thread's row: eight 16-byte reads, stage
// (rot + k) & 7 at step k.  Codes past the codebook are read as code 0 and counted.
__device__ __forceinline__ void att_gather(const AttRow &a, uint32_t K, uint32_t rot, uint32_t smem_table,
                                           float (&acc)[4], uint32_t &bad)
{
    uint32_t c0 = a.c0, c1 = a.c1, c2 = a.c2, c3 = a.c3;
    {
        const uint32_t m = __vmaxu2(__vmaxu2(c0, c1), __vmaxu2(c2, c3));
        if (max(m & 0xFFFFu, m >> 16) >= K) {
            uint32_t *cc[4] = {&c0, &c1, &c2, &c3};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t lo = *cc[c] & 0xFFFFu, hi = *cc[c] >> 16;
                if (lo >= K) { lo = 0; ++bad; }
                if (hi >= K) { hi = 0; ++bad; }
                *cc[c] = lo | (hi << 16);
            }
        }
    }
    // rotate the 8 halves left by `rot` so that step k finds its code at a fixed place
    if (rot & 4u) { const uint32_t t0 = c0, t1 = c1; c0 = c2; c1 = c3; c2 = t0; c3 = t1; }
    if (rot & 2u) { const uint32_t t0 = c0; c0 = c1; c1 = c2; c2 = c3; c3 = t0; }
    if (rot & 1u) {
        const uint32_t b0 = __funnelshift_r(c0, c1, 16), b1 = __funnelshift_r(c1, c2, 16);
        const uint32_t b2 = __funnelshift_r(c2, c3, 16), b3 = __funnelshift_r(c3, c0, 16);
        c0 = b0; c1 = b1; c2 = b2; c3 = b3;
    }
    const uint32_t cw[4] = {c0, c1, c2, c3};
    acc[0] = acc[1] = acc[2] = acc[3] = 0.0f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint32_t w = cw[k >> 1];
        const uint32_t line = (k & 1) ? ((w >> 9) & (0xFFFFu << 7)) : ((w << 7) & (0xFFFFu << 7));
        const uint32_t addr = smem_table + (line | (((rot + k) & 7u) * 16u));
        float f0, f1, f2, f3;
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(f0), "=f"(f1), "=f"(f2), "=f"(f3) : "r"(addr));
        acc[0] += f0; acc[1] += f1; acc[2] += f2; acc[3] += f3;
    }
}

// (cos, sin) of the rotary pairs of this thread's four channels at position `pos`:
// c[i], s[i] belong to place i (half-split pairs on strided groups and adjacent pairs on
// contiguous groups have two pairs in the thread: places 0 and 1 of c, s).
template <int LAYOUT, int ROPE>
__device__ __forceinline__ void att_cos_sin(const float2 *__restrict__ cos_sin, int positions, int pos, int sl, int g,
                                            float (&c)[4], float (&sn)[4])
{
    c[0] = c[1] = c[2] = c[3] = 1.0f;
    sn[0] = sn[1] = sn[2] = sn[3] = 0.0f;
    if (ROPE == 0) return;
    const float2 *cs = cos_sin + (size_t)min(max(pos, 0), positions - 1) * 64;
    if (ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED) {
        // places (0, 2) and (1, 3): channels 4 (2 sl + i) + g and 64 further on; that channel is the pair
#pragma unroll
        for (int i = 0; i < 2; ++i) { const float2 t = __ldg(cs + 4 * (2 * sl + i) + g); c[i] = t.x; sn[i] = t.y; }
    } else if (ROPE == 2 && LAYOUT == RVQ_GROUP_CONTIGUOUS) {
        // channels 32 g + 4 sl + i: pairs 16 g + 2 sl + i / 2, both halves in the thread
        const float4 t = __ldg(reinterpret_cast<const float4 *>(cs + 16 * g + 2 * sl));
        c[0] = t.x; sn[0] = t.y; c[1] = t.z; sn[1] = t.w;
    } else if (ROPE == 1) {
        // contiguous groups: channel 32 g + 4 sl + i and its partner in group g ^ 2; pairs 32 (g & 1) + 4 sl + i
        const float4 *p = reinterpret_cast<const float4 *>(cs + 32 * (g & 1) + 4 * sl);
        const float4 a = __ldg(p), b = __ldg(p + 1);
        c[0] = a.x; sn[0] = a.y; c[1] = a.z; sn[1] = a.w; c[2] = b.x; sn[2] = b.y; c[3] = b.z; sn[3] = b.w;
    } else {
        // strided groups, pairs (2k, 2k + 1): channels 4 e + g and 4 e + (g ^ 1), e = 4 sl + i; pair 2 e + g / 2
#pragma unroll
        for (int i = 0; i < 4; ++i) { const float2 t = __ldg(cs + 2 * (4 * sl + i) + (g >> 1)); c[i] = t.x; sn[i] = t.y; }
    }
}

// Step 1.  ROPE 0: keys as stored; 1: pairs (k, k + 64); 2: pairs (2k, 2k + 1).
template <int LAYOUT, int ROPE, int J>
__global__ void __launch_bounds__(kAttThreads, 1)
att_scores_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t tokens,
                  const float *__restrict__ cb, const float *__restrict__ q, const int32_t *__restrict__ position,
                  const float2 *__restrict__ cos_sin, int positions, float *__restrict__ scores, rvq_status *st)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int parts = gridDim.x / kAttSlices;
    if ((int)blockIdx.x >= parts * kAttSlices) return;
    const int sl = blockIdx.x % kAttSlices, part = blockIdx.x / kAttSlices;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, h = lane >> 2, g = lane & 3;
    att_fill_table<LAYOUT, ROPE>(s, cb, sl, reinterpret_cast<float4 *>(smem));
    // the query values that meet this thread's four channels, for the J query heads of its kv head
    float qr[J][4];
#pragma unroll
    for (int j = 0; j < J; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i)
            qr[j][i] = __ldg(q + (size_t)(h * J + j) * 128 + att_channel<LAYOUT>(g, att_element<LAYOUT, ROPE>(sl, i)));
    __syncthreads();
    const uint32_t smem_table = (uint32_t)__cvta_generic_to_shared(smem);
    uint32_t bad = 0;
    // Loads run ahead of their use: the codes, the deviation and the (cos, sin) values of the next token
    // are asked for while this one is gathered, and the position of the token after that (the address
    // of the (cos, sin) values hangs on it).
    const uint32_t T = (uint32_t)tokens, step = (uint32_t)parts * 32u, t0 = (uint32_t)part * 32u + (uint32_t)warp;
    AttRow next;
    float cn[4], sn[4];
    att_fetch(s, codes, std16, t0, T, lane, next);
    att_cos_sin<LAYOUT, ROPE>(cos_sin, positions, att_position(position, t0, T), sl, g, cn, sn);
    int pos_next = ROPE != 0 ? att_position(position, t0 + step, T) : 0;
    for (uint32_t t = t0; t < T; t += step) {
        const AttRow cur = next;
        float cc[4], ss[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { cc[i] = cn[i]; ss[i] = sn[i]; }
        att_cos_sin<LAYOUT, ROPE>(cos_sin, positions, pos_next, sl, g, cn, sn);
        if (ROPE != 0) pos_next = att_position(position, t + 2 * step, T);
        att_fetch(s, codes, std16, t + step, T, lane, next);
        float v[4];
        att_gather(cur, (uint32_t)s.K, (uint32_t)lane & 7u, smem_table, v, bad);
        const float sd = __half2float(__ushort_as_half(cur.sd));
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] *= sd;
        if (ROPE != 0) {
            if (ROPE == 1 && LAYOUT == RVQ_GROUP_STRIDED) {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float a = v[i], b = v[i + 2];
                    v[i] = a * cc[i] - b * ss[i];
                    v[i + 2] = b * cc[i] + a * ss[i];
                }
            } else if (ROPE == 2 && LAYOUT == RVQ_GROUP_CONTIGUOUS) {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float a = v[2 * i], b = v[2 * i + 1];
                    v[2 * i] = a * cc[i] - b * ss[i];
                    v[2 * i + 1] = b * cc[i] + a * ss[i];
                }
            } else {
                // the partner is the same place of group g ^ 2 (half-split pairs) or g ^ 1 (adjacent pairs)
                const int other = ROPE == 1 ? 2 : 1;
                const bool first = (g & other) == 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float o = __shfl_xor_sync(0xFFFFFFFFu, v[i], other);
                    v[i] = first ? v[i] * cc[i] - o * ss[i] : v[i] * cc[i] + o * ss[i];
                }
            }
        }
        float part_s[J];
#pragma unroll
        for (int j = 0; j < J; ++j) {
            float a = v[0] * qr[j][0];
            a = fmaf(v[1], qr[j][1], a);
            a = fmaf(v[2], qr[j][2], a);
            a = fmaf(v[3], qr[j][3], a);
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 1);
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 2);
            part_s[j] = a;
        }
        if (g == 0) {
            float *dst = scores + (size_t)(t * 8u + (uint32_t)h) * J;
            if (J == 4) atomicAdd(reinterpret_cast<float4 *>(dst), make_float4(part_s[0], part_s[1], part_s[J - 2], part_s[J - 1]));
            else if (J == 2) atomicAdd(reinterpret_cast<float2 *>(dst), make_float2(part_s[0], part_s[J - 1]));
            else atomicAdd(dst, part_s[0]);
        }
    }
    if (bad && st && sl == 0) atomicAdd(&st->bad_codes, bad);
}

// order-preserving map of a float onto unsigned integers (0 is below every float)
__device__ __forceinline__ uint32_t att_ordered(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float att_unordered(uint32_t u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

// Step 2: m[column] = max over the tokens of scale * s[token][column]; columns = 8 J (divides 1024).
__global__ void __launch_bounds__(kAttThreads)
att_max_kernel(const float *__restrict__ scores, int64_t tokens, int columns, float scale, uint32_t *__restrict__ m_ord)
{
    __shared__ float part[kAttThreads];
    const int col = threadIdx.x % columns, rows_per_block = kAttThreads / columns;
    float m = -INFINITY;
    for (int64_t t = (int64_t)blockIdx.x * rows_per_block + threadIdx.x / columns; t < tokens;
         t += (int64_t)gridDim.x * rows_per_block)
        m = fmaxf(m, scale * scores[t * columns + col]);
    part[threadIdx.x] = m;
    __syncthreads();
    if ((int)threadIdx.x < columns) {
        for (int r = 1; r < rows_per_block; ++r) m = fmaxf(m, part[r * columns + threadIdx.x]);
        if (m > -INFINITY) atomicMax(m_ord + threadIdx.x, att_ordered(m));
    }
}

// Step 3.
template <int LAYOUT, int J>
__global__ void __launch_bounds__(kAttThreads, 1)
att_values_kernel(Shape s, const void *__restrict__ codes, const uint16_t *__restrict__ std16, int64_t tokens,
                  const float *__restrict__ cb, const float *__restrict__ scores, const uint32_t *__restrict__ m_ord,
                  float scale, float *__restrict__ out_acc, float *__restrict__ weight_sum, rvq_status *st)
{
    extern __shared__ __align__(128) uint8_t smem[];
    const int parts = gridDim.x / kAttSlices;
    if ((int)blockIdx.x >= parts * kAttSlices) return;
    const int sl = blockIdx.x % kAttSlices, part = blockIdx.x / kAttSlices;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, h = lane >> 2;
    att_fill_table<LAYOUT, 0>(s, cb, sl, reinterpret_cast<float4 *>(smem));
    // exp(scale s - m) = 2^(s * scale log2(e) - m log2(e))
    constexpr float kLog2e = 1.4426950408889634f;
    const float sl2 = scale * kLog2e;
    __shared__ float mneg_s[32];                             // -m log2(e) per query head (read back per token: registers are short)
    if (threadIdx.x < 8 * J) mneg_s[threadIdx.x] = -att_unordered(m_ord[threadIdx.x]) * kLog2e;
    __syncthreads();
    const uint32_t smem_table = (uint32_t)__cvta_generic_to_shared(smem);
    uint32_t bad = 0;
    float acc[J][4], wsum[J];
#pragma unroll
    for (int j = 0; j < J; ++j) { wsum[j] = 0.0f; acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f; }
    const uint32_t T = (uint32_t)tokens, step = (uint32_t)parts * 32u;
    AttRow next;
    att_fetch(s, codes, std16, (uint32_t)part * 32u + (uint32_t)warp, T, lane, next);
    for (uint32_t t = (uint32_t)part * 32u + (uint32_t)warp; t < T; t += step) {
        const AttRow cur = next;
        // this token's scores, asked for before the gather
        float sc[J];
        {
            const float *src = scores + (size_t)(t * 8u + (uint32_t)h) * J;
            if (J == 4) { const float4 f = __ldg(reinterpret_cast<const float4 *>(src)); sc[0] = f.x; sc[1] = f.y; sc[J - 2] = f.z; sc[J - 1] = f.w; }
            else if (J == 2) { const float2 f = __ldg(reinterpret_cast<const float2 *>(src)); sc[0] = f.x; sc[J - 1] = f.y; }
            else sc[0] = __ldg(src);
        }
        att_fetch(s, codes, std16, t + step, T, lane, next);
        float v[4];
        att_gather(cur, (uint32_t)s.K, (uint32_t)lane & 7u, smem_table, v, bad);
        const float sd = __half2float(__ushort_as_half(cur.sd));
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] *= sd;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const float w = exp2f(fmaf(sc[j], sl2, mneg_s[h * J + j]));
            wsum[j] += w;
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[j][i] = fmaf(w, v[i], acc[j][i]);
        }
    }
    // sums over the CTA's warps (a lane is the same (head, group) in all of them), then one
    // reduction per value into global memory; the table's memory is free now
    __syncthreads();
    float *red = reinterpret_cast<float *>(smem);            // [5 J][32 warps][32 lanes]
#pragma unroll
    for (int j = 0; j < J; ++j) {
#pragma unroll
        for (int i = 0; i < 4; ++i) red[((j * 5 + i) * 32 + warp) * 32 + lane] = acc[j][i];
        red[((j * 5 + 4) * 32 + warp) * 32 + lane] = wsum[j];
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < 5 * J * 32; idx += kAttThreads) {
        const int ln = idx & 31, what = idx >> 5, j = what / 5, i = what % 5;
        float a = 0.0f;
        for (int w = 0; w < 32; ++w) a += red[(what * 32 + w) * 32 + ln];
        const int hh = ln >> 2, gg = ln & 3;
        if (i < 4)
            atomicAdd(out_acc + (size_t)(hh * J + j) * 128 + att_channel<LAYOUT>(gg, 4 * sl + i), a);
        else if (sl == 0 && gg == 0)
            atomicAdd(weight_sum + hh * J + j, a);
    }
    if (bad && st && sl == 0) atomicAdd(&st->bad_codes, bad);
}

// Step 4.
__global__ void att_finish_kernel(const float *__restrict__ out_acc, const float *__restrict__ weight_sum, int heads,
                                  float *__restrict__ out)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < heads * 128) out[idx] = out_acc[idx] / weight_sum[idx >> 7];
}

}  // namespace

// (token counts: the kernels index group rows, 32 per token, with 32-bit integers, and step past the end
// by up to two strides of at most 18 * 32 tokens)
constexpr int64_t kAttMaxTokens = (1LL << 26) - 4096;

bool attention_supported(const Shape &sk, const Shape &sv, int kv_heads, int q_heads, int64_t tokens)
{
    auto ok = [](const Shape &s) { return s.dim == 128 && s.gd == 32 && s.R <= 8 && s.K <= kAttMaxK; };
    const int J = kv_heads > 0 ? q_heads / kv_heads : 0;
    return ok(sk) && ok(sv) && kv_heads == 8 && q_heads == kv_heads * J && (J == 1 || J == 2 || J == 4) &&
           tokens <= kAttMaxTokens;
}

size_t attention_workspace_bytes(int64_t tokens, int q_heads)
{
    const size_t scores = ((size_t)tokens * q_heads * 4 + 255) / 256 * 256;
    return scores + 256 /* maxima */ + 256 /* weight sums */ + (size_t)q_heads * 128 * 4;
}

int launch_attention_decode(const Shape &sk, const Shape &sv, const float *q, int q_heads, const void *codes_k,
                            const uint16_t *std_k, const void *codes_v, const uint16_t *std_v, int64_t tokens,
                            const float *cb_k, const float *cb_v, const int32_t *position, const float *cos_sin,
                            int positions, int pairing, float scale, float *out, void *workspace, rvq_status *st,
                            cudaStream_t stream)
{
    const int J = q_heads / 8;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return RVQ_ERR_DEVICE;
    uint8_t *ws = reinterpret_cast<uint8_t *>(workspace);
    const size_t score_bytes = ((size_t)tokens * q_heads * 4 + 255) / 256 * 256;
    float *scores = reinterpret_cast<float *>(ws);
    uint32_t *m_ord = reinterpret_cast<uint32_t *>(ws + score_bytes);
    float *weight_sum = reinterpret_cast<float *>(ws + score_bytes + 256);
    float *out_acc = reinterpret_cast<float *>(ws + score_bytes + 512);
    if (cudaMemsetAsync(ws, 0, score_bytes + 512 + (size_t)q_heads * 128 * 4, stream) != cudaSuccess) return RVQ_ERR_LAUNCH;

    int parts = sms / kAttSlices;
    const int64_t tiles = (tokens + 31) / 32;
    if (parts > tiles) parts = (int)tiles;
    if (parts < 1) parts = 1;
    const int rope = cos_sin ? (pairing == RVQ_ROPE_HALVES ? 1 : 2) : 0;
    int rc = RVQ_OK;
    auto scores_launch = [&](auto kernel) -> int {
        const size_t smem = (size_t)sk.K * 128;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return RVQ_ERR_LAUNCH;
        kernel<<<parts * kAttSlices, kAttThreads, smem, stream>>>(sk, codes_k, std_k, tokens, cb_k, q, position,
                                                                   reinterpret_cast<const float2 *>(cos_sin), positions,
                                                                   scores, st);
        return check_launch();
    };
    auto values_launch = [&](auto kernel) -> int {
        size_t smem = (size_t)sv.K * 128;
        const size_t red = (size_t)5 * J * 32 * 32 * 4;
        if (smem < red) smem = red;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return RVQ_ERR_LAUNCH;
        kernel<<<parts * kAttSlices, kAttThreads, smem, stream>>>(sv, codes_v, std_v, tokens, cb_v, scores, m_ord, scale,
                                                                   out_acc, weight_sum, st);
        return check_launch();
    };
#define RVQ_ATT_S3(LAY, ROPE) (J == 4 ? scores_launch(att_scores_kernel<LAY, ROPE, 4>)                               \
                               : J == 2 ? scores_launch(att_scores_kernel<LAY, ROPE, 2>)                             \
                                        : scores_launch(att_scores_kernel<LAY, ROPE, 1>))
#define RVQ_ATT_S2(LAY) (rope == 0 ? RVQ_ATT_S3(LAY, 0) : rope == 1 ? RVQ_ATT_S3(LAY, 1) : RVQ_ATT_S3(LAY, 2))
    rc = sk.layout == RVQ_GROUP_CONTIGUOUS ? RVQ_ATT_S2(RVQ_GROUP_CONTIGUOUS) : RVQ_ATT_S2(RVQ_GROUP_STRIDED);
#undef RVQ_ATT_S2
#undef RVQ_ATT_S3
    if (rc != RVQ_OK) return rc;
    {
        int blocks = (int)((tokens * q_heads + kAttThreads - 1) / kAttThreads);
        if (blocks > sms * 2) blocks = sms * 2;
        if (blocks < 1) blocks = 1;
        att_max_kernel<<<blocks, kAttThreads, 0, stream>>>(scores, tokens, q_heads, scale, m_ord);
        if ((rc = check_launch()) != RVQ_OK) return rc;
    }
#define RVQ_ATT_V2(LAY) (J == 4 ? values_launch(att_values_kernel<LAY, 4>)                                           \
                         : J == 2 ? values_launch(att_values_kernel<LAY, 2>) : values_launch(att_values_kernel<LAY, 1>))
    rc = sv.layout == RVQ_GROUP_CONTIGUOUS ? RVQ_ATT_V2(RVQ_GROUP_CONTIGUOUS) : RVQ_ATT_V2(RVQ_GROUP_STRIDED);
#undef RVQ_ATT_V2
    if (rc != RVQ_OK) return rc;
    att_finish_kernel<<<(q_heads * 128 + 255) / 256, 256, 0, stream>>>(out_acc, weight_sum, q_heads, out);
    return check_launch();
}

}  // namespace rvq
