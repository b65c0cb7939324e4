// k-means initialisation of the codebooks (Section 3: every codebook starts
// from a k-means run on the first batch), stage after stage on that stage's inputs.
//
// The scaled group rows of the batch are written once to a float32 buffer
// [n][G][32]; stage r then runs Lloyd's iterations on it: the assignment is the
// tensor-core encoder at depth 1 over the buffer (taken raw: no deviation, no
// scaling) with the batch statistics accumulated in the same pass, the update
// moves every centroid to the mean of its rows (a centroid without rows stays).
// After the last iteration the rows are assigned once more and the chosen
// centroids are subtracted in place, which makes the buffer the next stage's input.
#include "prepared.cuh"

namespace rvq {

namespace {

size_t round256(size_t b) { return (b + 255) / 256 * 256; }

// The depth-1 problem of one stage: rows of 32 G float32 values, groups contiguous.
Shape stage_shape(const Shape &s)
{
    Shape t = s;
    t.R = 1; t.dtype = RVQ_F32; t.layout = RVQ_GROUP_CONTIGUOUS; t.bits = 16; t.elem_bytes = 4;
    t.per_vector = t.G;
    t.code_bytes = (t.G * 16 + 31) / 32 * 4;
    t.raw = 1;
    return t;
}

// One thread per group row: z[v][g][i] = x[v][channel(g, i)] / deviation(v)  (Section 2.2).
__global__ void __launch_bounds__(128)
kmeans_scale_kernel(Shape s, const void *__restrict__ x, int64_t n, int64_t stride, float *__restrict__ z, int vpb)
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
    float zr[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) zr[i] = xs[v_local * s.dim + channel_of(s.layout, s.G, 32, g, i)];
    const float dev = block_deviation<32>(zr, part, v_local, s.G, s.dim, s.ddof);
    const bool deg = deviation_is_degenerate(dev);
    if (gv >= n) return;
    float4 *o = reinterpret_cast<float4 *>(z + (gv * s.G + g) * 32);
#pragma unroll
    for (int q = 0; q < 8; ++q)
        o[q] = deg ? make_float4(0.f, 0.f, 0.f, 0.f)
                   : make_float4(zr[4 * q] / dev, zr[4 * q + 1] / dev, zr[4 * q + 2] / dev, zr[4 * q + 3] / dev);
}

// Centroid j starts as the row seed_rows[j] of the stage's input (a row number out of range reads row 0).
__global__ void __launch_bounds__(256)
kmeans_seed_kernel(const float *__restrict__ z, const int64_t *__restrict__ seed_rows, int64_t rows, int K,
                   float *__restrict__ cb)
{
    const int t = blockIdx.x * 256 + threadIdx.x;
    if (t >= K * 32) return;
    int64_t row = seed_rows[t >> 5];
    if (row < 0 || row >= rows) row = 0;
    cb[t] = z[row * 32 + (t & 31)];
}

// Lloyd's update: the mean of the rows of every centroid that has any.
__global__ void __launch_bounds__(256)
kmeans_update_kernel(const uint32_t *__restrict__ cnt, const float *__restrict__ sum, int K, float *__restrict__ cb)
{
    const int t = blockIdx.x * 256 + threadIdx.x;
    if (t >= K * 32) return;
    const uint32_t c = cnt[t >> 5];
    if (c) cb[t] = sum[t] / (float)c;
}

// z[row] -= centroid[code[row]]: the stage's residual becomes the next stage's input (Algorithm 1).
__global__ void __launch_bounds__(256)
kmeans_residual_kernel(float *__restrict__ z, const uint8_t *__restrict__ codes, const float *__restrict__ cb,
                       int64_t rows, int G, int code_bytes, int K)
{
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t >= rows * 8) return;
    const int64_t row = t >> 3;
    const int q = (int)(t & 7);
    const int64_t v = row / G;
    const int g = (int)(row - v * G);
    uint32_t j = *reinterpret_cast<const uint16_t *>(codes + v * code_bytes + g * 2);
    if (j >= (uint32_t)K) j = 0;
    float4 *p = reinterpret_cast<float4 *>(z + row * 32) + q;
    const float4 e = __ldg(reinterpret_cast<const float4 *>(cb + (size_t)j * 32) + q);
    float4 a = *p;
    a.x -= e.x; a.y -= e.y; a.z -= e.z; a.w -= e.w;
    *p = a;
}

struct Carve {
    float *z;
    uint8_t *codes;
    uint8_t *prep;
    uint32_t *cnt;
    float *sum;
    size_t total;
};

Carve carve(const Shape &s, int64_t n, void *ws)
{
    const Shape t = stage_shape(s);
    uint8_t *p = reinterpret_cast<uint8_t *>(ws);
    size_t off = 0;
    Carve c;
    c.z = reinterpret_cast<float *>(p + off); off += round256((size_t)n * s.G * 32 * sizeof(float));
    c.codes = p + off; off += round256((size_t)n * t.code_bytes);
    c.prep = p + off; off += round256(prepared_bytes(t));
    c.cnt = reinterpret_cast<uint32_t *>(p + off); off += round256((size_t)s.K * sizeof(uint32_t));
    c.sum = reinterpret_cast<float *>(p + off); off += round256((size_t)s.K * 32 * sizeof(float));
    c.total = off;
    return c;
}

}  // namespace

size_t kmeans_workspace_bytes(const Shape &s, int64_t n)
{
    if (!encode_tensor_supported(s) || n < 0) return 0;
    return carve(s, n, nullptr).total;
}

int launch_kmeans(const Shape &s, const void *x, int64_t n, int64_t stride, const int64_t *seed_rows,
                  int iterations, float *codebooks, void *prepared, void *workspace, rvq_status *st,
                  cudaStream_t stream)
{
    const Shape t = stage_shape(s);
    const Carve c = carve(s, n, workspace);
    const int64_t rows = n * s.G;
    const int vpb = 128 / s.G;
    {
        const size_t smem = ((size_t)vpb * s.dim + 128) * sizeof(float);
        const int64_t blocks = (n + vpb - 1) / vpb;
        if (cudaFuncSetAttribute(kmeans_scale_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return RVQ_ERR_LAUNCH;
        kmeans_scale_kernel<<<(unsigned)blocks, 128, smem, stream>>>(s, x, n, stride, c.z, vpb);
        int rc = check_launch();
        if (rc != RVQ_OK) return rc;
    }
    const int cells = (s.K * 32 + 255) / 256;
    for (int r = 0; r < s.R; ++r) {
        float *cb = codebooks + (size_t)r * s.K * 32;
        kmeans_seed_kernel<<<cells, 256, 0, stream>>>(c.z, seed_rows + (size_t)r * s.K, rows, s.K, cb);
        int rc = check_launch();
        if (rc != RVQ_OK) return rc;
        for (int it = 0; it <= iterations; ++it) {
            const bool last = it == iterations;          // the last pass only assigns, for the residual
            if (last && r + 1 == s.R) break;
            if ((rc = launch_prepare(t, cb, c.prep, stream)) != RVQ_OK) return rc;
            if (!last &&
                (cudaMemsetAsync(c.cnt, 0, (size_t)s.K * sizeof(uint32_t), stream) != cudaSuccess ||
                 cudaMemsetAsync(c.sum, 0, (size_t)s.K * 32 * sizeof(float), stream) != cudaSuccess))
                return RVQ_ERR_LAUNCH;
            rc = launch_encode_tensor(t, c.z, n, t.dim, cb, c.prep, c.codes, nullptr, st, stream,
                                      last ? nullptr : c.cnt, last ? nullptr : c.sum);
            if (rc != RVQ_OK) return rc;
            if (!last) {
                kmeans_update_kernel<<<cells, 256, 0, stream>>>(c.cnt, c.sum, s.K, cb);
                if ((rc = check_launch()) != RVQ_OK) return rc;
            }
        }
        if (r + 1 < s.R) {
            const int64_t blocks = (rows * 8 + 255) / 256;
            kmeans_residual_kernel<<<(unsigned)blocks, 256, 0, stream>>>(c.z, c.codes, cb, rows, s.G, t.code_bytes, s.K);
            if ((rc = check_launch()) != RVQ_OK) return rc;
        }
    }
    return launch_prepare(s, codebooks, prepared, stream);
}

}  // namespace rvq
