// extern "C" boundary of the RVQ library: argument checks on the host, then
// dispatch to the kernels.  No allocation, no synchronisation.  Process-wide
// state: the launch counter below, and (in ema.cu) the per-device address of
// the built-in scratch array of rvq_ema_update_static.
#include "prepared.cuh"
#include "rvq_selftest.h"

#include <atomic>

namespace rvq {

static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

static int ceil_log2(int k)
{
    int b = 0;
    while ((1 << b) < k) ++b;
    return b < 1 ? 1 : b;
}

int make_shape(const rvq_config *c, Shape *s)
{
    if (!c) return RVQ_ERR_BADARG;
    if (c->group_dim != 8 && c->group_dim != 16 && c->group_dim != 32 && c->group_dim != 64)
        return RVQ_ERR_UNSUPPORTED;
    if (c->dim < c->group_dim || c->dim > 1024 || c->dim % c->group_dim) return RVQ_ERR_BADARG;
    if (c->layout != RVQ_GROUP_CONTIGUOUS && c->layout != RVQ_GROUP_STRIDED) return RVQ_ERR_BADARG;
    if (c->depth < 1 || c->depth > 16) return RVQ_ERR_BADARG;
    if (c->codebook_size < 2 || c->codebook_size > 65536) return RVQ_ERR_BADARG;
    if (c->code_bits != 16 && c->code_bits != ceil_log2(c->codebook_size)) return RVQ_ERR_BADARG;
    if (c->x_dtype < RVQ_F32 || c->x_dtype > RVQ_F16) return RVQ_ERR_BADARG;
    if (c->std_ddof != 0 && c->std_ddof != 1) return RVQ_ERR_BADARG;
    s->dim = c->dim; s->gd = c->group_dim; s->G = c->dim / c->group_dim; s->layout = c->layout;
    s->R = c->depth; s->K = c->codebook_size; s->bits = c->code_bits; s->dtype = c->x_dtype;
    s->ddof = c->std_ddof;
    if (s->G > 128 || s->dim - s->ddof <= 0) return RVQ_ERR_UNSUPPORTED;
    s->per_vector = s->G * s->R;
    s->code_bytes = (s->per_vector * s->bits + 31) / 32 * 4;
    s->elem_bytes = c->x_dtype == RVQ_F32 ? 4 : 2;
    s->raw = 0;
    return RVQ_OK;
}

static int check_rows(const Shape &s, const void *p, int64_t n, int64_t stride)
{
    if (n < 0 || stride < s.dim) return RVQ_ERR_BADARG;
    if (n > 0 && !p) return RVQ_ERR_BADARG;
    if (!aligned16(p) || (stride * s.elem_bytes) % 16) return RVQ_ERR_ALIGN;
    return RVQ_OK;
}

}  // namespace rvq

using namespace rvq;

extern "C" {

const char *rvq_status_string(int code)
{
    switch (code) {
    case RVQ_OK: return "ok";
    case RVQ_ERR_BADARG: return "bad argument";
    case RVQ_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case RVQ_ERR_UNSUPPORTED: return "unsupported shape";
    case RVQ_ERR_WORKSPACE: return "workspace too small";
    case RVQ_ERR_LAUNCH: return "CUDA launch failed";
    case RVQ_ERR_DEVICE: return "no sm_100 device";
    case RVQ_ERR_STATIC_LIMIT: return "shape needs more scratch than the library's built-in array holds";
    default: return "unknown error";
    }
}

int rvq_version(void) { return 1000; }

uint64_t rvq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t rvq_code_bytes(const rvq_config *cfg)
{
    Shape s;
    return make_shape(cfg, &s) == RVQ_OK ? (size_t)s.code_bytes : 0;
}

size_t rvq_prepared_bytes(const rvq_config *cfg)
{
    Shape s;
    return make_shape(cfg, &s) == RVQ_OK ? prepared_bytes(s) : 0;
}

int rvq_prepare_codebooks(const rvq_config *cfg, const float *codebooks, void *prepared, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if (!codebooks || !prepared) return RVQ_ERR_BADARG;
    if (!aligned16(codebooks) || !aligned256(prepared)) return RVQ_ERR_ALIGN;
    return launch_prepare(s, codebooks, prepared, (cudaStream_t)stream);
}

size_t rvq_workspace_bytes(const rvq_config *cfg, int64_t n)
{
    Shape s;
    (void)n;
    return make_shape(cfg, &s) == RVQ_OK ? ema_workspace_bytes(s) : 0;
}

static int encode_common(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                         const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
                         float *stage_energy, rvq_status *status, void *stream, bool allow_tensor,
                         uint32_t *stat_cnt = nullptr, float *stat_sum = nullptr)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if ((rc = check_rows(s, x, n, x_row_stride)) != RVQ_OK) return rc;
    if (!codebooks || !prepared || (n > 0 && (!codes || !std_f16))) return RVQ_ERR_BADARG;
    if (!aligned16(codebooks) || !aligned16(codes) || !aligned256(prepared)) return RVQ_ERR_ALIGN;
    if (stage_energy && cudaMemsetAsync(stage_energy, 0, (size_t)s.R * sizeof(float), (cudaStream_t)stream) != cudaSuccess)
        return RVQ_ERR_LAUNCH;
    if (allow_tensor && encode_tensor_supported(s))
        return launch_encode_tensor(s, x, n, x_row_stride, codebooks, prepared, codes, std_f16, status,
                                    (cudaStream_t)stream, stat_cnt, stat_sum, stage_energy);
    return launch_encode_scalar(s, x, n, x_row_stride, codebooks, codes, std_f16, status, (cudaStream_t)stream,
                                stage_energy);
}

int rvq_encode(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
               const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
               float *stage_energy, void *workspace, size_t workspace_bytes, rvq_status *status, void *stream)
{
    (void)workspace; (void)workspace_bytes;
    return encode_common(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, stage_energy, status, stream, true);
}

int rvq_encode_stats(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                     const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
                     float *stage_energy, float *batch_count, float *batch_sum, void *workspace,
                     size_t workspace_bytes, rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if (!batch_count || !batch_sum || !workspace) return RVQ_ERR_BADARG;
    if (!aligned16(batch_sum) || !aligned256(workspace)) return RVQ_ERR_ALIGN;
    if (workspace_bytes < ema_stats_scratch_bytes(s)) return RVQ_ERR_WORKSPACE;
    if (!encode_tensor_supported(s)) {
        // shapes without the fused kernel: encode, then the separate statistics pass
        rc = encode_common(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, stage_energy, status, stream, true);
        if (rc != RVQ_OK) return rc;
        return launch_ema_stats(s, x, n, x_row_stride, codes, codebooks, batch_count, batch_sum, workspace,
                                status, (cudaStream_t)stream);
    }
    if ((rc = check_rows(s, x, n, x_row_stride)) != RVQ_OK) return rc;
    if (!codebooks || !prepared || (n > 0 && (!codes || !std_f16))) return RVQ_ERR_BADARG;
    if (!aligned16(codebooks) || !aligned16(codes) || !aligned256(prepared)) return RVQ_ERR_ALIGN;
    uint32_t *cnt = reinterpret_cast<uint32_t *>(workspace);
    const int bins = s.R * s.K;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(cnt, 0, (size_t)bins * sizeof(uint32_t), st) != cudaSuccess ||
        cudaMemsetAsync(batch_sum, 0, (size_t)bins * s.gd * sizeof(float), st) != cudaSuccess)
        return RVQ_ERR_LAUNCH;
    rc = encode_common(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, stage_energy, status, stream, true,
                       cnt, batch_sum);
    if (rc != RVQ_OK) return rc;
    return launch_stats_finish(s, cnt, codebooks, batch_sum, batch_count, encode_tensor_deferred_stages(s), st);
}

int rvq_selftest_encode_timeout(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                                const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
                                uint32_t wait_polls, rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if ((rc = check_rows(s, x, n, x_row_stride)) != RVQ_OK) return rc;
    if (!codebooks || !prepared || !status || (n > 0 && (!codes || !std_f16))) return RVQ_ERR_BADARG;
    if (!aligned16(codebooks) || !aligned16(codes) || !aligned256(prepared)) return RVQ_ERR_ALIGN;
    if (!encode_tensor_supported(s) || wait_polls < 1024u) return RVQ_ERR_UNSUPPORTED;
    return launch_encode_tensor(s, x, n, x_row_stride, codebooks, prepared, codes, std_f16, status,
                                (cudaStream_t)stream, nullptr, nullptr, nullptr, wait_polls, 1);
}

int rvq_encode_exact(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                     const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
                     float *stage_energy, rvq_status *status, void *stream)
{
    return encode_common(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, stage_energy, status, stream, false);
}

int rvq_decode(const rvq_config *cfg, const void *codes, const uint16_t *std_f16, int64_t n,
               const float *codebooks, const void *prepared, void *x_out, int64_t out_row_stride,
               rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if ((rc = check_rows(s, x_out, n, out_row_stride)) != RVQ_OK) return rc;
    if (!codebooks || !prepared || (n > 0 && (!codes || !std_f16))) return RVQ_ERR_BADARG;
    if (!aligned16(codebooks) || !aligned16(codes) || !aligned256(prepared)) return RVQ_ERR_ALIGN;
    if (decode_sliced_supported(s))
        return launch_decode_sliced(s, codes, std_f16, n, codebooks, prepared, x_out, out_row_stride, status, (cudaStream_t)stream);
    return launch_decode_gather(s, codes, std_f16, n, codebooks, x_out, out_row_stride, status, (cudaStream_t)stream);
}

int rvq_rope_table(int32_t dim, double base, int32_t positions, float *cos_sin, void *stream)
{
    if (dim < 2 || dim > 1024 || (dim & 1) || !(base > 1.0) || positions < 0 || (positions > 0 && !cos_sin))
        return RVQ_ERR_BADARG;
    if (!aligned16(cos_sin)) return RVQ_ERR_ALIGN;
    return launch_rope_table(dim, base, positions, cos_sin, (cudaStream_t)stream);
}

int rvq_decode_rope(const rvq_config *cfg, const void *codes, const uint16_t *std_f16, int64_t n,
                    const float *codebooks, const void *prepared, const int32_t *position,
                    int32_t vectors_per_position,
                    const float *cos_sin, int32_t positions, int32_t pairing, void *x_out,
                    int64_t out_row_stride, rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if ((rc = check_rows(s, x_out, n, out_row_stride)) != RVQ_OK) return rc;
    if (!codebooks || (n > 0 && (!codes || !std_f16 || !position || !cos_sin))) return RVQ_ERR_BADARG;
    if (vectors_per_position < 1 || positions < 1 || (pairing != RVQ_ROPE_HALVES && pairing != RVQ_ROPE_ADJACENT))
        return RVQ_ERR_BADARG;
    if (s.dim & 1) return RVQ_ERR_UNSUPPORTED;
    if (!aligned16(codebooks) || !aligned16(codes) || !aligned16(cos_sin) || !aligned256(prepared)) return RVQ_ERR_ALIGN;
    return launch_decode_rope(s, codes, std_f16, n, codebooks, prepared, position, vectors_per_position, cos_sin, positions,
                              pairing, x_out, out_row_stride, status, (cudaStream_t)stream);
}

size_t rvq_attention_workspace_bytes(int64_t tokens, int32_t q_heads)
{
    if (tokens < 1 || q_heads < 1 || q_heads > 32) return 0;
    return attention_workspace_bytes(tokens, q_heads);
}

int rvq_attention_decode(const rvq_config *cfg_k, const rvq_config *cfg_v, const float *q, int32_t q_heads,
                         const void *codes_k, const uint16_t *std_k, const void *codes_v, const uint16_t *std_v,
                         int64_t tokens, int32_t kv_heads, const float *codebooks_k, const float *codebooks_v,
                         const int32_t *position, const float *cos_sin, int32_t positions, int32_t pairing,
                         float scale, float *out, void *workspace, size_t workspace_bytes, rvq_status *status,
                         void *stream)
{
    Shape sk, sv;
    int rc = make_shape(cfg_k, &sk);
    if (rc != RVQ_OK) return rc;
    if ((rc = make_shape(cfg_v, &sv)) != RVQ_OK) return rc;
    if (!q || !codes_k || !std_k || !codes_v || !std_v || !codebooks_k || !codebooks_v || !out || !workspace)
        return RVQ_ERR_BADARG;
    if (tokens < 1 || q_heads < 1 || kv_heads < 1 || !(scale == scale)) return RVQ_ERR_BADARG;
    if (cos_sin && (positions < 1 || (pairing != RVQ_ROPE_HALVES && pairing != RVQ_ROPE_ADJACENT))) return RVQ_ERR_BADARG;
    if (!attention_supported(sk, sv, kv_heads, q_heads, tokens)) return RVQ_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(codes_k) || !aligned16(codes_v) || !aligned16(codebooks_k) || !aligned16(codebooks_v) ||
        !aligned16(cos_sin) || !aligned16(out) || !aligned256(workspace))
        return RVQ_ERR_ALIGN;
    if (workspace_bytes < attention_workspace_bytes(tokens, q_heads)) return RVQ_ERR_WORKSPACE;
    return launch_attention_decode(sk, sv, q, q_heads, codes_k, std_k, codes_v, std_v, tokens, codebooks_k, codebooks_v,
                                   position, cos_sin, positions, pairing, scale, out, workspace, status,
                                   (cudaStream_t)stream);
}

static int check_ema_common(const Shape &s, const void *x, int64_t n, int64_t stride, const void *codes,
                            const float *codebooks)
{
    int rc = check_rows(s, x, n, stride);
    if (rc != RVQ_OK) return rc;
    if (!codebooks || (n > 0 && !codes)) return RVQ_ERR_BADARG;
    if (!aligned16(codebooks) || !aligned16(codes)) return RVQ_ERR_ALIGN;
    return RVQ_OK;
}

int rvq_ema_stats(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                  const void *codes, const float *codebooks, float *batch_count, float *batch_sum,
                  void *workspace, size_t workspace_bytes, rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if ((rc = check_ema_common(s, x, n, x_row_stride, codes, codebooks)) != RVQ_OK) return rc;
    if (!batch_count || !batch_sum || !workspace) return RVQ_ERR_BADARG;
    if (!aligned16(batch_sum) || !aligned256(workspace)) return RVQ_ERR_ALIGN;
    if (workspace_bytes < ema_stats_scratch_bytes(s)) return RVQ_ERR_WORKSPACE;
    return launch_ema_stats(s, x, n, x_row_stride, codes, codebooks, batch_count, batch_sum, workspace,
                            status, (cudaStream_t)stream);
}

int rvq_ema_apply(const rvq_config *cfg, const float *batch_count, const float *batch_sum,
                  float *codebooks, float *ema_count, float *ema_sum, float decay, float eps,
                  void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if (!batch_count || !batch_sum || !codebooks || !ema_count || !ema_sum) return RVQ_ERR_BADARG;
    if (!(decay >= 0.0f && decay <= 1.0f) || !(eps >= 0.0f)) return RVQ_ERR_BADARG;
    return launch_ema_apply(s, batch_count, batch_sum, codebooks, ema_count, ema_sum, decay, eps,
                            (cudaStream_t)stream);
}

int rvq_ema_update(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                   const void *codes, float *codebooks, float *ema_count, float *ema_sum,
                   float *batch_count, float decay, float eps, void *workspace,
                   size_t workspace_bytes, rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if ((rc = check_ema_common(s, x, n, x_row_stride, codes, codebooks)) != RVQ_OK) return rc;
    if (!ema_count || !ema_sum || !workspace) return RVQ_ERR_BADARG;
    if (!(decay >= 0.0f && decay <= 1.0f) || !(eps >= 0.0f)) return RVQ_ERR_BADARG;
    if (!aligned16(ema_sum) || !aligned256(workspace)) return RVQ_ERR_ALIGN;
    if (workspace_bytes < ema_workspace_bytes(s)) return RVQ_ERR_WORKSPACE;
    uint8_t *ws = reinterpret_cast<uint8_t *>(workspace);
    float *bc = reinterpret_cast<float *>(ws + ema_stats_scratch_bytes(s));
    float *bs = reinterpret_cast<float *>(ws + ema_stats_scratch_bytes(s) +
                                          ((size_t)s.R * s.K * sizeof(float) + 255) / 256 * 256);
    rc = launch_ema_stats(s, x, n, x_row_stride, codes, codebooks, bc, bs, workspace, status, (cudaStream_t)stream);
    if (rc != RVQ_OK) return rc;
    if (batch_count &&
        cudaMemcpyAsync(batch_count, bc, (size_t)s.R * s.K * sizeof(float), cudaMemcpyDeviceToDevice,
                        (cudaStream_t)stream) != cudaSuccess)
        return RVQ_ERR_LAUNCH;
    return launch_ema_apply(s, bc, bs, codebooks, ema_count, ema_sum, decay, eps, (cudaStream_t)stream);
}

int rvq_learn_step(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                   float *codebooks, void *prepared, float *ema_count, float *ema_sum, void *codes,
                   uint16_t *std_f16, float *stage_energy, float decay, float eps, void *workspace,
                   size_t workspace_bytes, rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if (!ema_count || !ema_sum || !workspace || !codebooks || !prepared) return RVQ_ERR_BADARG;
    if (!(decay >= 0.0f && decay <= 1.0f) || !(eps >= 0.0f)) return RVQ_ERR_BADARG;
    if (!aligned16(ema_sum) || !aligned256(workspace)) return RVQ_ERR_ALIGN;
    if (workspace_bytes < ema_workspace_bytes(s)) return RVQ_ERR_WORKSPACE;
    // same carving as rvq_ema_update: counts | batch counts | batch sums
    uint8_t *ws = reinterpret_cast<uint8_t *>(workspace);
    float *bc = reinterpret_cast<float *>(ws + ema_stats_scratch_bytes(s));
    float *bs = reinterpret_cast<float *>(ws + ema_stats_scratch_bytes(s) +
                                          ((size_t)s.R * s.K * sizeof(float) + 255) / 256 * 256);
    rc = rvq_encode_stats(cfg, x, n, x_row_stride, codebooks, prepared, codes, std_f16, stage_energy, bc, bs,
                          workspace, workspace_bytes, status, stream);
    if (rc != RVQ_OK) return rc;
    rc = launch_ema_apply(s, bc, bs, codebooks, ema_count, ema_sum, decay, eps, (cudaStream_t)stream);
    if (rc != RVQ_OK) return rc;
    return launch_prepare(s, codebooks, prepared, (cudaStream_t)stream);
}

size_t rvq_kmeans_workspace_bytes(const rvq_config *cfg, int64_t n)
{
    Shape s;
    return make_shape(cfg, &s) == RVQ_OK ? kmeans_workspace_bytes(s, n) : 0;
}

int rvq_kmeans_init(const rvq_config *cfg, const void *x, int64_t n, int64_t x_row_stride,
                    const int64_t *seed_rows, int32_t iterations, float *codebooks, void *prepared,
                    void *workspace, size_t workspace_bytes, rvq_status *status, void *stream)
{
    Shape s;
    int rc = make_shape(cfg, &s);
    if (rc != RVQ_OK) return rc;
    if (!encode_tensor_supported(s)) return RVQ_ERR_UNSUPPORTED;
    if ((rc = check_rows(s, x, n, x_row_stride)) != RVQ_OK) return rc;
    if (n < 1 || !seed_rows || !codebooks || !prepared || !workspace) return RVQ_ERR_BADARG;
    if (iterations < 0 || iterations > 1000) return RVQ_ERR_BADARG;
    if (!aligned16(codebooks) || !aligned256(prepared) || !aligned256(workspace)) return RVQ_ERR_ALIGN;
    if (workspace_bytes < kmeans_workspace_bytes(s, n)) return RVQ_ERR_WORKSPACE;
    return launch_kmeans(s, x, n, x_row_stride, seed_rows, iterations, codebooks, prepared, workspace, status,
                         (cudaStream_t)stream);
}

}  // extern "C"
