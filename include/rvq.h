/*
 * rvq.h -- C ABI of the B200 residual-vector-quantization KV-cache library.
 *
 * The library implements the data-parallel part of "Residual vector
 * quantization for KV cache compression in large language model":
 *   - encode  (Section 2.2 + Algorithm 1): scale a head vector by its standard
 *     deviation, split its channels into groups (Section 3.1: contiguous, or
 *     channels d/d^ apart), run R greedy stages of nearest-code search and
 *     residual subtraction against one shared set of R codebooks;
 *   - decode  (Section 2.2, last sentence): sum the R chosen codes per group,
 *     un-group, multiply by the stored standard deviation (Section 3.2: kept in
 *     half precision);
 *   - EMA codebook update (Section 3: exponential moving average, decay 0.99).
 *
 * Conventions shared by every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller unless its
 *     comment says "host".  The library never allocates, frees or keeps a
 *     pointer after the call returns.  Work is enqueued on `stream` and the
 *     call returns without synchronising.
 *   - n     number of head vectors (tokens x heads); dim channels each.
 *     G = dim / group_dim groups per vector, R = depth, K = codebook_size.
 *   - codebooks: float32 [R][K][group_dim], row-major, 16-byte aligned.
 *   - x / x_out: n rows of `dim` contiguous elements of `x_dtype`; row v starts
 *     at element v * row_stride.  16-byte aligned base, row_stride * element
 *     size a multiple of 16 bytes.
 *   - codes: code_bits == 16: uint16 [n][G][R].  Otherwise code_bits must be
 *     ceil(log2 K) and each head vector is a little-endian bit stream, code
 *     number g*R+r at bit offset code_bits*(g*R+r), least significant bit
 *     first, padded to a multiple of 4 bytes (rvq_code_bytes()).
 *   - std: uint16 [n] holding IEEE binary16 bit patterns.
 *   - Return value: RVQ_OK or a negative rvq_error.  Argument errors are
 *     detected on the host before anything is launched.  Conditions found on
 *     the device are counted in the optional `rvq_status` block (device memory,
 *     zeroed by the caller, read by the caller after the stream has drained).
 */
#ifndef RVQ_H
#define RVQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { RVQ_F32 = 0, RVQ_BF16 = 1, RVQ_F16 = 2 } rvq_dtype;
typedef enum { RVQ_GROUP_CONTIGUOUS = 0, RVQ_GROUP_STRIDED = 1 } rvq_layout;

typedef enum {
    RVQ_OK = 0,
    RVQ_ERR_BADARG = -1,       /* null pointer, negative size, value out of range   */
    RVQ_ERR_ALIGN = -2,        /* pointer or stride not 16-byte aligned              */
    RVQ_ERR_UNSUPPORTED = -3,  /* shape outside what the kernels handle              */
    RVQ_ERR_WORKSPACE = -4,    /* workspace smaller than rvq_workspace_bytes()       */
    RVQ_ERR_LAUNCH = -5,       /* the CUDA runtime refused a launch or a copy        */
    RVQ_ERR_DEVICE = -6,       /* not an sm_100 device, or no device                 */
    RVQ_ERR_STATIC_LIMIT = -7  /* shape needs more than the library's built-in scratch */
} rvq_error;

/* Shape of one quantizer (Section 3: default dim 128, group_dim 32, depth 8,
 * codebook_size 2048). */
typedef struct rvq_config {
    int32_t dim;            /* channels per head vector, <= 1024, multiple of group_dim */
    int32_t group_dim;      /* d^: 8, 16, 32 or 64                                      */
    int32_t layout;         /* rvq_layout (Section 3.1)                                 */
    int32_t depth;          /* R, 1..16 (the paper's K)                                 */
    int32_t codebook_size;  /* K, 2..65536 (the paper's |C_i|)                          */
    int32_t code_bits;      /* 16, or ceil(log2 K) for the packed form (Section 3.2)    */
    int32_t x_dtype;        /* rvq_dtype of vectors in (encode, EMA) and out (decode)   */
    int32_t std_ddof;       /* 0: population deviation (default); 1: sample deviation   */
} rvq_config;

/* Device-side counters.  Zero the block before a call, read it after the
 * stream has drained.  Counters accumulate over calls. */
typedef struct rvq_status {
    uint32_t degenerate_vectors;  /* zero or non-finite deviation: codes 0, std 0         */
    uint32_t std_out_of_half;     /* deviation overflowed / underflowed binary16          */
    uint32_t rescored_rows;       /* (row, stage) pairs sent through the exact re-scoring */
    uint32_t exhaustive_rows;     /* (row, stage) pairs that fell back to a full scan     */
    uint32_t wait_timeouts;       /* bounded waits that gave up (result invalid if != 0)  */
    uint32_t bad_codes;           /* decode / EMA met a code >= K (treated as code 0)     */
    uint32_t reserved[2];
} rvq_status;

/* Text for a return value (host pointer to a static string). */
const char *rvq_status_string(int code);

/* Library version, major * 1000 + minor. */
int rvq_version(void);

/* Diagnostic: number of kernels this library has launched in this process so
 * far.  (Process-wide state of the library: this counter, and the per-device
 * address of the built-in scratch array that rvq_ema_update_static resolves on
 * its first call.) */
uint64_t rvq_launch_count(void);

/* Bytes of one head vector's codes in the configured storage form
 * (Section 3.2: G*R indices of code_bits bits).  0 on a bad config. */
size_t rvq_code_bytes(const rvq_config *cfg /* host */);

/* Size of the prepared-codebook block for this shape. 0 on a bad config. */
size_t rvq_prepared_bytes(const rvq_config *cfg /* host */);

/*
 * Derive, from the float32 codebooks, everything the kernels read instead of
 * them: half-precision copies in the tensor-core operand layout with their
 * squared norms and rounding-error bounds (Algorithm 1's argmin, expanded as
 * ||e||^2 - 2 z.e), and the fixed-point channel-sliced tables of the decoder.
 * `prepared` (device, 256-byte aligned, rvq_prepared_bytes() bytes) is
 * overwritten.  Must be called again after every change of the codebooks,
 * on the same stream or after synchronising.
 */
int rvq_prepare_codebooks(const rvq_config *cfg /* host */, const float *codebooks,
                          void *prepared, void *stream /* cudaStream_t */);

/* Scratch bytes rvq_encode / rvq_ema_stats / rvq_ema_update need for n head vectors. */
size_t rvq_workspace_bytes(const rvq_config *cfg /* host */, int64_t n);

/*
 * Encode (Section 2.2, Algorithm 1).  For each of the n head vectors: deviation
 * s over its dim channels (x is not centred), z = x / s, grouping, then for
 * r = 0..R-1: j = argmin_j ||z_r - C_r[j]||^2 under exact squared Euclidean
 * distance (lowest index on ties), z_{r+1} = z_r - C_r[j].
 *   x            in   n rows of x_dtype
 *   codebooks    in   float32 [R][K][group_dim]
 *   prepared     in   block written by rvq_prepare_codebooks for these codebooks
 *   codes        out  see "codes" above; rvq_code_bytes() * n bytes
 *   std_f16      out  binary16 rounding of s (the scaling itself uses s unrounded)
 *   stage_energy out  optional (may be NULL): float32 [R], overwritten; entry r is the sum over
 *                     all groups of all n head vectors of ||z_{r+1}||^2, the squared norm of the
 *                     residual that stage r leaves, in scaled units (after the division by s).
 *                     Entry R-1 is the quantization error of the batch: the quantity Section 3
 *                     watches while the codebooks are learnt.  Float32 atomics: the order of
 *                     the additions, and so the last bits, vary from call to call.
 *   workspace         rvq_workspace_bytes(cfg, n) bytes, 256-byte aligned; may be
 *                     NULL when that size is 0
 *   status            optional counters (may be NULL)
 * A vector whose deviation is zero or not finite gets codes 0 and std 0.
 */
int rvq_encode(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
               const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
               float *stage_energy, void *workspace, size_t workspace_bytes, rvq_status *status,
               void *stream /* cudaStream_t */);

/*
 * Encode and, in the same pass, the EMA statistics of this batch (Section 3:
 * the codebooks are learnt from the encoder's own assignments, batch after
 * batch).  Results are those of rvq_encode followed by rvq_ema_stats on the
 * codes it produced: the residual entering every stage is already in registers
 * when its code is chosen, so x is not read and re-scaled a second time.
 *   stage_energy out  optional [R], as under rvq_encode
 *   batch_count  out  float32 [R][K]             (overwritten)
 *   batch_sum    out  float32 [R][K][group_dim]  (overwritten; 16-byte aligned)
 *   workspace         rvq_workspace_bytes(cfg, n) bytes, 256-byte aligned
 * Follow with rvq_ema_apply (after summing over devices, if several).
 */
int rvq_encode_stats(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
                     const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
                     float *stage_energy, float *batch_count, float *batch_sum, void *workspace,
                     size_t workspace_bytes, rvq_status *status, void *stream /* cudaStream_t */);

/*
 * The same encode computed entirely in float32 on the CUDA cores (every
 * distance in the direct form sum((z - e)^2), no tensor cores, no prepared
 * operands).  Same arguments and results as rvq_encode; an order of magnitude
 * slower.  It serves shapes the tensor-core kernel does not cover and is the
 * on-device cross-check of rvq_encode: both emit identical codes.
 */
int rvq_encode_exact(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
                     const float *codebooks, const void *prepared, void *codes, uint16_t *std_f16,
                     float *stage_energy, rvq_status *status, void *stream /* cudaStream_t */);

/*
 * Decode (Section 2.2, last sentence; Section 3.2).  For every head vector and
 * channel c = channel(g, i): x_out[c] = std * sum_r C_r[code[g][r]][i], summed
 * in float32 and rounded once to x_dtype.  For groups of 32 (a power-of-two number
 * of them) with depth <= 8 the codebook entries are read from shared-memory tables: float32
 * copies (up to 3584 codes per stage) or, for 16-bit outputs and up to 3072
 * codes, 16-bit levels of each stage's value range kept in the prepared block.
 * With the levels the sum before the multiplication by std is within
 * err <= 1.04 * sum_r (max C_r - min C_r) * 2^-17 of the float32 one (levels of
 * each stage's own range), or within 4.1 * sum_r (max C_r - min C_r) * 2^-17 (levels
 * on a unit shared by the stages of one parity, which a decoder adds as packed
 * integers; four groups at depth 8).  The call looks at a sample of the deviations
 * and takes the coarsest table that keeps std * err below 0.9e-3, or the float32
 * tables; a single head vector whose std would still make std * err exceed 0.9e-3
 * gets the float32 sum instead, so the value before the final rounding is always
 * within 1e-3 of the exact one.  Other shapes gather the float32 codebooks from
 * global memory.
 *   codes, std_f16  in   as produced by rvq_encode
 *   x_out           out  n rows of x_dtype, row v at element v * out_row_stride
 * A code >= K is read as code 0 and counted in status->bad_codes.
 */
int rvq_decode(const rvq_config *cfg /* host */, const void *codes, const uint16_t *std_f16,
               int64_t n, const float *codebooks, const void *prepared, void *x_out,
               int64_t out_row_stride, rvq_status *status, void *stream /* cudaStream_t */);

/*
 * Decode followed by the rotary position embedding (Section 3: keys are
 * quantized before the rotation, so a key read back from the cache still needs
 * it; done here it costs no second pass over the keys).  With x^ the decoded
 * head vector in float32 (as under rvq_decode, before rounding), p its position
 * and (c_k, s_k) = cos_sin[p][k] for pair k:
 *   pairing RVQ_ROPE_HALVES    (a, b) = (x^[k], x^[k + dim/2])   (Llama checkpoints)
 *   pairing RVQ_ROPE_ADJACENT  (a, b) = (x^[2k], x^[2k + 1])     (RoFormer)
 *   a' = a c_k - b s_k ,  b' = b c_k + a s_k ,  rounded once to x_dtype.
 *   position              in  device int32: head vector v sits at position[v / vectors_per_position]
 *                             (vectors_per_position = number of KV heads for [token][head][dim] rows);
 *                             values outside [0, positions) are clamped into it
 *   cos_sin               in  device float32 [positions][dim/2][2], 16-byte aligned, e.g. from
 *                             rvq_rope_table
 *   prepared              in  block of rvq_prepare_codebooks for these codebooks, or NULL
 * Two or more groups of 32 (a power-of-two number) with depth <= 8: up to 3584 codes per stage float32
 * shared-memory tables (exact float32 sums); with 16-bit outputs and a prepared block also
 * the level tables described under rvq_decode (dim 128 at depth 8 with up to 1536 codes:
 * both kinds of level table, 8-channel slices, one launch; 1537..3072 codes: the per-stage
 * levels), chosen when the deviations are moderate (a head vector whose std would make
 * std * err exceed 0.6e-3 gets float32 sums, so the rotated value before the final
 * rounding stays within 1e-3 of the exact one).  Other shapes gather from global memory.
 */
enum { RVQ_ROPE_HALVES = 0, RVQ_ROPE_ADJACENT = 1 };
int rvq_decode_rope(const rvq_config *cfg /* host */, const void *codes, const uint16_t *std_f16,
                    int64_t n, const float *codebooks, const void *prepared,
                    const int32_t *position, int32_t vectors_per_position, const float *cos_sin, int32_t positions,
                    int32_t pairing, void *x_out, int64_t out_row_stride, rvq_status *status,
                    void *stream /* cudaStream_t */);

/* cos_sin[p][k] = (cos, sin)(p * base^(-2k/dim)) for p < positions, k < dim/2, evaluated in
 * double precision and rounded to float32 (the angles reach 1e5 radians at long context). */
int rvq_rope_table(int32_t dim, double base, int32_t positions, float *cos_sin /* device */,
                   void *stream /* cudaStream_t */);

/*
 * Attention of one new token over a compressed cache, without the decoded keys
 * and values ever reaching global memory (Section 1: loading the cache is what
 * bounds decoding at long context; Section 3: keys are quantized before the rotary
 * embedding, so they are rotated as they are read; Section 2.2: a cached vector is
 * std * sum of its codewords).  The paper gives no formula for this step; it is the
 * scaled dot-product attention of the models it quantizes.  Cache rows are
 * [token][kv head] (row t * kv_heads + h); query head i reads kv head
 * i / (q_heads / kv_heads).  With k^_t, v^_t the decoded head vectors of token t
 * (float32 sums, keys rotated as under rvq_decode_rope with pairing and cos_sin):
 *   s_t = scale * q_i . k^_t ;  w = softmax_t(s) ;  out_i = sum_t w_t v^_t.
 *   cfg_k, cfg_v   in   host: the two quantizers (dim 128, groups of 32, depth <= 8,
 *                       at most 1792 codes per stage; layouts and code widths may differ;
 *                       x_dtype is not used)
 *   q              in   device float32 [q_heads][128], already rotated to its own position
 *   codes_k, std_k, codes_v, std_v   in   as produced by rvq_encode, tokens * kv_heads rows
 *   tokens         in   1 .. 2^26 - 4096
 *   kv_heads       in   8;  q_heads 8, 16 or 32
 *   position       in   device int32 [tokens], or NULL: token t sits at position t
 *                       (values outside [0, positions) are clamped into it)
 *   cos_sin        in   device float32 [positions][64][2] (rvq_rope_table), or NULL:
 *                       the keys are used as stored
 *   out            out  device float32 [q_heads][128]
 *   workspace           rvq_attention_workspace_bytes(tokens, q_heads) bytes, 256-byte aligned
 * Arithmetic: float32 codeword tables in shared memory (exact float32 sums), float32
 * dot products and weights; the order of the float32 sums over tokens and channel
 * slices is not fixed (reductions in global memory).  Codes >= K are read as code 0
 * and counted in status->bad_codes.  Other shapes: RVQ_ERR_UNSUPPORTED.
 */
size_t rvq_attention_workspace_bytes(int64_t tokens, int32_t q_heads);
int rvq_attention_decode(const rvq_config *cfg_k /* host */, const rvq_config *cfg_v /* host */,
                         const float *q, int32_t q_heads, const void *codes_k, const uint16_t *std_k,
                         const void *codes_v, const uint16_t *std_v, int64_t tokens, int32_t kv_heads,
                         const float *codebooks_k, const float *codebooks_v, const int32_t *position,
                         const float *cos_sin, int32_t positions, int32_t pairing, float scale,
                         float *out, void *workspace, size_t workspace_bytes, rvq_status *status,
                         void *stream /* cudaStream_t */);

/*
 * One EMA codebook update (Section 3: the codebooks follow an exponential moving
 * average with decay 0.99; Section 2.1: EMA in place of the
 * codebook loss).  With n_r[j] the number of group rows whose stage-r code is j
 * and m_r[j] the sum of their stage-r inputs z_r (scaled space, rebuilt from x,
 * the codes and the codebooks passed in):
 *   N <- decay N + (1 - decay) n ;   M <- decay M + (1 - decay) m ;
 *   N^_j = (N_j + eps) * sum_j N / (sum_j N + K eps) ;   C_r[j] <- M_r[j] / N^_j.
 *   x, codes     in      the vectors and the codes rvq_encode chose for them
 *                        with these same codebooks
 *   codebooks    in/out  float32 [R][K][group_dim]
 *   ema_count    in/out  float32 [R][K]              (N)
 *   ema_sum      in/out  float32 [R][K][group_dim]   (M)
 *   batch_count  out     optional float32 [R][K]: n of this call (may be NULL)
 *   workspace            rvq_workspace_bytes(cfg, n) bytes, 256-byte aligned
 * The caller must call rvq_prepare_codebooks again before the next encode or
 * decode.  Equivalent to rvq_ema_stats followed by rvq_ema_apply.
 */
int rvq_ema_update(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
                   const void *codes, float *codebooks, float *ema_count, float *ema_sum,
                   float *batch_count, float decay, float eps, void *workspace,
                   size_t workspace_bytes, rvq_status *status, void *stream /* cudaStream_t */);

/*
 * The two halves of rvq_ema_update, for data-parallel codebook learning: every
 * device computes the statistics of its own vectors, the caller sums
 * batch_count and batch_sum over devices (the counts and sums of Section 3's
 * moving average are plain sums over vectors), then every device applies the
 * same update.
 *   batch_count  out  float32 [R][K]             n_r[j] of these n vectors
 *                     (exact while a bin holds fewer than 2^24 rows)
 *   batch_sum    out  float32 [R][K][group_dim]  m_r[j]; 16-byte aligned
 * Both are overwritten.  Workspace as for rvq_ema_update.
 */
int rvq_ema_stats(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
                  const void *codes, const float *codebooks, float *batch_count, float *batch_sum,
                  void *workspace, size_t workspace_bytes, rvq_status *status,
                  void *stream /* cudaStream_t */);

/* N, M and the codebooks updated in place from the given batch statistics
 * (formulas under rvq_ema_update). */
int rvq_ema_apply(const rvq_config *cfg /* host */, const float *batch_count,
                  const float *batch_sum, float *codebooks, float *ema_count, float *ema_sum,
                  float decay, float eps, void *stream /* cudaStream_t */);

/*
 * One codebook-learning step (Section 3: the codebooks follow the encoder's own
 * assignments by exponential moving average, batch after batch): the batch is
 * encoded with the current codebooks, the statistics of these assignments update
 * N, M and the codebooks as under rvq_ema_update, and the prepared block is
 * rebuilt for the new codebooks.  Same results as rvq_encode_stats, rvq_ema_apply
 * and rvq_prepare_codebooks called in turn.
 *   codebooks, prepared   in/out
 *   ema_count, ema_sum    in/out  N [R][K] and M [R][K][group_dim]
 *   codes, std_f16        out     the batch encoded with the codebooks as they came in
 *   stage_energy          out     optional [R], as under rvq_encode: the loss curve of the learning loop
 *   workspace                     rvq_workspace_bytes(cfg, n) bytes, 256-byte aligned
 */
int rvq_learn_step(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
                   float *codebooks, void *prepared, float *ema_count, float *ema_sum, void *codes,
                   uint16_t *std_f16, float *stage_energy, float decay, float eps, void *workspace,
                   size_t workspace_bytes, rvq_status *status, void *stream /* cudaStream_t */);

/*
 * k-means initialisation of the codebooks on one batch (Section 3: every codebook
 * starts from a k-means run; the paper gives no further detail, so the
 * variant is this library's: plain Lloyd iterations).  Stage r works on
 * the stage-r inputs of the batch -- the scaled group rows minus the centroids
 * chosen at the earlier stages -- starting from the rows seed_rows[r][0..K) of
 * that input: `iterations` times every row is assigned to its nearest centroid
 * (exact squared distance, lowest index on ties) and every centroid moves to the
 * mean of its rows; a centroid without rows stays where it is.
 *   seed_rows   in   device, int64 [R][K]: group row numbers v * G + g in
 *                    [0, n * G), drawn by the caller (the library draws no
 *                    random numbers); a number out of range reads row 0
 *   iterations  in   0..1000 (0: the codebooks are the seed rows)
 *   codebooks   out  float32 [R][K][group_dim]
 *   prepared    out  ready for rvq_encode / rvq_decode with these codebooks
 *   workspace        rvq_kmeans_workspace_bytes(cfg, n) bytes, 256-byte aligned:
 *                    the float32 stage inputs (n * dim * 4 bytes) and the
 *                    per-stage scratch
 * group_dim 32 with a power-of-two number of groups only
 * (RVQ_ERR_UNSUPPORTED otherwise).
 */
size_t rvq_kmeans_workspace_bytes(const rvq_config *cfg /* host */, int64_t n);
int rvq_kmeans_init(const rvq_config *cfg /* host */, const void *x, int64_t n, int64_t x_row_stride,
                    const int64_t *seed_rows, int32_t iterations, float *codebooks, void *prepared,
                    void *workspace, size_t workspace_bytes, rvq_status *status,
                    void *stream /* cudaStream_t */);

/*
 * rvq_ema_update without a workspace argument.  (The paper has no counterpart;
 * this exists for one kind of caller.)
 *
 * Who it is for: code that may not, or cannot, get device memory at the moment
 * it needs the update -- a plugin running inside a host application that owns
 * the allocator and hands out only the input and output buffers, a step inside
 * a region where cudaMalloc is forbidden because it synchronises the device, or
 * a process whose memory budget was fixed at start-up.  rvq_ema_update asks such
 * a caller for rvq_workspace_bytes() of scratch it has no way to provide.
 *
 * Here the scratch is a fixed array inside the library
 * (rvq_ema_static_scratch_bytes(), about 2.1 MiB; every GPU that loads the
 * library holds it until the process ends).  Shapes whose rvq_workspace_bytes()
 * is larger -- more than depth 8 x 2048 codes x 32 channels' worth -- are
 * refused with RVQ_ERR_STATIC_LIMIT and nothing is launched.  The call itself
 * allocates and frees nothing.
 *
 * Arguments, results and error codes are those of rvq_ema_update.  Differences:
 *   - The first call on each device looks up the array's device address (a
 *     runtime query, not a launch) and keeps it.  Make that first call outside
 *     any stream capture.  The kept address belongs to the device's primary
 *     context: after cudaDeviceReset the array lives elsewhere, so do not call
 *     this entry point on a device that has been reset since its first call.
 *   - All calls, on every stream, share the one array, and it still holds the
 *     previous call's numbers when the next begins; each call clears the parts
 *     it accumulates into.  Two calls that can overlap on the GPU (different
 *     streams without an ordering between them) corrupt each other: order them.
 */
int rvq_ema_update_static(const rvq_config *cfg /* host */, const void *x, int64_t n,
                          int64_t x_row_stride, const void *codes, float *codebooks,
                          float *ema_count, float *ema_sum, float *batch_count, float decay,
                          float eps, rvq_status *status, void *stream /* cudaStream_t */);

/* Size in bytes of the scratch array behind rvq_ema_update_static. */
size_t rvq_ema_static_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* RVQ_H */
