// Prepared-codebook block: what the kernels read instead of the float32
// codebooks.  Layout (all offsets multiples of 256 bytes):
//   header   256 bytes   magic, shape echo
// Further sections are appended by the kernels that need them.
#include "common.cuh"

namespace rvq {

struct PreparedHeader {
    uint32_t magic, R, K, gd;
};

size_t prepared_bytes(const Shape &s)
{
    (void)s;
    return 256;
}

__global__ void prepare_header_kernel(PreparedHeader *h, Shape s)
{
    h->magic = 0x52565131u;
    h->R = s.R; h->K = s.K; h->gd = s.gd;
}

int launch_prepare(const Shape &s, const float *cb, void *prepared, cudaStream_t stream)
{
    (void)cb;
    prepare_header_kernel<<<1, 1, 0, stream>>>(reinterpret_cast<PreparedHeader *>(prepared), s);
    return check_launch();
}

}  // namespace rvq
