// Online dictionary atoms ("Build dictionary": atoms sampled from the KV cache just
// computed; "NeuralDict": ReNorm keeps every atom at unit l2-norm).
//
// One warp per new atom: the sampled row of X is read once (coalesced), its squared norm
// is accumulated in fp32 (per-lane partial sums in channel order, then a butterfly over
// the lanes), and the row divided by the norm is written as the atom.  Row numbers outside
// [0, M) are clamped into range rather than read out of bounds.
#include "common.cuh"

namespace csr {
namespace {

template <int D_>
__global__ void dict_append_kernel(float* __restrict__ D_new, const void* __restrict__ X, int x_dtype, int64_t M,
                                   int64_t ldx, const int64_t* __restrict__ rows, int n_rows) {
    constexpr int PER = D_ / 32;                          // channels per lane
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i >= n_rows) return;
    int64_t r = rows[i];
    r = r < 0 ? 0 : (r >= M ? M - 1 : r);
    float v[PER];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const int64_t off = r * ldx + lane * PER + k;
        v[k] = load_elem(X, x_dtype, off);
        ss = fmaf(v[k], v[k], ss);
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float inv = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
#pragma unroll
    for (int k = 0; k < PER; ++k) D_new[(int64_t)i * D_ + lane * PER + k] = v[k] * inv;
}

}  // namespace

int launch_dict_append(float* D_new, int d, const void* X, int x_dtype, int64_t M, int64_t ldx, const int64_t* rows,
                       int n_rows, cudaStream_t stream) {
    const int wpb = 8;
    const int blocks = (n_rows + wpb - 1) / wpb;
    if (d == 128)
        dict_append_kernel<128><<<blocks, wpb * 32, 0, stream>>>(D_new, X, x_dtype, M, ldx, rows, n_rows);
    else
        dict_append_kernel<64><<<blocks, wpb * 32, 0, stream>>>(D_new, X, x_dtype, M, ldx, rows, n_rows);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "dict_append launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace csr
