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

// Largest | ||atom||_2 - 1 | over the dictionary: one warp per atom, fp32 sum of squares as in
// dict_append_kernel.  The deviations are non-negative floats, so their bit patterns order
// like integers and one atomicMax keeps the largest; NaN norms count as +inf.
template <int D_>
__global__ void norm_deviation_kernel(const float* __restrict__ D, int N, uint32_t* __restrict__ max_bits) {
    constexpr int PER = D_ / 32;
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const float v = D[(int64_t)n * D_ + lane * PER + k];
        ss = fmaf(v, v, ss);
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) {
        float dev = fabsf(sqrtf(ss) - 1.0f);
        if (!(dev == dev)) dev = __uint_as_float(0x7f800000u);
        atomicMax(max_bits, __float_as_uint(dev));
    }
}

// fp32 -> fp16 copy of the dictionary (round to nearest even), four values per thread.
__global__ void dict_to_f16_kernel(const float4* __restrict__ src, uint2* __restrict__ dst, int64_t n_vec4) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec4; i += (int64_t)gridDim.x * blockDim.x) {
        const float4 v = src[i];
        __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t*>(&lo);
        o.y = *reinterpret_cast<uint32_t*>(&hi);
        dst[i] = o;
    }
}

// Stored form of the coefficients ("Analysis for CSR": fp16 beside the 16-bit index): fp32 ->
// fp16, round to nearest even, eight values per thread (two 16-byte loads, one 16-byte store).
__global__ void pack_coef_kernel(const float4* __restrict__ src, uint4* __restrict__ dst, int64_t n8, const float* tail_src,
                                 __half* tail_dst, int tail) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride) {
        const float4 a = src[2 * i], b = src[2 * i + 1];
        __half2 h0 = __floats2half2_rn(a.x, a.y), h1 = __floats2half2_rn(a.z, a.w);
        __half2 h2 = __floats2half2_rn(b.x, b.y), h3 = __floats2half2_rn(b.z, b.w);
        uint4 u;
        u.x = *reinterpret_cast<uint32_t*>(&h0);
        u.y = *reinterpret_cast<uint32_t*>(&h1);
        u.z = *reinterpret_cast<uint32_t*>(&h2);
        u.w = *reinterpret_cast<uint32_t*>(&h3);
        dst[i] = u;
    }
    if (blockIdx.x == 0 && (int)threadIdx.x < tail) tail_dst[threadIdx.x] = __float2half_rn(tail_src[threadIdx.x]);
}

}  // namespace

int launch_pack_coef(const float* coef32, int64_t n, void* coef16, cudaStream_t stream) {
    if (n == 0) return CSR_OK;
    const int64_t n8 = n / 8;
    const int tail = (int)(n - 8 * n8);
    int64_t blocks = (n8 + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    pack_coef_kernel<<<(int)blocks, 256, 0, stream>>>(reinterpret_cast<const float4*>(coef32), reinterpret_cast<uint4*>(coef16),
                                                     n8, coef32 + 8 * n8, reinterpret_cast<__half*>(coef16) + 8 * n8, tail);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "pack_coef launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

int launch_dict_to_f16(const float* D, int N, int d, void* dst, cudaStream_t stream) {
    const int64_t n_vec4 = (int64_t)N * d / 4;
    int blocks = (int)((n_vec4 + 255) / 256);
    if (blocks > 4 * sm_count()) blocks = 4 * sm_count();
    dict_to_f16_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const float4*>(D), reinterpret_cast<uint2*>(dst), n_vec4);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "dict_to_f16 launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

int launch_dict_norm_deviation(const float* D, int N, int d, uint32_t* max_bits, cudaStream_t stream) {
    const int wpb = 8;
    const int blocks = (N + wpb - 1) / wpb;
    if (d == 128)
        norm_deviation_kernel<128><<<blocks, wpb * 32, 0, stream>>>(D, N, max_bits);
    else
        norm_deviation_kernel<64><<<blocks, wpb * 32, 0, stream>>>(D, N, max_bits);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "norm_deviation launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

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
