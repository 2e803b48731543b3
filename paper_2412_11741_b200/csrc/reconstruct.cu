// De-sparse (paper Eq. 12): X_hat[m,:] = sum_g coef[m][g] * D[idx[m][g]][:].
//
// One warp per output row.  The row's s codes are read once (lane g holds code g and
// g + 32), then every selected atom row is fetched with one coalesced request (d * 4
// bytes; the dictionary is at most a few MB and stays in L2) and accumulated in fp32 in
// the stored order.  HBM traffic per row is 4*s bytes of codes in and d * sizeof(out)
// bytes out; the gathers are L2 traffic.
#include "common.cuh"

namespace csr {
namespace {

constexpr int NT = 256;

template <int D_>
struct Vec;
template <>
struct Vec<128> {
    using T = float4;
};
template <>
struct Vec<64> {
    using T = float2;
};

__device__ __forceinline__ void axpy(float4& a, float c, const float4& v) {
    a.x = fmaf(c, v.x, a.x);
    a.y = fmaf(c, v.y, a.y);
    a.z = fmaf(c, v.z, a.z);
    a.w = fmaf(c, v.w, a.w);
}
__device__ __forceinline__ void axpy(float2& a, float c, const float2& v) {
    a.x = fmaf(c, v.x, a.x);
    a.y = fmaf(c, v.y, a.y);
}
__device__ __forceinline__ void zero(float4& a) { a = make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ void zero(float2& a) { a = make_float2(0.f, 0.f); }

// `off` is the element offset of the row inside X_hat; the lane writes its 4 (or 2) channels.
__device__ __forceinline__ void store_out(void* out, int out_dtype, int64_t off, int lane, const float4& a) {
    if (out_dtype == CSR_DTYPE_BF16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t*>(&lo);
        u.y = *reinterpret_cast<uint32_t*>(&hi);
        reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + off)[lane] = u;
    } else if (out_dtype == CSR_DTYPE_F16) {
        __half2 lo = __floats2half2_rn(a.x, a.y), hi = __floats2half2_rn(a.z, a.w);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t*>(&lo);
        u.y = *reinterpret_cast<uint32_t*>(&hi);
        reinterpret_cast<uint2*>(reinterpret_cast<__half*>(out) + off)[lane] = u;
    } else {
        reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + off)[lane] = a;
    }
}
__device__ __forceinline__ void store_out(void* out, int out_dtype, int64_t off, int lane, const float2& a) {
    if (out_dtype == CSR_DTYPE_BF16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(a.x, a.y);
        reinterpret_cast<uint32_t*>(reinterpret_cast<__nv_bfloat16*>(out) + off)[lane] = *reinterpret_cast<uint32_t*>(&v);
    } else if (out_dtype == CSR_DTYPE_F16) {
        __half2 v = __floats2half2_rn(a.x, a.y);
        reinterpret_cast<uint32_t*>(reinterpret_cast<__half*>(out) + off)[lane] = *reinterpret_cast<uint32_t*>(&v);
    } else {
        reinterpret_cast<float2*>(reinterpret_cast<float*>(out) + off)[lane] = a;
    }
}

template <int D_>
__global__ void __launch_bounds__(NT)
reconstruct_kernel(const float* __restrict__ D, const uint16_t* __restrict__ idx, const void* __restrict__ coef,
                   int coef_dtype, int64_t ldc, int64_t M, int N, int s, void* __restrict__ X_hat, int out_dtype,
                   int64_t ldxh) {
    using V = typename Vec<D_>::T;
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * (NT / 32) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (NT / 32);
    const V* Dv = reinterpret_cast<const V*>(D);
    for (int64_t m = warp0; m < M; m += nwarps) {
        int my_i[2] = {0, 0};
        float my_c[2] = {0.f, 0.f};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int g = lane + 32 * h;
            if (g < s) {
                int i = idx[m * ldc + g];
                my_i[h] = i < N ? i : N - 1;
                my_c[h] = (coef_dtype == CSR_DTYPE_F16)
                              ? __half2float(reinterpret_cast<const __half*>(coef)[m * ldc + g])
                              : reinterpret_cast<const float*>(coef)[m * ldc + g];
            }
        }
        V acc;
        zero(acc);
        for (int g0 = 0; g0 < s; g0 += 4) {
            V v[4];
            float c[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int g = g0 + u;
                const int src = g & 31;
                const int i = (g < 32) ? __shfl_sync(0xffffffffu, my_i[0], src) : __shfl_sync(0xffffffffu, my_i[1], src);
                c[u] = (g < 32) ? __shfl_sync(0xffffffffu, my_c[0], src) : __shfl_sync(0xffffffffu, my_c[1], src);
                if (g >= s) c[u] = 0.f;
                v[u] = Dv[(int64_t)i * 32 + lane];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (g0 + u < s) axpy(acc, c[u], v[u]);
        }
        store_out(X_hat, out_dtype, m * ldxh, lane, acc);
    }
}

}  // namespace

int launch_reconstruct(const ReconstructArgs& a) {
    if (a.M == 0) return CSR_OK;
    const int64_t warps_needed = a.M;
    int64_t blocks = (warps_needed + (NT / 32) - 1) / (NT / 32);
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (a.d == 128)
        reconstruct_kernel<128><<<(int)blocks, NT, 0, a.stream>>>(a.D, a.idx, a.coef, a.coef_dtype, a.ld_code, a.M,
                                                                  a.N, a.s, a.X_hat, a.out_dtype, a.ld_xhat);
    else
        reconstruct_kernel<64><<<(int)blocks, NT, 0, a.stream>>>(a.D, a.idx, a.coef, a.coef_dtype, a.ld_code, a.M,
                                                                 a.N, a.s, a.X_hat, a.out_dtype, a.ld_xhat);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "reconstruct launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace csr
