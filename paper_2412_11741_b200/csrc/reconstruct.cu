// De-sparse (paper Eq. 12): X_hat[m,:] = sum_g coef[m][g] * D[idx[m][g]][:].
//
// HBM traffic per row is 4*s bytes of codes in and d * sizeof(out) bytes out; the s atom rows a
// row needs are gathered from the dictionary, which is a few MB and stays in L2, so from about
// s = 4 up the kernel is bound by the L2 -> SM gather (s * d * sizeof(atom) bytes per row), not
// by HBM.  Two things follow:
//   - the atoms can be gathered from the bf16 copy of a prepared dictionary (csr_dict_create)
//     instead of the fp32 master: half the gathered bytes;
//   - what is left is latency: a CTA works on blocks of 64 rows whose codes are staged through
//     shared memory with cp.async one block ahead (one coalesced stream instead of a dependent
//     load per row), and a warp keeps the gathers of several rows in flight: every lane moves
//     16 bytes of an atom, so an atom row takes 32, 16 or 8 lanes and a warp instruction serves
//     1, 2 or 4 rows.
// Accumulation is fp32 in the stored order g = 0 .. s-1 (repeated atoms accumulate).
#include "common.cuh"

namespace csr {
namespace {

constexpr int NT = 256;
constexpr int RB = 64;                                    // rows per block of a CTA
constexpr int PP = 2;                                     // passes (rows) a lane works on together
constexpr int INFLIGHT = 4;                               // gathers per row issued before their first use

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem))),
                 "l"(gmem)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// The 16 bytes of an atom a lane holds, as channels in fp32.
template <bool BF16>
struct Piece;
template <>
struct Piece<false> {
    static constexpr int CH = 4;
    static __device__ __forceinline__ void axpy(float (&a)[4], float c, const uint4& v) {
        a[0] = fmaf(c, __uint_as_float(v.x), a[0]);
        a[1] = fmaf(c, __uint_as_float(v.y), a[1]);
        a[2] = fmaf(c, __uint_as_float(v.z), a[2]);
        a[3] = fmaf(c, __uint_as_float(v.w), a[3]);
    }
};
template <>
struct Piece<true> {
    static constexpr int CH = 8;
    static __device__ __forceinline__ void axpy(float (&a)[8], float c, const uint4& v) {
        a[0] = fmaf(c, __uint_as_float(v.x << 16), a[0]);
        a[1] = fmaf(c, __uint_as_float(v.x & 0xFFFF0000u), a[1]);
        a[2] = fmaf(c, __uint_as_float(v.y << 16), a[2]);
        a[3] = fmaf(c, __uint_as_float(v.y & 0xFFFF0000u), a[3]);
        a[4] = fmaf(c, __uint_as_float(v.z << 16), a[4]);
        a[5] = fmaf(c, __uint_as_float(v.z & 0xFFFF0000u), a[5]);
        a[6] = fmaf(c, __uint_as_float(v.w << 16), a[6]);
        a[7] = fmaf(c, __uint_as_float(v.w & 0xFFFF0000u), a[7]);
    }
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi, int out_dtype) {
    if (out_dtype == CSR_DTYPE_BF16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// CH consecutive channels of one row, starting at element `off` of X_hat.
template <int CH>
__device__ __forceinline__ void store_out(void* out, int out_dtype, int64_t off, const float (&a)[CH]) {
    if (out_dtype == CSR_DTYPE_F32) {
        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + off);
#pragma unroll
        for (int q = 0; q < CH / 4; ++q) dst[q] = make_float4(a[4 * q], a[4 * q + 1], a[4 * q + 2], a[4 * q + 3]);
    } else if constexpr (CH == 8) {
        uint4 u;
        u.x = pack2(a[0], a[1], out_dtype);
        u.y = pack2(a[2], a[3], out_dtype);
        u.z = pack2(a[4], a[5], out_dtype);
        u.w = pack2(a[6], a[7], out_dtype);
        *reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(out) + off) = u;
    } else {
        uint2 u;
        u.x = pack2(a[0], a[1], out_dtype);
        u.y = pack2(a[2], a[3], out_dtype);
        *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(out) + off) = u;
    }
}

// Codes of rows [row0, row0 + RB) into shared memory as [RB][s].  `fast`: the block lies inside
// dense, 16-byte aligned code arrays, so it is one contiguous run per array and moves with
// cp.async; otherwise element by element (row strides, the ragged last block).
__device__ __forceinline__ void stage_codes(uint16_t* s_idx, unsigned char* s_coef, const uint16_t* __restrict__ idx,
                                            const void* __restrict__ coef, int cbytes, int64_t ldc, int64_t row0, int rows,
                                            int s, bool fast) {
    if (fast) {
        const int n_i = RB * s * 2 / 16, n_c = RB * s * cbytes / 16;
        const char* gi = reinterpret_cast<const char*>(idx + row0 * s);
        const char* gc = static_cast<const char*>(coef) + row0 * s * cbytes;
        for (int q = threadIdx.x; q < n_i; q += NT) cp_async16(reinterpret_cast<char*>(s_idx) + 16 * q, gi + 16 * q);
        for (int q = threadIdx.x; q < n_c; q += NT) cp_async16(s_coef + 16 * q, gc + 16 * q);
    } else {
        for (int q = threadIdx.x; q < rows * s; q += NT) {
            const int r = q / s, g = q - r * s;
            s_idx[q] = idx[(row0 + r) * ldc + g];
            if (cbytes == 2)
                reinterpret_cast<uint16_t*>(s_coef)[q] = reinterpret_cast<const uint16_t*>(coef)[(row0 + r) * ldc + g];
            else
                reinterpret_cast<float*>(s_coef)[q] = reinterpret_cast<const float*>(coef)[(row0 + r) * ldc + g];
        }
    }
}

template <int D_, bool BF16>
__global__ void __launch_bounds__(NT)
reconstruct_kernel(const void* __restrict__ Dict, const uint16_t* __restrict__ idx, const void* __restrict__ coef,
                   int coef_dtype, int64_t ldc, int64_t M, int N, int s, void* __restrict__ X_hat, int out_dtype,
                   int64_t ldxh, int dense_codes) {
    using P = Piece<BF16>;
    constexpr int CH = P::CH;                             // channels per lane
    constexpr int LPR = D_ / CH;                          // lanes per row: 32, 16 or 8
    constexpr int RPP = 32 / LPR;                         // rows per warp pass
    constexpr int PASSES = RB / (NT / 32) / RPP;          // passes of a warp per block: 8, 4 or 2
    static_assert(PASSES % PP == 0, "passes are taken PP at a time");
    extern __shared__ __align__(16) unsigned char smem[];
    const int cbytes = coef_dtype == CSR_DTYPE_F16 ? 2 : 4;
    const int stride_i = RB * s * 2, stride_c = RB * s * cbytes;      // multiples of 16 bytes
    auto s_idx = [&](int which) { return reinterpret_cast<uint16_t*>(smem + which * stride_i); };
    auto s_coef = [&](int which) { return smem + 2 * stride_i + which * stride_c; };

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane / LPR, l = lane % LPR;
    const uint4* Dv = static_cast<const uint4*>(Dict);     // an atom row is LPR pieces of 16 bytes
    const int64_t n_blocks = (M + RB - 1) / RB;

    auto block_fast = [&](int64_t b) { return dense_codes && (b + 1) * RB <= M; };
    int buf = 0;
    if ((int64_t)blockIdx.x < n_blocks) {
        const int64_t b = blockIdx.x;
        stage_codes(s_idx(0), s_coef(0), idx, coef, cbytes, ldc, b * RB, (int)min((int64_t)RB, M - b * RB), s, block_fast(b));
    }
    cp_async_commit();
    for (int64_t b = blockIdx.x; b < n_blocks; b += gridDim.x, buf ^= 1) {
        const int64_t nb = b + gridDim.x;
        if (nb < n_blocks)
            stage_codes(s_idx(buf ^ 1), s_coef(buf ^ 1), idx, coef, cbytes, ldc, nb * RB, (int)min((int64_t)RB, M - nb * RB), s,
                        block_fast(nb));
        cp_async_commit();
        cp_async_wait<1>();                               // this block's codes have landed (the next may be in flight)
        __syncthreads();
        const uint16_t* ci = s_idx(buf);
        const unsigned char* cc = s_coef(buf);
#pragma unroll 1
        for (int p = 0; p < PASSES; p += PP) {
            int r[PP];
            bool valid[PP];
            float acc[PP][CH];
#pragma unroll
            for (int w = 0; w < PP; ++w) {
                r[w] = (warp * PASSES + p + w) * RPP + sub;       // row inside the block
                valid[w] = b * RB + r[w] < M;
#pragma unroll
                for (int k = 0; k < CH; ++k) acc[w][k] = 0.f;
            }
            for (int g0 = 0; g0 < s; g0 += INFLIGHT) {
                uint4 v[PP][INFLIGHT];
                float c[PP][INFLIGHT];
#pragma unroll
                for (int w = 0; w < PP; ++w)
#pragma unroll
                    for (int u = 0; u < INFLIGHT; ++u) {
                        const int g = g0 + u;
                        v[w][u] = make_uint4(0u, 0u, 0u, 0u);
                        c[w][u] = 0.f;
                        if (g < s && valid[w]) {
                            int i = ci[r[w] * s + g];
                            i = i < N ? i : N - 1;
                            c[w][u] = cbytes == 2 ? __half2float(reinterpret_cast<const __half*>(cc)[r[w] * s + g])
                                                  : reinterpret_cast<const float*>(cc)[r[w] * s + g];
                            v[w][u] = __ldg(Dv + (int64_t)i * LPR + l);
                        }
                    }
#pragma unroll
                for (int w = 0; w < PP; ++w)
#pragma unroll
                    for (int u = 0; u < INFLIGHT; ++u)
                        if (g0 + u < s) P::axpy(acc[w], c[w][u], v[w][u]);
            }
#pragma unroll
            for (int w = 0; w < PP; ++w)
                if (valid[w]) store_out<CH>(X_hat, out_dtype, (b * RB + r[w]) * ldxh + l * CH, acc[w]);
        }
        __syncthreads();                                   // the buffer may be refilled
    }
    cp_async_wait<0>();
}

template <int D_, bool BF16>
int launch_t(const ReconstructArgs& a, const void* dict) {
    const int cbytes = a.coef_dtype == CSR_DTYPE_F16 ? 2 : 4;
    const size_t smem = 2 * (size_t)RB * a.s * (2 + cbytes);
    const int64_t n_blocks = (a.M + RB - 1) / RB;
    static int ctas_per_sm[64] = {};                       // per device; what the occupancy calculator says for smem = 0
    int dev = 0;
    cudaGetDevice(&dev);
    dev = (dev >= 0 && dev < 64) ? dev : 0;
    int per_sm = ctas_per_sm[dev];
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, reconstruct_kernel<D_, BF16>, NT, 0) != cudaSuccess || per_sm < 1)
            per_sm = 4;
        ctas_per_sm[dev] = per_sm;
    }
    // shared memory may hold fewer CTAs than the registers do (227 KB per SM)
    int fit = smem ? (int)((size_t)(227 * 1024) / (smem + 1024)) : per_sm;
    if (fit < 1) fit = 1;
    const int64_t cap = (int64_t)sm_count() * (per_sm < fit ? per_sm : fit);
    const int grid = (int)(n_blocks < cap ? n_blocks : cap);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(reconstruct_kernel<D_, BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    const uintptr_t pi = reinterpret_cast<uintptr_t>(a.idx), pc = reinterpret_cast<uintptr_t>(a.coef);
    const int dense = a.ld_code == a.s && pi % 16 == 0 && pc % 16 == 0;
    reconstruct_kernel<D_, BF16><<<grid, NT, smem, a.stream>>>(dict, a.idx, a.coef, a.coef_dtype, a.ld_code, a.M, a.N, a.s,
                                                              a.X_hat, a.out_dtype, a.ld_xhat, dense);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "reconstruct launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace

int launch_reconstruct(const ReconstructArgs& a) {
    if (a.M == 0) return CSR_OK;
    if (a.dict_bf16) return a.d == 128 ? launch_t<128, true>(a, a.dict_bf16) : launch_t<64, true>(a, a.dict_bf16);
    return a.d == 128 ? launch_t<128, false>(a, a.D) : launch_t<64, false>(a, a.D);
}

}  // namespace csr
