// De-sparse (paper Eq. 12): X_hat[m,:] = sum_g coef[m][g] * D[idx[m][g]][:].
//
// HBM traffic per row is 4*s bytes of codes in and d * sizeof(out) bytes out; the s atom rows a
// row needs are gathered from the dictionary, which is a few MB and stays in L2, so from about
// s = 4 up the kernel is bound by the L2 -> SM gather (s * d * sizeof(atom) bytes per row), not
// by HBM.  Two things follow:
//   - the atoms can be gathered from the fp16 copy of a prepared dictionary (csr_dict_create)
//     instead of the fp32 master: half the gathered bytes, and with fp16 coefficients (the
//     stored form) the products need no unpacking at all: fma.rn.f32.f16 multiplies two fp16
//     values exactly and accumulates in fp32;
//   - what is left is latency: every warp works on units of 16 consecutive rows whose codes it
//     stages through its own piece of shared memory with cp.async one unit ahead (one coalesced
//     stream instead of a dependent load per row; no block-wide barrier anywhere), and it keeps
//     the gathers of several rows in flight: every lane moves 16 bytes of an atom, so an atom
//     row takes 32, 16 or 8 lanes and a warp instruction serves 1, 2 or 4 rows.
// Accumulation is fp32 in the stored order g = 0 .. s-1 (repeated atoms accumulate).
#include <type_traits>

#include "common.cuh"

namespace csr {
namespace {

constexpr int NT = 256;
constexpr int RW = 16;                                    // rows per unit of a warp
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

// The 16 bytes of an atom a lane holds: four fp32 channels, or eight fp16 channels.
template <bool F16>
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
// acc0 += c * low half of w, acc1 += c * high half of w: fp16 x fp16 products are exact in
// fp32, the sum is rounded once (the same value as fmaf on the widened operands).
__device__ __forceinline__ void fma2_f16(float& acc0, float& acc1, uint32_t w, uint16_t c) {
    asm("{\n"
        ".reg .b16 lo, hi;\n"
        "mov.b32 {lo, hi}, %2;\n"
        "fma.rn.f32.f16 %0, lo, %3, %0;\n"
        "fma.rn.f32.f16 %1, hi, %3, %1;\n"
        "}\n"
        : "+f"(acc0), "+f"(acc1)
        : "r"(w), "h"(c));
}
template <>
struct Piece<true> {
    static constexpr int CH = 8;
    // fp32 coefficient: the atom's halves are widened first
    static __device__ __forceinline__ void axpy(float (&a)[8], float c, const uint4& v) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[q]));
            a[2 * q] = fmaf(c, f.x, a[2 * q]);
            a[2 * q + 1] = fmaf(c, f.y, a[2 * q + 1]);
        }
    }
    // fp16 coefficient, as stored
    static __device__ __forceinline__ void axpy(float (&a)[8], uint16_t c, const uint4& v) {
        fma2_f16(a[0], a[1], v.x, c);
        fma2_f16(a[2], a[3], v.y, c);
        fma2_f16(a[4], a[5], v.z, c);
        fma2_f16(a[6], a[7], v.w, c);
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

// Codes of rows [row0, row0 + RW) into the warp's shared memory as [RW][s].  `fast`: the unit lies
// inside dense, 16-byte aligned code arrays, so it is one contiguous run per array and moves with
// cp.async; otherwise element by element (row strides, the ragged last unit).
__device__ __forceinline__ void stage_codes(uint16_t* s_idx, unsigned char* s_coef, const uint16_t* __restrict__ idx,
                                            const void* __restrict__ coef, int cbytes, int64_t ldc, int64_t row0, int rows,
                                            int s, bool fast, int lane) {
    if (fast) {
        const int n_i = RW * s * 2 / 16, n_c = RW * s * cbytes / 16;
        const char* gi = reinterpret_cast<const char*>(idx + row0 * s);
        const char* gc = static_cast<const char*>(coef) + row0 * s * cbytes;
        for (int q = lane; q < n_i; q += 32) cp_async16(reinterpret_cast<char*>(s_idx) + 16 * q, gi + 16 * q);
        for (int q = lane; q < n_c; q += 32) cp_async16(s_coef + 16 * q, gc + 16 * q);
    } else {
        for (int q = lane; q < rows * s; q += 32) {
            const int r = q / s, g = q - r * s;
            s_idx[q] = idx[(row0 + r) * ldc + g];
            if (cbytes == 2)
                reinterpret_cast<uint16_t*>(s_coef)[q] = reinterpret_cast<const uint16_t*>(coef)[(row0 + r) * ldc + g];
            else
                reinterpret_cast<float*>(s_coef)[q] = reinterpret_cast<const float*>(coef)[(row0 + r) * ldc + g];
        }
    }
}

// Rows r[0..PP) of the staged block, one gather step at a time (any s, rows past M skipped).
template <int CH, int LPR, typename P>
__device__ __forceinline__ void rows_generic(const uint4* __restrict__ Dl, const uint16_t* ci, const unsigned char* cc,
                                             int cbytes, int s, int N, const int (&r)[PP], const bool (&valid)[PP],
                                             float (&acc)[PP][CH], [[maybe_unused]] uint32_t* status) {
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
                    const int i = min(static_cast<int>(ci[r[w] * s + g]), N - 1);
#ifdef CSR_DEBUG_CHECKS
                    if (static_cast<int>(ci[r[w] * s + g]) >= N) atomicOr(status, kStatusBounds);
#endif
                    c[w][u] = cbytes == 2 ? __half2float(reinterpret_cast<const __half*>(cc)[r[w] * s + g])
                                          : reinterpret_cast<const float*>(cc)[r[w] * s + g];
                    v[w][u] = __ldg(Dl + static_cast<size_t>(i) * LPR);
                }
            }
#pragma unroll
        for (int w = 0; w < PP; ++w)
#pragma unroll
            for (int u = 0; u < INFLIGHT; ++u)
                if (g0 + u < s) P::axpy(acc[w], c[w][u], v[w][u]);
    }
}

// The same for s a multiple of four and rows that all exist: the codes of four steps come out
// of shared memory with one 8-byte load per array (16 bytes for fp32 coefficients), and nothing
// is predicated.
template <int CH, int LPR, typename P, bool COEF16>
__device__ __forceinline__ void rows_by_four(const uint4* __restrict__ Dl, const uint16_t* ci, const unsigned char* cc, int s,
                                             int N, const int (&r)[PP], float (&acc)[PP][CH], [[maybe_unused]] uint32_t* status) {
    static_assert(INFLIGHT == 4, "four steps per trip");
    constexpr bool RAW16 = COEF16 && CH == 8;             // fp16 coefficients meet fp16 atoms: no conversion
    using CoefT = typename std::conditional<RAW16, uint16_t, float>::type;
    const int nmax = N - 1;
    for (int g0 = 0; g0 < s; g0 += 4) {
        uint4 v[PP][4];
        CoefT c[PP][4];
#pragma unroll
        for (int w = 0; w < PP; ++w) {
            const uint2 iw = *reinterpret_cast<const uint2*>(ci + r[w] * s + g0);
            if constexpr (RAW16) {
                const uint2 cw = *reinterpret_cast<const uint2*>(cc + (r[w] * s + g0) * 2);
                c[w][0] = static_cast<uint16_t>(cw.x & 0xFFFFu);
                c[w][1] = static_cast<uint16_t>(cw.x >> 16);
                c[w][2] = static_cast<uint16_t>(cw.y & 0xFFFFu);
                c[w][3] = static_cast<uint16_t>(cw.y >> 16);
            } else if constexpr (COEF16) {
                const uint2 cw = *reinterpret_cast<const uint2*>(cc + (r[w] * s + g0) * 2);
                const float2 c01 = __half22float2(*reinterpret_cast<const __half2*>(&cw.x));
                const float2 c23 = __half22float2(*reinterpret_cast<const __half2*>(&cw.y));
                c[w][0] = c01.x;
                c[w][1] = c01.y;
                c[w][2] = c23.x;
                c[w][3] = c23.y;
            } else {
                const float4 cw = *reinterpret_cast<const float4*>(cc + (r[w] * s + g0) * 4);
                c[w][0] = cw.x;
                c[w][1] = cw.y;
                c[w][2] = cw.z;
                c[w][3] = cw.w;
            }
            const int i0 = min(static_cast<int>(iw.x & 0xFFFFu), nmax), i1 = min(static_cast<int>(iw.x >> 16), nmax);
            const int i2 = min(static_cast<int>(iw.y & 0xFFFFu), nmax), i3 = min(static_cast<int>(iw.y >> 16), nmax);
#ifdef CSR_DEBUG_CHECKS
            if (static_cast<int>(max(max(iw.x & 0xFFFFu, iw.x >> 16), max(iw.y & 0xFFFFu, iw.y >> 16))) > nmax)
                atomicOr(status, kStatusBounds);
#endif
            v[w][0] = __ldg(Dl + static_cast<uint32_t>(i0 * LPR));
            v[w][1] = __ldg(Dl + static_cast<uint32_t>(i1 * LPR));
            v[w][2] = __ldg(Dl + static_cast<uint32_t>(i2 * LPR));
            v[w][3] = __ldg(Dl + static_cast<uint32_t>(i3 * LPR));
        }
#pragma unroll
        for (int w = 0; w < PP; ++w)
#pragma unroll
            for (int u = 0; u < 4; ++u) P::axpy(acc[w], c[w][u], v[w][u]);
    }
}

template <int D_, bool F16>
__global__ void __launch_bounds__(NT, F16 ? 3 : 4)
reconstruct_kernel(const void* __restrict__ Dict, const uint16_t* __restrict__ idx, const void* __restrict__ coef,
                   int coef_dtype, int64_t ldc, int64_t M, int N, int s, void* __restrict__ X_hat, int out_dtype,
                   int64_t ldxh, int dense_codes, uint32_t* status) {
    using P = Piece<F16>;
    constexpr int CH = P::CH;                             // channels per lane
    constexpr int LPR = D_ / CH;                          // lanes per row: 32, 16 or 8
    constexpr int RPP = 32 / LPR;                         // rows per warp pass
    constexpr int PASSES = RW / RPP;                      // passes per unit: 16, 8 or 4
    static_assert(PASSES % PP == 0, "passes are taken PP at a time");
    extern __shared__ __align__(16) unsigned char smem[];
    const int cbytes = coef_dtype == CSR_DTYPE_F16 ? 2 : 4;
    const int stride_i = RW * s * 2, stride_c = RW * s * cbytes;      // multiples of 16 bytes
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* mine = smem + warp * 2 * (stride_i + stride_c);   // this warp's two buffers of [idx | coef]
    auto s_idx = [&](int which) { return reinterpret_cast<uint16_t*>(mine + which * (stride_i + stride_c)); };
    auto s_coef = [&](int which) { return mine + which * (stride_i + stride_c) + stride_i; };

    const int sub = lane / LPR, l = lane % LPR;
    const uint4* Dl = static_cast<const uint4*>(Dict) + l;  // this lane's 16 bytes of atom 0; an atom row is LPR pieces
    const int64_t n_units = (M + RW - 1) / RW;
    const int64_t unit_step = (int64_t)gridDim.x * (NT / 32);
    const bool by_four = (s & 3) == 0;

    auto unit_fast = [&](int64_t u) { return dense_codes && (u + 1) * RW <= M; };
    int64_t u = (int64_t)blockIdx.x * (NT / 32) + warp;
    int buf = 0;
    if (u < n_units) stage_codes(s_idx(0), s_coef(0), idx, coef, cbytes, ldc, u * RW, (int)min((int64_t)RW, M - u * RW), s, unit_fast(u), lane);
    cp_async_commit();
    for (; u < n_units; u += unit_step, buf ^= 1) {
        const int64_t nu = u + unit_step;
        if (nu < n_units)
            stage_codes(s_idx(buf ^ 1), s_coef(buf ^ 1), idx, coef, cbytes, ldc, nu * RW, (int)min((int64_t)RW, M - nu * RW), s,
                        unit_fast(nu), lane);
        cp_async_commit();
        cp_async_wait<1>();                               // this unit's codes have landed (the next may be in flight)
        __syncwarp();
        const uint16_t* ci = s_idx(buf);
        const unsigned char* cc = s_coef(buf);
        const bool whole = (u + 1) * RW <= M;
#pragma unroll 1
        for (int p = 0; p < PASSES; p += PP) {
            int r[PP];
            bool valid[PP];
            float acc[PP][CH];
#pragma unroll
            for (int w = 0; w < PP; ++w) {
                r[w] = (p + w) * RPP + sub;               // row inside the unit
                valid[w] = u * RW + r[w] < M;
#pragma unroll
                for (int k = 0; k < CH; ++k) acc[w][k] = 0.f;
            }
            if (whole && by_four) {
                if (cbytes == 2)
                    rows_by_four<CH, LPR, P, true>(Dl, ci, cc, s, N, r, acc, status);
                else
                    rows_by_four<CH, LPR, P, false>(Dl, ci, cc, s, N, r, acc, status);
            } else {
                rows_generic<CH, LPR, P>(Dl, ci, cc, cbytes, s, N, r, valid, acc, status);
            }
#pragma unroll
            for (int w = 0; w < PP; ++w)
                if (valid[w]) store_out<CH>(X_hat, out_dtype, (u * RW + r[w]) * ldxh + l * CH, acc[w]);
        }
        __syncwarp();                                      // the buffer may be refilled
    }
    cp_async_wait<0>();
}

template <int D_, bool F16>
int launch_t(const ReconstructArgs& a, const void* dict) {
    const int cbytes = a.coef_dtype == CSR_DTYPE_F16 ? 2 : 4;
    const size_t smem = (size_t)(NT / 32) * 2 * RW * a.s * (2 + cbytes);
    const int64_t n_blocks = ((a.M + RW - 1) / RW + NT / 32 - 1) / (NT / 32);
    static int ctas_per_sm[64] = {};                       // per device; what the occupancy calculator says for smem = 0
    int dev = 0;
    cudaGetDevice(&dev);
    dev = (dev >= 0 && dev < 64) ? dev : 0;
    int per_sm = ctas_per_sm[dev];
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, reconstruct_kernel<D_, F16>, NT, 0) != cudaSuccess || per_sm < 1)
            per_sm = 4;
        ctas_per_sm[dev] = per_sm;
    }
    // shared memory may hold fewer CTAs than the registers do (227 KB per SM)
    int fit = smem ? (int)((size_t)(227 * 1024) / (smem + 1024)) : per_sm;
    if (fit < 1) fit = 1;
    const int64_t cap = (int64_t)sm_count() * (per_sm < fit ? per_sm : fit);
    const int grid = (int)(n_blocks < cap ? n_blocks : cap);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(reconstruct_kernel<D_, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    const uintptr_t pi = reinterpret_cast<uintptr_t>(a.idx), pc = reinterpret_cast<uintptr_t>(a.coef);
    const int dense = a.ld_code == a.s && pi % 16 == 0 && pc % 16 == 0;
    reconstruct_kernel<D_, F16><<<grid, NT, smem, a.stream>>>(dict, a.idx, a.coef, a.coef_dtype, a.ld_code, a.M, a.N, a.s,
                                                              a.X_hat, a.out_dtype, a.ld_xhat, dense, a.status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "reconstruct launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace

int launch_reconstruct(const ReconstructArgs& a) {
    if (a.M == 0) return CSR_OK;
    if (a.dict_f16) return a.d == 128 ? launch_t<128, true>(a, a.dict_f16) : launch_t<64, true>(a, a.dict_f16);
    return a.d == 128 ? launch_t<128, false>(a, a.D) : launch_t<64, false>(a, a.D);
}

}  // namespace csr
