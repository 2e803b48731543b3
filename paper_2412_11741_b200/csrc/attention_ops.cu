// Attention straight from the codes ("De-Sparse to restore": the restored tensor
// X~ = D r of Eq. 12 "will be used in the attention score calculation").  Because X~ is
// linear in the atoms, neither product needs X~ in memory:
//
//   scores[t] = scale * q . x~_t   = sum_g coef[t][g] * p[idx[t][g]],    p = scale * D q
//   out       = sum_t w[t] * x~_t  = sum_n a[n] * D[n][:],               a[n] = sum_{(t,g): idx[t][g] = n} w[t] coef[t][g]
//
// HBM traffic per token is the 4*s bytes of its code (plus 4 bytes per query head of score
// or weight) instead of the 2*d bytes of a restored bf16 row written and read again.
//
// key_scores: (1) p = scale * Q D^T for all B*H query heads, a small fp32 GEMM written to a
// scratch array [B*H][N] (channels summed in ascending order); (2) one CTA per (code stream,
// token range) copies its heads' rows of p into shared memory, streams the codes, one
// thread per token, and sums the s terms in stored order.
// value_mix: (1) one CTA per (code stream, token range) scatters w * coef into a[head][N] in
// shared memory with atomic adds while it streams the codes and then adds its a to the
// scratch array [B*H][N] with global atomic adds; (2) out = a D, a small fp32 GEMM (split
// over atoms with atomic adds when there are few heads).  Atomic fp32 adds make value_mix
// reproducible only to rounding.
#include "common.cuh"

namespace csr {
namespace {

constexpr int NT = 256;
constexpr int NTS = 1024;   // threads of the code-streaming kernels (one CTA per SM: shared memory)

__device__ __forceinline__ float load_coef(const void* coef, int coef_dtype, int64_t off) {
    return coef_dtype == CSR_DTYPE_F16 ? __half2float(reinterpret_cast<const __half*>(coef)[off])
                                       : reinterpret_cast<const float*>(coef)[off];
}
__device__ __forceinline__ float load_q(const void* Q, int q_dtype, int64_t off) {
    return q_dtype == CSR_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(Q)[off])
                                     : reinterpret_cast<const float*>(Q)[off];
}

// ---- P[r][n] = scale * Q[r][:] . D[n][:]  (r = b*H + h) -----------------------------------
// CTA = 64 atoms x all rows, 16 rows at a time; thread = (atom, group of 4 rows).
constexpr int PA = 64;    // atoms per CTA
constexpr int PR = 16;    // rows per pass
constexpr int QROWS = 64; // rows per CTA (grid.y)
template <int D_>
__global__ void __launch_bounds__(NT)
qd_kernel(const float* __restrict__ D, int N, const void* __restrict__ Q, int q_dtype, int R, float scale,
          float* __restrict__ P) {
    __shared__ float Ds[PA][D_ + 1];
    __shared__ __align__(16) float Qs[PR][D_];
    const int n0 = blockIdx.x * PA;
    for (int f = threadIdx.x; f < PA * D_; f += NT) {
        const int a = f / D_, k = f % D_;
        Ds[a][k] = (n0 + a < N) ? D[(int64_t)(n0 + a) * D_ + k] : 0.f;
    }
    const int a = threadIdx.x % PA, rg = threadIdx.x / PA;     // rows rg*4 .. rg*4+3 of the pass
    const int r_end = min(R, (int)(blockIdx.y + 1) * QROWS);
    for (int r0 = blockIdx.y * QROWS; r0 < r_end; r0 += PR) {
        __syncthreads();
        for (int f = threadIdx.x; f < PR * D_; f += NT) {
            const int r = f / D_, k = f % D_;
            Qs[r][k] = (r0 + r < R) ? load_q(Q, q_dtype, (int64_t)(r0 + r) * D_ + k) : 0.f;
        }
        __syncthreads();
        float acc[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = 0.f;
        for (int k = 0; k < D_; k += 4) {
            const float d0 = Ds[a][k], d1 = Ds[a][k + 1], d2 = Ds[a][k + 2], d3 = Ds[a][k + 3];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 q = *reinterpret_cast<const float4*>(&Qs[rg * 4 + i][k]);
                acc[i] = fmaf(q.w, d3, fmaf(q.z, d2, fmaf(q.y, d1, fmaf(q.x, d0, acc[i]))));
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = r0 + rg * 4 + i;
            if (r < R && n0 + a < N) P[(int64_t)r * N + n0 + a] = scale * acc[i];
        }
    }
}

// ---- out[r][:] (+)= sum_{n in slice} A[r][n] * D[n][:] ------------------------------------
// CTA = 16 rows x one atom slice; thread = (channel, group of rows).
constexpr int OR = 16;    // rows per CTA
constexpr int OA = 64;    // atoms per staged block
template <int D_>
__global__ void __launch_bounds__(NT)
ad_kernel(const float* __restrict__ D, int N, const float* __restrict__ A, int R, int atoms_per_slice, int use_atomics,
          float* __restrict__ out) {
    __shared__ float Ds[OA][D_];
    __shared__ __align__(16) float As[OR][OA];
    constexpr int RG = NT / D_;            // row groups (2 or 4)
    constexpr int RPT = OR / RG;           // rows per thread (8 or 4)
    const int c = threadIdx.x % D_, rg = threadIdx.x / D_;
    const int r0 = blockIdx.x * OR;
    const int nb = blockIdx.y * atoms_per_slice;
    const int ne = min(nb + atoms_per_slice, N);
    float acc[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) acc[i] = 0.f;
    for (int n0 = nb; n0 < ne; n0 += OA) {
        __syncthreads();
        for (int f = threadIdx.x; f < OA * D_; f += NT) {
            const int a = f / D_, k = f % D_;
            Ds[a][k] = (n0 + a < ne) ? D[(int64_t)(n0 + a) * D_ + k] : 0.f;
        }
        for (int f = threadIdx.x; f < OR * OA; f += NT) {
            const int r = f / OA, a = f % OA;
            As[r][a] = (r0 + r < R && n0 + a < ne) ? A[(int64_t)(r0 + r) * N + n0 + a] : 0.f;
        }
        __syncthreads();
        for (int a = 0; a < OA; a += 4) {
            const float d0 = Ds[a][c], d1 = Ds[a + 1][c], d2 = Ds[a + 2][c], d3 = Ds[a + 3][c];
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const float4 w = *reinterpret_cast<const float4*>(&As[rg * RPT + i][a]);
                acc[i] = fmaf(w.w, d3, fmaf(w.z, d2, fmaf(w.y, d1, fmaf(w.x, d0, acc[i]))));
            }
        }
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = r0 + rg * RPT + i;
        if (r < R) {
            if (use_atomics)
                atomicAdd(&out[(int64_t)r * D_ + c], acc[i]);
            else
                out[(int64_t)r * D_ + c] = acc[i];
        }
    }
}

// Eight consecutive codes of one token (16-byte loads; the caller guarantees s % 8 == 0 and
// 16-byte aligned arrays, so every block of eight starts on a 16-byte boundary).
__device__ __forceinline__ void load_codes8(const uint16_t* idx, const void* coef, int coef_dtype, int64_t off, int (&i)[8],
                                            float (&c)[8]) {
    const uint4 iv = *reinterpret_cast<const uint4*>(idx + off);
    i[0] = iv.x & 0xFFFF; i[1] = iv.x >> 16; i[2] = iv.y & 0xFFFF; i[3] = iv.y >> 16;
    i[4] = iv.z & 0xFFFF; i[5] = iv.z >> 16; i[6] = iv.w & 0xFFFF; i[7] = iv.w >> 16;
    if (coef_dtype == CSR_DTYPE_F16) {
        const uint4 cv = *reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(coef) + off);
        const __half2* h = reinterpret_cast<const __half2*>(&cv);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(h[j]);
            c[2 * j] = f.x;
            c[2 * j + 1] = f.y;
        }
    } else {
        const float4 a = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(coef) + off);
        const float4 b = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(coef) + off + 4);
        c[0] = a.x; c[1] = a.y; c[2] = a.z; c[3] = a.w; c[4] = b.x; c[5] = b.y; c[6] = b.z; c[7] = b.w;
    }
}

// ---- code streams --------------------------------------------------------------------------
// blockIdx.x = code stream, blockIdx.y = token range; dynamic smem: HG * N floats.
__global__ void __launch_bounds__(NTS)
key_scores_kernel(const float* __restrict__ P, int N, int H, int HG, const uint16_t* __restrict__ idx,
                  const void* __restrict__ coef, int coef_dtype, int64_t T, int s, int vec, int64_t tokens_per_cta,
                  float* __restrict__ scores) {
    extern __shared__ __align__(16) float p[];             // [HG][N]
    const int b = blockIdx.x;
    const int64_t t0 = (int64_t)blockIdx.y * tokens_per_cta;
    const int64_t t1 = t0 + tokens_per_cta < T ? t0 + tokens_per_cta : T;
    for (int h0 = 0; h0 < H; h0 += HG) {
        const int hg = H - h0 < HG ? H - h0 : HG;
        __syncthreads();
        const float* src = P + ((int64_t)b * H + h0) * N;
        for (int j = threadIdx.x; j < hg * N; j += NTS) p[j] = src[j];
        __syncthreads();
        for (int64_t t = t0 + threadIdx.x; t < t1; t += NTS) {
            const int64_t o = ((int64_t)b * T + t) * s;
            float acc[8];
#pragma unroll
            for (int h = 0; h < 8; ++h) acc[h] = 0.f;
            if (vec) {
                for (int g0 = 0; g0 < s; g0 += 8) {
                    int i8[8];
                    float c8[8];
                    load_codes8(idx, coef, coef_dtype, o + g0, i8, c8);
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const int i = i8[g] < N ? i8[g] : N - 1;
#pragma unroll
                        for (int h = 0; h < 8; ++h)
                            if (h < hg) acc[h] = fmaf(c8[g], p[h * N + i], acc[h]);
                    }
                }
            } else {
                for (int g = 0; g < s; ++g) {
                    int i = idx[o + g];
                    i = i < N ? i : N - 1;
                    const float c = load_coef(coef, coef_dtype, o + g);
#pragma unroll
                    for (int h = 0; h < 8; ++h)
                        if (h < hg) acc[h] = fmaf(c, p[h * N + i], acc[h]);
                }
            }
#pragma unroll
            for (int h = 0; h < 8; ++h)
                if (h < hg) scores[((int64_t)b * H + h0 + h) * T + t] = acc[h];
        }
    }
}

__global__ void __launch_bounds__(NTS)
value_scatter_kernel(int N, const float* __restrict__ W, int H, int HG, const uint16_t* __restrict__ idx,
                     const void* __restrict__ coef, int coef_dtype, int64_t T, int s, int vec, int64_t tokens_per_cta,
                     float* __restrict__ A) {
    extern __shared__ __align__(16) float a[];             // [HG][N]
    const int b = blockIdx.x;
    const int64_t t0 = (int64_t)blockIdx.y * tokens_per_cta;
    const int64_t t1 = t0 + tokens_per_cta < T ? t0 + tokens_per_cta : T;
    for (int h0 = 0; h0 < H; h0 += HG) {
        const int hg = H - h0 < HG ? H - h0 : HG;
        __syncthreads();
        for (int j = threadIdx.x; j < hg * N; j += NTS) a[j] = 0.f;
        __syncthreads();
        for (int64_t t = t0 + threadIdx.x; t < t1; t += NTS) {
            const int64_t o = ((int64_t)b * T + t) * s;
            float w[8];
#pragma unroll
            for (int h = 0; h < 8; ++h) w[h] = h < hg ? W[((int64_t)b * H + h0 + h) * T + t] : 0.f;
            if (vec) {
                for (int g0 = 0; g0 < s; g0 += 8) {
                    int i8[8];
                    float c8[8];
                    load_codes8(idx, coef, coef_dtype, o + g0, i8, c8);
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const int i = i8[g] < N ? i8[g] : N - 1;
#pragma unroll
                        for (int h = 0; h < 8; ++h)
                            if (h < hg) atomicAdd(&a[h * N + i], w[h] * c8[g]);
                    }
                }
            } else {
                for (int g = 0; g < s; ++g) {
                    int i = idx[o + g];
                    i = i < N ? i : N - 1;
                    const float c = load_coef(coef, coef_dtype, o + g);
#pragma unroll
                    for (int h = 0; h < 8; ++h)
                        if (h < hg) atomicAdd(&a[h * N + i], w[h] * c);
                }
            }
        }
        __syncthreads();
        float* dst = A + ((int64_t)b * H + h0) * N;
        for (int j = threadIdx.x; j < hg * N; j += NTS)
            if (a[j] != 0.f) atomicAdd(&dst[j], a[j]);
    }
}

// Query heads whose N-vectors fit in shared memory together (at most 8).
int head_group(int N, int H) {
    int hg = (200 * 1024) / (N * 4);
    if (hg > 8) hg = 8;
    if (hg > H) hg = H;
    return hg;
}

// Token ranges per code stream: enough CTAs to fill the GPU about twice, at least 1024 tokens each.
int64_t tokens_per_cta(int B, int64_t T) {
    int64_t splits = (2 * (int64_t)sm_count() + B - 1) / B;
    if (splits < 1) splits = 1;
    int64_t per = (T + splits - 1) / splits;
    if (per < 1024) per = 1024;
    return per;
}

}  // namespace

size_t attn_scratch_bytes(int B, int H, int N) { return (size_t)B * H * N * sizeof(float); }

int launch_key_scores(const AttnArgs& a, float* P) {
    if (a.B == 0 || a.T == 0 || a.H == 0) return CSR_OK;
    const int hg = head_group(a.N, a.H);
    if (hg < 1) return fail(CSR_ERR_UNSUPPORTED, "N = %d: one head's N fp32 values do not fit in shared memory", a.N);
    const int R = a.B * a.H;
    const dim3 pgrid((a.N + PA - 1) / PA, (R + QROWS - 1) / QROWS);
    if (a.d == 128)
        qd_kernel<128><<<pgrid, NT, 0, a.stream>>>(a.D, a.N, a.Q, a.q_dtype, R, a.scale, P);
    else
        qd_kernel<64><<<pgrid, NT, 0, a.stream>>>(a.D, a.N, a.Q, a.q_dtype, R, a.scale, P);
    const size_t smem = (size_t)hg * a.N * 4;
    const int64_t per = tokens_per_cta(a.B, a.T);
    const dim3 grid(a.B, (unsigned)((a.T + per - 1) / per));
    cudaError_t e = cudaFuncSetAttribute(key_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
        key_scores_kernel<<<grid, NTS, smem, a.stream>>>(P, a.N, a.H, hg, a.idx, a.coef, a.coef_dtype, a.T, a.s, a.s % 8 == 0,
                                                         per, a.out);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "key_scores launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

int launch_value_mix(const AttnArgs& a, float* A) {
    if (a.B == 0 || a.H == 0) return CSR_OK;
    const int R = a.B * a.H;
    if (a.T == 0) {
        cudaError_t e0 = cudaMemsetAsync(a.out, 0, (size_t)R * a.d * sizeof(float), a.stream);
        if (e0 != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e0));
        return CSR_OK;
    }
    const int hg = head_group(a.N, a.H);
    if (hg < 1) return fail(CSR_ERR_UNSUPPORTED, "N = %d: one head's N fp32 values do not fit in shared memory", a.N);
    cudaError_t e = cudaMemsetAsync(A, 0, attn_scratch_bytes(a.B, a.H, a.N), a.stream);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    const size_t smem = (size_t)hg * a.N * 4;
    const int64_t per = tokens_per_cta(a.B, a.T);
    const dim3 grid(a.B, (unsigned)((a.T + per - 1) / per));
    e = cudaFuncSetAttribute(value_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
        value_scatter_kernel<<<grid, NTS, smem, a.stream>>>(a.N, static_cast<const float*>(a.Q), a.H, hg, a.idx, a.coef,
                                                            a.coef_dtype, a.T, a.s, a.s % 8 == 0, per, A);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "value_scatter launch: %s", cudaGetErrorString(e));
    // out = A D: row blocks of 16; with few row blocks the atoms are split over CTAs as well
    const int row_blocks = (R + OR - 1) / OR;
    int slices = 4 * sm_count() / row_blocks;
    const int max_slices = (a.N + 255) / 256;
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    int per_slice = ((a.N + slices - 1) / slices + OA - 1) / OA * OA;
    slices = (a.N + per_slice - 1) / per_slice;
    if (slices > 1) {
        e = cudaMemsetAsync(a.out, 0, (size_t)R * a.d * sizeof(float), a.stream);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    }
    const dim3 ogrid(row_blocks, slices);
    if (a.d == 128)
        ad_kernel<128><<<ogrid, NT, 0, a.stream>>>(a.D, a.N, A, R, per_slice, slices > 1, a.out);
    else
        ad_kernel<64><<<ogrid, NT, 0, a.stream>>>(a.D, a.N, A, R, per_slice, slices > 1, a.out);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "value_mix launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace csr
