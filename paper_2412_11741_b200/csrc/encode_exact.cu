// Correctness-mode matching pursuit (paper Eq. 2-4) on the plain ALUs.
//
// One CTA owns a tile of 64 input rows for all s iterations.  Per iteration it sweeps the
// dictionary in tiles of 128 atoms: an fp32 register-tiled product (each thread 4 rows x
// 8 atoms, fp32 FMA, k ascending) gives the correlations, and every thread keeps, for
// each of its rows, the largest and second largest |correlation| seen so far.  Nothing
// of the M x N correlation matrix is written anywhere.
//
// fp32 rounding can reorder two correlations that are closer than about
// 2 * 128 * 2^-24 * ||R||.  A row whose two largest values are inside that band is
// re-scored: one warp recomputes all N correlations of that row in fp64 and takes the
// arg-max with the lowest-index tie rule.  The coefficient (Eq. 2, signed) is always an
// fp64 dot product of the fp64 residual with the fp32 atom, and the residual update
// (Eq. 4) is fp64; the fp32 copy of the residual that feeds the next sweep is rounded
// from it.
#include "common.cuh"

namespace csr {
namespace {

constexpr int BM = 64;        // rows per CTA
constexpr int BN = 128;       // atoms per dictionary tile
constexpr int BK = 16;        // channels per staged chunk
constexpr int NT = 256;       // threads per CTA
constexpr int AS_LD = BM + 4; // leading dimension of the transposed fp32 residual
constexpr int BS_LD = BN + 4;
// |fp32 dot - exact dot| <= d * 2^-24 * ||R|| * ||atom|| for d <= 128 sequential FMAs plus
// the rounding of R itself; two candidates can therefore swap when closer than twice that.
constexpr float kBandRel = 1.6e-5f;

template <int D_>
struct Smem {
    double Rd[BM][D_];          // fp64 residual, row-major
    float As[D_][AS_LD];        // fp32 residual, transposed: As[k][row]
    float Bs[2][BK][BS_LD];     // staged dictionary chunk, transposed: Bs[k][atom]
    float best[BM];
    float second[BM];
    int bidx[BM];
    float band[BM];
};

__device__ __forceinline__ float load_x(const void* X, int x_dtype, int64_t off) {
    if (x_dtype == CSR_DTYPE_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(X)[off]);
    return reinterpret_cast<const float*>(X)[off];
}

struct Top2 {
    float best, second;
    int idx;
};

__device__ __forceinline__ void top2_push(Top2& t, float a, int n) {
    if (a > t.best) {
        t.second = t.best;
        t.best = a;
        t.idx = n;
    } else if (a > t.second) {
        t.second = a;
    }
}

__device__ __forceinline__ void top2_merge(Top2& t, float ob, float os, int oi) {
    bool other_wins = (ob > t.best) || (ob == t.best && oi < t.idx);
    float loser = other_wins ? t.best : ob;
    float sec = fmaxf(fmaxf(t.second, os), loser);
    if (other_wins) {
        t.best = ob;
        t.idx = oi;
    }
    t.second = sec;
}

template <int D_>
__global__ void __launch_bounds__(NT, 1)
encode_exact_kernel(const float* __restrict__ D, const void* __restrict__ X, int x_dtype, int64_t ldx, int64_t M, int N,
                    int s, uint16_t* __restrict__ out_idx, void* __restrict__ out_coef, int coef_dtype, int64_t ldc) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem<D_>& sm = *reinterpret_cast<Smem<D_>*>(smem_raw);

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int tx = tid & 15;   // atom group
    const int ty = tid >> 4;   // row group: rows ty*4 .. ty*4+3
    const int64_t n_tiles = (M + BM - 1) / BM;
    const int n_btiles = (N + BN - 1) / BN;
    constexpr int KCH = D_ / BK;

    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t row0 = tile * BM;
        __syncthreads();
        // R_0 = x
        for (int r = warp; r < BM; r += NT / 32) {
            const int64_t m = row0 + r;
            double nn = 0.0;
            for (int k = lane; k < D_; k += 32) {
                float v = (m < M) ? load_x(X, x_dtype, m * ldx + k) : 0.f;
                sm.Rd[r][k] = (double)v;
                sm.As[k][r] = v;
                nn += (double)v * (double)v;
            }
            for (int o = 16; o; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
            if (lane == 0) sm.band[r] = kBandRel * (float)sqrt(nn);
        }
        __syncthreads();

        for (int g = 0; g < s; ++g) {
            Top2 top[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) top[i] = Top2{-1.f, -1.f, 0};

            // ---- sweep over the dictionary (Eq. 2-3) ----
            const int total_chunks = n_btiles * KCH;
            float4 stage[2];
            auto gload = [&](int chunk) {
                const int bt = chunk / KCH, kc = chunk % KCH;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int f = tid + i * NT;
                    const int atom = f >> 2, kq = f & 3;
                    const int n = bt * BN + atom;
                    stage[i] = (n < N) ? *reinterpret_cast<const float4*>(D + (int64_t)n * D_ + kc * BK + kq * 4)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            };
            auto sstore = [&](int buf) {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int f = tid + i * NT;
                    const int atom = f >> 2, kq = f & 3;
                    sm.Bs[buf][kq * 4 + 0][atom] = stage[i].x;
                    sm.Bs[buf][kq * 4 + 1][atom] = stage[i].y;
                    sm.Bs[buf][kq * 4 + 2][atom] = stage[i].z;
                    sm.Bs[buf][kq * 4 + 3][atom] = stage[i].w;
                }
            };
            gload(0);
            sstore(0);
            __syncthreads();
            float acc[4][8];
            for (int chunk = 0; chunk < total_chunks; ++chunk) {
                const int buf = chunk & 1;
                const int kc = chunk % KCH;
                if (kc == 0) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
                }
                if (chunk + 1 < total_chunks) gload(chunk + 1);
#pragma unroll
                for (int k = 0; k < BK; ++k) {
                    const float4 a4 = *reinterpret_cast<const float4*>(&sm.As[kc * BK + k][ty * 4]);
                    const float4 b0 = *reinterpret_cast<const float4*>(&sm.Bs[buf][k][tx * 4]);
                    const float4 b1 = *reinterpret_cast<const float4*>(&sm.Bs[buf][k][64 + tx * 4]);
                    const float a[4] = {a4.x, a4.y, a4.z, a4.w};
                    const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
                }
                if (kc == KCH - 1) {
                    const int nb = (chunk / KCH) * BN;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int n = nb + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
                        if (n < N) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) top2_push(top[i], fabsf(acc[i][j]), n);
                        }
                    }
                }
                if (chunk + 1 < total_chunks) sstore(buf ^ 1);
                __syncthreads();
            }
            // Each thread visited its atoms in ascending order, so its strict ">" kept the
            // lowest index among equal values; top2_merge applies the same rule across the
            // 16 threads that share a row.  Equal fp32 values are re-scored in fp64 anyway.
#pragma unroll
            for (int i = 0; i < 4; ++i) {
#pragma unroll
                for (int o = 8; o; o >>= 1) {
                    const float ob = __shfl_xor_sync(0xffffffffu, top[i].best, o);
                    const float os = __shfl_xor_sync(0xffffffffu, top[i].second, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, top[i].idx, o);
                    top2_merge(top[i], ob, os, oi);
                }
                if (tx == 0) {
                    sm.best[ty * 4 + i] = top[i].best;
                    sm.second[ty * 4 + i] = top[i].second;
                    sm.bidx[ty * 4 + i] = top[i].idx;
                }
            }
            __syncthreads();

            // ---- pick, coefficient and residual update (Eq. 2-4), one warp per row ----
            for (int r = warp; r < BM; r += NT / 32) {
                const int64_t m = row0 + r;
                if (m >= M) continue;
                int bi = sm.bidx[r];
                const bool unresolved = (N > 1) && (sm.best[r] - sm.second[r] <= sm.band[r]);
                const double* Rr = sm.Rd[r];
                if (unresolved) {
                    double bb = -1.0;
                    int bn = 0;
                    for (int n = lane; n < N; n += 32) {
                        const float4* dn = reinterpret_cast<const float4*>(D + (int64_t)n * D_);
                        double c = 0.0;
#pragma unroll 4
                        for (int q = 0; q < D_ / 4; ++q) {
                            const float4 v = dn[q];
                            c = fma(Rr[4 * q + 0], (double)v.x, c);
                            c = fma(Rr[4 * q + 1], (double)v.y, c);
                            c = fma(Rr[4 * q + 2], (double)v.z, c);
                            c = fma(Rr[4 * q + 3], (double)v.w, c);
                        }
                        const double a = fabs(c);
                        if (a > bb) {
                            bb = a;
                            bn = n;
                        }
                    }
                    for (int o = 16; o; o >>= 1) {
                        const double ob = __shfl_xor_sync(0xffffffffu, bb, o);
                        const int on = __shfl_xor_sync(0xffffffffu, bn, o);
                        if (ob > bb || (ob == bb && on < bn)) {
                            bb = ob;
                            bn = on;
                        }
                    }
                    bi = bn;
                }
                const float* db = D + (int64_t)bi * D_;
                double part = 0.0;
                for (int k = lane; k < D_; k += 32) part = fma(Rr[k], (double)db[k], part);
                for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                const double c = part;
                double nn = 0.0;
                for (int k = lane; k < D_; k += 32) {
                    const double v = sm.Rd[r][k] - c * (double)db[k];
                    sm.Rd[r][k] = v;
                    sm.As[k][r] = (float)v;
                    nn += v * v;
                }
                for (int o = 16; o; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
                if (lane == 0) {
                    sm.band[r] = kBandRel * (float)sqrt(nn);
                    out_idx[m * ldc + g] = (uint16_t)bi;
                    const float cf = (float)c;
                    if (coef_dtype == CSR_DTYPE_F16)
                        reinterpret_cast<__half*>(out_coef)[m * ldc + g] = __float2half_rn(cf);
                    else
                        reinterpret_cast<float*>(out_coef)[m * ldc + g] = cf;
                }
            }
            __syncthreads();
        }
    }
}

}  // namespace

int launch_encode_exact(const EncodeArgs& a) {
    const int64_t n_tiles = (a.M + BM - 1) / BM;
    if (n_tiles == 0) return CSR_OK;
    const int grid = (int)(n_tiles < (int64_t)sm_count() ? n_tiles : (int64_t)sm_count());
    cudaError_t e;
    if (a.d == 128) {
        const size_t smem = sizeof(Smem<128>);
        e = cudaFuncSetAttribute(encode_exact_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        encode_exact_kernel<128><<<grid, NT, smem, a.stream>>>(a.D, a.X, a.x_dtype, a.ldx, a.M, a.N, a.s,
                                                               a.out_idx, a.out_coef, a.coef_dtype, a.ld_code);
    } else {
        const size_t smem = sizeof(Smem<64>);
        e = cudaFuncSetAttribute(encode_exact_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        encode_exact_kernel<64><<<grid, NT, smem, a.stream>>>(a.D, a.X, a.x_dtype, a.ldx, a.M, a.N, a.s,
                                                              a.out_idx, a.out_coef, a.coef_dtype, a.ld_code);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "encode_exact launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace csr
