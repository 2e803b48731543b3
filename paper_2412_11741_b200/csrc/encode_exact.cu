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
// re-scored by the whole CTA: an fp32 pass collects the atoms within the band of the
// maximum, their correlations are recomputed in fp64 and the largest is taken, as an
// arg-max with the lowest-index tie rule.  The coefficient (Eq. 2, signed) is always an
// fp64 dot product of the fp64 residual with the fp32 atom, and the residual update
// (Eq. 4) is fp64; the fp32 copy of the residual that feeds the next sweep is rounded
// from it.
#include "exact_common.cuh"

namespace csr {
namespace {

using namespace exact;

template <int D_>
struct Smem {
    double Rd[BM][D_];          // fp64 residual, row-major
    float As[D_][AS_LD];        // fp32 residual, transposed: As[k][row]
    float Bs[2][BK][BS_LD];     // staged dictionary chunk, transposed: Bs[k][atom]
    float best[BM];
    float second[BM];
    int bidx[BM];
    float band[BM];
    RescoreSmem rs;
};

template <int D_>
__global__ void __launch_bounds__(NT, 2)
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
            sweep_tiles<D_>(D, N, 0, n_btiles, sm.As, sm.Bs, top);
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

            // ---- rows that fp32 cannot decide are re-scored by the whole CTA ----
            for (int r = 0; r < BM; ++r) {
                const bool unresolved = (row0 + r < M) && (N > 1) && (sm.best[r] > 0.f) &&
                                        (sm.best[r] - sm.second[r] <= sm.band[r]);
                if (!unresolved) continue;                // uniform over the CTA
                const int bn = rescore_cta<D_>(D, N, sm.Rd[r], sm.best[r], sm.band[r], sm.rs);
                if (tid == 0) sm.bidx[r] = bn;
                __syncthreads();
            }
            // ---- pick, coefficient and residual update (Eq. 2-4), one warp per row ----
            for (int r = warp; r < BM; r += NT / 32) {
                const int64_t m = row0 + r;
                if (m >= M) continue;
                const int bi = sm.best[r] > 0.f ? sm.bidx[r] : 0;   // an all-zero sweep picks atom 0
                const double* Rr = sm.Rd[r];
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
    const int64_t resident = 2 * (int64_t)sm_count();   // two CTAs per SM
    const int grid = (int)(n_tiles < resident ? n_tiles : resident);
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
