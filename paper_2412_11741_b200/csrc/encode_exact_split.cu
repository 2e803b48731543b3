// Correctness-mode matching pursuit (paper Eq. 2-4) for FEW rows: the encode of the
// vectors one decoding step adds ("De-Sparse to restore": new keys and values are encoded
// as they are produced).
//
// With few rows the one-CTA-per-row-tile encoder leaves most of the GPU idle and takes
// s * N * d serial FMAs per lane.  Here the dictionary is split across CTAs instead: per
// iteration one launch sweeps (row tile, dictionary slice) pairs on all SMs and writes each
// row's two largest |correlations| of every slice; a second, small launch merges the slices
// per row (lowest atom among equal values), re-scores unresolved rows in fp64, takes the
// fp64 coefficient, updates the fp64 residual and writes the fp32 residual the next sweep
// reads.  Arithmetic, summation order and tie rules are those of the one-CTA encoder, so
// both return identical codes.  Kernels of consecutive iterations are ordered by the
// stream; no kernel waits on another.
//
// Scratch per row (global, L2 resident): fp64 residual (8d B), fp32 residual (4d B), band
// (4 B), and 12 B per dictionary slice.
#include "exact_common.cuh"

namespace csr {
namespace {

using namespace exact;

struct Partial {
    float best, second;
    int idx;
};

template <int D_>
struct SplitSmem {
    float As[D_][AS_LD];
    float Bs[2][BK][BS_LD];
};

// R_0 = x: fp64 and fp32 copies of the residual and the band inside which fp32 cannot order
// two correlations.  One warp per row.
template <int D_>
__global__ void split_init_kernel(const void* __restrict__ X, int x_dtype, int64_t ldx, int64_t M, double* __restrict__ Rd,
                                  float* __restrict__ Rf, float* __restrict__ band) {
    const int lane = threadIdx.x & 31;
    const int64_t m = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (m >= M) return;
    double nn = 0.0;
    for (int k = lane; k < D_; k += 32) {
        const float v = load_x(X, x_dtype, m * ldx + k);
        Rd[m * D_ + k] = (double)v;
        Rf[m * D_ + k] = v;
        nn += (double)v * (double)v;
    }
    for (int o = 16; o; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
    if (lane == 0) band[m] = kBandRel * (float)sqrt(nn);
}

// blockIdx.x = row tile, blockIdx.y = dictionary slice (tiles_per_slice tiles of 128 atoms).
template <int D_>
__global__ void __launch_bounds__(NT, 1)
split_sweep_kernel(const float* __restrict__ D, const float* __restrict__ Rf, int64_t M, int N, int tiles_per_slice,
                   Partial* __restrict__ part) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SplitSmem<D_>& sm = *reinterpret_cast<SplitSmem<D_>*>(smem_raw);
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t row0 = (int64_t)blockIdx.x * BM;
    const int n_btiles = (N + BN - 1) / BN;
    const int bt0 = blockIdx.y * tiles_per_slice;
    const int bt1 = min(bt0 + tiles_per_slice, n_btiles);
    // fp32 residual tile, transposed
    for (int f = tid; f < BM * (D_ / 4); f += NT) {
        const int r = f / (D_ / 4), q = f % (D_ / 4);
        const int64_t m = row0 + r;
        const float4 v = (m < M) ? *reinterpret_cast<const float4*>(Rf + m * D_ + 4 * q) : make_float4(0.f, 0.f, 0.f, 0.f);
        sm.As[4 * q + 0][r] = v.x;
        sm.As[4 * q + 1][r] = v.y;
        sm.As[4 * q + 2][r] = v.z;
        sm.As[4 * q + 3][r] = v.w;
    }
    __syncthreads();
    Top2 top[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) top[i] = Top2{-1.f, -1.f, 0};
    sweep_tiles<D_>(D, N, bt0, bt1, sm.As, sm.Bs, top);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int o = 8; o; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, top[i].best, o);
            const float os = __shfl_xor_sync(0xffffffffu, top[i].second, o);
            const int oi = __shfl_xor_sync(0xffffffffu, top[i].idx, o);
            top2_merge(top[i], ob, os, oi);
        }
        const int64_t m = row0 + ty * 4 + i;
        if (tx == 0 && m < M) part[m * gridDim.y + blockIdx.y] = Partial{top[i].best, top[i].second, top[i].idx};
    }
}

// Eight rows per CTA, one warp each: merge the slices, pick (Eq. 2-3), coefficient and
// residual update (Eq. 4).  A row whose two largest fp32 values are too close to call is
// re-scored by the whole CTA, because one warp alone would hold up the whole iteration.
// An all-zero sweep (zero residual) picks atom 0 without re-scoring.
constexpr int UPD_ROWS = NT / 32;

template <int D_>
__global__ void __launch_bounds__(NT)
split_update_kernel(const float* __restrict__ D, int N, int64_t M, int n_slices, const Partial* __restrict__ part,
                    double* __restrict__ Rd, float* __restrict__ Rf, float* __restrict__ band, int g,
                    uint16_t* __restrict__ out_idx, void* __restrict__ out_coef, int coef_dtype, int64_t ldc) {
    __shared__ int pick[UPD_ROWS];
    __shared__ int unresolved[UPD_ROWS];
    __shared__ float sbest[UPD_ROWS];
    __shared__ RescoreSmem rs;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t m = (int64_t)blockIdx.x * UPD_ROWS + warp;
    if (m < M) {
        Top2 t{-1.f, -1.f, 0};
        for (int j = lane; j < n_slices; j += 32) {
            const Partial p = part[m * n_slices + j];
            if (p.best >= 0.f) top2_merge(t, p.best, p.second, p.idx);
        }
        for (int o = 16; o; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, t.best, o);
            const float os = __shfl_xor_sync(0xffffffffu, t.second, o);
            const int oi = __shfl_xor_sync(0xffffffffu, t.idx, o);
            top2_merge(t, ob, os, oi);
        }
        if (lane == 0) {
            pick[warp] = t.best > 0.f ? t.idx : 0;
            sbest[warp] = t.best;
            unresolved[warp] = (N > 1 && t.best > 0.f && t.best - t.second <= band[m]) ? 1 : 0;
        }
    } else if (lane == 0) {
        unresolved[warp] = 0;
    }
    __syncthreads();
    for (int r = 0; r < UPD_ROWS; ++r) {
        if (!unresolved[r]) continue;                     // uniform over the CTA
        const int64_t mr = (int64_t)blockIdx.x * UPD_ROWS + r;
        const int bn = rescore_cta<D_>(D, N, Rd + mr * D_, sbest[r], band[mr], rs);
        if (threadIdx.x == 0) pick[r] = bn;
        __syncthreads();
    }
    if (m >= M) return;
    double* Rr = Rd + m * D_;
    const int bi = pick[warp];
    const float* db = D + (int64_t)bi * D_;
    double part_c = 0.0;
    for (int k = lane; k < D_; k += 32) part_c = fma(Rr[k], (double)db[k], part_c);
    for (int o = 16; o; o >>= 1) part_c += __shfl_xor_sync(0xffffffffu, part_c, o);
    const double c = part_c;
    double nn = 0.0;
    for (int k = lane; k < D_; k += 32) {
        const double v = Rr[k] - c * (double)db[k];
        Rr[k] = v;
        Rf[m * D_ + k] = (float)v;
        nn += v * v;
    }
    for (int o = 16; o; o >>= 1) nn += __shfl_xor_sync(0xffffffffu, nn, o);
    if (lane == 0) {
        band[m] = kBandRel * (float)sqrt(nn);
        out_idx[m * ldc + g] = (uint16_t)bi;
        const float cf = (float)c;
        if (coef_dtype == CSR_DTYPE_F16)
            reinterpret_cast<__half*>(out_coef)[m * ldc + g] = __float2half_rn(cf);
        else
            reinterpret_cast<float*>(out_coef)[m * ldc + g] = cf;
    }
}

struct Plan {
    int n_tiles, n_slices, tiles_per_slice;
};

// Slices are whole 128-atom tiles; as many as fill the GPU once, none empty.
Plan make_plan(int64_t M, int N) {
    Plan p;
    p.n_tiles = (int)((M + BM - 1) / BM);
    const int n_btiles = (N + BN - 1) / BN;
    int want = sm_count() / p.n_tiles;
    if (want < 1) want = 1;
    if (want > n_btiles) want = n_btiles;
    p.tiles_per_slice = (n_btiles + want - 1) / want;
    p.n_slices = (n_btiles + p.tiles_per_slice - 1) / p.tiles_per_slice;
    return p;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

template <int D_>
int run(const EncodeArgs& a, void* scratch, const Plan& pl) {
    char* base = static_cast<char*>(scratch);
    double* Rd = reinterpret_cast<double*>(base);
    base += align256((size_t)a.M * D_ * 8);
    float* Rf = reinterpret_cast<float*>(base);
    base += align256((size_t)a.M * D_ * 4);
    float* band = reinterpret_cast<float*>(base);
    base += align256((size_t)a.M * 4);
    Partial* part = reinterpret_cast<Partial*>(base);
    const size_t smem = sizeof(SplitSmem<D_>);
    cudaError_t e = cudaFuncSetAttribute(split_sweep_kernel<D_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const int wpb = 4;
    const int row_blocks = (int)((a.M + wpb - 1) / wpb);
    const int upd_blocks = (int)((a.M + UPD_ROWS - 1) / UPD_ROWS);
    split_init_kernel<D_><<<row_blocks, wpb * 32, 0, a.stream>>>(a.X, a.x_dtype, a.ldx, a.M, Rd, Rf, band);
    for (int g = 0; g < a.s; ++g) {
        split_sweep_kernel<D_><<<dim3(pl.n_tiles, pl.n_slices), NT, smem, a.stream>>>(a.D, Rf, a.M, a.N, pl.tiles_per_slice,
                                                                                      part);
        split_update_kernel<D_><<<upd_blocks, UPD_ROWS * 32, 0, a.stream>>>(a.D, a.N, a.M, pl.n_slices, part, Rd, Rf, band,
                                                                            g, a.out_idx, a.out_coef, a.coef_dtype,
                                                                            a.ld_code);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "encode_exact_split launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace

bool encode_exact_split_applies(int64_t M, int N) {
    if (M <= 0) return false;
    const int64_t n_tiles = (M + BM - 1) / BM;
    // worth it while a row tile per CTA would leave at least half of the SMs idle
    return n_tiles * 2 <= sm_count() && N > BN;
}

size_t encode_exact_split_scratch_bytes(int64_t M, int d, int N) {
    const Plan pl = make_plan(M, N);
    return align256((size_t)M * d * 8) + align256((size_t)M * d * 4) + align256((size_t)M * 4) +
           align256((size_t)M * pl.n_slices * sizeof(Partial));
}

int launch_encode_exact_split(const EncodeArgs& a, void* scratch) {
    if (a.M == 0) return CSR_OK;
    const Plan pl = make_plan(a.M, a.N);
    if (a.d == 128) return run<128>(a, scratch, pl);
    return run<64>(a, scratch, pl);
}

}  // namespace csr
