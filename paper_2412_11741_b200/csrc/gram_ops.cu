// Diversity loss of the dictionary training step ("NeuralDict": L_div = ||I - W^T W||_F^2 / N^2
// with one atom per column of W, i.e. ||D D^T - I||_F^2 / N^2 for D [N][d]) and its gradient
// (4 / N^2) (D D^T - I) D, both products on the tcgen05 tensor cores.
//
// The step's result must agree with an fp64 evaluation to about 1e-6 of an atom's entries, which
// plain bf16 (or tf32) operands do not give.  Every fp32 operand x is therefore split into
// hi = bf16(x) and lo = bf16(x - hi) (x = hi + lo to about 2^-17 relative), and a product a * b is
// taken as hi_a hi_b + hi_a lo_b + lo_a hi_b: three tcgen05.mma per K-step into one fp32
// accumulator in tensor memory (the dropped lo_a lo_b term is below 2^-16 of the product).
//
//   split_dict_kernel   D -> (Dh, Dl) [Np][d] and their transposes (DTh, DTl) [d][Np], Np = N
//                       rounded up to 128 atoms (the padding atoms are zero);
//   gram_kernel         a CTA keeps a block of 128 atoms i (hi and lo) in shared memory and
//                       sweeps blocks of 128 atoms j (TMA, two buffers): acc = D_i D_j^T, then the
//                       epilogue takes acc out of tensor memory, subtracts the identity, adds
//                       the squares to L_div and writes G - I, split again into hi and lo, to a
//                       scratch array [R][Np] (R rows per pass, sized to stay near the L2);
//   grad_kernel         grad[i][:] = (4 / N^2) sum_j (G - I)[i][j] D[j][:]: A = the scratch array
//                       (K = j contiguous), B = the transposed dictionary; the K range is cut into
//                       slices so that every SM has work, the slices' results are added with
//                       vector atomics.
// Warp roles in both kernels: warps 0-3 epilogue (thread = accumulator row = TMEM lane), warp 4
// TMA producer, warp 5 TMEM owner and MMA issuer.  Every wait is bounded, as in the encoder.
#include <cuda.h>

#include "common.cuh"
#include "tcgen05_common.cuh"

namespace csr {
namespace {

using namespace tc;

constexpr int GM = 128;                                   // rows of a tile = TMEM lanes
constexpr int KBLK = 64;                                  // K elements per shared-memory block (128-byte rows)
constexpr int NT = 192;
constexpr int PRODUCER_WARP = 4;
constexpr int MMA_WARP = 5;
constexpr int BLK_BYTES = GM * KBLK * 2;                  // 128 rows x 128 bytes = 16 KB

__device__ __forceinline__ uint32_t bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---------------------------------------------------------------------------------------
// operand split
// ---------------------------------------------------------------------------------------
// A 32 x 32 tile of D per block of 32 x 8 threads: hi and lo row-major as they are read,
// transposed through shared memory so that both layouts are written coalesced.
__global__ void split_dict_kernel(const float* __restrict__ D, int N, int d, int Np, __nv_bfloat16* __restrict__ Dh,
                                  __nv_bfloat16* __restrict__ Dl, __nv_bfloat16* __restrict__ DTh,
                                  __nv_bfloat16* __restrict__ DTl) {
    __shared__ __nv_bfloat16 th[32][33], tl[32][33];
    const int n0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;
    for (int r = ty; r < 32; r += 8) {
        const int n = n0 + r, c = c0 + tx;
        const float x = n < N ? D[(int64_t)n * d + c] : 0.f;
        const __nv_bfloat16 h = __float2bfloat16_rn(x);
        const __nv_bfloat16 l = __float2bfloat16_rn(x - __bfloat162float(h));
        Dh[(int64_t)n * d + c] = h;
        Dl[(int64_t)n * d + c] = l;
        th[r][tx] = h;
        tl[r][tx] = l;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int c = c0 + r, n = n0 + tx;
        DTh[(int64_t)c * Np + n] = th[tx][r];
        DTl[(int64_t)c * Np + n] = tl[tx][r];
    }
}

// ---------------------------------------------------------------------------------------
// G - I = D_i D_j^T - I, its squares, and its hi / lo split
// ---------------------------------------------------------------------------------------
template <int D_>
struct GramSmem {
    static constexpr int KB = D_ / KBLK;                  // K blocks of the whole contraction
    alignas(1024) uint8_t A[2][KB][BLK_BYTES];            // [hi, lo] of the atoms i (resident)
    alignas(1024) uint8_t B[2][2][KB][BLK_BYTES];         // [buffer][hi, lo] of the atoms j
    uint64_t a_full, b_full[2], b_empty[2], acc_full[2], acc_empty[2], drained;
    uint32_t tmem_base;
    volatile uint32_t abort;
};

template <int D_>
__global__ void __launch_bounds__(NT, 1)
gram_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_l, int N, int Np, int row0,
            int n_jsplit, __nv_bfloat16* __restrict__ Gh, __nv_bfloat16* __restrict__ Gl, double* __restrict__ losses,
            uint32_t* status, unsigned long long wait_limit_ns) {
    using S = GramSmem<D_>;
    constexpr int KB = S::KB;
    constexpr uint32_t kIdesc = instr_desc_bf16(GM, GM);
    constexpr uint32_t kTmemCols = 256;                   // two accumulators of 128 columns
    extern __shared__ uint8_t smem_raw[];
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ib = blockIdx.x / n_jsplit, js = blockIdx.x % n_jsplit;
    const int i0 = row0 + ib * GM;                        // first atom of this CTA's rows
    const int JT = Np / GM;
    const int jt0 = (int)((int64_t)JT * js / n_jsplit), jt1 = (int)((int64_t)JT * (js + 1) / n_jsplit);
    const WaitCtx wc{&sm.abort, status, wait_limit_ns};

    if (threadIdx.x == 0) {
        mbar_init(&sm.a_full, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.b_full[b], 1);
            mbar_init(&sm.b_empty[b], 1);
            mbar_init(&sm.acc_full[b], 1);
            mbar_init(&sm.acc_empty[b], 4);
        }
        mbar_init(&sm.drained, 1);
        sm.abort = 0;
        fence_barrier_init();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm.tmem_base;

    if (warp == PRODUCER_WARP) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_h)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_l)) : "memory");
            mbar_expect_tx(&sm.a_full, 2 * KB * BLK_BYTES);
            for (int kb = 0; kb < KB; ++kb) {
                tma_load_2d(&sm.A[0][kb][0], &map_h, kb * KBLK, i0, &sm.a_full);
                tma_load_2d(&sm.A[1][kb][0], &map_l, kb * KBLK, i0, &sm.a_full);
            }
            bool ok = true;
            uint32_t n = 0;
            for (int jt = jt0; jt < jt1 && ok; ++jt, ++n) {
                const int b = n & 1;
                if (!wait_bounded(&sm.b_empty[b], ((n >> 1) & 1) ^ 1, wc)) {
                    ok = false;
                    break;
                }
                mbar_expect_tx(&sm.b_full[b], 2 * KB * BLK_BYTES);
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(&sm.B[b][0][kb][0], &map_h, kb * KBLK, jt * GM, &sm.b_full[b]);
                    tma_load_2d(&sm.B[b][1][kb][0], &map_l, kb * KBLK, jt * GM, &sm.b_full[b]);
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA goes away
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(&sm.a_full, 0))
                    if (globaltimer_ns() - t0 > 20000000ull) break;
                for (uint32_t q = n > 2 ? n - 2 : 0; q < n; ++q) {
                    const unsigned long long t1 = globaltimer_ns();
                    while (!mbar_try_wait(&sm.b_full[q & 1], (q >> 1) & 1))
                        if (globaltimer_ns() - t1 > 20000000ull) break;
                }
            }
        }
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            bool ok = wait_bounded(&sm.a_full, 0, wc);
            uint32_t n = 0;
            for (int jt = jt0; jt < jt1 && ok; ++jt, ++n) {
                const int b = n & 1;
                if (!wait_bounded(&sm.b_full[b], (n >> 1) & 1, wc) || !wait_bounded(&sm.acc_empty[b], ((n >> 1) & 1) ^ 1, wc)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + b * GM;
#pragma unroll
                for (int kb = 0; kb < KB; ++kb) {
                    const uint64_t ah = make_smem_desc(smem_u32(&sm.A[0][kb][0])), al = make_smem_desc(smem_u32(&sm.A[1][kb][0]));
                    const uint64_t bh = make_smem_desc(smem_u32(&sm.B[b][0][kb][0])), bl = make_smem_desc(smem_u32(&sm.B[b][1][kb][0]));
#pragma unroll
                    for (int k = 0; k < KBLK / 16; ++k) {
                        const uint64_t off = static_cast<uint64_t>((k * 32) >> 4);       // 16 elements = 32 bytes
                        umma_bf16(d_tmem, ah + off, bh + off, kIdesc, (kb | k) ? 1u : 0u);
                        umma_bf16(d_tmem, ah + off, bl + off, kIdesc, 1u);
                        umma_bf16(d_tmem, al + off, bh + off, kIdesc, 1u);
                    }
                }
                umma_commit(&sm.b_empty[b]);
                umma_commit(&sm.acc_full[b]);
            }
            if (!ok) {
                umma_commit(&sm.drained);
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(&sm.drained, 0))
                    if (globaltimer_ns() - t0 > 20000000ull) break;
            }
        }
    } else {
        // epilogue: thread = row r of the tile = atom i0 + r
        const int r = warp * 32 + lane;
        const int i = i0 + r;
        const size_t grow = static_cast<size_t>(ib * GM + r) * Np;    // this row inside the scratch arrays
        float lsum = 0.f;
        uint32_t n = 0;
        bool ok = true;
        for (int jt = jt0; jt < jt1 && ok; ++jt, ++n) {
            const int b = n & 1;
            bool got = wait_bounded(&sm.acc_full[b], (n >> 1) & 1, wc);
            got = __all_sync(0xffffffffu, got);
            if (!got) {
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + b * GM;
            const bool diagonal = jt * GM == i0;          // this tile holds (i, i) for every row: column r
#pragma unroll 1
            for (int c = 0; c < GM / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(taddr + c * 32, v);
                tmem_wait_ld(v);
                if (diagonal && c == warp && i < N) {
#pragma unroll
                    for (int k = 0; k < 32; ++k)
                        if (k == lane) v[k] = __float_as_uint(__uint_as_float(v[k]) - 1.0f);
                }
                uint32_t hi[16], lo[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const float x0 = __uint_as_float(v[2 * k]), x1 = __uint_as_float(v[2 * k + 1]);
                    lsum = fmaf(x0, x0, lsum);
                    lsum = fmaf(x1, x1, lsum);
                    hi[k] = bf16x2(x0, x1);
                    lo[k] = bf16x2(x0 - __uint_as_float(hi[k] << 16), x1 - __uint_as_float(hi[k] & 0xFFFF0000u));
                }
                uint4* dh = reinterpret_cast<uint4*>(Gh + grow + jt * GM + c * 32);
                uint4* dl = reinterpret_cast<uint4*>(Gl + grow + jt * GM + c * 32);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    dh[q] = make_uint4(hi[4 * q], hi[4 * q + 1], hi[4 * q + 2], hi[4 * q + 3]);
                    dl[q] = make_uint4(lo[4 * q], lo[4 * q + 1], lo[4 * q + 2], lo[4 * q + 3]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.acc_empty[b]);
        }
        double ls = static_cast<double>(lsum);
        for (int o = 16; o; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
        if (lane == 0 && ok) atomicAdd(&losses[1], ls / (static_cast<double>(N) * static_cast<double>(N)));
    }

    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------
// grad = (4 / N^2) (G - I) D
// ---------------------------------------------------------------------------------------
constexpr int GRAD_STAGES = 3;
template <int D_>
struct GradSmem {
    static constexpr int B_BYTES = D_ * KBLK * 2;         // D_ channels x 128 bytes
    alignas(1024) uint8_t A[GRAD_STAGES][2][BLK_BYTES];   // [stage][hi, lo] of 128 rows of G - I, 64 atoms j
    alignas(1024) uint8_t B[GRAD_STAGES][2][B_BYTES];     // [stage][hi, lo] of D^T, the same 64 atoms j
    uint64_t full[GRAD_STAGES], empty[GRAD_STAGES], acc_full, drained;
    uint32_t tmem_base;
    volatile uint32_t abort;
};

template <int D_>
__global__ void __launch_bounds__(NT, 1)
grad_kernel(const __grid_constant__ CUtensorMap map_gh, const __grid_constant__ CUtensorMap map_gl,
            const __grid_constant__ CUtensorMap map_th, const __grid_constant__ CUtensorMap map_tl, int N, int Np, int row0,
            int n_ksplit, float* __restrict__ grad, uint32_t* status, unsigned long long wait_limit_ns) {
    using S = GradSmem<D_>;
    constexpr uint32_t kIdesc = instr_desc_bf16(GM, D_);
    constexpr uint32_t kTmemCols = D_;                    // 128 or 64: a power of two >= 32
    extern __shared__ uint8_t smem_raw[];
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ib = blockIdx.x / n_ksplit, ks = blockIdx.x % n_ksplit;
    const int KT = Np / KBLK;                             // K blocks of the whole contraction (atoms j)
    const int kb0 = (int)((int64_t)KT * ks / n_ksplit), kb1 = (int)((int64_t)KT * (ks + 1) / n_ksplit);
    const WaitCtx wc{&sm.abort, status, wait_limit_ns};

    if (threadIdx.x == 0) {
        for (int st = 0; st < GRAD_STAGES; ++st) {
            mbar_init(&sm.full[st], 1);
            mbar_init(&sm.empty[st], 1);
        }
        mbar_init(&sm.acc_full, 1);
        mbar_init(&sm.drained, 1);
        sm.abort = 0;
        fence_barrier_init();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm.tmem_base;

    if (warp == PRODUCER_WARP) {
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_gh)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_gl)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_th)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_tl)) : "memory");
            bool ok = true;
            uint32_t p = 0;
            for (int kb = kb0; kb < kb1 && ok; ++kb, ++p) {
                const int st = p % GRAD_STAGES;
                if (!wait_bounded(&sm.empty[st], ((p / GRAD_STAGES) & 1) ^ 1, wc)) {
                    ok = false;
                    break;
                }
                mbar_expect_tx(&sm.full[st], 2 * BLK_BYTES + 2 * S::B_BYTES);
                tma_load_2d(&sm.A[st][0][0], &map_gh, kb * KBLK, ib * GM, &sm.full[st]);
                tma_load_2d(&sm.A[st][1][0], &map_gl, kb * KBLK, ib * GM, &sm.full[st]);
                tma_load_2d(&sm.B[st][0][0], &map_th, kb * KBLK, 0, &sm.full[st]);
                tma_load_2d(&sm.B[st][1][0], &map_tl, kb * KBLK, 0, &sm.full[st]);
            }
            if (!ok) {
                for (uint32_t q = p > GRAD_STAGES ? p - GRAD_STAGES : 0; q < p; ++q) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(&sm.full[q % GRAD_STAGES], (q / GRAD_STAGES) & 1))
                        if (globaltimer_ns() - t0 > 20000000ull) break;
                }
            }
        }
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            bool ok = true;
            uint32_t p = 0;
            for (int kb = kb0; kb < kb1 && ok; ++kb, ++p) {
                const int st = p % GRAD_STAGES;
                if (!wait_bounded(&sm.full[st], (p / GRAD_STAGES) & 1, wc)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint64_t ah = make_smem_desc(smem_u32(&sm.A[st][0][0])), al = make_smem_desc(smem_u32(&sm.A[st][1][0]));
                const uint64_t bh = make_smem_desc(smem_u32(&sm.B[st][0][0])), bl = make_smem_desc(smem_u32(&sm.B[st][1][0]));
#pragma unroll
                for (int k = 0; k < KBLK / 16; ++k) {
                    const uint64_t off = static_cast<uint64_t>((k * 32) >> 4);
                    umma_bf16(tmem_base, ah + off, bh + off, kIdesc, (p | k) ? 1u : 0u);
                    umma_bf16(tmem_base, ah + off, bl + off, kIdesc, 1u);
                    umma_bf16(tmem_base, al + off, bh + off, kIdesc, 1u);
                }
                umma_commit(&sm.empty[st]);
            }
            if (ok) {
                umma_commit(&sm.acc_full);
            } else {
                umma_commit(&sm.drained);
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(&sm.drained, 0))
                    if (globaltimer_ns() - t0 > 20000000ull) break;
            }
        }
    } else if (kb1 > kb0) {
        const int r = warp * 32 + lane;
        const int i = row0 + ib * GM + r;
        bool got = wait_bounded(&sm.acc_full, 0, wc);
        got = __all_sync(0xffffffffu, got);
        if (got) {
            tc_fence_after();
            const float scale = 4.0f / (static_cast<float>(N) * static_cast<float>(N));
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
#pragma unroll 1
            for (int c = 0; c < D_ / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(taddr + c * 32, v);
                tmem_wait_ld(v);
                if (i < N) {
                    float4* dst = reinterpret_cast<float4*>(grad + static_cast<size_t>(i) * D_ + c * 32);
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 add = make_float4(scale * __uint_as_float(v[4 * q]), scale * __uint_as_float(v[4 * q + 1]),
                                                       scale * __uint_as_float(v[4 * q + 2]), scale * __uint_as_float(v[4 * q + 3]));
                        atomicAdd(dst + q, add);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static const EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

// bf16 matrix [rows][cols] (cols contiguous), boxes of box_rows x 64 columns, 128-byte swizzle.
int make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const cuuint64_t gdim[2] = {cols, rows};
    const cuuint64_t gstride[1] = {cols * 2};
    const cuuint32_t box[2] = {KBLK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return CSR_OK;
}

size_t align1k(size_t x) { return (x + 1023) / 1024 * 1024; }
int padded(int N) { return (N + GM - 1) / GM * GM; }
// rows of G - I held in scratch per pass: all of them up to 64 MiB (hi + lo), else as many blocks of
// 128 as fit
int pass_rows(int N) {
    const int Np = padded(N);
    const size_t budget = static_cast<size_t>(64) << 20;
    size_t rows = budget / (static_cast<size_t>(Np) * 4) / GM * GM;
    if (rows < GM) rows = GM;
    return rows < static_cast<size_t>(Np) ? static_cast<int>(rows) : Np;
}

template <int D_>
int run(const float* D, int N, float* grad_div, double* losses, void* scratch, uint32_t* status, cudaStream_t stream) {
    const int Np = padded(N), R = pass_rows(N);
    const size_t dict_b = align1k(static_cast<size_t>(Np) * D_ * 2), g_b = align1k(static_cast<size_t>(R) * Np * 2);
    char* q = static_cast<char*>(scratch);
    __nv_bfloat16* Dh = reinterpret_cast<__nv_bfloat16*>(q);
    __nv_bfloat16* Dl = reinterpret_cast<__nv_bfloat16*>(q + dict_b);
    __nv_bfloat16* DTh = reinterpret_cast<__nv_bfloat16*>(q + 2 * dict_b);
    __nv_bfloat16* DTl = reinterpret_cast<__nv_bfloat16*>(q + 3 * dict_b);
    __nv_bfloat16* Gh = reinterpret_cast<__nv_bfloat16*>(q + 4 * dict_b);
    __nv_bfloat16* Gl = reinterpret_cast<__nv_bfloat16*>(q + 4 * dict_b + g_b);
    split_dict_kernel<<<dim3(Np / 32, D_ / 32), dim3(32, 8), 0, stream>>>(D, N, D_, Np, Dh, Dl, DTh, DTl);
    CUtensorMap m_dh, m_dl, m_th, m_tl, m_gh, m_gl;
    if (int rc = make_map(&m_dh, Dh, Np, D_, GM)) return rc;
    if (int rc = make_map(&m_dl, Dl, Np, D_, GM)) return rc;
    if (int rc = make_map(&m_th, DTh, D_, Np, D_)) return rc;
    if (int rc = make_map(&m_tl, DTl, D_, Np, D_)) return rc;
    if (int rc = make_map(&m_gh, Gh, R, Np, GM)) return rc;
    if (int rc = make_map(&m_gl, Gl, R, Np, GM)) return rc;
    const size_t smem_gram = sizeof(GramSmem<D_>) + 1024, smem_grad = sizeof(GradSmem<D_>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(gram_kernel<D_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_gram);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(grad_kernel<D_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_grad);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const unsigned long long limit = options().wait_limit_ns;
    const int sms = sm_count();
    for (int row0 = 0; row0 < Np; row0 += R) {
        const int rows = Np - row0 < R ? Np - row0 : R;
        const int n_ib = rows / GM;
        int split = sms / n_ib;                           // as many CTAs per block of rows as fill the GPU once
        if (split < 1) split = 1;
        int jsplit = split < Np / GM ? split : Np / GM;
        int ksplit = split < 8 ? split : 8;
        if (ksplit > Np / KBLK) ksplit = Np / KBLK;
        gram_kernel<D_><<<n_ib * jsplit, NT, smem_gram, stream>>>(m_dh, m_dl, N, Np, row0, jsplit, Gh, Gl, losses, status, limit);
        grad_kernel<D_><<<n_ib * ksplit, NT, smem_grad, stream>>>(m_gh, m_gl, m_th, m_tl, N, Np, row0, ksplit, grad_div, status,
                                                                  limit);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "diversity gradient launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace

size_t div_grad_scratch_bytes(int N, int d) {
    const int Np = padded(N);
    return 4 * align1k(static_cast<size_t>(Np) * d * 2) + 2 * align1k(static_cast<size_t>(pass_rows(N)) * Np * 2) + 1024;
}

int launch_div_grad(const float* D, int N, int d, float* grad_div, double* losses, void* scratch, uint32_t* status,
                    cudaStream_t stream) {
    void* aligned = reinterpret_cast<void*>((reinterpret_cast<uintptr_t>(scratch) + 1023) & ~static_cast<uintptr_t>(1023));
    return d == 128 ? run<128>(D, N, grad_div, losses, aligned, status, stream) : run<64>(D, N, grad_div, losses, aligned, status, stream);
}

}  // namespace csr
