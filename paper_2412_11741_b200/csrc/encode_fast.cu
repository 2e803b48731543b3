// Fast matching pursuit (paper Eq. 2-4) on the sm_100a tensor cores.
//
// One persistent CTA per SM owns two tiles of 128 input rows at a time and keeps their
// residuals on chip for all s iterations:
//
//   - the residual tiles live in shared memory as bf16, in the K-major 128-byte-swizzled
//     layout tcgen05.mma reads (operand A);
//   - the bf16 copy of the dictionary (a few MB, L2 resident) streams through a ring of
//     shared-memory stages, 128 atoms per stage, fetched by TMA (operand B); each stage
//     is used by both row tiles, so every dictionary byte fetched feeds 256 rows;
//   - tcgen05.mma (M=128, N=128, K=16, bf16 x bf16 -> fp32) writes the 128 x 128
//     correlations of (row tile, atom tile) into one of four TMEM accumulators
//     (2 row tiles x 2 buffers x 128 columns = all 512 columns);
//   - eight epilogue warps (four per row tile, one thread per row) pull the
//     accumulators out with tcgen05.ld and keep a running arg-max of |correlation| per
//     row: each value's sign bit is cleared and its low 7 mantissa bits are replaced by
//     127 - column, so that one 3-input integer max per two values finds both the
//     largest magnitude and where it was.  The M x N correlations never leave the SM;
//   - at the end of a sweep every epilogue thread gathers its winning atom (bf16, from
//     L2), recomputes the signed coefficient as an fp32 dot product with its residual
//     row, subtracts coefficient * atom, writes the bf16 residual back into the operand
//     tile and releases the MMA warp for the next iteration;
//   - codes are collected per thread and written as 16-byte vectors (uint16 index,
//     fp16 or fp32 coefficient).
//
// Warp roles: warps 0-3 epilogue of row tile 0, warps 4-7 epilogue of row tile 1 (warp w
// reads TMEM lanes 32*(w%4) .. +31), warp 8 TMA producer, warp 9 TMEM owner and MMA
// issuer.  All hand-offs are mbarriers; every wait is bounded by a wall-clock limit,
// after which the CTA raises a flag in the status word, lets its copies land, frees
// its TMEM and exits.
#include <cuda.h>

#include "common.cuh"

namespace csr {
namespace {

constexpr int TILE_M = 128;
constexpr int TILE_N = 128;
constexpr int UMMA_K = 16;
constexpr int STAGES = 4;
constexpr int NT = 320;
constexpr int PRODUCER_WARP = 8;
constexpr int MMA_WARP = 9;
constexpr uint32_t TMEM_COLS = 512;
constexpr int CODE_BLOCK = 8;                         // codes collected before a flush
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // 2 s per wait

// ---------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t* dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 operands, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier gets one arrival once every tcgen05.mma issued so far by this thread is done.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// Waits for this thread's outstanding tcgen05.ld.  The registers are passed through the
// statement so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&v)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]), "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
                 :
                 : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes with
// the 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t desc = 0;
    desc |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    desc |= static_cast<uint64_t>(1) << 16;                  // leading byte offset (unused with swizzle)
    desc |= static_cast<uint64_t>(1024 >> 4) << 32;          // stride byte offset between 8-row groups
    desc |= static_cast<uint64_t>(1) << 46;                  // descriptor version of sm_100
    desc |= static_cast<uint64_t>(2) << 61;                  // 128-byte swizzle
    return desc;
}

// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((TILE_N >> 3) << 17) | ((TILE_M >> 4) << 24);

// ---------------------------------------------------------------------------------------
// shared memory
// ---------------------------------------------------------------------------------------
template <int D_>
struct FastSmem {
    static constexpr int kTileBytes = TILE_M * D_ * 2;   // one operand tile (A or B)
    alignas(1024) uint8_t A[2][kTileBytes];
    alignas(1024) uint8_t B[STAGES][kTileBytes];
    alignas(16) uint16_t code_idx[2 * TILE_M][CODE_BLOCK];
    alignas(16) float code_coef[2 * TILE_M][CODE_BLOCK];
    uint64_t full_b[STAGES];
    uint64_t empty_b[STAGES];
    uint64_t acc_full[2][2];
    uint64_t acc_empty[2][2];
    uint64_t res_ready[2];
    uint64_t drained;
    uint32_t tmem_base;
    volatile uint32_t abort;
};

struct WaitCtx {
    volatile uint32_t* abort;
    uint32_t* status;
};

// Waits for the phase with the given parity; gives up after WAIT_LIMIT_NS or when another
// thread of the CTA has given up.
__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, const WaitCtx& w) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1; it < (1u << 28); ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (*w.abort) return false;
            if (globaltimer_ns() - t0 > WAIT_LIMIT_NS) break;
        }
    }
    *w.abort = 1;
    atomicOr(w.status, kStatusTimeout);
    return false;
}

// Byte offset of 16-byte chunk `chunk` (8 channels) of row `r` inside an operand tile.
template <int D_>
__device__ __forceinline__ uint32_t swz_off(int r, int chunk) {
    const int khalf = chunk >> 3, cc = chunk & 7;
    return khalf * (TILE_M * 128) + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
}

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// max over 32 packed keys (|value| with the low 7 bits replaced by 127 - column)
template <int COL0>
__device__ __forceinline__ uint32_t chunk_key_max(const uint32_t (&v)[32], uint32_t m) {
    uint32_t m0 = m, m1 = 0, m2 = 0, m3 = 0;
#pragma unroll
    for (int j = 0; j < 32; j += 8) {
#define CSR_KEY(J) ((v[(J)] & 0x7FFFFF80u) | static_cast<uint32_t>(127 - (COL0 + (J))))
        m0 = __vimax3_u32(m0, CSR_KEY(j + 0), CSR_KEY(j + 1));
        m1 = __vimax3_u32(m1, CSR_KEY(j + 2), CSR_KEY(j + 3));
        m2 = __vimax3_u32(m2, CSR_KEY(j + 4), CSR_KEY(j + 5));
        m3 = __vimax3_u32(m3, CSR_KEY(j + 6), CSR_KEY(j + 7));
#undef CSR_KEY
    }
    return __vimax3_u32(__vimax3_u32(m0, m1, m2), m3, 0u);
}

// ---------------------------------------------------------------------------------------
// dictionary preparation: fp32 -> bf16 copy, same [N][d] layout
// ---------------------------------------------------------------------------------------
__global__ void dict_to_bf16_kernel(const float4* __restrict__ src, uint2* __restrict__ dst, int64_t n_vec4) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec4; i += (int64_t)gridDim.x * blockDim.x) {
        const float4 v = src[i];
        uint2 o;
        o.x = pack_bf16(v.x, v.y);
        o.y = pack_bf16(v.z, v.w);
        dst[i] = o;
    }
}

// ---------------------------------------------------------------------------------------
// the encoder
// ---------------------------------------------------------------------------------------
template <int D_>
__global__ void __launch_bounds__(NT, 1)
encode_fast_kernel(const __grid_constant__ CUtensorMap tmap_d, const uint16_t* __restrict__ Db,
                   const void* __restrict__ X, int x_dtype, int64_t M, int N, int s, uint16_t* __restrict__ out_idx,
                   void* __restrict__ out_coef, int coef_dtype, uint32_t* status) {
    using S = FastSmem<D_>;
    extern __shared__ uint8_t smem_raw[];
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int T = N / TILE_N;                               // dictionary tiles per sweep
    const int64_t n_pairs = (M + 2 * TILE_M - 1) / (2 * TILE_M);
    constexpr int KSTEPS = D_ / UMMA_K;
    constexpr int CHUNKS = D_ / 8;                          // 16-byte chunks per row
    constexpr uint32_t kStageBytes = S::kTileBytes;
    const WaitCtx wc{&sm.abort, status};

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(&sm.full_b[i], 1);
            mbar_init(&sm.empty_b[i], 1);
        }
        for (int t = 0; t < 2; ++t) {
            for (int b = 0; b < 2; ++b) {
                mbar_init(&sm.acc_full[t][b], 1);
                mbar_init(&sm.acc_empty[t][b], 4);
            }
            mbar_init(&sm.res_ready[t], TILE_M);
        }
        mbar_init(&sm.drained, 1);
        sm.abort = 0;
        fence_barrier_init();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(&sm.tmem_base, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm.tmem_base;

    if (warp == PRODUCER_WARP) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_d)) : "memory");
            uint32_t p = 0;
            bool ok = true;
            for (int64_t pair = blockIdx.x; pair < n_pairs && ok; pair += gridDim.x) {
                for (int g = 0; g < s && ok; ++g) {
                    for (int t = 0; t < T; ++t, ++p) {
                        const int stage = p % STAGES;
                        if (!wait_bounded(&sm.empty_b[stage], ((p / STAGES) & 1) ^ 1, wc)) {
                            ok = false;
                            break;
                        }
                        mbar_expect_tx(&sm.full_b[stage], kStageBytes);
#pragma unroll
                        for (int h = 0; h < D_ / 64; ++h)
                            tma_load_2d(&sm.B[stage][h * (TILE_N * 128)], &tmap_d, h * 64, t * TILE_N,
                                        &sm.full_b[stage]);
                    }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA goes away
                const uint32_t first = p > STAGES ? p - STAGES : 0;
                for (uint32_t q = first; q < p; ++q) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(&sm.full_b[q % STAGES], (q / STAGES) & 1))
                        if (globaltimer_ns() - t0 > 20000000ull) break;
                }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            uint32_t p = 0, accn = 0, steps = 0;
            bool ok = true;
            for (int64_t pair = blockIdx.x; pair < n_pairs && ok; pair += gridDim.x) {
                for (int g = 0; g < s && ok; ++g, ++steps) {
                    for (int t = 0; t < T && ok; ++t, ++p, ++accn) {
                        const int stage = p % STAGES;
                        const uint32_t buf = accn & 1;
                        if (!wait_bounded(&sm.full_b[stage], (p / STAGES) & 1, wc)) {
                            ok = false;
                            break;
                        }
                        for (int tile = 0; tile < 2; ++tile) {
                            if (t == 0 && !wait_bounded(&sm.res_ready[tile], steps & 1, wc)) {
                                ok = false;
                                break;
                            }
                            if (!wait_bounded(&sm.acc_empty[tile][buf], ((accn >> 1) & 1) ^ 1, wc)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after();
                            const uint32_t d_tmem = tmem_base + (tile * 2 + buf) * TILE_N;
                            const uint64_t a0 = make_smem_desc(smem_u32(&sm.A[tile][0]));
                            const uint64_t b0 = make_smem_desc(smem_u32(&sm.B[stage][0]));
#pragma unroll
                            for (int k = 0; k < KSTEPS; ++k) {
                                // 16 channels = 32 bytes inside a 128-byte swizzled row; the
                                // second 64-channel half is a separate block of TILE_M rows
                                const uint64_t off = static_cast<uint64_t>(((k >> 2) * (TILE_M * 128) + (k & 3) * 32) >> 4);
                                umma_bf16(d_tmem, a0 + off, b0 + off, kInstrDesc, k > 0 ? 1u : 0u);
                            }
                            umma_commit(&sm.acc_full[tile][buf]);
                        }
                        if (ok) umma_commit(&sm.empty_b[stage]);
                    }
                }
            }
            if (!ok) {
                // wait (bounded) until the tensor core has stopped writing TMEM
                umma_commit(&sm.drained);
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(&sm.drained, 0))
                    if (globaltimer_ns() - t0 > 20000000ull) break;
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int tile = warp >> 2;
        const int q = warp & 3;
        const int r = q * 32 + lane;                      // row inside the tile == TMEM lane
        const int slot = tile * TILE_M + r;               // row inside the CTA's pair
        uint8_t* Atile = &sm.A[tile][0];
        uint32_t accn = 0;
        bool ok = true;
        for (int64_t pair = blockIdx.x; pair < n_pairs && ok; pair += gridDim.x) {
            const int64_t m = pair * (2 * TILE_M) + slot;
            const bool valid = m < M;
            // ---- R_0 = x, rounded to bf16, into the operand tile ----
            if (x_dtype == CSR_DTYPE_BF16) {
                const uint4* src = reinterpret_cast<const uint4*>(X) + m * CHUNKS;
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (valid) v = __ldg(src + c);
                    *reinterpret_cast<uint4*>(Atile + swz_off<D_>(r, c)) = v;
                }
            } else {
                const float4* src = reinterpret_cast<const float4*>(X) + m * (CHUNKS * 2);
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
                    if (valid) {
                        a = __ldg(src + 2 * c);
                        b = __ldg(src + 2 * c + 1);
                    }
                    uint4 v;
                    v.x = pack_bf16(a.x, a.y);
                    v.y = pack_bf16(a.z, a.w);
                    v.z = pack_bf16(b.x, b.y);
                    v.w = pack_bf16(b.z, b.w);
                    *reinterpret_cast<uint4*>(Atile + swz_off<D_>(r, c)) = v;
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(&sm.res_ready[tile]);

            for (int g = 0; g < s && ok; ++g) {
                // ---- sweep: running arg-max of |correlation| over all atom tiles ----
                uint32_t best_key = 0, best_t = 0;
                for (int t = 0; t < T; ++t, ++accn) {
                    const uint32_t buf = accn & 1;
                    bool got = wait_bounded(&sm.acc_full[tile][buf], (accn >> 1) & 1, wc);
                    got = __all_sync(0xffffffffu, got);
                    if (!got) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + (tile * 2 + buf) * TILE_N;
                    uint32_t va[32], vb[32];
                    uint32_t key = 0;
                    tmem_ld32(taddr + 0, va);
                    tmem_wait_ld(va);
                    tmem_ld32(taddr + 32, vb);
                    key = chunk_key_max<0>(va, key);
                    tmem_wait_ld(vb);
                    tmem_ld32(taddr + 64, va);
                    key = chunk_key_max<32>(vb, key);
                    tmem_wait_ld(va);
                    tmem_ld32(taddr + 96, vb);
                    key = chunk_key_max<64>(va, key);
                    tmem_wait_ld(vb);
                    // every column of this accumulator is in registers: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.acc_empty[tile][buf]);
                    key = chunk_key_max<96>(vb, key);
                    if (key > best_key) {
                        best_key = key;
                        best_t = t;
                    }
                }
                if (!ok) break;
                // ---- pick, signed coefficient, residual update ----
                const int n = best_t * TILE_N + (127 - static_cast<int>(best_key & 127u));
                const uint4* arow = reinterpret_cast<const uint4*>(Db + static_cast<size_t>(n) * D_);
                uint4 atom[CHUNKS];
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) atom[c] = __ldg(arow + c);
                float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    const uint4 rv = *reinterpret_cast<const uint4*>(Atile + swz_off<D_>(r, c));
                    c0 = fmaf(bf_lo(rv.x), bf_lo(atom[c].x), c0);
                    c1 = fmaf(bf_hi(rv.x), bf_hi(atom[c].x), c1);
                    c2 = fmaf(bf_lo(rv.y), bf_lo(atom[c].y), c2);
                    c3 = fmaf(bf_hi(rv.y), bf_hi(atom[c].y), c3);
                    c0 = fmaf(bf_lo(rv.z), bf_lo(atom[c].z), c0);
                    c1 = fmaf(bf_hi(rv.z), bf_hi(atom[c].z), c1);
                    c2 = fmaf(bf_lo(rv.w), bf_lo(atom[c].w), c2);
                    c3 = fmaf(bf_hi(rv.w), bf_hi(atom[c].w), c3);
                }
                const float coef = (c0 + c1) + (c2 + c3);
                if (g + 1 < s) {
#pragma unroll
                    for (int c = 0; c < CHUNKS; ++c) {
                        uint4* p4 = reinterpret_cast<uint4*>(Atile + swz_off<D_>(r, c));
                        uint4 rv = *p4;
                        rv.x = pack_bf16(fmaf(-coef, bf_lo(atom[c].x), bf_lo(rv.x)), fmaf(-coef, bf_hi(atom[c].x), bf_hi(rv.x)));
                        rv.y = pack_bf16(fmaf(-coef, bf_lo(atom[c].y), bf_lo(rv.y)), fmaf(-coef, bf_hi(atom[c].y), bf_hi(rv.y)));
                        rv.z = pack_bf16(fmaf(-coef, bf_lo(atom[c].z), bf_lo(rv.z)), fmaf(-coef, bf_hi(atom[c].z), bf_hi(rv.z)));
                        rv.w = pack_bf16(fmaf(-coef, bf_lo(atom[c].w), bf_lo(rv.w)), fmaf(-coef, bf_hi(atom[c].w), bf_hi(rv.w)));
                        *p4 = rv;
                    }
                    fence_proxy_async_smem();
                    mbar_arrive(&sm.res_ready[tile]);
                }
                // ---- collect the code; flush eight at a time ----
                const int gi = g & (CODE_BLOCK - 1);
                sm.code_idx[slot][gi] = static_cast<uint16_t>(n);
                sm.code_coef[slot][gi] = coef;
                if ((gi == CODE_BLOCK - 1 || g == s - 1) && valid) {
                    const int g0 = g - gi;
                    const int64_t o = m * s + g0;
                    if (gi == CODE_BLOCK - 1 && (s & 7) == 0) {
                        *reinterpret_cast<uint4*>(out_idx + o) = *reinterpret_cast<const uint4*>(&sm.code_idx[slot][0]);
                        const float4 f0 = *reinterpret_cast<const float4*>(&sm.code_coef[slot][0]);
                        const float4 f1 = *reinterpret_cast<const float4*>(&sm.code_coef[slot][4]);
                        if (coef_dtype == CSR_DTYPE_F16) {
                            __half2 h0 = __floats2half2_rn(f0.x, f0.y), h1 = __floats2half2_rn(f0.z, f0.w);
                            __half2 h2 = __floats2half2_rn(f1.x, f1.y), h3 = __floats2half2_rn(f1.z, f1.w);
                            uint4 u;
                            u.x = *reinterpret_cast<uint32_t*>(&h0);
                            u.y = *reinterpret_cast<uint32_t*>(&h1);
                            u.z = *reinterpret_cast<uint32_t*>(&h2);
                            u.w = *reinterpret_cast<uint32_t*>(&h3);
                            *reinterpret_cast<uint4*>(reinterpret_cast<__half*>(out_coef) + o) = u;
                        } else {
                            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(out_coef) + o);
                            dst[0] = f0;
                            dst[1] = f1;
                        }
                    } else {
                        for (int j = 0; j <= gi; ++j) {
                            out_idx[o + j] = sm.code_idx[slot][j];
                            if (coef_dtype == CSR_DTYPE_F16)
                                reinterpret_cast<__half*>(out_coef)[o + j] = __float2half_rn(sm.code_coef[slot][j]);
                            else
                                reinterpret_cast<float*>(out_coef)[o + j] = sm.code_coef[slot][j];
                        }
                    }
                }
            }
        }
    }

    // ------------------------------ teardown ------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

template <int D_>
int launch(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status) {
    const size_t smem = sizeof(FastSmem<D_>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(encode_fast_kernel<D_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const int64_t n_pairs = (a.M + 2 * TILE_M - 1) / (2 * TILE_M);
    const int grid = (int)(n_pairs < (int64_t)sm_count() ? n_pairs : (int64_t)sm_count());
    encode_fast_kernel<D_><<<grid, NT, smem, a.stream>>>(tmap, Db, a.X, a.x_dtype, a.M, a.N, a.s, a.out_idx, a.out_coef,
                                                        a.coef_dtype, status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "encode_fast launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace

size_t encode_fast_workspace_bytes(int d, int N) { return (size_t)N * (size_t)d * 2; }

int launch_encode_fast(const EncodeArgs& a, void* workspace, uint32_t* status) {
    if (a.M == 0) return CSR_OK;
    if ((reinterpret_cast<uintptr_t>(workspace) & 1023u) != 0)
        return fail(CSR_ERR_ALIGNMENT, "internal: dictionary scratch not 1024-byte aligned");
    EncodeTiledFn encode = get_encode_tiled();
    if (!encode) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");

    // bf16 copy of the dictionary
    const int64_t n_vec4 = (int64_t)a.N * a.d / 4;
    int blocks = (int)((n_vec4 + 255) / 256);
    if (blocks > 4 * sm_count()) blocks = 4 * sm_count();
    dict_to_bf16_kernel<<<blocks, 256, 0, a.stream>>>(reinterpret_cast<const float4*>(a.D),
                                                      reinterpret_cast<uint2*>(workspace), n_vec4);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "dict_to_bf16 launch: %s", cudaGetErrorString(e));

    CUtensorMap tmap;
    const cuuint64_t gdim[2] = {(cuuint64_t)a.d, (cuuint64_t)a.N};
    const cuuint64_t gstride[1] = {(cuuint64_t)a.d * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)TILE_N};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, workspace, gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);

    const uint16_t* Db = static_cast<const uint16_t*>(workspace);
    if (a.d == 128) return launch<128>(a, tmap, Db, status);
    return launch<64>(a, tmap, Db, status);
}

}  // namespace csr
