// Correctness-mode matching pursuit (paper Eq. 2-4) with the sweep on the sm_100a tensor cores.
//
// The picks must be those of an fp64 evaluation of the pursuit.  A bf16 product cannot decide
// them, but three can bound them: with r = rh + rl and d = dh + dl (each part bf16, the low part
// the rounded remainder), rh*dh + rl*dh + rh*dl differs from r*d by at most 3 * 2^-18 |r d| per
// channel, so the sum over the channels is within 1.2e-5 ||R|| ||d|| of the exact correlation; the
// tensor core adds the exact bf16 products in fp32.  Every correlation of a sweep is therefore
// known to within a band of a few 1e-5 ||R||, which decides all rows but the few whose two
// largest |correlations| are closer than that; for those the candidates are re-scored in fp64.
//
// One persistent CTA per SM owns two tiles of 128 rows for all s iterations:
//   - the fp64 residuals live in a per-CTA scratch area in global memory (256 KB, L2 resident);
//     their bf16 high and low parts are the tcgen05.mma A operands in shared memory (K-major,
//     128-byte swizzle, 2 row tiles x 2 parts);
//   - the dictionary's high and low parts (two bf16 arrays made once per call) stream through a
//     ring of 32 KB stages fetched by TMA: 64 channels of 256 atoms of one part per stage.  A
//     stage of high parts feeds four groups of MMAs (both parts of both row tiles), a stage of low
//     parts two (the high parts of both row tiles);
//   - each row tile has one 256-column fp32 accumulator in TMEM.  All eight epilogue warps drain
//     every accumulator: warp w reads the 32 TMEM lanes of w % 4 and the 128 columns of w / 4, i.e.
//     all of them sit in registers after one round of loads and the accumulator goes straight back
//     to the tensor core.  Each thread keeps the four largest keys of its half row, a key being
//     |value| with its seven lowest mantissa bits replaced by the column's tag, and where the
//     largest three came from.  Groups of four values are first reduced to their largest
//     magnitude and only groups within the band of the running maximum are inserted;
//   - at the end of a sweep the halves are merged through shared memory, and each warp settles
//     its 32 rows, eight lanes per row: rows whose best and second-best keys are further apart
//     than the band take the best; rows where only the second is inside the band compare the two
//     or three in fp64; rows where the fourth is inside too (about one in 10^6) are re-scored by the warp
//     over the whole dictionary (fp32 filter, then fp64).  Coefficient (Eq. 2, signed) and
//     residual update (Eq. 4) are fp64, as in the plain-ALU encoder.
// Warp roles: 0-7 epilogue, 8 TMA producer, 9 TMEM owner and MMA issuer.  All waits are bounded.
#include <cuda.h>

#include "common.cuh"
#include "tcgen05_common.cuh"

namespace csr {
namespace {

using namespace tc;

constexpr int TILE_M = 128;
constexpr int TILE_N = 256;
constexpr int UMMA_K = 16;
constexpr int STAGE_CH = 64;
constexpr int NT = 320;
constexpr int PRODUCER_WARP = 8;
constexpr int MMA_WARP = 9;
constexpr int ROWS = 2 * TILE_M;                          // rows a CTA holds at a time
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t kInstrDesc = instr_desc_bf16(TILE_M, TILE_N);
constexpr uint32_t kKeyMask = 0x7FFFFF80u;                // |value| without its seven lowest mantissa bits
constexpr uint32_t FULL = 0xffffffffu;
#ifndef CSR_TC_GROUP128
#define CSR_TC_GROUP128 2                                 // measured: 12-17 % faster than 1 at d = 128
#endif
// Half-width of the undecided zone relative to ||R||: twice the error of a tensor-core
// correlation (the split's 1.2e-5 plus the fp32 accumulation of 3 d products in groups of 16)
// plus the 2^-16 relative truncation of the keys.
constexpr float kBandRel = 1.0f / 4096.0f;

template <int D_>
struct TcSmem {
    static constexpr int kStages = D_ == 128 ? 3 : 4;
    static constexpr int kATileBytes = TILE_M * D_ * 2;          // one part of one row tile
    static constexpr int kStageBytes = TILE_N * STAGE_CH * 2;
    alignas(1024) uint8_t A[2][2][kATileBytes];                  // [row tile][high, low]
    alignas(1024) uint8_t B[kStages][kStageBytes];
    uint32_t xchg[5][TILE_M];                                    // one half's top four of a row tile (and the rows' bands)
    uint64_t full_b[kStages];
    uint64_t empty_b[kStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t res_ready;
    uint64_t drained;
    uint32_t tmem_base;
    volatile uint32_t abort;
};

__device__ __forceinline__ uint32_t swz_off(int r, int chunk) {
    const int kblock = chunk >> 3, cc = chunk & 7;
    return kblock * (TILE_M * 128) + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
}

// The four largest keys seen, in descending order, and the places (2 * dictionary tile + column
// half) the first three came from.
struct Top4 {
    uint32_t k0, k1, k2, k3;
    uint32_t i0, i1, i2;
};

__device__ __forceinline__ void top4_insert(Top4& q, uint32_t k, uint32_t id) {
    const bool p0 = k > q.k0, p1 = k > q.k1, p2 = k > q.k2;
    q.k3 = p2 ? q.k2 : max(q.k3, k);
    q.k2 = p1 ? q.k1 : (p2 ? k : q.k2);
    q.i2 = p1 ? q.i1 : (p2 ? id : q.i2);
    q.k1 = p0 ? q.k0 : (p1 ? k : q.k1);
    q.i1 = p0 ? q.i0 : (p1 ? id : q.i1);
    q.k0 = p0 ? k : q.k0;
    q.i0 = p0 ? id : q.i0;
}
// max(|a|, |b|, |c|)
__device__ __forceinline__ float absmax3(float a, float b, float c) {
    float r;
    asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// The filter's slow path, one copy for all groups: inserts the group's values (magnitudes a0..a3,
// `tag` = tag of the first) from the largest down until what is left is below the rising
// threshold: one trip for nearly every lane that gets here.  Returns the new state and threshold.
struct Top4Thr {
    Top4 q;
    float thr;
};
__device__ __noinline__ Top4Thr insert_group(Top4 q, float thr, float a0, float a1, float a2, float a3, uint32_t tag, uint32_t id,
                                             float band) {
    float gm = fmaxf(fmaxf(a0, a1), fmaxf(a2, a3));
#pragma unroll 1
    for (int trip = 0; trip < 4 && gm >= thr; ++trip) {
        // position of the largest magnitude left (the lowest column among equals)
        const uint32_t pos = a0 == gm ? 0u : (a1 == gm ? 1u : (a2 == gm ? 2u : 3u));
        top4_insert(q, (__float_as_uint(gm) & kKeyMask) | (tag - pos), id);
        a0 = pos == 0u ? -1.f : a0;
        a1 = pos == 1u ? -1.f : a1;
        a2 = pos == 2u ? -1.f : a2;
        a3 = pos == 3u ? -1.f : a3;
        thr = __uint_as_float(q.k0 & kKeyMask) - band;
        gm = fmaxf(fmaxf(a0, a1), fmaxf(a2, a3));
    }
    return Top4Thr{q, thr};
}

// Folds 32 columns of this thread's 128 into its top four; `tag0` is the tag of v[0] (tags fall
// with the column so that the lowest column wins among equal magnitudes).  Four values at a
// time are first reduced to their largest magnitude (two instructions) and only a group that
// reaches `thr`, the running maximum less the band, is inserted (a call: the sweep's code has
// to stay small enough for the instruction cache): whatever ends up within the band of the
// final maximum was within the band of the running one when it came by, so what the filter
// drops can never matter.
template <int J = 0>
__device__ __forceinline__ void chunk_top4(const uint32_t (&v)[32], Top4& q, uint32_t id, uint32_t tag0, float& thr, float band) {
    if constexpr (J < 32) {
        // eight values per test (one branch), four per call
        float ga = absmax3(__uint_as_float(v[J]), __uint_as_float(v[J + 1]), __uint_as_float(v[J + 2]));
        ga = fmaxf(ga, fabsf(__uint_as_float(v[J + 3])));
        float gb = absmax3(__uint_as_float(v[J + 4]), __uint_as_float(v[J + 5]), __uint_as_float(v[J + 6]));
        gb = fmaxf(gb, fabsf(__uint_as_float(v[J + 7])));
        if (fmaxf(ga, gb) >= thr) {
            if (ga >= thr) {
                const Top4Thr r = insert_group(q, thr, fabsf(__uint_as_float(v[J])), fabsf(__uint_as_float(v[J + 1])),
                                               fabsf(__uint_as_float(v[J + 2])), fabsf(__uint_as_float(v[J + 3])), tag0 - J, id, band);
                q = r.q;
                thr = r.thr;
            }
            if (gb >= thr) {
                const Top4Thr r = insert_group(q, thr, fabsf(__uint_as_float(v[J + 4])), fabsf(__uint_as_float(v[J + 5])),
                                               fabsf(__uint_as_float(v[J + 6])), fabsf(__uint_as_float(v[J + 7])), tag0 - J - 4, id, band);
                q = r.q;
                thr = r.thr;
            }
        }
        chunk_top4<J + 8>(v, q, id, tag0, thr, band);
    }
}

// Pulls this thread's 128 columns of an accumulator into registers, hands the accumulator back
// and folds the values into `q`.  `band`: that of the row, a little widened; negative for a row
// that is all zero (nothing is inserted and atom 0 is taken).
__device__ __forceinline__ void drain_half(uint32_t taddr, Top4& q, uint32_t id, float band, uint64_t* acc_empty, int lane) {
    uint32_t v0[32], v1[32], v2[32], v3[32];
    tmem_ld32(taddr + 0, v0);
    tmem_ld32(taddr + 32, v1);
    tmem_ld32(taddr + 64, v2);
    tmem_ld32(taddr + 96, v3);
    tmem_wait_ld(v0);
    reg_fence(v1);
    reg_fence(v2);
    reg_fence(v3);
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(acc_empty);
    float thr = __uint_as_float(q.k0 & kKeyMask) - band;
    chunk_top4(v0, q, id, 127u, thr, band);
    chunk_top4(v1, q, id, 95u, thr, band);
    chunk_top4(v2, q, id, 63u, thr, band);
    chunk_top4(v3, q, id, 31u, thr, band);
}

__device__ __forceinline__ unsigned long long compose(uint32_t key, uint32_t id) {
    return (static_cast<unsigned long long>(key) << 16) | id;
}
// Folds the other column half's top four (keys o0..o3, ids packed ten bits each in oi) into `a`.
__device__ __forceinline__ void top4_merge(Top4& a, uint32_t o0, uint32_t o1, uint32_t o2, uint32_t o3, uint32_t oi) {
    unsigned long long K0 = compose(a.k0, a.i0), K1 = compose(a.k1, a.i1), K2 = compose(a.k2, a.i2), K3 = compose(a.k3, 0);
    const unsigned long long in[4] = {compose(o0, oi & 1023u), compose(o1, (oi >> 10) & 1023u), compose(o2, (oi >> 20) & 1023u),
                                      compose(o3, 0)};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const unsigned long long k = in[i];
        const unsigned long long x = k < K0 ? k : K0;
        K0 = k < K0 ? K0 : k;
        const unsigned long long y = x < K1 ? x : K1;
        K1 = x < K1 ? K1 : x;
        const unsigned long long z = y < K2 ? y : K2;
        K2 = y < K2 ? K2 : y;
        K3 = K3 < z ? z : K3;
    }
    a.k0 = static_cast<uint32_t>(K0 >> 16);
    a.i0 = static_cast<uint32_t>(K0 & 0xFFFFu);
    a.k1 = static_cast<uint32_t>(K1 >> 16);
    a.i1 = static_cast<uint32_t>(K1 & 0xFFFFu);
    a.k2 = static_cast<uint32_t>(K2 >> 16);
    a.i2 = static_cast<uint32_t>(K2 & 0xFFFFu);
    a.k3 = static_cast<uint32_t>(K3 >> 16);
}
__device__ __forceinline__ int atom_of(uint32_t key, uint32_t id) {
    return static_cast<int>(id) * 128 + (127 - static_cast<int>(key & 127u));
}

// Barrier of the 256 epilogue threads that also tells every one of them whether any of them
// passed `pred`.
__device__ __forceinline__ bool epilogue_barrier_any(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 q, %1, 0;\n"
        "bar.red.or.pred p, 1, 256, q;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(r)
        : "r"(static_cast<uint32_t>(pred))
        : "memory");
    return r != 0;
}
__device__ __forceinline__ void epilogue_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ double group8_sum(double v) {
    v += __shfl_xor_sync(FULL, v, 1);
    v += __shfl_xor_sync(FULL, v, 2);
    v += __shfl_xor_sync(FULL, v, 4);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    return v;
}

// The eight lanes that share a row own its channels in pairs: lane l8 has channels 2 (8 k + l8)
// and the next one, k = 0 .. CH / 2 - 1, so that one load or store instruction of the eight lanes
// covers one contiguous run (whole 32-byte sectors of the fp64 row).
// CH channels of one atom (fp32 master copy), as this lane's slice.
template <int CH>
__device__ __forceinline__ void load_atom(const float* __restrict__ atom, int l8, float (&a)[CH]) {
#pragma unroll
    for (int k = 0; k < CH / 2; ++k) {
        const float2 v = __ldg(reinterpret_cast<const float2*>(atom) + 8 * k + l8);
        a[2 * k] = v.x;
        a[2 * k + 1] = v.y;
    }
}
// (four running sums: a single chain of fp64 FMAs would wait out the pipe's latency CH times)
template <int CH>
__device__ __forceinline__ double slice_dot(const double (&R)[CH], const float (&a)[CH]) {
    double c0 = 0.0, c1 = 0.0, c2 = 0.0, c3 = 0.0;
#pragma unroll
    for (int k = 0; k < CH; k += 4) {
        c0 = fma(R[k], static_cast<double>(a[k]), c0);
        c1 = fma(R[k + 1], static_cast<double>(a[k + 1]), c1);
        c2 = fma(R[k + 2], static_cast<double>(a[k + 2]), c2);
        c3 = fma(R[k + 3], static_cast<double>(a[k + 3]), c3);
    }
    return (c0 + c1) + (c2 + c3);
}

// Writes this lane's CH residual values: fp64 to the scratch row (`row`: its first element), bf16
// high and low parts into the operand tiles.  Returns the lane's share of ||R||^2.
template <int CH>
__device__ __forceinline__ double store_residual(const double (&R)[CH], double* __restrict__ row, uint8_t* Ahi, uint8_t* Alo,
                                                 int r, int l8) {
    double n0 = 0.0, n1 = 0.0;
#pragma unroll
    for (int k = 0; k < CH / 2; ++k) {
        reinterpret_cast<double2*>(row)[8 * k + l8] = make_double2(R[2 * k], R[2 * k + 1]);
        n0 = fma(R[2 * k], R[2 * k], n0);
        n1 = fma(R[2 * k + 1], R[2 * k + 1], n1);
        const float f0 = static_cast<float>(R[2 * k]), f1 = static_cast<float>(R[2 * k + 1]);
        const __nv_bfloat16 h0 = __float2bfloat16_rn(f0), h1 = __float2bfloat16_rn(f1);
        const __nv_bfloat16 l0 = __float2bfloat16_rn(f0 - __bfloat162float(h0));
        const __nv_bfloat16 l1 = __float2bfloat16_rn(f1 - __bfloat162float(h1));
        // channels 2 (8 k + l8), +1: 16-byte chunk 2 k + l8 / 4 of the row, word l8 % 4 of it
        const uint32_t off = swz_off(r, 2 * k + (l8 >> 2)) + (l8 & 3) * 4;
        *reinterpret_cast<uint32_t*>(Ahi + off) =
            static_cast<uint32_t>(__bfloat16_as_ushort(h0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16);
        *reinterpret_cast<uint32_t*>(Alo + off) =
            static_cast<uint32_t>(__bfloat16_as_ushort(l0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(l1)) << 16);
    }
    return n0 + n1;
}

// Elements `off` and `off + 1` of X widened to fp64.
__device__ __forceinline__ void load_x2(const void* X, int x_dtype, int64_t off, double& x0, double& x1) {
    if (x_dtype == CSR_DTYPE_F32) {
        const float2 v = __ldg(reinterpret_cast<const float2*>(reinterpret_cast<const float*>(X) + off));
        x0 = v.x;
        x1 = v.y;
    } else {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(reinterpret_cast<const uint16_t*>(X) + off));
        if (x_dtype == CSR_DTYPE_BF16) {
            x0 = __uint_as_float(w << 16);
            x1 = __uint_as_float(w & 0xFFFF0000u);
        } else {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
            x0 = f.x;
            x1 = f.y;
        }
    }
}

// Arg-max of |R . d_n| over the whole dictionary for one row, by one warp (all lanes call).  The
// true arg-max has an fp32 value of at least `thresh` (the tensor-core maximum less the band and
// the fp32 rounding), so an fp32 pass collects those atoms, one per lane, and their fp64
// correlations decide, the lowest atom among equal values.  More than 32 candidates (copies of
// one atom): every atom is scored in fp64.
template <int D_>
__device__ __noinline__ int rescore_row(const float* __restrict__ D, int N, const double* __restrict__ Rrow, float thresh, int lane) {
    constexpr int PER = D_ / 32;
    double R[PER];
    float rf[PER];
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        R[k] = Rrow[lane * PER + k];
        rf[k] = static_cast<float>(R[k]);
    }
    int mine = 0, count = 0;
    for (int n0 = 0; n0 < N; n0 += 8) {
        float c[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int n = min(n0 + u, N - 1);
            float a[PER];
            if constexpr (PER == 4) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(D + static_cast<int64_t>(n) * D_) + lane);
                a[0] = v.x, a[1] = v.y, a[2] = v.z, a[3] = v.w;
            } else {
                const float2 v = __ldg(reinterpret_cast<const float2*>(D + static_cast<int64_t>(n) * D_) + lane);
                a[0] = v.x, a[1] = v.y;
            }
            float p = 0.f;
#pragma unroll
            for (int k = 0; k < PER; ++k) p = fmaf(rf[k], a[k], p);
            c[u] = p;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            for (int o = 16; o; o >>= 1) c[u] += __shfl_xor_sync(FULL, c[u], o);
            if (n0 + u < N && !(fabsf(c[u]) < thresh)) {  // (NaN counts as a candidate)
                if (lane == (count & 31)) mine = n0 + u;
                ++count;
            }
        }
    }
    double best = -1.0;
    int bn = 0;
    const bool all = count > 32;
    const int todo = all ? N : count;
    for (int j = 0; j < todo; ++j) {
        const int n = all ? j : __shfl_sync(FULL, mine, j);
        double p = 0.0;
#pragma unroll
        for (int k = 0; k < PER; ++k) p = fma(R[k], static_cast<double>(__ldg(D + static_cast<int64_t>(n) * D_ + lane * PER + k)), p);
        const double a = fabs(warp_sum(p));
        if (a > best || (a == best && n < bn)) {
            best = a;
            bn = n;
        }
    }
    return bn;
}

template <int D_>
__global__ void __launch_bounds__(NT, 1)
encode_exact_tc_kernel(const __grid_constant__ CUtensorMap tmap_hi, const __grid_constant__ CUtensorMap tmap_lo,
                       const float* __restrict__ D, const void* __restrict__ X, int x_dtype, int64_t ldx, int64_t M, int N, int s,
                       uint16_t* __restrict__ out_idx, void* __restrict__ out_coef, int coef_dtype, int64_t ldc,
                       double* __restrict__ Rd_all, uint32_t* status, [[maybe_unused]] uint32_t* diag,
                       unsigned long long wait_limit_ns) {
    using S = TcSmem<D_>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    if ((smem_u32(smem_raw) & 1023u) != 0) {              // the swizzled tiles need this; never seen otherwise
        if (threadIdx.x == 0) atomicOr(status, kStatusLayout);
        return;
    }
    S& sm = *reinterpret_cast<S*>(smem_raw);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int T = (N + TILE_N - 1) / TILE_N;
    const int64_t n_pairs = (M + ROWS - 1) / ROWS;
    constexpr int KH = D_ / STAGE_CH;                       // 64-channel blocks per row
    constexpr int KSTEPS = STAGE_CH / UMMA_K;
    constexpr int STAGES = S::kStages;
    constexpr int NSTG = 2 * KH;                            // stages per dictionary tile
    constexpr int GROUP = STAGES >= NSTG + 2 ? NSTG : CSR_TC_GROUP128;
    static_assert(GROUP < STAGES && NSTG % GROUP == 0, "a group of stages must fit the ring with one stage to spare");
    const WaitCtx wc{&sm.abort, status, wait_limit_ns};

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(&sm.full_b[i], 1);
            mbar_init(&sm.empty_b[i], 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&sm.acc_full[t], 1);
            mbar_init(&sm.acc_empty[t], 8);
        }
        mbar_init(&sm.res_ready, ROWS);
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
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_hi)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_lo)) : "memory");
            uint32_t p = 0;
            bool ok = true;
            for (int64_t pair = blockIdx.x; pair < n_pairs && ok; pair += gridDim.x) {
                for (int g = 0; g < s && ok; ++g) {
                    for (int t = 0; t < T && ok; ++t) {
                        for (int hp = 0; hp < 2 * KH; ++hp, ++p) {
                            const int stage = p % STAGES;
                            if (!wait_bounded_suspended(&sm.empty_b[stage], ((p / STAGES) & 1) ^ 1, wc, 2000)) {
                                ok = false;
                                break;
                            }
                            // atoms past N arrive as zeros and count as bytes
                            mbar_expect_tx(&sm.full_b[stage], S::kStageBytes);
                            tma_load_2d(&sm.B[stage][0], (hp & 1) ? &tmap_lo : &tmap_hi, (hp >> 1) * STAGE_CH, t * TILE_N,
                                        &sm.full_b[stage]);
                        }
                    }
                }
            }
            if (!ok) {                                    // let the copies already issued land
                const uint32_t first = p > STAGES ? p - STAGES : 0;
                for (uint32_t qq = first; qq < p; ++qq) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(&sm.full_b[qq % STAGES], (qq / STAGES) & 1))
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
                    if (!wait_bounded_suspended(&sm.res_ready, steps & 1, wc, 4000)) {
                        ok = false;
                        break;
                    }
                    // A dictionary tile is NSTG stages (high and low parts of each 64-channel block).
                    // Each row tile takes GROUP stages in a row before the other takes the same ones,
                    // and a stage goes back to the producer after the second row tile's use: the
                    // larger the group, the further apart the two accumulators complete (the epilogue
                    // drains them one after the other), at the price of a shorter prefetch distance.
                    for (int t = 0; t < T && ok; ++t, ++accn, p += NSTG) {
                        for (int hp0 = 0; hp0 < NSTG && ok; hp0 += GROUP) {
                            for (int tile = 0; tile < 2 && ok; ++tile) {
                                for (int hp = hp0; hp < hp0 + GROUP; ++hp) {
                                    const uint32_t ps = p + hp;
                                    const int stage = ps % STAGES;
                                    const int h = hp >> 1;
                                    const bool low = hp & 1;      // this stage holds low parts of the atoms
                                    if (tile == 0 && !wait_bounded_suspended(&sm.full_b[stage], (ps / STAGES) & 1, wc, 1000)) {
                                        ok = false;
                                        break;
                                    }
                                    if (hp == 0 && !wait_bounded_suspended(&sm.acc_empty[tile], (accn & 1) ^ 1, wc, 1000)) {
                                        ok = false;
                                        break;
                                    }
                                    tc_fence_after();
                                    const uint64_t b0 = make_smem_desc(smem_u32(&sm.B[stage][0]));
                                    const uint32_t d_tmem = tmem_base + tile * TILE_N;
                                    const uint64_t ah = make_smem_desc(smem_u32(&sm.A[tile][0][h * (TILE_M * 128)]));
                                    const uint64_t al = make_smem_desc(smem_u32(&sm.A[tile][1][h * (TILE_M * 128)]));
#pragma unroll
                                    for (int k = 0; k < KSTEPS; ++k) {
                                        const uint64_t off = static_cast<uint64_t>((k * 32) >> 4);
                                        umma_bf16(d_tmem, ah + off, b0 + off, kInstrDesc, (hp | k) ? 1u : 0u);
                                    }
                                    if (!low) {
#pragma unroll
                                        for (int k = 0; k < KSTEPS; ++k) {
                                            const uint64_t off = static_cast<uint64_t>((k * 32) >> 4);
                                            umma_bf16(d_tmem, al + off, b0 + off, kInstrDesc, 1u);
                                        }
                                    }
                                    if (tile == 1) umma_commit(&sm.empty_b[stage]);
                                    if (hp == NSTG - 1) umma_commit(&sm.acc_full[tile]);
                                }
                            }
                        }
                    }
                }
            }
            if (!ok) {
                umma_commit(&sm.drained);
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(&sm.drained, 0))
                    if (globaltimer_ns() - t0 > 20000000ull) break;
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        constexpr int CH = D_ / 8;                          // channels per lane when eight lanes share a row
        const int q = warp & 3;                             // TMEM lane quarter
        const int half = warp >> 2;                         // column half drained by this warp
        const int own_tile = warp >> 2;                     // row tile whose rows this warp settles
        const int r_own = q * 32 + lane;                    // this lane's row in either tile
        const int l8 = lane & 7, grp = lane >> 3;
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + half * 128;
        double* Rd_cta = Rd_all + static_cast<int64_t>(blockIdx.x) * ROWS * D_;
        uint8_t* Ahi = &sm.A[own_tile][0][0];
        uint8_t* Alo = &sm.A[own_tile][1][0];
        uint32_t accn = 0;
        bool ok = true;
        for (int64_t pair = blockIdx.x; pair < n_pairs && ok; pair += gridDim.x) {
            float band = 0.f;                               // of row r_own of tile own_tile
            // ---- R_0 = x ----
#pragma unroll 1
            for (int p = 0; p < 8; ++p) {
                const int r = q * 32 + 4 * p + grp;
                const int64_t m = pair * ROWS + own_tile * TILE_M + r;
                double R[CH];
                if (m < M) {
#pragma unroll
                    for (int k = 0; k < CH / 2; ++k) load_x2(X, x_dtype, m * ldx + 2 * (8 * k + l8), R[2 * k], R[2 * k + 1]);
                } else {
#pragma unroll
                    for (int k = 0; k < CH; ++k) R[k] = 0.0;
                }
                double nn = store_residual<CH>(R, Rd_cta + static_cast<int64_t>(own_tile * TILE_M + r) * D_, Ahi, Alo, r, l8);
                nn = group8_sum(nn);
                const float nn_o = static_cast<float>(__shfl_sync(FULL, nn, (lane & 3) * 8));
                if ((lane >> 2) == p) band = kBandRel * sqrtf(nn_o) * 1.001f;
            }
            fence_proxy_async_smem();
            mbar_arrive(&sm.res_ready);

            for (int g = 0; g < s && ok; ++g) {
                // ---- sweep: top four keys of this thread's half of two rows ----
                Top4 st[2] = {Top4{0u, 0u, 0u, 0u, 0u, 0u, 0u}, Top4{0u, 0u, 0u, 0u, 0u, 0u, 0u}};
                // the filter's bands of this thread's two rows: its own and the one the warp of the
                // other row tile left in shared memory
                float* band_x = reinterpret_cast<float*>(&sm.xchg[0][0]);
                band_x[own_tile * TILE_M + r_own] = band;
                epilogue_barrier();
                const float band_other = band_x[(own_tile ^ 1) * TILE_M + r_own];
                epilogue_barrier();
                const float fb_own = band > 0.f ? band * 1.0625f : -1.f;
                const float fb_other = band_other > 0.f ? band_other * 1.0625f : -1.f;
                const float fband[2] = {own_tile == 0 ? fb_own : fb_other, own_tile == 0 ? fb_other : fb_own};
                for (int t = 0; t < T && ok; ++t, ++accn) {
#pragma unroll 1
                    for (int a = 0; a < 2; ++a) {           // (rolled: one copy of the drain's code)
                        bool got = wait_bounded_suspended(&sm.acc_full[a], accn & 1, wc, 2000);
                        got = __all_sync(FULL, got);
                        if (!got) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        Top4 qa = a ? st[1] : st[0];
                        drain_half(taddr + a * TILE_N, qa, static_cast<uint32_t>(2 * t + half), a ? fband[1] : fband[0],
                                   &sm.acc_empty[a], lane);
                        if (a)
                            st[1] = qa;
                        else
                            st[0] = qa;
                    }
                }
                // ---- merge the column halves: warps 0-3 end up with row tile 0, warps 4-7 with row tile 1 ----
                auto post = [&](const Top4& o) {
                    sm.xchg[0][r_own] = o.k0;
                    sm.xchg[1][r_own] = o.k1;
                    sm.xchg[2][r_own] = o.k2;
                    sm.xchg[3][r_own] = o.k3;
                    sm.xchg[4][r_own] = o.i0 | (o.i1 << 10) | (o.i2 << 20);
                };
                auto take = [&](Top4& mine_) {
                    top4_merge(mine_, sm.xchg[0][r_own], sm.xchg[1][r_own], sm.xchg[2][r_own], sm.xchg[3][r_own], sm.xchg[4][r_own]);
                };
                if (half == 1) post(st[0]);
                if (epilogue_barrier_any(!ok || sm.abort != 0)) {
                    ok = false;
                    break;
                }
                if (half == 0) take(st[0]);
                epilogue_barrier();
                if (half == 0) post(st[1]);
                epilogue_barrier();
                if (half == 1) take(st[1]);
                epilogue_barrier();                         // (the exchange area is rewritten before the next sweep)
                const Top4 mine = own_tile ? st[1] : st[0];
                const float v0 = __uint_as_float(mine.k0 & kKeyMask);
                int my_n1 = atom_of(mine.k0, mine.i0);
                if (!(v0 > 0.f) || my_n1 >= N) my_n1 = 0;   // an all-zero sweep picks atom 0
                const int my_n2 = min(atom_of(mine.k1, mine.i1), N - 1), my_n3 = min(atom_of(mine.k2, mine.i2), N - 1);
                // bits 0, 1, 2: the second, third, fourth largest key is inside the band (NaN counts as inside)
                int my_flags = 0;
                if (v0 > 0.f && N > 1) {
                    if (!(v0 - __uint_as_float(mine.k1 & kKeyMask) > band)) my_flags |= 1;
                    if (!(v0 - __uint_as_float(mine.k2 & kKeyMask) > band)) my_flags |= 2;
                    if (!(v0 - __uint_as_float(mine.k3 & kKeyMask) > band)) my_flags |= 4;
                }
                const float my_thresh = v0 - 1.5f * band;

                // ---- settle the 32 rows of this warp, eight lanes per row, four rows per pass; the
                // next pass's residual rows and atoms are requested before this pass is worked on
                // (one copy of the code: it has to stay in the instruction cache next to the sweep) ----
                auto fetch = [&](int p, int& n, int& flags, double (&R)[CH], float (&a)[CH]) {
                    const int src = 4 * p + grp;
                    n = __shfl_sync(FULL, my_n1, src);
                    flags = __shfl_sync(FULL, my_flags, src);
                    const double* Rrow = Rd_cta + static_cast<int64_t>(own_tile * TILE_M + q * 32 + src) * D_;
#pragma unroll
                    for (int k = 0; k < CH / 2; ++k) {
                        const double2 v = reinterpret_cast<const double2*>(Rrow)[8 * k + l8];
                        R[2 * k] = v.x;
                        R[2 * k + 1] = v.y;
                    }
                    load_atom<CH>(D + static_cast<int64_t>(n) * D_, l8, a);
                };
                int n, flags;
                double R[CH];
                float a[CH];
                fetch(0, n, flags, R, a);
#pragma unroll 1
                for (int p = 0; p < 8; ++p) {
                    int n_nx = 0, flags_nx = 0;
                    double R_nx[CH];
                    float a_nx[CH];
                    if (p + 1 < 8) {
                        fetch(p + 1, n_nx, flags_nx, R_nx, a_nx);
                    } else {
#pragma unroll
                        for (int k = 0; k < CH; ++k) {
                            R_nx[k] = 0.0;
                            a_nx[k] = 0.f;
                        }
                    }
                    const int src = 4 * p + grp;
                    const int r = q * 32 + src;
                    const int64_t m = pair * ROWS + own_tile * TILE_M + r;
                    double* Rrow = Rd_cta + static_cast<int64_t>(own_tile * TILE_M + r) * D_;
                    if (__any_sync(FULL, flags != 0)) {
                        // some row of this pass is not decided by its largest key alone
                        const int n_first = n;
                        if (__any_sync(FULL, flags & 4)) {
                            for (int j = 0; j < 4; ++j) {   // four keys inside the band: the whole dictionary, by the warp
                                const int fj = __shfl_sync(FULL, flags, 8 * j);
                                const float th = __shfl_sync(FULL, my_thresh, 4 * p + j);
                                if (fj & 4) {
                                    const int nr = rescore_row<D_>(D, N, Rd_cta + static_cast<int64_t>(own_tile * TILE_M + q * 32 + 4 * p + j) * D_, th, lane);
                                    if (grp == j) n = nr;
                                }
                            }
                        }
                        const bool cmp = (flags & 4) == 0 && flags != 0;   // this lane's row compares two or three
                        if (__any_sync(FULL, cmp)) {
                            double cbest = fabs(group8_sum(slice_dot<CH>(R, a)));
                            int nbest = n;
#pragma unroll 1
                            for (int cand = 0; cand < 2; ++cand) {
                                if (cand == 1 && !__any_sync(FULL, cmp && (flags & 2))) break;
                                const int nc = __shfl_sync(FULL, cand ? my_n3 : my_n2, src);
                                float ax[CH];
                                load_atom<CH>(D + static_cast<int64_t>(nc) * D_, l8, ax);
                                const double cc = fabs(group8_sum(slice_dot<CH>(R, ax)));
                                if ((cand == 0 || (flags & 2)) && (cc > cbest || (cc == cbest && nc < nbest))) {
                                    cbest = cc;
                                    nbest = nc;
                                }
                            }
                            if (cmp) n = nbest;
                        }
                        if (__any_sync(FULL, n != n_first)) load_atom<CH>(D + static_cast<int64_t>(n) * D_, l8, a);
                    }
                    const double c = group8_sum(slice_dot<CH>(R, a));
#ifdef CSR_DEBUG_CHECKS
                    {   // largest |tensor-core value - fp64 value| / ||R|| seen, as float bits
                        const float vbo = __shfl_sync(FULL, v0, src), bo = __shfl_sync(FULL, band, src);
                        if (l8 == 0 && m < M && flags == 0 && bo > 0.f) {
                            const float rel = fabsf(vbo - static_cast<float>(fabs(c))) / (bo / kBandRel);
                            atomicMax(diag, __float_as_uint(rel));
                        }
                    }
#endif
                    if (l8 == 0 && m < M) {
                        out_idx[m * ldc + g] = static_cast<uint16_t>(n);
                        const float cf = static_cast<float>(c);
                        if (coef_dtype == CSR_DTYPE_F16)
                            reinterpret_cast<__half*>(out_coef)[m * ldc + g] = __float2half_rn(cf);
                        else
                            reinterpret_cast<float*>(out_coef)[m * ldc + g] = cf;
                    }
                    if (g + 1 < s) {
#pragma unroll
                        for (int k = 0; k < CH; ++k) R[k] = fma(-c, static_cast<double>(a[k]), R[k]);
                        double nn = store_residual<CH>(R, Rrow, Ahi, Alo, r, l8);
                        nn = group8_sum(nn);
                        const float nn_o = static_cast<float>(__shfl_sync(FULL, nn, (lane & 3) * 8));
                        if ((lane >> 2) == p) band = kBandRel * sqrtf(nn_o) * 1.001f;
                    }
                    n = n_nx;
                    flags = flags_nx;
#pragma unroll
                    for (int k = 0; k < CH; ++k) {
                        R[k] = R_nx[k];
                        a[k] = a_nx[k];
                    }
                }
                if (g + 1 < s) {
                    fence_proxy_async_smem();
                    mbar_arrive(&sm.res_ready);
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

// D (fp32, [N][d]) -> its bf16 high part and the bf16 rounding of the remainder, same layout.
__global__ void split_dict_kernel(const float4* __restrict__ D, uint2* __restrict__ hi, uint2* __restrict__ lo, int64_t n_vec4) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec4; i += (int64_t)gridDim.x * blockDim.x) {
        const float4 v = D[i];
        const float f[4] = {v.x, v.y, v.z, v.w};
        uint32_t h[4], l[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const __nv_bfloat16 hk = __float2bfloat16_rn(f[k]);
            h[k] = __bfloat16_as_ushort(hk);
            l[k] = __bfloat16_as_ushort(__float2bfloat16_rn(f[k] - __bfloat162float(hk)));
        }
        hi[i] = make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
        lo[i] = make_uint2(l[0] | (l[1] << 16), l[2] | (l[3] << 16));
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn tensor_map_encoder() {
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

// One bf16 part of the dictionary, [N][d]: boxes of 256 atoms x 64 channels, 128-byte swizzle;
// atoms past N read as zeros.
int part_map(CUtensorMap* map, void* base, int N, int d) {
    EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const cuuint64_t gdim[2] = {(cuuint64_t)d, (cuuint64_t)N};
    const cuuint64_t gstride[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {STAGE_CH, (cuuint32_t)TILE_N};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, gdim, gstride, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return CSR_OK;
}

size_t align1k(size_t x) { return (x + 1023) / 1024 * 1024; }
int ctas_for(int64_t M) {
    const int64_t n_pairs = (M + ROWS - 1) / ROWS;
    const int64_t sms = sm_count();
    return (int)(n_pairs < sms ? n_pairs : sms);
}

template <int D_>
int run(const EncodeArgs& a, const CUtensorMap& mh, const CUtensorMap& ml, double* Rd, uint32_t* status, uint32_t* diag) {
    const size_t smem = sizeof(TcSmem<D_>);
    cudaError_t e = cudaFuncSetAttribute(encode_exact_tc_kernel<D_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const int grid = ctas_for(a.M);
    encode_exact_tc_kernel<D_><<<grid, NT, smem, a.stream>>>(mh, ml, a.D, a.X, a.x_dtype, a.ldx, a.M, a.N, a.s, a.out_idx,
                                                                     a.out_coef, a.coef_dtype, a.ld_code, Rd, status, diag,
                                                                     options().wait_limit_ns);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "encode_exact_tc launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace

size_t encode_exact_tc_scratch_bytes(int64_t M, int d, int N) {
    return 2 * align1k((size_t)N * d * 2) + (size_t)ctas_for(M) * ROWS * d * sizeof(double);
}

int launch_encode_exact_tc(const EncodeArgs& a, void* scratch, uint32_t* status, uint32_t* diag) {
    if (a.M == 0) return CSR_OK;
    if ((reinterpret_cast<uintptr_t>(scratch) & 1023u) != 0)
        return fail(CSR_ERR_ALIGNMENT, "internal: exact-mode scratch not 1024-byte aligned");
    char* base = static_cast<char*>(scratch);
    const size_t part = align1k((size_t)a.N * a.d * 2);
    void* hi = base;
    void* lo = base + part;
    double* Rd = reinterpret_cast<double*>(base + 2 * part);
    const int64_t n_vec4 = (int64_t)a.N * a.d / 4;
    int blocks = (int)((n_vec4 + 255) / 256);
    if (blocks > 4 * sm_count()) blocks = 4 * sm_count();
    split_dict_kernel<<<blocks, 256, 0, a.stream>>>(reinterpret_cast<const float4*>(a.D), static_cast<uint2*>(hi),
                                                    static_cast<uint2*>(lo), n_vec4);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "split_dict launch: %s", cudaGetErrorString(e));
    CUtensorMap mh, ml;
    if (int rc = part_map(&mh, hi, a.N, a.d)) return rc;
    if (int rc = part_map(&ml, lo, a.N, a.d)) return rc;
    if (a.d == 128) return run<128>(a, mh, ml, Rd, status, diag);
    return run<64>(a, mh, ml, Rd, status, diag);
}

}  // namespace csr
