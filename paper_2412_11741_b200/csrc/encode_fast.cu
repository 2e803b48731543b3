// Fast matching pursuit (paper Eq. 2-4) on the sm_100a tensor cores.
//
// One persistent CTA per SM owns two tiles of 128 input rows at a time and keeps their
// residuals on chip for all s iterations:
//
//   - the residual tiles live in shared memory as bf16, in the K-major 128-byte-swizzled
//     layout tcgen05.mma reads (operand A);
//   - the bf16 copy of the dictionary (a few MB, L2 resident) streams through a ring of
//     shared-memory stages fetched by TMA (operand B).  A stage holds 64 channels of 256
//     atoms (32 KB); every stage feeds both row tiles, so each dictionary byte fetched
//     from L2 serves 256 rows;
//   - tcgen05.mma (M = 128, N = 256, K = 16, bf16 x bf16 -> fp32) writes the 128 x 256
//     correlations of (row tile, atom tile) into that row tile's TMEM accumulator (2 row
//     tiles x 256 columns = all 512 columns).  N = 256 per instruction is what keeps the
//     tensor pipe fed: with N = 128 the operand reads from shared memory (A and B per
//     instruction) need the whole shared-memory bandwidth and the pipe starves;
//   - eight epilogue warps (four per row tile, one thread per row) pull the
//     accumulators out with tcgen05.ld and keep a running arg-max of |correlation| per
//     row.  The plain-ALU work per correlation value is what bounds the kernel next to
//     the tensor pipe, so it is cut in two levels: groups of G adjacent atoms are first
//     reduced to max |value| with 3-input floating-point maxima (absolute value is an
//     operand modifier, half an instruction per value), then the group maximum's low
//     mantissa bits are replaced by a group tag (one logic instruction per group) and a
//     3-input integer max per two groups tracks the largest magnitude and where it was.
//     The first half of an accumulator is processed while its second half is already on
//     its way into registers, so the accumulator is handed back to the tensor core after
//     half of the arithmetic; the two row tiles alternate on the tensor pipe.  The M x N
//     correlations never leave the SM;
//   - at the end of a sweep the four warps of a row tile resolve their rows' picks
//     cooperatively: eight lanes per row gather the G atoms of the row's winning group
//     (bf16, from L2, 128 contiguous bytes or more per request), recompute the G signed
//     correlations as fp32 dot products with the residual row, take the largest in
//     magnitude as (index, coefficient), subtract coefficient * atom and write the bf16
//     residual back into the operand tile; then the MMA warp is released for the next
//     iteration;
//   - codes are collected in shared memory and written as 16-byte vectors (uint16 index,
//     fp16 or fp32 coefficient).
//
// Warp roles: warps 0-3 epilogue of row tile 0, warps 4-7 epilogue of row tile 1 (warp w
// reads TMEM lanes 32*(w%4) .. +31), warp 8 TMA producer, warp 9 TMEM owner and MMA
// issuer.  All hand-offs are mbarriers; every wait is bounded by a wall-clock limit,
// after which the CTA raises a flag in the status word, lets its copies land, frees
// its TMEM and exits.
//
// Few rows (the vectors one decoding step adds) would leave all but a few SMs idle, each of
// them sweeping the whole dictionary s times.  Three instantiations of the kernel cover
// that case (template argument CL):
//   CL = 0  the kernel above; with n_splits > 1 it sweeps only a slice of the dictionary for
//           ONE iteration and leaves the rows' maxima to split_pick_kernel (a launch pair
//           per iteration: the fallback where clusters cannot be launched);
//   CL = 1  n_splits CTAs form a thread-block cluster, hold the same pair of row tiles and
//           each sweep a slice; after every sweep the rows' maxima are exchanged through
//           distributed shared memory (st.async credited to the peers' mbarriers: gather at
//           the CTA that merges a row, merged value back to everyone) and every CTA makes
//           the same pick and update, so all s iterations run in one launch;
//   CL = 2  the same with at most 128 rows in all: both accumulators and both epilogue warp
//           groups serve the one row tile, and the other row tile's shared memory holds
//           exchange buffers large enough for a one-hop all-to-all.
// The codes are the same bits in every case.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "tcgen05_common.cuh"

namespace csr {
namespace {

using namespace tc;

constexpr int TILE_M = 128;
constexpr int TILE_N = 256;                           // atoms per accumulator / per MMA instruction
constexpr int UMMA_K = 16;
constexpr int STAGE_CH = 64;                          // channels per dictionary stage (one 128-byte row)
constexpr int STAGES = 4;
constexpr int NT = 320;
constexpr int PRODUCER_WARP = 8;
constexpr int MMA_WARP = 9;
constexpr uint32_t TMEM_COLS = 512;
constexpr int CODE_BLOCK = 8;                         // codes collected before a flush


// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = 256.
constexpr uint32_t kInstrDesc = instr_desc_bf16(TILE_M, TILE_N);

// ---------------------------------------------------------------------------------------
// shared memory
// ---------------------------------------------------------------------------------------
template <int D_>
struct FastSmem {
    static constexpr int kATileBytes = TILE_M * D_ * 2;          // residual tile: D_/64 blocks of 128 rows x 128 B
    static constexpr int kStageBytes = TILE_N * STAGE_CH * 2;    // 256 atoms x 64 channels
    alignas(1024) uint8_t A[2][kATileBytes];
    alignas(1024) uint8_t B[STAGES][kStageBytes];
    alignas(16) uint16_t code_idx[2 * TILE_M][CODE_BLOCK];
    alignas(16) float code_coef[2 * TILE_M][CODE_BLOCK];
    uint64_t full_b[STAGES];
    uint64_t empty_b[STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t res_ready[2];
    uint64_t drained;
    uint64_t pair_bar;                                 // CL == 2: second warp group's result is in xout
    uint64_t pick_bar;                                 // CL == 2: the rows' picks are in xin (for the second group)
    uint64_t xbar[2];                                  // cluster exchange: gathered / merged, one phase per iteration each
    unsigned long long xin[2 * TILE_M];                // cluster exchange: (key, ~tile) of the rows this CTA merges, per source CTA
                                                       // (CL == 2: the rows' winning atoms, for the second warp group)
    unsigned long long xout[2 * TILE_M];               // cluster exchange: merged (key, ~tile) of every row
                                                       // (CL == 2: the second warp group's maxima)
    uint32_t tmem_base;
    volatile uint32_t abort;
};


// Byte offset of 16-byte chunk `chunk` (8 channels) of row `r` inside a residual tile.
__device__ __forceinline__ uint32_t swz_off(int r, int chunk) {
    const int khalf = chunk >> 3, cc = chunk & 7;
    return khalf * (TILE_M * 128) + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
}

// First atom of the group a (key, tile) pair names.  Whatever the keys say (NaN correlations can
// make a zero-filled column past the dictionary win) the gather that follows stays inside the
// padded bf16 copy; a build with CSR_DEBUG_CHECKS also records that the clamp was needed.
template <int G>
__device__ __forceinline__ int candidate_start(uint32_t best_key, uint32_t best_t, int N, [[maybe_unused]] uint32_t* status) {
    constexpr int NG = TILE_N / G;
    const int n0 = static_cast<int>(best_t) * TILE_N + (NG - 1 - static_cast<int>(best_key & static_cast<uint32_t>(NG - 1))) * G;
    const int last = ((N + 7) / 8) * 8 - G;
#ifdef CSR_DEBUG_CHECKS
    if (n0 > last || n0 < 0) atomicOr(status, kStatusBounds);
#endif
    return min(n0, last);
}

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// (a & mask) | TAG as one logic instruction: the mask is a kernel argument (so it sits in
// a register) and the tag is the instruction's immediate.
template <uint32_t TAG>
__device__ __forceinline__ uint32_t mask_tag(uint32_t a, uint32_t mask) {
    uint32_t r;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "n"(TAG));
    return r;
}
// max(|a|, |b|, |c|)
__device__ __forceinline__ float absmax3(float a, float b, float c) {
    float r;
    asm("max.abs.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Key of the group of G values starting at v[J] (column COL0 + J of the accumulator):
// max |value| with its low bits replaced by the tag of the group (higher tag = lower
// column, so that the lowest column wins ties).
template <int G, int COL0, int J>
__device__ __forceinline__ uint32_t group_key(const uint32_t (&v)[32], uint32_t mask) {
    constexpr uint32_t kTag = static_cast<uint32_t>(TILE_N / G - 1 - (COL0 + J) / G);
    if constexpr (G == 1) {
        return mask_tag<kTag>(v[J], mask);                // the mask also clears the sign
    } else {
        float gm;
        if constexpr (G == 2) {
            gm = fmaxf(fabsf(__uint_as_float(v[J])), fabsf(__uint_as_float(v[J + 1])));
        } else if constexpr (G == 4) {
            gm = fmaxf(absmax3(__uint_as_float(v[J]), __uint_as_float(v[J + 1]), __uint_as_float(v[J + 2])),
                       fabsf(__uint_as_float(v[J + 3])));
        } else {
            const float t1 = absmax3(__uint_as_float(v[J]), __uint_as_float(v[J + 1]), __uint_as_float(v[J + 2]));
            const float t2 = absmax3(__uint_as_float(v[J + 3]), __uint_as_float(v[J + 4]), __uint_as_float(v[J + 5]));
            gm = fmaxf(t2, absmax3(__uint_as_float(v[J + 6]), __uint_as_float(v[J + 7]), t1));
        }
        return mask_tag<kTag>(__float_as_uint(gm), mask);
    }
}

// Running key maxima (two independent chains) over the 32 / G groups of a 32-column chunk.
template <int G, int COL0, int J = 0>
__device__ __forceinline__ void chunk_key_max(const uint32_t (&v)[32], uint32_t mask, uint32_t& m0, uint32_t& m1) {
    if constexpr (J < 32) {
        m0 = __vimax3_u32(m0, group_key<G, COL0, J>(v, mask), group_key<G, COL0, J + G>(v, mask));
        m1 = __vimax3_u32(m1, group_key<G, COL0, J + 2 * G>(v, mask), group_key<G, COL0, J + 3 * G>(v, mask));
        chunk_key_max<G, COL0, J + 4 * G>(v, mask, m0, m1);
    }
}

// even += lo(r) * lo(a), odd += hi(r) * hi(a) for one word of two bf16 values each: the product of
// two bf16 values is exact in fp32 and the sum is rounded once (the value fmaf gives on the widened
// operands), and the mixed-precision instruction takes the 16-bit halves as they are.
__device__ __forceinline__ void fma2_bf16(float& even, float& odd, uint32_t r, uint32_t a) {
    asm("{\n"
        ".reg .b16 rl, rh, al, ah;\n"
        "mov.b32 {rl, rh}, %2;\n"
        "mov.b32 {al, ah}, %3;\n"
        "fma.rn.f32.bf16 %0, rl, al, %0;\n"
        "fma.rn.f32.bf16 %1, rh, ah, %1;\n"
        "}\n"
        : "+f"(even), "+f"(odd)
        : "r"(r), "r"(a));
}
// fp32 dot product of eight bf16 pairs (one 16-byte chunk of a residual row and of an atom)
__device__ __forceinline__ void dot8(const uint4& rv, const uint4& av, float& even, float& odd) {
    fma2_bf16(even, odd, rv.x, av.x);
    fma2_bf16(even, odd, rv.y, av.y);
    fma2_bf16(even, odd, rv.z, av.z);
    fma2_bf16(even, odd, rv.w, av.w);
}
// r -= coef * a on one 16-byte chunk, rounded back to bf16
__device__ __forceinline__ uint4 axpy8(const uint4& rv, const uint4& av, float coef) {
    uint4 o;
    o.x = pack_bf16(fmaf(-coef, bf_lo(av.x), bf_lo(rv.x)), fmaf(-coef, bf_hi(av.x), bf_hi(rv.x)));
    o.y = pack_bf16(fmaf(-coef, bf_lo(av.y), bf_lo(rv.y)), fmaf(-coef, bf_hi(av.y), bf_hi(rv.y)));
    o.z = pack_bf16(fmaf(-coef, bf_lo(av.z), bf_lo(rv.z)), fmaf(-coef, bf_hi(av.z), bf_hi(rv.z)));
    o.w = pack_bf16(fmaf(-coef, bf_lo(av.w), bf_lo(rv.w)), fmaf(-coef, bf_hi(av.w), bf_hi(rv.w)));
    return o;
}

// End of a sweep for the 32 rows of one epilogue warp (Eq. 2-4).  Lane i enters with the
// first atom `n0` of the winning group of row q*32 + i.  Eight lanes work on one row (four
// rows per pass, eight passes): each lane gathers its 1/8 of the G candidate atoms (one
// contiguous run of G * 2 * D_ bytes per row), the G signed correlations with the row's
// residual are rebuilt as fp32 dot products and summed over the eight lanes, the largest
// in magnitude (lowest atom on ties) gives the index and the coefficient, and, unless
// this was the last iteration, the residual row in the operand tile becomes
// R - coef * atom.  The code goes to the row's slot in the shared-memory staging arrays.
// With SKIP, groups of (at most four) passes none of whose rows is set in `row_mask` (bit i =
// row i of the warp's 32 is a row of X) are left out: with few rows the pick is on the
// critical path of every iteration.
template <int D_, int G, bool SKIP = false>
__device__ __forceinline__ void pick_and_update(uint8_t* Atile, int q, int lane, const uint16_t* __restrict__ Db,
                                                int n0, bool update, uint16_t (*code_idx)[CODE_BLOCK],
                                                float (*code_coef)[CODE_BLOCK], int gi, uint32_t row_mask = 0xffffffffu) {
    constexpr int CH = D_ / 64;                           // 16-byte chunks per lane per atom
    constexpr int APR = D_ / 8;                           // 16-byte chunks per atom row
    constexpr int LPP = G * CH;                           // gathered chunks per lane per pass
    constexpr int WAVE0 = (32 / LPP) < 8 ? (32 / LPP) : 8;
    constexpr int WAVE = SKIP && WAVE0 > 4 ? 4 : WAVE0;   // passes whose gathers are in flight together
    const int sub = lane >> 3, l8 = lane & 7;
#pragma unroll
    for (int w0 = 0; w0 < 8; w0 += WAVE) {
        if (SKIP && ((row_mask >> (w0 * 4)) & ((1ull << (4 * WAVE)) - 1)) == 0) continue;
        uint4 atom[WAVE][G][CH];
        int base[WAVE];
#pragma unroll
        for (int it = 0; it < WAVE; ++it) {
            base[it] = __shfl_sync(0xffffffffu, n0, (w0 + it) * 4 + sub);
            const uint4* src = reinterpret_cast<const uint4*>(Db + static_cast<size_t>(base[it]) * D_) + l8 * CH;
#pragma unroll
            for (int j = 0; j < G; ++j)
#pragma unroll
                for (int c = 0; c < CH; ++c) atom[it][j][c] = __ldg(src + j * APR + c);
        }
#pragma unroll
        for (int it = 0; it < WAVE; ++it) {
            const int i = (w0 + it) * 4 + sub;            // row inside the warp's 32
            const int r = q * 32 + i;                     // row inside the tile
            uint4 rv[CH];
#pragma unroll
            for (int c = 0; c < CH; ++c) rv[c] = *reinterpret_cast<const uint4*>(Atile + swz_off(r, l8 * CH + c));
            float dot[G];
#pragma unroll
            for (int j = 0; j < G; ++j) {
                float ev = 0.f, od = 0.f;
#pragma unroll
                for (int c = 0; c < CH; ++c) dot8(rv[c], atom[it][j][c], ev, od);
                dot[j] = ev + od;
            }
#pragma unroll
            for (int m = 1; m < 8; m <<= 1)
#pragma unroll
                for (int j = 0; j < G; ++j) dot[j] += __shfl_xor_sync(0xffffffffu, dot[j], m);
            float coef = dot[0];
            int jb = 0;
#pragma unroll
            for (int j = 1; j < G; ++j)
                if (fabsf(dot[j]) > fabsf(coef)) {
                    coef = dot[j];
                    jb = j;
                }
            if (update) {
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    uint4 av = atom[it][0][c];
#pragma unroll
                    for (int j = 1; j < G; ++j)
                        if (jb == j) av = atom[it][j][c];
                    *reinterpret_cast<uint4*>(Atile + swz_off(r, l8 * CH + c)) = axpy8(rv[c], av, coef);
                }
            }
            if (l8 == 0) {
                code_idx[r][gi] = static_cast<uint16_t>(base[it] + jb);
                code_coef[r][gi] = coef;
            }
        }
    }
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
// few rows: the dictionary is split across CTAs, one iteration per launch
// ---------------------------------------------------------------------------------------
// R_0 = x rounded to bf16, dense [M][d]; one thread per 16-byte chunk of eight channels.
template <int D_>
__global__ void rows_to_bf16_kernel(const void* __restrict__ X, int x_dtype, int64_t ldx, int64_t M, uint4* __restrict__ Rb) {
    constexpr int CHUNKS = D_ / 8;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M * CHUNKS) return;
    const int64_t m = i / CHUNKS;
    const int c = (int)(i % CHUNKS);
    uint4 v;
    if (x_dtype == CSR_DTYPE_BF16) {
        v = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(X) + m * ldx + 8 * c);
    } else {
        float f[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) f[k] = load_elem(X, x_dtype, m * ldx + 8 * c + k);
        v.x = pack_bf16(f[0], f[1]);
        v.y = pack_bf16(f[2], f[3]);
        v.z = pack_bf16(f[4], f[5]);
        v.w = pack_bf16(f[6], f[7]);
    }
    Rb[i] = v;
}

// Pick of one iteration for the split sweep: merges a row's per-CTA (key, tile) pairs (largest
// key, lowest tile among equal keys: the order in which one CTA would have met them), then
// does exactly what pick_and_update does, on the residual rows kept in global memory.
// Eight lanes per row, four rows per warp.
template <int D_, int G>
__global__ void __launch_bounds__(128)
split_pick_kernel(const uint16_t* __restrict__ Db, int N, uint4* __restrict__ Rb, const uint2* __restrict__ partial,
                  int n_splits, int64_t M, int g, int update, uint16_t* __restrict__ out_idx, void* __restrict__ out_coef, int coef_dtype,
                  int64_t ldc) {
    constexpr int CH = D_ / 64;
    constexpr int APR = D_ / 8;
    constexpr int NG = TILE_N / G;
    const int lane = threadIdx.x & 31, sub = lane >> 3, l8 = lane & 7;
    const int64_t m = ((int64_t)blockIdx.x * 4 + (threadIdx.x >> 5)) * 4 + sub;
    const bool valid = m < M;
    uint32_t key = 0, t = 0;
    if (valid) {
        for (int j = l8; j < n_splits; j += 8) {
            const uint2 pr = partial[m * n_splits + j];
            if (pr.x > key || (pr.x == key && pr.y < t)) {
                key = pr.x;
                t = pr.y;
            }
        }
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
        const uint32_t ok = __shfl_xor_sync(0xffffffffu, key, o), ot = __shfl_xor_sync(0xffffffffu, t, o);
        if (ok > key || (ok == key && ot < t)) {
            key = ok;
            t = ot;
        }
    }
    const int n0 = min(static_cast<int>(t) * TILE_N + (NG - 1 - static_cast<int>(key & static_cast<uint32_t>(NG - 1))) * G,
                       ((N + 7) / 8) * 8 - G);     // as in the one-launch kernel: never past the padded copy
    const int64_t mr = valid ? m : 0;
    uint4 atom[G][CH], rv[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        rv[c] = Rb[mr * APR + l8 * CH + c];
#pragma unroll
        for (int j = 0; j < G; ++j)
            atom[j][c] = __ldg(reinterpret_cast<const uint4*>(Db + static_cast<size_t>(n0) * D_) + j * APR + l8 * CH + c);
    }
    float dot[G];
#pragma unroll
    for (int j = 0; j < G; ++j) {
        float ev = 0.f, od = 0.f;
#pragma unroll
        for (int c = 0; c < CH; ++c) dot8(rv[c], atom[j][c], ev, od);
        dot[j] = ev + od;
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1)
#pragma unroll
        for (int j = 0; j < G; ++j) dot[j] += __shfl_xor_sync(0xffffffffu, dot[j], o);
    if (!valid) return;
    float coef = dot[0];
    int jb = 0;
#pragma unroll
    for (int j = 1; j < G; ++j)
        if (fabsf(dot[j]) > fabsf(coef)) {
            coef = dot[j];
            jb = j;
        }
    if (update) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            uint4 av = atom[0][c];
#pragma unroll
            for (int j = 1; j < G; ++j)
                if (jb == j) av = atom[j][c];
            Rb[m * APR + l8 * CH + c] = axpy8(rv[c], av, coef);
        }
    }
    if (l8 == 0) {
        out_idx[m * ldc + g] = static_cast<uint16_t>(n0 + jb);
        if (coef_dtype == CSR_DTYPE_F16)
            reinterpret_cast<__half*>(out_coef)[m * ldc + g] = __float2half_rn(coef);
        else
            reinterpret_cast<float*>(out_coef)[m * ldc + g] = coef;
    }
}

// ---------------------------------------------------------------------------------------
// the encoder
// ---------------------------------------------------------------------------------------
template <int D_, int G, int CL>
__global__ void __launch_bounds__(NT, 1)
encode_fast_kernel(const __grid_constant__ CUtensorMap tmap_d, const uint16_t* __restrict__ Db,
                   const void* __restrict__ X, int x_dtype, int64_t ldx, int64_t M, int N, int s,
                   uint16_t* __restrict__ out_idx, void* __restrict__ out_coef, int coef_dtype, int64_t ldc, int vec_codes,
                   uint32_t key_mask, uint32_t* status, int n_splits, uint2* __restrict__ partial,
                   unsigned long long wait_limit_ns) {
    using S = FastSmem<D_>;
    extern __shared__ uint8_t smem_raw[];
    S& sm = *reinterpret_cast<S*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int T = (N + TILE_N - 1) / TILE_N;                // dictionary tiles per sweep (the last may be half)
    const int64_t n_pairs = (M + 2 * TILE_M - 1) / (2 * TILE_M);
    // Few rows (n_splits > 1): n_splits CTAs share one pair of row tiles, CTA j sweeping the
    // dictionary tiles j, j + n_splits, ...
    //  - CL: the n_splits CTAs are one thread-block cluster and run all s iterations.
    //    After each sweep every row's best (key, tile) is max-reduced into every CTA's shared
    //    memory, every CTA then makes the same pick and the same residual update on its own
    //    copy of the rows, and CTA 0 of the cluster writes the codes.
    //    CL == 2: at most TILE_M rows in all (one decoding step of a small batch).  Only the
    //    first row tile exists; the two accumulators take the CTA's dictionary tiles in turn
    //    and the second group of epilogue warps drains the second accumulator for the same
    //    rows; the unused second row tile holds the exchange buffers, large enough for every
    //    CTA to hear from every CTA directly (one hop).
    //  - otherwise ONE iteration per launch (s == 1 is passed): each row's best (key, tile) goes
    //    to `partial` and the pick kernel takes over.
    const int t_begin = n_splits > 1 ? (int)(blockIdx.x % n_splits) : 0;
    const int t_step = n_splits > 1 ? n_splits : 1;
    const int64_t pair_first = n_splits > 1 ? blockIdx.x / n_splits : blockIdx.x;
    const int64_t pair_step = n_splits > 1 ? gridDim.x / n_splits : gridDim.x;
    constexpr int KH = D_ / STAGE_CH;                       // stages per dictionary tile
    constexpr int KSTEPS = STAGE_CH / UMMA_K;               // MMAs per stage
    constexpr int CHUNKS = D_ / 8;                          // 16-byte chunks per row
    constexpr int NG = TILE_N / G;                          // arg-max groups per accumulator
    const WaitCtx wc{&sm.abort, status, wait_limit_ns};

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(&sm.full_b[i], 1);
            mbar_init(&sm.empty_b[i], 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&sm.acc_full[t], 1);
            mbar_init(&sm.acc_empty[t], 4);
            // (with one tile of rows both warp groups update rows of it)
            mbar_init(&sm.res_ready[t], CL == 2 ? 2 * TILE_M : TILE_M);
        }
        mbar_init(&sm.drained, 1);
        if constexpr (CL == 1) {
            // one phase per iteration: this thread arms it with the bytes the peers will send
            mbar_init(&sm.xbar[0], 1);
            mbar_init(&sm.xbar[1], 1);
            mbar_expect_tx(&sm.xbar[0], 2 * TILE_M * 8);
            mbar_expect_tx(&sm.xbar[1], 2 * TILE_M * 8);
        }
        if constexpr (CL == 2) {
            mbar_init(&sm.xbar[0], 1);
            mbar_expect_tx(&sm.xbar[0], static_cast<uint32_t>(n_splits) * TILE_M * 8);
            mbar_init(&sm.pair_bar, TILE_M);
            mbar_init(&sm.pick_bar, TILE_M);
        }
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
    // no CTA touches a peer's barrier or words before every peer has set them up
    if constexpr (CL) cluster_sync_all();

    if (warp == PRODUCER_WARP) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_d)) : "memory");
            uint32_t p = 0;
            bool ok = true;
            for (int64_t pair = pair_first; pair < n_pairs && ok; pair += pair_step) {
                for (int g = 0; g < s && ok; ++g) {
                    for (int t = t_begin; t < T && ok; t += t_step) {
                        for (int h = 0; h < KH; ++h, ++p) {
                            const int stage = p % STAGES;
                            if (!wait_bounded(&sm.empty_b[stage], ((p / STAGES) & 1) ^ 1, wc)) {
                                ok = false;
                                break;
                            }
                            // rows past N (a half tile at the end) arrive as zeros and count as bytes
                            mbar_expect_tx(&sm.full_b[stage], S::kStageBytes);
                            tma_load_2d(&sm.B[stage][0], &tmap_d, h * STAGE_CH, t * TILE_N, &sm.full_b[stage]);
                        }
                    }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA goes away
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
        if (lane == 0 && CL == 2) {
            // one row tile; the CTA's dictionary tiles go to the two accumulators in turn
            uint32_t p = 0, accn[2] = {0u, 0u};
            bool ok = true;
            for (int g = 0; g < s && ok; ++g) {
                if (!wait_bounded(&sm.res_ready[0], g & 1, wc)) {
                    ok = false;
                    break;
                }
                int j = 0;
                for (int t = t_begin; t < T && ok; t += t_step, p += KH, ++j) {
                    const int acc = j & 1;
                    if (!wait_bounded(&sm.acc_empty[acc], (accn[acc] & 1) ^ 1, wc)) {
                        ok = false;
                        break;
                    }
                    const uint32_t d_tmem = tmem_base + acc * TILE_N;
#pragma unroll
                    for (int h = 0; h < KH; ++h) {
                        const uint32_t ps = p + h;
                        const int stage = ps % STAGES;
                        if (!wait_bounded(&sm.full_b[stage], (ps / STAGES) & 1, wc)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint64_t a0 = make_smem_desc(smem_u32(&sm.A[0][h * (TILE_M * 128)]));
                        const uint64_t b0 = make_smem_desc(smem_u32(&sm.B[stage][0]));
#pragma unroll
                        for (int k = 0; k < KSTEPS; ++k) {
                            const uint64_t off = static_cast<uint64_t>((k * 32) >> 4);
                            umma_bf16(d_tmem, a0 + off, b0 + off, kInstrDesc, (h | k) ? 1u : 0u);
                        }
                        umma_commit(&sm.empty_b[stage]);
                    }
                    if (ok) {
                        umma_commit(&sm.acc_full[acc]);
                        ++accn[acc];
                    }
                }
            }
            if (!ok) {
                umma_commit(&sm.drained);
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(&sm.drained, 0))
                    if (globaltimer_ns() - t0 > 20000000ull) break;
            }
        } else if (lane == 0) {
            uint32_t p = 0, accn = 0, steps = 0;
            bool ok = true;
            for (int64_t pair = pair_first; pair < n_pairs && ok; pair += pair_step) {
                for (int g = 0; g < s && ok; ++g, ++steps) {
                    for (int t = t_begin; t < T && ok; t += t_step, p += KH, ++accn) {
                        for (int tile = 0; tile < 2 && ok; ++tile) {
                            if (t == t_begin && !wait_bounded(&sm.res_ready[tile], steps & 1, wc)) {
                                ok = false;
                                break;
                            }
                            if (!wait_bounded(&sm.acc_empty[tile], (accn & 1) ^ 1, wc)) {
                                ok = false;
                                break;
                            }
                            const uint32_t d_tmem = tmem_base + tile * TILE_N;
#pragma unroll
                            for (int h = 0; h < KH; ++h) {
                                const uint32_t ps = p + h;
                                const int stage = ps % STAGES;
                                if (tile == 0 && !wait_bounded(&sm.full_b[stage], (ps / STAGES) & 1, wc)) {
                                    ok = false;
                                    break;
                                }
                                tc_fence_after();
                                const uint64_t a0 = make_smem_desc(smem_u32(&sm.A[tile][h * (TILE_M * 128)]));
                                const uint64_t b0 = make_smem_desc(smem_u32(&sm.B[stage][0]));
#pragma unroll
                                for (int k = 0; k < KSTEPS; ++k) {
                                    // 16 channels = 32 bytes inside a 128-byte swizzled row
                                    const uint64_t off = static_cast<uint64_t>((k * 32) >> 4);
                                    umma_bf16(d_tmem, a0 + off, b0 + off, kInstrDesc, (h | k) ? 1u : 0u);
                                }
                                // the second row tile is the last reader of a stage
                                if (tile == 1) umma_commit(&sm.empty_b[stage]);
                            }
                            if (ok) umma_commit(&sm.acc_full[tile]);
                        }
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
        const int acc = warp >> 2;                        // the accumulator this warp drains
        const int tile = CL == 2 ? 0 : acc;               // the row tile its rows belong to
        const int q = warp & 3;
        const int r = q * 32 + lane;                      // row inside the tile == TMEM lane
        const int slot = tile * TILE_M + r;               // row inside the CTA's pair
        uint8_t* Atile = &sm.A[tile][0];
        uint16_t (*code_idx)[CODE_BLOCK] = &sm.code_idx[tile * TILE_M];
        float (*code_coef)[CODE_BLOCK] = &sm.code_coef[tile * TILE_M];
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * TILE_N;
        uint32_t accn = 0;
        [[maybe_unused]] uint32_t xn = 0;
        bool ok = true;
        const bool writes_codes = !CL || t_begin == 0;
        for (int64_t pair = pair_first; pair < n_pairs && ok; pair += pair_step) {
            const int64_t m = pair * (2 * TILE_M) + slot;
            const bool valid = m < M;
            uint32_t row_mask = 0xffffffffu;
            if constexpr (CL) row_mask = __ballot_sync(0xffffffffu, valid);
            // ---- R_0 = x, rounded to bf16, into the operand tile ----
            if (CL == 2 && acc == 1) {
                // the second warp group has no rows of its own
            } else if (x_dtype == CSR_DTYPE_BF16) {
                const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(X) + m * ldx);
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (valid) v = __ldg(src + c);
                    *reinterpret_cast<uint4*>(Atile + swz_off(r, c)) = v;
                }
            } else if (x_dtype == CSR_DTYPE_F16) {
                const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(X) + m * ldx);
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    uint4 h = make_uint4(0u, 0u, 0u, 0u);
                    if (valid) h = __ldg(src + c);
                    const __half2* hp = reinterpret_cast<const __half2*>(&h);
                    const float2 f0 = __half22float2(hp[0]), f1 = __half22float2(hp[1]);
                    const float2 f2 = __half22float2(hp[2]), f3 = __half22float2(hp[3]);
                    uint4 v;
                    v.x = pack_bf16(f0.x, f0.y);
                    v.y = pack_bf16(f1.x, f1.y);
                    v.z = pack_bf16(f2.x, f2.y);
                    v.w = pack_bf16(f3.x, f3.y);
                    *reinterpret_cast<uint4*>(Atile + swz_off(r, c)) = v;
                }
            } else {
                const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(X) + m * ldx);
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
                    *reinterpret_cast<uint4*>(Atile + swz_off(r, c)) = v;
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(&sm.res_ready[tile]);

            for (int g = 0; g < s && ok; ++g) {
                // ---- sweep: running arg-max of |correlation| over all atom tiles ----
                uint32_t best_key = 0, best_t = 0;
                [[maybe_unused]] int n0_other = 0;
                for (int t = t_begin + (CL == 2 ? acc * t_step : 0); t < T; t += (CL == 2 ? 2 : 1) * t_step, ++accn) {
                    bool got = wait_bounded(&sm.acc_full[acc], accn & 1, wc);
                    got = __all_sync(0xffffffffu, got);
                    if (!got) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    uint32_t v0[32], v1[32], v2[32], v3[32];
                    uint32_t k0 = 0, k1 = 0;
                    tmem_ld32(taddr + 0, v0);
                    tmem_ld32(taddr + 32, v1);
                    tmem_ld32(taddr + 64, v2);
                    tmem_ld32(taddr + 96, v3);
                    tmem_wait_ld(v0);
                    reg_fence(v1);
                    reg_fence(v2);
                    reg_fence(v3);
                    chunk_key_max<G, 0>(v0, key_mask, k0, k1);
                    tmem_ld32(taddr + 128, v0);
                    chunk_key_max<G, 32>(v1, key_mask, k0, k1);
                    tmem_ld32(taddr + 160, v1);
                    chunk_key_max<G, 64>(v2, key_mask, k0, k1);
                    tmem_ld32(taddr + 192, v2);
                    chunk_key_max<G, 96>(v3, key_mask, k0, k1);
                    tmem_ld32(taddr + 224, v3);
                    tmem_wait_ld(v0);
                    reg_fence(v1);
                    reg_fence(v2);
                    reg_fence(v3);
                    // every column of this accumulator is in registers: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.acc_empty[acc]);
                    chunk_key_max<G, 128>(v0, key_mask, k0, k1);
                    chunk_key_max<G, 160>(v1, key_mask, k0, k1);
                    chunk_key_max<G, 192>(v2, key_mask, k0, k1);
                    chunk_key_max<G, 224>(v3, key_mask, k0, k1);
                    const uint32_t key = k0 > k1 ? k0 : k1;
                    if (key > best_key) {
                        best_key = key;
                        best_t = t;
                    }
                }
                if (!ok) break;
                if (!CL && partial) {                       // split sweep: the pick kernel takes over
                    if (valid) partial[m * n_splits + t_begin] = make_uint2(best_key, best_t);
                    continue;
                }
                if constexpr (CL == 2) {
                    // ---- the row's best over this CTA's tiles (both accumulators), then over the
                    // whole dictionary: every CTA sends its (key, ~tile) of the row to every CTA.
                    // The entries are double-buffered by iteration: a peer writes iteration g + 2's
                    // only after it has heard this CTA's iteration g + 1, which the thread that
                    // reads the entries sends after it has read iteration g's. ----
                    unsigned long long mine = (static_cast<unsigned long long>(best_key) << 32) | (0xFFFFFFFFu - best_t);
                    // (a CTA with a single dictionary tile has no use for the second group, which
                    // would otherwise run ahead of the first: nothing paces it but its sweep)
                    const bool two_groups = t_begin + t_step < T;
                    int* pick_n0 = reinterpret_cast<int*>(&sm.xin[0]);
                    bool got = true;
                    if (acc == 1) {
                        if (two_groups) {
                            sm.xout[r] = mine;
                            mbar_arrive(&sm.pair_bar);
                        }
                        // the second half of every warp's rows is picked and updated by this group
                        got = wait_bounded(&sm.pick_bar, xn & 1, wc);
                    } else if (two_groups) {
                        got = wait_bounded(&sm.pair_bar, xn & 1, wc);
                    }
                    if (got && acc == 0) {
                        if (two_groups) {
                            const unsigned long long other = *reinterpret_cast<volatile unsigned long long*>(&sm.xout[r]);
                            mine = other > mine ? other : mine;
                        }
                        constexpr int XMAX = FastSmem<D_>::kATileBytes / (2 * TILE_M * 8);   // CTAs the buffers hold
                        unsigned long long* xg = reinterpret_cast<unsigned long long*>(&sm.A[1][0]) + (xn & 1) * XMAX * TILE_M;
                        const uint32_t dst = smem_u32(&xg[t_begin * TILE_M + r]), bar = smem_u32(&sm.xbar[0]);
                        for (int c = 0; c < n_splits; ++c) st_async_u64(map_to_cta(dst, c), mine, map_to_cta(bar, c));
                        got = wait_bounded_cluster(&sm.xbar[0], xn & 1, wc);
                        if (got) {
                            if (r == 0) mbar_expect_tx(&sm.xbar[0], static_cast<uint32_t>(n_splits) * TILE_M * 8);
                            unsigned long long top = 0ull;
                            for (int c = 0; c < n_splits; ++c) {
                                const unsigned long long v = *reinterpret_cast<volatile unsigned long long*>(&xg[c * TILE_M + r]);
                                top = v > top ? v : top;
                            }
                            mine = top;
                        }
                    }
                    got = __all_sync(0xffffffffu, got);
                    if (!got) {
                        ok = false;
                        break;
                    }
                    ++xn;
                    best_key = static_cast<uint32_t>(mine >> 32);
                    best_t = 0xFFFFFFFFu - static_cast<uint32_t>(mine);
                    if (acc == 0) {
                        pick_n0[r] = candidate_start<G>(best_key, best_t, N, status);
                        mbar_arrive(&sm.pick_bar);
                        row_mask &= 0x0000FFFFu;
                    } else {
                        n0_other = *reinterpret_cast<volatile int*>(&pick_n0[r]);
                        row_mask &= 0xFFFF0000u;
                    }
                }
                if constexpr (CL == 1) {
                    // ---- every CTA of the cluster learns the row's best over the whole dictionary:
                    // the highest key and, among equal keys, the lowest tile.  Row i of the pair is
                    // merged by CTA i % n_splits: gather there, merge, send the result to everyone.
                    // Both buffers are single.  An entry of xin is overwritten by a peer that has
                    // seen this iteration's merged rows from all of this CTA's merging threads,
                    // each of which read its entries first; an entry of xout is overwritten by a
                    // peer that has received the next iteration's key from the one thread that
                    // reads it. ----
                    const unsigned long long mine =
                        (static_cast<unsigned long long>(best_key) << 32) | (0xFFFFFFFFu - best_t);
                    const int per_cta = 2 * TILE_M / n_splits;        // rows merged by one CTA
                    {
                        const uint32_t o = static_cast<uint32_t>(slot % n_splits);
                        st_async_u64(map_to_cta(smem_u32(&sm.xin[t_begin * per_cta + slot / n_splits]), o), mine,
                                     map_to_cta(smem_u32(&sm.xbar[0]), o));
                    }
                    bool got = true;
                    if (slot < per_cta) {
                        got = wait_bounded_cluster(&sm.xbar[0], xn & 1, wc);
                        if (got) {
                            if (slot == 0) mbar_expect_tx(&sm.xbar[0], 2 * TILE_M * 8);       // the next iteration's
                            unsigned long long top = 0ull;
                            for (int c = 0; c < n_splits; ++c) {
                                const unsigned long long v =
                                    *reinterpret_cast<volatile unsigned long long*>(&sm.xin[c * per_cta + slot]);
                                top = v > top ? v : top;
                            }
                            const uint32_t dst = smem_u32(&sm.xout[slot * n_splits + t_begin]), bar = smem_u32(&sm.xbar[1]);
                            for (int c = 0; c < n_splits; ++c) st_async_u64(map_to_cta(dst, c), top, map_to_cta(bar, c));
                        }
                    }
                    if (got) got = wait_bounded_cluster(&sm.xbar[1], xn & 1, wc);
                    got = __all_sync(0xffffffffu, got);
                    if (!got) {
                        ok = false;
                        break;
                    }
                    if (slot == 0) mbar_expect_tx(&sm.xbar[1], 2 * TILE_M * 8);               // the next iteration's
                    const unsigned long long all = *reinterpret_cast<volatile unsigned long long*>(&sm.xout[slot]);
                    ++xn;
                    best_key = static_cast<uint32_t>(all >> 32);
                    best_t = 0xFFFFFFFFu - static_cast<uint32_t>(all);
                }
                // ---- pick, signed coefficient, residual update ----
                const int gi = g & (CODE_BLOCK - 1);
                int n0 = candidate_start<G>(best_key, best_t, N, status);
                if (CL == 2 && acc == 1) n0 = n0_other;
                if constexpr (CL)
                    pick_and_update<D_, G, true>(Atile, q, lane, Db, n0, g + 1 < s, code_idx, code_coef, gi, row_mask);
                else
                    pick_and_update<D_, G>(Atile, q, lane, Db, n0, g + 1 < s, code_idx, code_coef, gi);
                if (g + 1 < s) {
                    fence_proxy_async_smem();
                    mbar_arrive(&sm.res_ready[tile]);
                }
                __syncwarp();
                // ---- flush the collected codes eight at a time ----
                if ((gi == CODE_BLOCK - 1 || g == s - 1) && valid && writes_codes && (CL != 2 || (lane < 16) == (acc == 0))) {
                    const int g0 = g - gi;
                    const int64_t o = m * ldc + g0;
                    if (gi == CODE_BLOCK - 1 && vec_codes) {
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
                __syncwarp();
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
    // a CTA's shared memory must outlive its peers' last writes to it
    if constexpr (CL) cluster_sync_all();
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_tiled() {
    static const EncodeTiledFn fn = [] {               // initialised once, also with concurrent callers
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

constexpr int kClusterLaunchRefused = 1;                  // internal: not a CSR_ERR_* code

template <int D_, int G>
void cluster_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int cluster_ctas, int grid, size_t smem,
                    cudaStream_t stream) {
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(NT, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster_ctas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

// How many clusters of `cluster_ctas` CTAs of the encoder the device holds at once (0: none,
// or clusters of that size cannot be launched here).  Asked once per size.
template <int D_, int G>
int max_clusters(int cluster_ctas) {
    static int cached_dev[64][17] = {};                // per device: 0 = not asked yet, -1 = none
    static std::mutex mu;
    int dev = 0;
    if (cluster_ctas < 2 || cluster_ctas > 16 || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    std::lock_guard<std::mutex> lk(mu);
    int* cached = cached_dev[dev];                     // (function attributes are per device as well)
    if (cached[cluster_ctas] == 0) {
        const size_t smem = sizeof(FastSmem<D_>) + 1024;
        int n = 0;
        bool good = cudaFuncSetAttribute(encode_fast_kernel<D_, G, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem) == cudaSuccess;
        if (good && cluster_ctas > 8)
            good = cudaFuncSetAttribute(encode_fast_kernel<D_, G, 1>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) ==
                       cudaSuccess &&
                   cudaFuncSetAttribute(encode_fast_kernel<D_, G, 2>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) ==
                       cudaSuccess;
        if (good) {
            cudaLaunchConfig_t cfg = {};
            cudaLaunchAttribute attr[1];
            cluster_config<D_, G>(cfg, attr, cluster_ctas, cluster_ctas, smem, 0);
            good = cudaOccupancyMaxActiveClusters(&n, encode_fast_kernel<D_, G, 1>, &cfg) == cudaSuccess;
        }
        if (!good) {
            cudaGetLastError();                        // a refusal is an answer, not a failure of the call
            n = 0;
        }
        cached[cluster_ctas] = n > 0 ? n : -1;
    }
    return cached[cluster_ctas] > 0 ? cached[cluster_ctas] : 0;
}

template <int D_, int G>
int launch(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status, int n_splits,
           uint2* partial, int cluster_grid = 0) {
    const size_t smem = sizeof(FastSmem<D_>) + 1024;
    // at most one tile of rows in all: the clustered kernel that spends both accumulators on it
    const bool one_tile = cluster_grid > 0 && a.M <= TILE_M && n_splits <= FastSmem<D_>::kATileBytes / (2 * TILE_M * 8);
    cudaError_t e =
        cluster_grid > 0
            ? cudaFuncSetAttribute(one_tile ? encode_fast_kernel<D_, G, 2> : encode_fast_kernel<D_, G, 1>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
            : cudaFuncSetAttribute(encode_fast_kernel<D_, G, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    const int64_t n_pairs = (a.M + 2 * TILE_M - 1) / (2 * TILE_M);
    const int grid = n_splits > 1 ? (int)(n_pairs * n_splits)
                                  : (int)(n_pairs < (int64_t)sm_count() ? n_pairs : (int64_t)sm_count());
    // keys keep the magnitude bits above the group tag; with G == 1 the key is built from the
    // raw value, so the mask clears the sign bit as well
    const uint32_t key_mask = (G == 1 ? 0x7FFFFFFFu : 0xFFFFFFFFu) & ~static_cast<uint32_t>(TILE_N / G - 1);
    // 16-byte code stores need eight codes per flush and 16-byte aligned rows in both arrays
    const uintptr_t ci = reinterpret_cast<uintptr_t>(a.out_idx), cc = reinterpret_cast<uintptr_t>(a.out_coef);
    const int vec_codes = (a.s % 8 == 0) && (a.ld_code % 8 == 0) && (ci % 16 == 0) && (cc % 16 == 0);
    const unsigned long long wait_limit = options().wait_limit_ns;
    if (cluster_grid > 0) {
        // n_splits CTAs per cluster, cluster_grid CTAs in all
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        cluster_config<D_, G>(cfg, attr, n_splits, cluster_grid, smem, a.stream);
        e = cudaLaunchKernelEx(&cfg, one_tile ? encode_fast_kernel<D_, G, 2> : encode_fast_kernel<D_, G, 1>, tmap, Db, a.X, a.x_dtype, a.ldx, a.M, a.N, a.s, a.out_idx,
                               a.out_coef, a.coef_dtype, a.ld_code, vec_codes, key_mask, status, n_splits,
                               static_cast<uint2*>(nullptr), wait_limit);
        if (e != cudaSuccess) {
            // refused at launch (nothing ran): the caller takes another path
            cudaGetLastError();
            return kClusterLaunchRefused;
        }
        return CSR_OK;
    }
    encode_fast_kernel<D_, G, 0><<<grid, NT, smem, a.stream>>>(tmap, Db, a.X, a.x_dtype, a.ldx, a.M, a.N, a.s, a.out_idx,
                                                           a.out_coef, a.coef_dtype, a.ld_code, vec_codes, key_mask,
                                                           status, n_splits, partial, wait_limit);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "encode_fast launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

// Atoms per arg-max group.  Larger groups save arg-max arithmetic during the sweep (which
// grows with N) and cost a wider gather at the end of every sweep (which does not); the
// defaults are where the measured crossovers lie.  The option "fast_group" (1, 2, 4 or 8)
// overrides them; it is a tuning knob only: every setting picks, per row, an atom whose bf16
// correlation is the largest to within the width of the group tag.
int group_size(int d, int N) {
    const int v = options().fast_group;
    if (v == 1 || v == 2 || v == 4 || v == 8) return v;
    if (d == 64) return N <= 2048 ? 2 : 4;
    return 1;
}

template <int D_>
int launch_d(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status) {
    switch (group_size(D_, a.N)) {
        case 1: return launch<D_, 1>(a, tmap, Db, status, 0, nullptr);
        case 2: return launch<D_, 2>(a, tmap, Db, status, 0, nullptr);
        case 8: return launch<D_, 8>(a, tmap, Db, status, 0, nullptr);
        default: return launch<D_, 4>(a, tmap, Db, status, 0, nullptr);
    }
}

// Few rows, one launch: clusters of CTAs share a pair of row tiles.  Picks the cluster size
// whose modelled time per iteration (about 1.6 us per 256-atom tile swept plus about 3.5 us
// for the exchange and the pick, over as many rounds as the device needs to hold all pairs)
// is lowest, and returns 0 when one CTA per pair over the whole dictionary (about 1.55 us
// per tile, measured) is no slower, or when the estimate exceeds `budget_us` (what another
// path is expected to take).  *grid gets the CTAs to launch.
template <int D_, int G>
int cluster_split(int64_t M, int N, float budget_us, int* grid) {
    const int64_t n_pairs = (M + 2 * TILE_M - 1) / (2 * TILE_M);
    const int T = (N + TILE_N - 1) / TILE_N;
    if (n_pairs < 1 || T < 2) return 0;
    float best = 0.f;
    int best_ns = 0;
    for (int ns = 16; ns >= 2; ns >>= 1) {
        if (ns > T) continue;
        // one tile of rows: the exchange buffers (the unused row tile) bound the cluster size
        if (M <= TILE_M && ns > FastSmem<D_>::kATileBytes / (2 * TILE_M * 8)) continue;
        const int nc = max_clusters<D_, G>(ns);
        if (nc < 1) continue;
        const int64_t rounds = (n_pairs + nc - 1) / nc;
        const float est = (float)rounds * (1.6f * ((T + ns - 1) / ns) + 3.5f);
        if (best_ns == 0 || est < best) {
            best = est;
            best_ns = ns;
            *grid = (int)(n_pairs < nc ? n_pairs : nc) * ns;
        }
    }
    if (best_ns == 0 || best > budget_us) return 0;
    const int64_t whole_rounds = (n_pairs + sm_count() - 1) / sm_count();
    return (float)whole_rounds * 1.55f * T > 1.15f * best ? best_ns : 0;
}

template <int D_>
int launch_clustered_g(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status, float budget_us,
                       bool* done);

// *done says whether the clustered launch took the job; a launch the driver refuses leaves
// it to the other paths.
template <int D_>
int launch_clustered(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status, float budget_us,
                     bool* done) {
    const int rc = launch_clustered_g<D_>(a, tmap, Db, status, budget_us, done);
    if (rc == kClusterLaunchRefused) {
        *done = false;
        return CSR_OK;
    }
    return rc;
}

template <int D_>
int launch_clustered_g(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status, float budget_us,
                       bool* done) {
    int grid = 0, ns = 0;
    *done = false;
    switch (group_size(D_, a.N)) {
        case 1:
            if ((ns = cluster_split<D_, 1>(a.M, a.N, budget_us, &grid)) == 0) return CSR_OK;
            *done = true;
            return launch<D_, 1>(a, tmap, Db, status, ns, nullptr, grid);
        case 2:
            if ((ns = cluster_split<D_, 2>(a.M, a.N, budget_us, &grid)) == 0) return CSR_OK;
            *done = true;
            return launch<D_, 2>(a, tmap, Db, status, ns, nullptr, grid);
        case 8:
            if ((ns = cluster_split<D_, 8>(a.M, a.N, budget_us, &grid)) == 0) return CSR_OK;
            *done = true;
            return launch<D_, 8>(a, tmap, Db, status, ns, nullptr, grid);
        default:
            if ((ns = cluster_split<D_, 4>(a.M, a.N, budget_us, &grid)) == 0) return CSR_OK;
            *done = true;
            return launch<D_, 4>(a, tmap, Db, status, ns, nullptr, grid);
    }
}

// Few rows: how many CTAs share a pair of row tiles (1 = the whole dictionary per CTA);
// *per_iter_us gets the modelled time of one iteration.
int split_count(int64_t M, int N, float* per_iter_us = nullptr) {
    const int64_t n_pairs = (M + 2 * TILE_M - 1) / (2 * TILE_M);
    const int T = (N + TILE_N - 1) / TILE_N;
    if (n_pairs < 1 || n_pairs * 2 > sm_count() || T < 2) return 1;
    int ns = (int)(sm_count() / n_pairs);
    if (ns > T) ns = T;
    if (ns > 32) ns = 32;
    // Worth it only if an iteration's sweep over all T tiles by one CTA (about 1.55 us per
    // tile, measured) outlasts two launches (about 12 us) plus the sweep of a slice.
    const float whole = 1.55f * T, sliced = 12.f + 1.6f * ((T + ns - 1) / ns);
    if (per_iter_us) *per_iter_us = sliced;
    return whole > 1.2f * sliced ? ns : 1;
}
size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// One launch of the sweep (every CTA a slice of the dictionary, s = 1) and one of the pick
// per iteration; the residual rows live in global memory as bf16 in between.
template <int D_, int G>
int run_split_g(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status, void* scratch) {
    const int ns = split_count(a.M, a.N);
    uint4* Rb = static_cast<uint4*>(scratch);
    uint2* partial = reinterpret_cast<uint2*>(static_cast<char*>(scratch) + align256((size_t)a.M * D_ * 2));
    const int64_t chunks = a.M * (D_ / 8);
    rows_to_bf16_kernel<D_><<<(unsigned)((chunks + 255) / 256), 256, 0, a.stream>>>(a.X, a.x_dtype, a.ldx, a.M, Rb);
    EncodeArgs b = a;
    b.X = Rb;
    b.x_dtype = CSR_DTYPE_BF16;
    b.ldx = D_;
    b.s = 1;
    const unsigned pick_blocks = (unsigned)((a.M + 15) / 16);
    for (int g = 0; g < a.s; ++g) {
        if (int rc = launch<D_, G>(b, tmap, Db, status, ns, partial)) return rc;
        split_pick_kernel<D_, G><<<pick_blocks, 128, 0, a.stream>>>(Db, a.N, Rb, partial, ns, a.M, g, g + 1 < a.s, a.out_idx, a.out_coef,
                                                                a.coef_dtype, a.ld_code);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "encode_fast split launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

template <int D_>
int run_split(const EncodeArgs& a, const CUtensorMap& tmap, const uint16_t* Db, uint32_t* status, void* scratch) {
    switch (group_size(D_, a.N)) {
        case 1: return run_split_g<D_, 1>(a, tmap, Db, status, scratch);
        case 2: return run_split_g<D_, 2>(a, tmap, Db, status, scratch);
        case 8: return run_split_g<D_, 8>(a, tmap, Db, status, scratch);
        default: return run_split_g<D_, 4>(a, tmap, Db, status, scratch);
    }
}

}  // namespace

bool encode_fast_split_applies(int64_t M, int N) { return M > 0 && split_count(M, N) > 1; }
size_t encode_fast_split_scratch_bytes(int64_t M, int d, int N) {
    return align256((size_t)M * d * 2) + align256((size_t)M * split_count(M, N) * sizeof(uint2));
}

// The bf16 copy holds N rounded up to a multiple of 8 atoms; the extra rows are zero, so a
// group of up to 8 candidate atoms never reaches past the copy.
static int padded_atoms(int N) { return (N + 7) / 8 * 8; }
size_t encode_fast_workspace_bytes(int d, int N) { return (size_t)padded_atoms(N) * (size_t)d * 2; }

int prepare_fast_dictionary(const float* D, int N, int d, void* workspace, cudaStream_t stream) {
    if ((reinterpret_cast<uintptr_t>(workspace) & 1023u) != 0)
        return fail(CSR_ERR_ALIGNMENT, "internal: dictionary scratch not 1024-byte aligned");
    const int64_t n_vec4 = (int64_t)N * d / 4;
    int blocks = (int)((n_vec4 + 255) / 256);
    if (blocks > 4 * sm_count()) blocks = 4 * sm_count();
    dict_to_bf16_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const float4*>(D), reinterpret_cast<uint2*>(workspace),
                                                    n_vec4);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "dict_to_bf16 launch: %s", cudaGetErrorString(e));
    const int n_pad = padded_atoms(N);
    if (n_pad > N) {
        e = cudaMemsetAsync(static_cast<char*>(workspace) + (size_t)N * d * 2, 0, (size_t)(n_pad - N) * d * 2, stream);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    }
    return CSR_OK;
}

int launch_encode_fast(const EncodeArgs& a, void* workspace, uint32_t* status) {
    if (a.M == 0) return CSR_OK;
    if (int rc = prepare_fast_dictionary(a.D, a.N, a.d, workspace, a.stream)) return rc;
    return launch_encode_fast_prepared(a, workspace, status, nullptr);
}

int launch_encode_fast_prepared(const EncodeArgs& a, const void* dict_bf16, uint32_t* status, void* split_scratch) {
    if (a.M == 0) return CSR_OK;
    void* workspace = const_cast<void*>(dict_bf16);
    if ((reinterpret_cast<uintptr_t>(workspace) & 1023u) != 0)
        return fail(CSR_ERR_ALIGNMENT, "internal: dictionary scratch not 1024-byte aligned");
    EncodeTiledFn encode = get_encode_tiled();
    if (!encode) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const int n_pad = padded_atoms(a.N);

    // rows past the padded copy (the rest of the last 256-atom tile) are filled with zeros by TMA
    CUtensorMap tmap;
    const cuuint64_t gdim[2] = {(cuuint64_t)a.d, (cuuint64_t)n_pad};
    const cuuint64_t gstride[1] = {(cuuint64_t)a.d * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)TILE_N};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, workspace, gdim, gstride, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(CSR_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);

    const uint16_t* Db = static_cast<const uint16_t*>(workspace);
    // few rows: one launch of CTA clusters that share the dictionary (needs no scratch) ...
    // (unless the launch-per-iteration split below, which can spread a pair of row tiles over more
    // than 16 CTAs, is expected to be faster: very large dictionaries)
    if (options().fast_split == 0) {
        float budget = 3.0e38f;
        if (split_scratch && split_count(a.M, a.N, &budget) <= 1) budget = 3.0e38f;
        bool done = false;
        const int rc = a.d == 128 ? launch_clustered<128>(a, tmap, Db, status, budget, &done)
                                  : launch_clustered<64>(a, tmap, Db, status, budget, &done);
        if (rc != CSR_OK || done) return rc;
    }
    // ... else, with scratch, a sweep launch and a pick launch per iteration
    if (split_scratch) {
        if (a.d == 128) return run_split<128>(a, tmap, Db, status, split_scratch);
        return run_split<64>(a, tmap, Db, status, split_scratch);
    }
    if (a.d == 128) return launch_d<128>(a, tmap, Db, status);
    return launch_d<64>(a, tmap, Db, status);
}

}  // namespace csr
