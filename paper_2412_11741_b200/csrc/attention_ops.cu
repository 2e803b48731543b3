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
// scratch array [B][N][H] (a stream's heads side by side per atom; channels summed in
// ascending order); (2) one CTA per (code stream, token range) copies its heads' part of p
// into shared memory, streams the codes, one thread per token, and sums the s terms in
// stored order.
// value_mix: (1) every code stream is cut into `pieces` token ranges, one CTA each, which
// scatters w * coef into a[head][N] in shared memory with atomic adds while it streams the
// codes and then stores its a to the scratch array [B][pieces][H][N]; (2) out = a D with the
// pieces summed in order on the way in, a small fp32 GEMM (split into slices of the atoms
// when there are few heads; the slices' partial results are then added in slice order by
// add_slices_kernel).  The tables are accumulated in fixed point (see value_scatter_kernel),
// and every floating-point sum is taken in a fixed order, so the result is the same bits on
// every run.
#include "exact_common.cuh"

namespace csr {
namespace {

constexpr int NT = 256;
constexpr int NTS = 1024;   // threads of the code-streaming kernels (one CTA per SM: shared memory)

__device__ __forceinline__ float load_coef(const void* coef, int coef_dtype, int64_t off) {
    return coef_dtype == CSR_DTYPE_F16 ? __half2float(reinterpret_cast<const __half*>(coef)[off])
                                       : reinterpret_cast<const float*>(coef)[off];
}
__device__ __forceinline__ float load_q(const void* Q, int q_dtype, int64_t off) { return load_elem(Q, q_dtype, off); }

// ---- P[b][n][h] = scale * Q[r][:] . D[n][:]  (r = b*H + h) --------------------------------
// CTA = 64 rows x one 128-atom tile of the dictionary, on the register-tiled product the
// exact encoder sweeps with (thread = 4 rows x 8 atoms, channels summed in ascending order).
template <int D_>
__global__ void __launch_bounds__(NT)
qd_kernel(const float* __restrict__ D, int N, const void* __restrict__ Q, int q_dtype, int R, int H, float scale,
          float* __restrict__ P) {
    __shared__ __align__(16) float As[D_][exact::AS_LD];              // As[k][row]
    __shared__ __align__(16) float Bs[2][exact::BK][exact::BS_LD];
    const int r0 = blockIdx.y * exact::BM;
    for (int f = threadIdx.x; f < exact::BM * D_; f += NT) {
        const int r = f / D_, k = f % D_;
        As[k][r] = (r0 + r < R) ? load_q(Q, q_dtype, (int64_t)(r0 + r) * D_ + k) : 0.f;
    }
    __syncthreads();
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    exact::sweep_tiles_fn<D_>(D, N, blockIdx.x, blockIdx.x + 1, As, Bs, [&](int bt, const float (&acc)[4][8]) {
        const int rr = r0 + ty * 4;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int n = bt * exact::BN + (j >> 2) * 64 + tx * 4 + (j & 3);
            if (n >= N) continue;
            if (H == 4 && rr + 3 < R) {                   // the four rows are one stream's four heads
                float4 v;
                v.x = scale * acc[0][j];
                v.y = scale * acc[1][j];
                v.z = scale * acc[2][j];
                v.w = scale * acc[3][j];
                *reinterpret_cast<float4*>(P + ((int64_t)(rr / 4) * N + n) * 4) = v;
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = rr + i;
                    if (r < R) P[((int64_t)(r / H) * N + n) * H + r % H] = scale * acc[i][j];
                }
            }
        }
    });
}

// ---- part[slice][r][:] = sum_{n in slice} (sum_pieces A[b][piece][h][n]) * D[n][:] ----------
// CTA = 64 rows x all channels x one slice of the atoms; thread = 4 rows x 8 (d = 128) or 4
// (d = 64) channels.  The slice is taken 64 atoms at a time: all of a tile's loads are issued
// together (one memory latency per tile, several CTAs per SM to cover it), then the tile is
// multiplied out of shared memory, atoms in ascending order.  With more than one slice a
// second kernel adds the slices in order, so the result does not depend on the schedule.
constexpr int OR = 64;    // rows per CTA
constexpr int OA = 64;    // atoms per tile
template <int D_>
struct AdSmem {
    float As[OA][OR + 4];      // As[atom][row]
    float Bs[OA][D_ + 4];      // Bs[atom][channel]
};
template <int D_>
__global__ void __launch_bounds__(NT, 3)
ad_kernel(const float* __restrict__ D, int N, const float* __restrict__ A, int R, int H, int pieces, int atoms_per_slice,
          float* __restrict__ part) {
    extern __shared__ __align__(16) unsigned char ad_raw[];
    AdSmem<D_>& sm = *reinterpret_cast<AdSmem<D_>*>(ad_raw);
    constexpr int CPT = D_ / 16;                          // channels per thread: 8 or 4
    constexpr int DV = OA * D_ / 4 / NT;                  // float4 of D per thread per tile: 8 or 4
    constexpr int AV = OA * OR / 4 / NT;                  // float4 of A per thread per tile: 4
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int r0 = blockIdx.y * OR;
    const int nb = blockIdx.x * atoms_per_slice;
    const int ne = min(nb + atoms_per_slice, N);
    const int64_t piece_stride = (int64_t)H * N;
    const bool vec_a = (N % 4) == 0;                       // rows of A start on 16-byte boundaries
    float acc[4][CPT];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < CPT; ++j) acc[i][j] = 0.f;
    for (int n0 = nb; n0 < ne; n0 += OA) {
        // ---- stage the tile: A (pieces summed in order, transposed) and D ----
        float4 av[AV];
#pragma unroll
        for (int u = 0; u < AV; ++u) av[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int pc = 0; pc < pieces; ++pc) {
#pragma unroll
            for (int u = 0; u < AV; ++u) {
                // float4 index: consecutive lanes take consecutive rows (the transposed stores
                // below are then free of bank conflicts), atoms 4 * (f / 64) ..
                const int f = tid + u * NT;
                const int r = r0 + f % OR, n = n0 + 4 * (f / OR);
                if (r >= R || n >= ne) continue;
                const float* src = A + (((int64_t)(r / H) * pieces + pc) * H + r % H) * N + n;
                float4 v;
                if (vec_a && n + 3 < ne) {
                    v = *reinterpret_cast<const float4*>(src);
                } else {
                    v.x = src[0];
                    v.y = n + 1 < ne ? src[1] : 0.f;
                    v.z = n + 2 < ne ? src[2] : 0.f;
                    v.w = n + 3 < ne ? src[3] : 0.f;
                }
                av[u].x += v.x;
                av[u].y += v.y;
                av[u].z += v.z;
                av[u].w += v.w;
            }
        }
        float4 dv[DV];
#pragma unroll
        for (int u = 0; u < DV; ++u) {
            const int f = tid + u * NT;
            const int atom = f / (D_ / 4), c4 = f % (D_ / 4);
            dv[u] = (n0 + atom < ne) ? *reinterpret_cast<const float4*>(D + (int64_t)(n0 + atom) * D_ + c4 * 4)
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        __syncthreads();                                   // the previous tile has been used
#pragma unroll
        for (int u = 0; u < AV; ++u) {
            const int f = tid + u * NT;
            const int r = f % OR, a4 = 4 * (f / OR);
            sm.As[a4 + 0][r] = av[u].x;
            sm.As[a4 + 1][r] = av[u].y;
            sm.As[a4 + 2][r] = av[u].z;
            sm.As[a4 + 3][r] = av[u].w;
        }
#pragma unroll
        for (int u = 0; u < DV; ++u) {
            const int f = tid + u * NT;
            *reinterpret_cast<float4*>(&sm.Bs[f / (D_ / 4)][(f % (D_ / 4)) * 4]) = dv[u];
        }
        __syncthreads();
        // ---- multiply ----
#pragma unroll 8
        for (int k = 0; k < OA; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&sm.As[k][ty * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            float bch[CPT];
#pragma unroll
            for (int q = 0; q < CPT / 4; ++q) {
                const float4 b4 = *reinterpret_cast<const float4*>(&sm.Bs[k][q * 64 + tx * 4]);
                bch[4 * q + 0] = b4.x;
                bch[4 * q + 1] = b4.y;
                bch[4 * q + 2] = b4.z;
                bch[4 * q + 3] = b4.w;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < CPT; ++j) acc[i][j] = fmaf(a[i], bch[j], acc[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty * 4 + i;
        if (r >= R) continue;
        float* dst = part + ((int64_t)blockIdx.x * R + r) * D_;
#pragma unroll
        for (int q = 0; q < CPT / 4; ++q)
            *reinterpret_cast<float4*>(dst + q * 64 + tx * 4) =
                make_float4(acc[i][4 * q + 0], acc[i][4 * q + 1], acc[i][4 * q + 2], acc[i][4 * q + 3]);
    }
}

// out[j] = part[0][j] + part[1][j] + ... in this order
__global__ void __launch_bounds__(NT)
add_slices_kernel(const float* __restrict__ part, int slices, int64_t n, float* __restrict__ out) {
    const int64_t j = (int64_t)blockIdx.x * NT + threadIdx.x;
    if (j >= n) return;
    float v = 0.f;
    for (int sl = 0; sl < slices; ++sl) v += part[(int64_t)sl * n + j];
    out[j] = v;
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
// Work = (code stream, chunk of CHUNK_T tokens); each persistent CTA takes a contiguous,
// balanced range of it, so it changes stream (and reloads its shared-memory table) at most
// a few times.  The table is interleaved, tab[atom][HGP] with HGP = 1, 2, 4 or 8 query heads
// side by side, so that one vector access per stored entry serves all heads of the group.
constexpr int CHUNK_T = 1024;

template <int HGP>
struct HeadVec {
    float v[HGP];
};
template <int HGP>
__device__ __forceinline__ HeadVec<HGP> load_heads(const float* p) {
    HeadVec<HGP> r;
    if constexpr (HGP == 1) {
        r.v[0] = p[0];
    } else if constexpr (HGP == 2) {
        const float2 t = *reinterpret_cast<const float2*>(p);
        r.v[0] = t.x;
        r.v[1] = t.y;
    } else {
#pragma unroll
        for (int q = 0; q < HGP / 4; ++q) {
            const float4 t = *reinterpret_cast<const float4*>(p + 4 * q);
            r.v[4 * q + 0] = t.x;
            r.v[4 * q + 1] = t.y;
            r.v[4 * q + 2] = t.z;
            r.v[4 * q + 3] = t.w;
        }
    }
    return r;
}

// Calls f(g, atom, coef) for the s stored entries of the token whose codes start at `o`.
template <typename F>
__device__ __forceinline__ void for_each_code(const uint16_t* idx, const void* coef, int coef_dtype, int64_t o, int s, int N,
                                              int vec, F&& f) {
    if (vec) {
        for (int g0 = 0; g0 < s; g0 += 8) {
            int i8[8];
            float c8[8];
            load_codes8(idx, coef, coef_dtype, o + g0, i8, c8);
#pragma unroll
            for (int g = 0; g < 8; ++g) f(i8[g] < N ? i8[g] : N - 1, c8[g]);
        }
    } else {
        for (int g = 0; g < s; ++g) {
            const int i = idx[o + g];
            f(i < N ? i : N - 1, load_coef(coef, coef_dtype, o + g));
        }
    }
}

template <int HGP>
__global__ void __launch_bounds__(NTS)
key_scores_kernel(const float* __restrict__ P, int N, int B, int H, const uint16_t* __restrict__ idx,
                  const void* __restrict__ coef, int coef_dtype, int64_t T, int s, int vec, float* __restrict__ scores) {
    extern __shared__ __align__(16) float tab[];           // [N][HGP]
    const int64_t chunks_per_b = (T + CHUNK_T - 1) / CHUNK_T;
    const int64_t total = (int64_t)B * chunks_per_b;
    const int64_t w0 = total * blockIdx.x / gridDim.x, w1 = total * (blockIdx.x + 1) / gridDim.x;
    for (int h0 = 0; h0 < H; h0 += HGP) {
        const int hg = H - h0 < HGP ? H - h0 : HGP;
        int cur_b = -1;
        for (int64_t w = w0; w < w1; ++w) {
            const int b = (int)(w / chunks_per_b);
            if (b != cur_b) {
                __syncthreads();
                const float* src = P + (int64_t)b * N * H;           // [N][H]
                if (HGP == H && HGP >= 4) {                          // the whole stream's table, as it lies
                    const float4* s4 = reinterpret_cast<const float4*>(src);
                    float4* t4 = reinterpret_cast<float4*>(tab);
                    const int n4 = N * HGP / 4;
#pragma unroll 8
                    for (int j = threadIdx.x; j < n4; j += NTS) t4[j] = s4[j];
                } else {
                    for (int j = threadIdx.x; j < N * HGP; j += NTS) {
                        const int n = j / HGP, h = j % HGP;
                        tab[j] = h < hg ? src[(int64_t)n * H + h0 + h] : 0.f;
                    }
                }
                __syncthreads();
                cur_b = b;
            }
            const int64_t t = (w % chunks_per_b) * CHUNK_T + threadIdx.x;
            if (t >= T) continue;
            float acc[HGP];
#pragma unroll
            for (int h = 0; h < HGP; ++h) acc[h] = 0.f;
            for_each_code(idx, coef, coef_dtype, ((int64_t)b * T + t) * s, s, N, vec, [&](int i, float c) {
                const HeadVec<HGP> pv = load_heads<HGP>(tab + i * HGP);
#pragma unroll
                for (int h = 0; h < HGP; ++h) acc[h] = fmaf(c, pv.v[h], acc[h]);
            });
#pragma unroll
            for (int h = 0; h < HGP; ++h)
                if (h < hg) scores[((int64_t)b * H + h0 + h) * T + t] = acc[h];
        }
    }
}

// Block-wide maximum / sum of one value per thread (NTS threads), returned to every thread;
// the order of the additions is fixed.
__device__ __forceinline__ float block_max(float v, float* red) {
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int j = 1; j < NTS / 32; ++j) r = fmaxf(r, red[j]);
    return r;
}
__device__ __forceinline__ float block_sum(float v, float* red) {
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
    for (int j = 0; j < NTS / 32; ++j) r += red[j];
    return r;
}

// Unit of work = (code stream, piece): a contiguous range of the stream's token chunks.  The
// CTA owns the unit's table, so its result is stored, not added.
//
// The table is accumulated in 32-bit fixed point: integer shared-memory atomics run at more
// than twice the rate of fp32 ones (measured 17.5 against 7.7 per ns per SM), and integer
// addition does not depend on the order, so the table is the same on every run.  A first
// pass over the unit's weights and coefficients gives, per head, S = sum |w_t| and
// U = max over tokens of sum_g |coef[t][g]| (a token's entries may all name one atom); no
// table entry can exceed S * U in magnitude, and the scale is the power
// of two that maps S * U to at most 2^29, which leaves the rounding of the individual terms
// (half a unit each) far inside the 32-bit range.  Each term w * coef is rounded once to
// fp32, as a floating-point accumulation would, and once to the grid, whose step is
// 2^-29 * S * U or finer.  A unit whose S or U is not finite falls back to fp32 atomics, so
// that NaN and Inf still reach the output.
template <int HGP>
__global__ void __launch_bounds__(NTS)
value_scatter_kernel(int N, const float* __restrict__ W, int B, int H, const uint16_t* __restrict__ idx,
                     const void* __restrict__ coef, int coef_dtype, int64_t T, int s, int vec, int pieces,
                     float* __restrict__ A) {
    extern __shared__ __align__(16) float tab[];           // [HGP][N]: scalar atomics want the heads apart
    __shared__ float red[NTS / 32];
    int* itab = reinterpret_cast<int*>(tab);
    const int64_t chunks_per_b = (T + CHUNK_T - 1) / CHUNK_T;
    const int64_t units = (int64_t)B * pieces;
    for (int64_t unit = blockIdx.x; unit < units; unit += gridDim.x) {
        const int b = (int)(unit / pieces), piece = (int)(unit % pieces);
        const int64_t c0 = chunks_per_b * piece / pieces, c1 = chunks_per_b * (piece + 1) / pieces;
        for (int h0 = 0; h0 < H; h0 += HGP) {
            const int hg = H - h0 < HGP ? H - h0 : HGP;
            __syncthreads();
            for (int j = threadIdx.x; j < N * HGP; j += NTS) tab[j] = 0.f;    // +0.0f and integer 0 share their bits
            // ---- pass 1: bounds ----
            float umax = 0.f, sw[HGP];
#pragma unroll
            for (int h = 0; h < HGP; ++h) sw[h] = 0.f;
            for (int64_t c = c0; c < c1; ++c) {
                const int64_t t = c * CHUNK_T + threadIdx.x;
                if (t >= T) continue;
#pragma unroll
                for (int h = 0; h < HGP; ++h)
                    if (h < hg) sw[h] += fabsf(W[((int64_t)b * H + h0 + h) * T + t]);
                float l1 = 0.f;                            // all of a token's entries may name the same atom
                for_each_code(idx, coef, coef_dtype, ((int64_t)b * T + t) * s, s, N, vec,
                              [&](int, float cf) { l1 += fabsf(cf); });
                umax = l1 == l1 ? fmaxf(umax, l1) : INFINITY;
            }
            umax = block_max(umax, red);
            float scale[HGP], inv_scale[HGP];
            // (the half-unit roundings of the terms must stay far inside the range too)
            bool fixed_point = umax < INFINITY && (c1 - c0) * CHUNK_T * static_cast<int64_t>(s) <= (1ll << 30);
#pragma unroll
            for (int h = 0; h < HGP; ++h) {
                const float S = block_sum(sw[h], red);
                const float bound = S * umax;
                if (!(bound < INFINITY)) fixed_point = false;                 // Inf or NaN
                int e = 0;
                if (bound > 0.f) e = 29 - (ilogbf(bound) + 1);                // 2^e * bound <= 2^29
                e = e > 96 ? 96 : e < -96 ? -96 : e;
                scale[h] = ldexpf(1.f, e);
                inv_scale[h] = ldexpf(1.f, -e);
            }
            __syncthreads();
            // ---- pass 2: scatter ----
            for (int64_t c = c0; c < c1; ++c) {
                const int64_t t = c * CHUNK_T + threadIdx.x;
                if (t >= T) continue;
                float wv[HGP];
#pragma unroll
                for (int h = 0; h < HGP; ++h) wv[h] = h < hg ? W[((int64_t)b * H + h0 + h) * T + t] : 0.f;
                if (fixed_point) {
#pragma unroll
                    for (int h = 0; h < HGP; ++h) wv[h] *= scale[h];          // exact: a power of two
                    for_each_code(idx, coef, coef_dtype, ((int64_t)b * T + t) * s, s, N, vec, [&](int i, float cf) {
#pragma unroll
                        for (int h = 0; h < HGP; ++h)
                            if (h < hg) atomicAdd(&itab[h * N + i], __float2int_rn(wv[h] * cf));
                    });
                } else {
                    for_each_code(idx, coef, coef_dtype, ((int64_t)b * T + t) * s, s, N, vec, [&](int i, float cf) {
#pragma unroll
                        for (int h = 0; h < HGP; ++h)
                            if (h < hg) atomicAdd(&tab[h * N + i], wv[h] * cf);
                    });
                }
            }
            __syncthreads();
            float* dst = A + ((unit * H) + h0) * N;         // rows h0 .. h0+hg-1 of this unit, [H][N]
            if (fixed_point) {
#pragma unroll
                for (int h = 0; h < HGP; ++h)
                    if (h < hg)
                        for (int j = threadIdx.x; j < N; j += NTS) dst[h * N + j] = static_cast<float>(itab[h * N + j]) * inv_scale[h];
            } else {
                for (int j = threadIdx.x; j < hg * N; j += NTS) dst[j] = tab[j];
            }
        }
    }
}

// Softmax over the T scores of one (stream, head) row, in place; one CTA per row, fp32, the
// maximum subtracted first; the row is read three times (maximum, sum, result) and written once.  Rows are a few tens of KB and were just written: they come
// from L2.
__global__ void __launch_bounds__(NT)
softmax_rows_kernel(float* __restrict__ S, int64_t T) {
    __shared__ float red[NT / 32];
    __shared__ float bcast;
    float* row = S + (int64_t)blockIdx.x * T;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float mx = -INFINITY;
    for (int64_t t = threadIdx.x; t < T; t += NT) mx = fmaxf(mx, row[t]);
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
        float m = red[0];
        for (int j = 1; j < NT / 32; ++j) m = fmaxf(m, red[j]);
        bcast = m;
    }
    __syncthreads();
    mx = bcast;
    float sum = 0.f;
    for (int64_t t = threadIdx.x; t < T; t += NT) sum += __expf(row[t] - mx);
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    __syncthreads();
    if (lane == 0) red[warp] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int j = 0; j < NT / 32; ++j) t += red[j];
        bcast = 1.0f / t;
    }
    __syncthreads();
    const float inv = bcast;
    for (int64_t t = threadIdx.x; t < T; t += NT) row[t] = __expf(row[t] - mx) * inv;
}

// Query heads whose N-vectors fit in shared memory side by side: 8, 4, 2 or 1 (0 = none fits).
int head_group(int N, int H) {
    int hgp = 8;
    while (hgp > 1 && (hgp / 2 >= H || (size_t)hgp * N * 4 > 200 * 1024)) hgp /= 2;
    return (size_t)hgp * N * 4 > 200 * 1024 ? 0 : hgp;
}

int stream_grid(int B, int64_t T) {
    const int64_t total = (int64_t)B * ((T + CHUNK_T - 1) / CHUNK_T);
    return (int)(total < (int64_t)sm_count() ? total : (int64_t)sm_count());
}

template <int HGP>
cudaError_t run_key_scores(const AttnArgs& a, const float* P) {
    const size_t smem = (size_t)HGP * a.N * 4;
    cudaError_t e = cudaFuncSetAttribute(key_scores_kernel<HGP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    key_scores_kernel<HGP><<<stream_grid(a.B, a.T), NTS, smem, a.stream>>>(P, a.N, a.B, a.H, a.idx, a.coef, a.coef_dtype,
                                                                          a.T, a.s, a.s % 8 == 0, a.out);
    return cudaGetLastError();
}

// Token ranges a code stream is cut into for value_mix: enough to give every SM a unit, no
// more than there are chunks.
int value_pieces(int B, int64_t T) {
    const int64_t chunks_per_b = (T + CHUNK_T - 1) / CHUNK_T;
    int64_t k = B > 0 ? sm_count() / B : 1;
    if (k > chunks_per_b) k = chunks_per_b;
    return k < 1 ? 1 : (int)k;
}

template <int HGP>
cudaError_t run_value_scatter(const AttnArgs& a, float* A, int pieces) {
    const size_t smem = (size_t)HGP * a.N * 4;
    cudaError_t e = cudaFuncSetAttribute(value_scatter_kernel<HGP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t units = (int64_t)a.B * pieces;
    const int grid = (int)(units < (int64_t)sm_count() ? units : (int64_t)sm_count());
    value_scatter_kernel<HGP><<<grid, NTS, smem, a.stream>>>(a.N, static_cast<const float*>(a.Q), a.B, a.H, a.idx, a.coef,
                                                            a.coef_dtype, a.T, a.s, a.s % 8 == 0, pieces, A);
    return cudaGetLastError();
}

}  // namespace

// tables of the value mix (the larger use) + the per-slice outputs of its second step
size_t attn_scratch_bytes(int B, int H, int N, int64_t T) {
    const size_t slices_max = 4 * (size_t)sm_count();
    return ((size_t)B * value_pieces(B, T) * H * N + 4 + slices_max * (size_t)B * H * 128) * sizeof(float);
}

int launch_key_scores(const AttnArgs& a, float* P) {
    if (a.B == 0 || a.T == 0 || a.H == 0) return CSR_OK;
    const int hg = head_group(a.N, a.H);
    if (hg < 1) return fail(CSR_ERR_UNSUPPORTED, "N = %d: one head's N fp32 values do not fit in shared memory", a.N);
    const int R = a.B * a.H;
    const dim3 pgrid((a.N + exact::BN - 1) / exact::BN, (R + exact::BM - 1) / exact::BM);
    if (a.d == 128)
        qd_kernel<128><<<pgrid, NT, 0, a.stream>>>(a.D, a.N, a.Q, a.q_dtype, R, a.H, a.scale, P);
    else
        qd_kernel<64><<<pgrid, NT, 0, a.stream>>>(a.D, a.N, a.Q, a.q_dtype, R, a.H, a.scale, P);
    cudaError_t e = hg == 8 ? run_key_scores<8>(a, P) : hg == 4 ? run_key_scores<4>(a, P)
                    : hg == 2 ? run_key_scores<2>(a, P) : run_key_scores<1>(a, P);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "key_scores launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

int launch_softmax_rows(float* S, int64_t rows, int64_t T, cudaStream_t stream) {
    if (rows == 0 || T == 0) return CSR_OK;
    softmax_rows_kernel<<<(unsigned)rows, NT, 0, stream>>>(S, T);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "softmax launch: %s", cudaGetErrorString(e));
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
    const int pieces = value_pieces(a.B, a.T);
    cudaError_t e = hg == 8 ? run_value_scatter<8>(a, A, pieces) : hg == 4 ? run_value_scatter<4>(a, A, pieces)
                    : hg == 2 ? run_value_scatter<2>(a, A, pieces) : run_value_scatter<1>(a, A, pieces);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "value_scatter launch: %s", cudaGetErrorString(e));
    // out = A D: row blocks of 64; the atoms are split over CTAs as well (four CTAs per SM: each
    // waits for its next chunk of atoms most of the time)
    const int row_blocks = (R + OR - 1) / OR;
    int slices = 4 * sm_count() / row_blocks;
    const int max_slices = (a.N + 63) / 64;
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    const int per_slice = ((a.N + slices - 1) / slices + OA - 1) / OA * OA;
    slices = (a.N + per_slice - 1) / per_slice;
    float* part = slices > 1 ? A + ((size_t)a.B * pieces * a.H * a.N + 3) / 4 * 4 : a.out;      // 16-byte aligned
    const dim3 ogrid(slices, row_blocks);
    cudaError_t e2;
    if (a.d == 128) {
        e2 = cudaFuncSetAttribute(ad_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AdSmem<128>));
        ad_kernel<128><<<ogrid, NT, sizeof(AdSmem<128>), a.stream>>>(a.D, a.N, A, R, a.H, pieces, per_slice, part);
    } else {
        e2 = cudaFuncSetAttribute(ad_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AdSmem<64>));
        ad_kernel<64><<<ogrid, NT, sizeof(AdSmem<64>), a.stream>>>(a.D, a.N, A, R, a.H, pieces, per_slice, part);
    }
    if (e2 != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e2));
    if (slices > 1) {
        const int64_t n = (int64_t)R * a.d;
        add_slices_kernel<<<(unsigned)((n + NT - 1) / NT), NT, 0, a.stream>>>(part, slices, n, a.out);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "value_mix launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace csr
