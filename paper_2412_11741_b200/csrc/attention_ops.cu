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
// pieces summed in order on the way in, a small fp32 GEMM (split over atoms with atomic
// adds when there are few heads).  The tables are accumulated in fixed point (see
// value_scatter_kernel) and are the same on every run; the split over atoms of step (2),
// when it is used, still adds in an order that varies.
#include "common.cuh"

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
// CTA = 64 atoms x 64 rows; thread = 4 rows x 4 atoms; channels staged 32 at a time,
// transposed, and summed in ascending order.
constexpr int PA = 64;    // atoms per CTA
constexpr int QROWS = 64; // rows per CTA (grid.y)
constexpr int PK = 32;    // channels per staged block
template <int D_>
__global__ void __launch_bounds__(NT)
qd_kernel(const float* __restrict__ D, int N, const void* __restrict__ Q, int q_dtype, int R, int H, float scale,
          float* __restrict__ P) {
    __shared__ __align__(16) float Ds[PK][PA + 4];         // Ds[k][atom]
    __shared__ __align__(16) float Qs[PK][QROWS + 4];      // Qs[k][row]
    const int n0 = blockIdx.x * PA, r0 = blockIdx.y * QROWS;
    const int ta = (threadIdx.x & 15) * 4, tr = (threadIdx.x >> 4) * 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < D_; k0 += PK) {
        __syncthreads();
        for (int f = threadIdx.x; f < PA * PK; f += NT) {
            const int a = f / PK, k = f % PK;
            Ds[k][a] = (n0 + a < N) ? D[(int64_t)(n0 + a) * D_ + k0 + k] : 0.f;
        }
        for (int f = threadIdx.x; f < QROWS * PK; f += NT) {
            const int r = f / PK, k = f % PK;
            Qs[k][r] = (r0 + r < R) ? load_q(Q, q_dtype, (int64_t)(r0 + r) * D_ + k0 + k) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int k = 0; k < PK; ++k) {
            const float4 dv = *reinterpret_cast<const float4*>(&Ds[k][ta]);
            const float4 qv = *reinterpret_cast<const float4*>(&Qs[k][tr]);
            const float d[4] = {dv.x, dv.y, dv.z, dv.w};
            const float q[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(q[i], d[j], acc[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + tr + i;
        if (r < R) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (n0 + ta + j < N) P[((int64_t)(r / H) * N + n0 + ta + j) * H + r % H] = scale * acc[i][j];
        }
    }
}

// ---- out[r][:] (+)= sum_{n in slice} (sum_pieces A[b][piece][h][n]) * D[n][:] ---------------
// CTA = 16 rows x one atom slice; thread = (channel, group of rows).
constexpr int OR = 16;    // rows per CTA
constexpr int OA = 64;    // atoms per staged block
template <int D_>
__global__ void __launch_bounds__(NT)
ad_kernel(const float* __restrict__ D, int N, const float* __restrict__ A, int R, int H, int pieces, int atoms_per_slice,
          int use_atomics, float* __restrict__ out) {
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
            float v = 0.f;
            if (r0 + r < R && n0 + a < ne) {                // row (b, h): the stream's pieces in order
                const int64_t bb = (r0 + r) / H, hh = (r0 + r) % H;
                for (int pc = 0; pc < pieces; ++pc) v += A[((bb * pieces + pc) * H + hh) * N + n0 + a];
            }
            As[r][a] = v;
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
// U = max |coef|; no table entry can exceed S * U in magnitude, and the scale is the power
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
                for_each_code(idx, coef, coef_dtype, ((int64_t)b * T + t) * s, s, N, vec,
                              [&](int, float cf) { umax = fmaxf(umax, fabsf(cf)); if (cf != cf) umax = INFINITY; });
            }
            umax = block_max(umax, red);
            float scale[HGP], inv_scale[HGP];
            bool fixed_point = umax < INFINITY;
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
// maximum subtracted first.  Rows are a few tens of KB and were just written: they come
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
    for (int64_t t = threadIdx.x; t < T; t += NT) {
        const float e = __expf(row[t] - mx);
        row[t] = e;
        sum += e;
    }
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
    for (int64_t t = threadIdx.x; t < T; t += NT) row[t] *= inv;
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

size_t attn_scratch_bytes(int B, int H, int N, int64_t T) {
    return (size_t)B * value_pieces(B, T) * H * N * sizeof(float);
}

int launch_key_scores(const AttnArgs& a, float* P) {
    if (a.B == 0 || a.T == 0 || a.H == 0) return CSR_OK;
    const int hg = head_group(a.N, a.H);
    if (hg < 1) return fail(CSR_ERR_UNSUPPORTED, "N = %d: one head's N fp32 values do not fit in shared memory", a.N);
    const int R = a.B * a.H;
    const dim3 pgrid((a.N + PA - 1) / PA, (R + QROWS - 1) / QROWS);
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
        ad_kernel<128><<<ogrid, NT, 0, a.stream>>>(a.D, a.N, A, R, a.H, pieces, per_slice, slices > 1, a.out);
    else
        ad_kernel<64><<<ogrid, NT, 0, a.stream>>>(a.D, a.N, A, R, a.H, pieces, per_slice, slices > 1, a.out);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "value_mix launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace csr
