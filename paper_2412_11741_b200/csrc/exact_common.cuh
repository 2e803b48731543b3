// Pieces shared by the two correctness-mode encoders (one CTA per row tile for all atoms;
// dictionary split across CTAs for few rows): tile constants, the top-2 bookkeeping, the
// fp32 sweep and the fp64 re-scoring.
#pragma once

#include "common.cuh"

namespace csr {
namespace exact {

constexpr int BM = 64;        // rows per CTA
constexpr int BN = 128;       // atoms per dictionary tile
constexpr int BK = 8;         // channels per staged chunk (small: two CTAs of the row-tile encoder fit one SM)
constexpr int NT = 256;       // threads per CTA
constexpr int AS_LD = BM + 4; // leading dimension of the transposed fp32 residual
constexpr int BS_LD = BN + 4;
// |fp32 dot - exact dot| <= d * 2^-24 * ||R|| * ||atom|| for d <= 128 sequential FMAs plus
// the rounding of R itself; two candidates can therefore swap when closer than twice that.
constexpr float kBandRel = 1.6e-5f;

__device__ __forceinline__ float load_x(const void* X, int x_dtype, int64_t off) { return load_elem(X, x_dtype, off); }

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

// The same bookkeeping without branches (NaN values count as ties and send the row to the
// fp64 re-scoring instead of being skipped).
__device__ __forceinline__ void top2_push_fast(Top2& t, float a, int n) {
    t.second = fmaxf(t.second, fminf(a, t.best));
    const bool p = a > t.best;
    t.best = fmaxf(a, t.best);
    t.idx = p ? n : t.idx;
}

// Products of the 64 rows whose fp32 values sit transposed in As with the atoms of dictionary
// tiles [bt0, bt1) (128 atoms each): fp32 register-tiled, each thread 4 rows x 8 atoms, k
// ascending.  Thread (tx, ty) = (tid & 15, tid >> 4) ends every tile with acc[i][j] = the
// product of row ty*4 + i with atom bt*128 + (j >> 2)*64 + tx*4 + (j & 3) and hands it to
// on_tile(bt, acc).  Bs is the double-buffered staging area of dictionary chunks (8 channels
// each; the next chunk waits in registers while the current one is used).  Ends with a
// __syncthreads.
template <int D_, typename TileFn>
__device__ __forceinline__ void sweep_tiles_fn(const float* __restrict__ D, int N, int bt0, int bt1,
                                               const float (*As)[AS_LD], float (*Bs)[BK][BS_LD], TileFn&& on_tile) {
    static_assert(BK == 8 && NT == 2 * BN, "two threads stage one atom's eight channels");
    constexpr int KCH = D_ / BK;                          // chunks per tile (even)
    const int tid = threadIdx.x;
    const int tx = tid & 15;   // atom group
    const int ty = tid >> 4;   // row group: rows ty*4 .. ty*4+3
    if (bt1 <= bt0) return;
    const int satom = tid >> 1, skq = (tid & 1) * 4;       // staged: channels skq .. skq+3 of atom satom
    float4 stage;
    auto gload = [&](const float* src, bool in_range) {
        stage = in_range ? *reinterpret_cast<const float4*>(src) : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    auto sstore = [&](float (*B)[BS_LD]) {
        B[skq + 0][satom] = stage.x;
        B[skq + 1][satom] = stage.y;
        B[skq + 2][satom] = stage.z;
        B[skq + 3][satom] = stage.w;
    };
    float acc[4][8];
    auto compute8 = [&](const float (*B)[BS_LD], const float (*A)[AS_LD]) {
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&A[k][ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&B[k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&B[k][64 + tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    };
    const float* src = D + ((int64_t)bt0 * BN + satom) * D_ + skq;
    bool in_range = bt0 * BN + satom < N;
    gload(src, in_range);
    sstore(Bs[0]);
    __syncthreads();
    for (int bt = bt0; bt < bt1; ++bt) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
        const bool last_tile = bt + 1 == bt1;
#pragma unroll 1
        for (int c = 0; c < KCH; c += 2) {
            // here: Bs[0] holds chunk c of the tile
            src += BK;
            gload(src, in_range);                         // chunk c + 1 (KCH is even)
            compute8(Bs[0], As + c * BK);
            sstore(Bs[1]);
            __syncthreads();
            const bool more = !(last_tile && c + 2 == KCH);
            if (more) {                                   // chunk c + 2, or the next tile's first
                if (c + 2 == KCH) {
                    src += (int64_t)BN * D_ - (KCH - 1) * BK;
                    in_range = (bt + 1) * BN + satom < N;
                } else {
                    src += BK;
                }
                gload(src, in_range);
            }
            compute8(Bs[1], As + (c + 1) * BK);
            if (more) sstore(Bs[0]);
            __syncthreads();
        }
        on_tile(bt, acc);
    }
}

// The sweep of Eq. 2-3: every thread keeps the two largest |correlations| of its rows.
template <int D_>
__device__ __forceinline__ void sweep_tiles(const float* __restrict__ D, int N, int bt0, int bt1,
                                            const float (*As)[AS_LD], float (*Bs)[BK][BS_LD], Top2 (&top)[4]) {
    const int tx = threadIdx.x & 15;
    sweep_tiles_fn<D_>(D, N, bt0, bt1, As, Bs, [&](int bt, const float (&acc)[4][8]) {
        const int nb = bt * BN + tx * 4;
        if ((bt + 1) * BN <= N) {                         // a whole tile: no atom to leave out
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int i = 0; i < 4; ++i) top2_push_fast(top[i], fabsf(acc[i][j]), nb + (j >> 2) * 64 + (j & 3));
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int n = nb + (j >> 2) * 64 + (j & 3);
                if (n < N) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) top2_push_fast(top[i], fabsf(acc[i][j]), n);
                }
            }
        }
    });
}

// Re-scoring of a row whose two largest fp32 |correlations| are too close to call, by the
// whole CTA (all threads must call; blockDim.x = NT).  The true arg-max can only be an atom
// whose fp32 value lies within the rounding band of the fp32 maximum, so a cheap fp32 pass
// over all atoms (one warp per atom, lanes over channels, coalesced) first collects those
// candidates; each candidate's correlation is then taken in fp64 (channels in ascending
// order, one thread per candidate) and the largest wins, the lowest atom among equal
// values.  Should the candidates overflow the list (many copies of one atom), every atom is
// scored in fp64 instead.  Returns the pick to all threads.
constexpr int RESCORE_CAP = 64;

struct RescoreSmem {
    double val[RESCORE_CAP];
    int cand[RESCORE_CAP];
    int count;
    int pick;
    double wbest[NT / 32];
    int widx[NT / 32];
};

template <int PER>
struct LaneVec;
template <>
struct LaneVec<4> {
    using T = float4;
};
template <>
struct LaneVec<2> {
    using T = float2;
};
__device__ __forceinline__ float lane_dot(const float (&r)[4], const float4& v) {
    return fmaf(r[3], v.w, fmaf(r[2], v.z, fmaf(r[1], v.y, r[0] * v.x)));
}
__device__ __forceinline__ float lane_dot(const float (&r)[2], const float2& v) { return fmaf(r[1], v.y, r[0] * v.x); }

template <int D_>
__device__ __forceinline__ double dot_fp64(const double* Rr, const float* __restrict__ dn) {
    double c = 0.0;
#pragma unroll 4
    for (int q = 0; q < D_ / 4; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(dn + 4 * q);
        c = fma(Rr[4 * q + 0], (double)v.x, c);
        c = fma(Rr[4 * q + 1], (double)v.y, c);
        c = fma(Rr[4 * q + 2], (double)v.z, c);
        c = fma(Rr[4 * q + 3], (double)v.w, c);
    }
    return c;
}

template <int D_>
__device__ __forceinline__ int rescore_cta(const float* __restrict__ D, int N, const double* Rr, float best, float band,
                                           RescoreSmem& rs) {
    constexpr int PER = D_ / 32;                          // channels per lane in the fp32 pass
    constexpr int UNR = 8;                                // atoms in flight per warp
    using V = typename LaneVec<PER>::T;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) rs.count = 0;
    __syncthreads();
    float rf[PER];
#pragma unroll
    for (int k = 0; k < PER; ++k) rf[k] = (float)Rr[lane * PER + k];
    const float thresh = best - 1.5f * band;
    for (int n0 = warp * UNR; n0 < N; n0 += (NT / 32) * UNR) {
        V v[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int n = min(n0 + u, N - 1);
            v[u] = *reinterpret_cast<const V*>(D + (int64_t)n * D_ + lane * PER);
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            float c = lane_dot(rf, v[u]);
            for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
            if (lane == 0 && n0 + u < N && fabsf(c) >= thresh) {
                const int slot = atomicAdd(&rs.count, 1);
                if (slot < RESCORE_CAP) rs.cand[slot] = n0 + u;
            }
        }
    }
    __syncthreads();
    const int count = rs.count;
    if (count <= RESCORE_CAP) {
        if (threadIdx.x < count) rs.val[threadIdx.x] = fabs(dot_fp64<D_>(Rr, D + (int64_t)rs.cand[threadIdx.x] * D_));
        __syncthreads();
        if (threadIdx.x == 0) {
            double bb = -1.0;
            int bn = 0;
            for (int j = 0; j < count; ++j)
                if (rs.val[j] > bb || (rs.val[j] == bb && rs.cand[j] < bn)) {
                    bb = rs.val[j];
                    bn = rs.cand[j];
                }
            rs.pick = bn;
        }
    } else {
        double bb = -1.0;
        int bn = 0;
        for (int n = threadIdx.x; n < N; n += NT) {
            const double a = fabs(dot_fp64<D_>(Rr, D + (int64_t)n * D_));
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
        if (lane == 0) {
            rs.wbest[warp] = bb;
            rs.widx[warp] = bn;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int j = 0; j < NT / 32; ++j)
                if (rs.wbest[j] > bb || (rs.wbest[j] == bb && rs.widx[j] < bn)) {
                    bb = rs.wbest[j];
                    bn = rs.widx[j];
                }
            rs.pick = bn;
        }
    }
    __syncthreads();
    return rs.pick;
}

}  // namespace exact
}  // namespace csr
