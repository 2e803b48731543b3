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

// Sweep of dictionary tiles [bt0, bt1) (128 atoms each) for the 64 rows whose fp32 residual
// sits transposed in As (Eq. 2-3): fp32 register-tiled products, each thread 4 rows x 8
// atoms, k ascending; every thread keeps the two largest |correlations| of its rows.
// Bs is the double-buffered staging area of dictionary chunks.  Ends with a __syncthreads.
template <int D_>
__device__ __forceinline__ void sweep_tiles(const float* __restrict__ D, int N, int bt0, int bt1,
                                            const float (*As)[AS_LD], float (*Bs)[BK][BS_LD], Top2 (&top)[4]) {
    constexpr int KCH = D_ / BK;
    const int tid = threadIdx.x;
    const int tx = tid & 15;   // atom group
    const int ty = tid >> 4;   // row group: rows ty*4 .. ty*4+3
    const int total_chunks = (bt1 - bt0) * KCH;
    if (total_chunks <= 0) return;
    constexpr int KQ = BK / 4;                            // float4 per atom per chunk
    constexpr int FPT = BN * KQ / NT;                     // float4 staged per thread
    float4 stage[FPT];
    auto gload = [&](int chunk) {
        const int bt = bt0 + chunk / KCH, kc = chunk % KCH;
#pragma unroll
        for (int i = 0; i < FPT; ++i) {
            const int f = tid + i * NT;
            const int atom = f / KQ, kq = f % KQ;
            const int n = bt * BN + atom;
            stage[i] = (n < N) ? *reinterpret_cast<const float4*>(D + (int64_t)n * D_ + kc * BK + kq * 4)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    auto sstore = [&](int buf) {
#pragma unroll
        for (int i = 0; i < FPT; ++i) {
            const int f = tid + i * NT;
            const int atom = f / KQ, kq = f % KQ;
            Bs[buf][kq * 4 + 0][atom] = stage[i].x;
            Bs[buf][kq * 4 + 1][atom] = stage[i].y;
            Bs[buf][kq * 4 + 2][atom] = stage[i].z;
            Bs[buf][kq * 4 + 3][atom] = stage[i].w;
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
            const float4 a4 = *reinterpret_cast<const float4*>(&As[kc * BK + k][ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][k][64 + tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (kc == KCH - 1) {
            const int nb = (bt0 + chunk / KCH) * BN;
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
