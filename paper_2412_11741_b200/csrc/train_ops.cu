// One training step of the offline dictionary ("NeuralDict", Algorithm 1, procedure
// TrainNeurDict; the MSE loss, the diversity loss L_div = ||I - W^T W||_F^2 / N^2, the complete
// loss L = L_MSE + beta * L_div and ReNorm).  The sparse codes of the batch are computed by
// the matching-pursuit encoder before these kernels run and are held fixed while the loss
// is differentiated (the alternating scheme of dictionary learning), so with
// e_x = x - W r(x):
//
//   dL_MSE / d d_n = -2 * sum over (x, g) with i_g(x) = n of  c_g(x) * e_x
//   dL_div / d d_n = (4 / N^2) * sum_j (G[n][j] - delta_nj) * d_j,      G = D D^T
//
//   mse_grad_kernel   one warp per row: restores x^ from the codes, forms e = x - x^, adds
//                     ||e||^2 to the loss (fp64 atomic) and scatters -2 c_g e into the
//                     gradient rows of the s selected atoms (fp32 atomic adds).
//   div_grad_kernel   one CTA per block of 64 atoms: sweeps all atoms in blocks of 64,
//                     forms the 64 x 64 block of G - I in shared memory (never in global
//                     memory), adds its squares to L_div and multiplies it into the
//                     gradient block held in registers (both products register-tiled).
//                     No atomics except the loss.
//   update_kernel     one warp per atom: d_n <- ReNorm(d_n - lr * (g_mse + beta * g_div)).
#include "common.cuh"

namespace csr {
namespace {

__device__ __forceinline__ float load_x(const void* X, int x_dtype, int64_t off) { return load_elem(X, x_dtype, off); }

template <int D_>
__global__ void __launch_bounds__(256)
mse_grad_kernel(const float* __restrict__ D, int N, const void* __restrict__ X, int x_dtype, int64_t M, int s,
                const uint16_t* __restrict__ idx, const float* __restrict__ coef, float* __restrict__ grad,
                double* __restrict__ losses) {
    constexpr int PER = D_ / 32;
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    double local = 0.0;
    for (int64_t m = warp0; m < M; m += nwarps) {
        float e[PER];
#pragma unroll
        for (int k = 0; k < PER; ++k) e[k] = load_x(X, x_dtype, m * D_ + lane * PER + k);
        for (int g = 0; g < s; ++g) {                     // e = x - sum_g c_g d_{i_g}, stored order
            int i = idx[m * s + g];
            i = i < N ? i : N - 1;
            const float c = coef[m * s + g];
            const float* dn = D + (int64_t)i * D_ + lane * PER;
#pragma unroll
            for (int k = 0; k < PER; ++k) e[k] = fmaf(-c, dn[k], e[k]);
        }
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < PER; ++k) ss = fmaf(e[k], e[k], ss);
        for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        local += (double)ss;
        for (int g = 0; g < s; ++g) {
            int i = idx[m * s + g];
            i = i < N ? i : N - 1;
            const float c2 = -2.f * coef[m * s + g];
            float* gn = grad + (int64_t)i * D_ + lane * PER;
#pragma unroll
            for (int k = 0; k < PER; ++k) atomicAdd(gn + k, c2 * e[k]);
        }
    }
    if (lane == 0 && local != 0.0) atomicAdd(&losses[0], local);
}

// CTA = 64 atoms (rows i) against all atoms in blocks of 64 (rows j); 256 threads.  Both
// products are register-tiled with 16-byte shared-memory operand loads: the block of
// G = Di Dj^T from transposed copies of the two tiles (thread = 4 x 4, channels ascending),
// the gradient block (G - I) Dj from G^T and the row-major tile (thread = 4 rows x 8 or 4
// channels, atoms ascending).  The next tile of atoms waits in registers meanwhile.
constexpr int GB = 64;
template <int D_>
struct DivSmem {
    float DiT[D_][GB + 4];     // [channel][atom i]
    float DjT[D_][GB + 4];     // [channel][atom j]; once the block of G is in registers its first
                               // GB rows hold (G - I) transposed, [atom j][atom i]
    float Dj[GB][D_ + 4];      // [atom j][channel]
};
// gridDim.y halves of the atoms j share a block of atoms i; each adds its part of the gradient
// (two addends on zeroed memory: the sum does not depend on which comes first).
template <int D_>
__global__ void __launch_bounds__(256, 2)
div_grad_kernel(const float* __restrict__ D, int N, float* __restrict__ grad_div, double* __restrict__ losses) {
    extern __shared__ __align__(16) unsigned char div_raw[];
    DivSmem<D_>& sm = *reinterpret_cast<DivSmem<D_>*>(div_raw);
    constexpr int V = GB * D_ / 4 / 256;                  // float4 of a tile per thread: 8 or 4
    constexpr int CPT = D_ / 16;                          // gradient channels per thread: 8 or 4
    const int tid = threadIdx.x;
    const int i0 = blockIdx.x * GB;
    float4 st[V];
    auto gload = [&](int r0) {
#pragma unroll
        for (int u = 0; u < V; ++u) {
            const int f = tid + u * 256, r = f % GB, c4 = f / GB;     // lanes along the atoms: see sstore
            st[u] = (r0 + r < N) ? *reinterpret_cast<const float4*>(D + (int64_t)(r0 + r) * D_ + 4 * c4)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    auto sstore = [&](float (*T)[GB + 4], bool row_major) {
#pragma unroll
        for (int u = 0; u < V; ++u) {
            // consecutive lanes hold consecutive atoms of the same four channels, so the four
            // transposed stores and the row-major one are free of bank conflicts
            const int f = tid + u * 256, r = f % GB, c4 = f / GB;
            T[4 * c4 + 0][r] = st[u].x;
            T[4 * c4 + 1][r] = st[u].y;
            T[4 * c4 + 2][r] = st[u].z;
            T[4 * c4 + 3][r] = st[u].w;
            if (row_major) *reinterpret_cast<float4*>(&sm.Dj[r][4 * c4]) = st[u];
        }
    };
    gload(i0);
    sstore(sm.DiT, false);
    gload((int)((int64_t)((N + GB - 1) / GB) * blockIdx.y / gridDim.y) * GB);
    // G block: thread owns rows pr .. pr+3, columns pc .. pc+3; gradient block: rows pr .. pr+3,
    // channels tx*4 .. +3 (and 64 + tx*4 .. +3 when d = 128)
    const int tx = tid & 15, pr = (tid >> 4) * 4, pc = tx * 4;
    float acc[4][CPT];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < CPT; ++c) acc[a][c] = 0.f;
    double lsum = 0.0;
    float (*GsT)[GB + 4] = sm.DjT;
    const int jblocks = (N + GB - 1) / GB;
    const int jb0 = jblocks * blockIdx.y / gridDim.y, jb1 = jblocks * (blockIdx.y + 1) / gridDim.y;
    for (int j0 = jb0 * GB; j0 < jb1 * GB; j0 += GB) {
        __syncthreads();                                   // the previous tile has been used
        sstore(sm.DjT, true);
        __syncthreads();
        if (j0 + GB < jb1 * GB) gload(j0 + GB);
        float g[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) g[a][b] = 0.f;
#pragma unroll 8
        for (int k = 0; k < D_; ++k) {
            const float4 xv = *reinterpret_cast<const float4*>(&sm.DiT[k][pr]);
            const float4 yv = *reinterpret_cast<const float4*>(&sm.DjT[k][pc]);
            const float x[4] = {xv.x, xv.y, xv.z, xv.w};
            const float y[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) g[a][b] = fmaf(x[a], y[b], g[a][b]);
        }
        __syncthreads();                                   // every thread is done with DjT
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + pr + a, j = j0 + pc + b;
                float v = g[a][b] - (i == j ? 1.f : 0.f);
                if (i >= N || j >= N) v = 0.f;
                GsT[pc + b][pr + a] = v;
                lsum += (double)v * (double)v;
            }
        __syncthreads();
        // acc[row][c] += sum_j (G - I)[row][j] * Dj[j][c]
#pragma unroll 4
        for (int j = 0; j < GB; ++j) {
            const float4 wv = *reinterpret_cast<const float4*>(&GsT[j][pr]);
            const float w[4] = {wv.x, wv.y, wv.z, wv.w};
            float dch[CPT];
#pragma unroll
            for (int q = 0; q < CPT / 4; ++q) {
                const float4 dv = *reinterpret_cast<const float4*>(&sm.Dj[j][q * 64 + tx * 4]);
                dch[4 * q + 0] = dv.x;
                dch[4 * q + 1] = dv.y;
                dch[4 * q + 2] = dv.z;
                dch[4 * q + 3] = dv.w;
            }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < CPT; ++c) acc[a][c] = fmaf(w[a], dch[c], acc[a][c]);
        }
    }
    const float scale = 4.0f / ((float)N * (float)N);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        if (i0 + pr + a >= N) continue;
        float* dst = grad_div + (int64_t)(i0 + pr + a) * D_;
#pragma unroll
        for (int c = 0; c < CPT; ++c) atomicAdd(dst + (c >> 2) * 64 + tx * 4 + (c & 3), scale * acc[a][c]);
    }
    for (int o = 16; o; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
    if ((tid & 31) == 0) atomicAdd(&losses[1], lsum / ((double)N * (double)N));
}

template <int D_>
__global__ void update_kernel(float* __restrict__ D, int N, const float* __restrict__ grad_mse,
                              const float* __restrict__ grad_div, float lr, float beta) {
    constexpr int PER = D_ / 32;
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    float w[PER];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        const int64_t o = (int64_t)n * D_ + lane * PER + k;
        w[k] = D[o] - lr * fmaf(beta, grad_div[o], grad_mse[o]);
        ss = fmaf(w[k], w[k], ss);
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float inv = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;
#pragma unroll
    for (int k = 0; k < PER; ++k) D[(int64_t)n * D_ + lane * PER + k] = w[k] * inv;
}

template <int D_>
int run(const TrainArgs& a) {
    const size_t gbytes = (size_t)a.N * D_ * sizeof(float);
    cudaError_t e = cudaMemsetAsync(a.grad_mse, 0, gbytes, a.stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(a.losses, 0, 2 * sizeof(double), a.stream);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    if (a.M > 0) {
        int64_t blocks = (a.M + 7) / 8;
        const int64_t cap = (int64_t)sm_count() * 8;
        if (blocks > cap) blocks = cap;
        mse_grad_kernel<D_><<<(int)blocks, 256, 0, a.stream>>>(a.D, a.N, a.X, a.x_dtype, a.M, a.s, a.idx, a.coef,
                                                              a.grad_mse, a.losses);
    }
    const size_t smem = sizeof(DivSmem<D_>);
    e = cudaFuncSetAttribute(div_grad_kernel<D_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    e = cudaMemsetAsync(a.grad_div, 0, gbytes, a.stream);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    div_grad_kernel<D_><<<dim3((a.N + GB - 1) / GB, 2), 256, smem, a.stream>>>(a.D, a.N, a.grad_div, a.losses);
    update_kernel<D_><<<(a.N + 7) / 8, 256, 0, a.stream>>>(a.D, a.N, a.grad_mse, a.grad_div, a.lr, a.beta);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "dict_train launch: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace

int launch_dict_train(const TrainArgs& a) {
    if (a.d == 128) return run<128>(a);
    return run<64>(a);
}

}  // namespace csr
