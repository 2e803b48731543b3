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
//   diversity term    both products (D D^T - I, and that times D) run on the tensor cores with
//                     split bf16 operands: gram_ops.cu.
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
    e = cudaMemsetAsync(a.grad_div, 0, gbytes, a.stream);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    if (int rc = launch_div_grad(a.D, a.N, D_, a.grad_div, a.losses, a.div_scratch, a.status, a.stream)) return rc;
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
