// Shared declarations of the libcsr translation units (host-side plumbing only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "csr.h"

namespace csr {

// Records the calling thread's last error message and returns `code`.
int fail(int code, const char* fmt, ...);

// Device status word written by kernels whose bounded waits expire.
constexpr uint32_t kStatusTimeout = 1u;
// Raised only by a library built with CSR_DEBUG_CHECKS (python -m paper_2412_11741_b200.build
// --debug): an index about to be used for a gather was out of range and has been clamped.
constexpr uint32_t kStatusBounds = 2u;
// A kernel found its dynamic shared memory not 1024-byte aligned and did nothing.
constexpr uint32_t kStatusLayout = 4u;

// Process-wide switches set through csr_set_option (plain loads on the call path).
struct Options {
    int fast_group;                     // 0 = chosen by the library; 1, 2, 4, 8 = atoms per arg-max group
    int fast_split;                     // 0 = chosen by the library; 1 = one CTA per pair of row tiles over the whole
                                        // dictionary; 2 = few rows split the dictionary without clusters
    int exact_split;                    // 0 = chosen by the library; 1 = the row-tile encoder also with few rows
    int exact_engine;                   // 0 = chosen by the library; 1 = plain-ALU encoders only; 2 = the tensor-core
                                        // encoder also with few rows
    unsigned long long wait_limit_ns;   // bound of every device-side wait
};
Options options();

struct EncodeArgs {
    const float* D;
    const void* X;
    int x_dtype;
    int coef_dtype;
    int64_t M;
    int d, N, s;
    uint16_t* out_idx;
    void* out_coef;
    int64_t ldx;       // elements between consecutive rows of X (>= d)
    int64_t ld_code;   // elements between consecutive rows of out_idx and of out_coef (>= s)
    cudaStream_t stream;
};

// fp32-operand matching pursuit with fp64 re-scoring of unresolved picks.
int launch_encode_exact(const EncodeArgs& a);

// The same encoder for few rows (the vectors one decoding step adds): the dictionary is
// split across CTAs, two launches per iteration; identical codes.  `scratch` must hold
// encode_exact_split_scratch_bytes() bytes, 256-byte aligned.
bool encode_exact_split_applies(int64_t M, int N);
size_t encode_exact_split_scratch_bytes(int64_t M, int d, int N);
int launch_encode_exact_split(const EncodeArgs& a, void* scratch);

// The same picks with the sweep on the tensor cores (three bf16 products per correlation bound
// it to a band; rows inside the band are re-scored in fp64).  `scratch`:
// encode_exact_tc_scratch_bytes() bytes, 1024-byte aligned; `status` receives kStatusTimeout;
// `diag` is a device word that a build with CSR_DEBUG_CHECKS raises to the largest error of a
// tensor-core correlation seen, relative to ||R|| (float bits).
size_t encode_exact_tc_scratch_bytes(int64_t M, int d, int N);
int launch_encode_exact_tc(const EncodeArgs& a, void* scratch, uint32_t* status, uint32_t* diag);

// tcgen05 bf16 matching pursuit.  `workspace` holds the bf16 copy of D (N*d*2 bytes,
// 1024-byte aligned); `status` is a device word that receives kStatusTimeout.
int launch_encode_fast(const EncodeArgs& a, void* workspace, uint32_t* status);
size_t encode_fast_workspace_bytes(int d, int N);
// fp32 -> fp16 copy of D (round to nearest even), same [N][d] layout: the de-sparse kernel's gather source.
int launch_dict_to_f16(const float* D, int N, int d, void* dst, cudaStream_t stream);
// The two halves of launch_encode_fast: build the bf16 copy once, encode against it many times.
int prepare_fast_dictionary(const float* D, int N, int d, void* workspace, cudaStream_t stream);
// With few rows the dictionary is split across the CTAs of thread-block clusters (one launch,
// no scratch).  Where clusters cannot be launched, `split_scratch`
// (encode_fast_split_scratch_bytes(), 256-byte aligned) lets it be split across CTAs with one
// sweep launch and one pick launch per iteration; NULL = one CTA per pair of row tiles over
// the whole dictionary.  Identical codes in all three.
int launch_encode_fast_prepared(const EncodeArgs& a, const void* dict_bf16, uint32_t* status, void* split_scratch);
bool encode_fast_split_applies(int64_t M, int N);
size_t encode_fast_split_scratch_bytes(int64_t M, int d, int N);

struct ReconstructArgs {
    const float* D;
    const void* dict_f16;    // fp16 copy of D ([N][d]) to gather from instead, or NULL
    const uint16_t* idx;
    const void* coef;
    int coef_dtype;
    int out_dtype;
    int64_t M;
    int d, N, s;
    void* X_hat;
    int64_t ld_code;   // elements between consecutive rows of idx and of coef (>= s)
    int64_t ld_xhat;   // elements between consecutive rows of X_hat (>= d)
    uint32_t* status;  // debug builds: the word that records a clamped index; else NULL
    cudaStream_t stream;
};
int launch_reconstruct(const ReconstructArgs& a);

// D_new[i][:] = X[rows[i]][:] / ||X[rows[i]][:]||_2 for i < n_rows (zero rows stay zero).
int launch_dict_append(float* D_new, int d, const void* X, int x_dtype, int64_t M, int64_t ldx, const int64_t* rows,
                       int n_rows, cudaStream_t stream);

// *max_bits (zeroed by the caller) receives the bit pattern of max_n | ||D[n]||_2 - 1 |.
int launch_dict_norm_deviation(const float* D, int N, int d, uint32_t* max_bits, cudaStream_t stream);

// Attention straight from the codes.  key_scores: Q = queries [B][H][d] (q_dtype), out = scores
// [B][H][T].  value_mix: Q = attention weights [B][H][T] fp32, out = [B][H][d] fp32.
struct AttnArgs {
    const float* D;
    int N, d;
    const void* Q;
    int q_dtype;
    int B, H;
    const uint16_t* idx;   // [B][T][s]
    const void* coef;      // [B][T][s]
    int coef_dtype;
    int64_t T;
    int s;
    float scale;
    float* out;
    cudaStream_t stream;
};
// `scratch` holds attn_scratch_bytes() bytes: the fp32 array of per-atom partial products
// ([B][N][H] for the scores, [B][pieces][H][N] for the value mix).
size_t attn_scratch_bytes(int B, int H, int N, int64_t T);
int launch_key_scores(const AttnArgs& a, float* scratch);
int launch_value_mix(const AttnArgs& a, float* scratch);
int launch_softmax_rows(float* S, int64_t rows, int64_t T, cudaStream_t stream);   // in place, fp32

// Gradient step of the dictionary on one batch whose codes (idx, fp32 coef, dense [M][s])
// are given; losses[0] = L_MSE, losses[1] = L_div of the dictionary before the update.
struct TrainArgs {
    float* D;
    int N, d;
    const void* X;
    int x_dtype;
    int64_t M;
    int s;
    const uint16_t* idx;
    const float* coef;
    float* grad_mse;   // [N][d] scratch
    float* grad_div;   // [N][d] scratch
    double* losses;    // [2]
    float lr, beta;
    void* div_scratch;  // div_grad_scratch_bytes(N, d) bytes for the diversity gradient's operands
    uint32_t* status;   // device word raised by a bounded wait that expires
    cudaStream_t stream;
};
int launch_dict_train(const TrainArgs& a);

// Diversity loss and gradient on the tensor cores: losses[1] += ||D D^T - I||_F^2 / N^2 and
// grad_div (zeroed by the caller) += (4 / N^2) (D D^T - I) D.
size_t div_grad_scratch_bytes(int N, int d);
int launch_div_grad(const float* D, int N, int d, float* grad_div, double* losses, void* scratch, uint32_t* status,
                    cudaStream_t stream);

// Element `off` of an array of dtype F32, BF16 or F16, widened exactly to fp32.
__device__ __forceinline__ float load_elem(const void* p, int dtype, int64_t off) {
    if (dtype == CSR_DTYPE_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[off]);
    if (dtype == CSR_DTYPE_F16) return __half2float(reinterpret_cast<const __half*>(p)[off]);
    return reinterpret_cast<const float*>(p)[off];
}
inline bool valid_x_dtype(int t) { return t == CSR_DTYPE_F32 || t == CSR_DTYPE_BF16 || t == CSR_DTYPE_F16; }
inline size_t dtype_size(int t) { return t == CSR_DTYPE_F32 ? 4 : 2; }

// fp32 coefficients -> stored fp16 form (round to nearest even), n values.
int launch_pack_coef(const float* coef32, int64_t n, void* coef16, cudaStream_t stream);

int sm_count();

}  // namespace csr
