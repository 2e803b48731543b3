/*
 * libcsr — sparse codec of CSR ("Cache Sparse Representation") for NVIDIA B200 (sm_100a).
 *
 * The codec turns every dense key/value head vector x (d channels) into s
 * (atom index, coefficient) pairs over a fixed dictionary D of N unit-norm atoms by
 * greedy matching pursuit, and turns such pairs back into dense vectors.
 *
 * Conventions shared by every entry point
 *   - All functions return an int status: CSR_OK (0) or a negative CSR_ERR_* code.
 *     csr_last_error_string() returns the message of the calling thread's last failure.
 *     No exception crosses this boundary and no argument error is undefined behaviour.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the
 *     caller.  The library neither frees nor keeps caller pointers after a call's work
 *     has finished on its stream.
 *   - Calls are asynchronous with respect to the host: work is enqueued on the given
 *     CUDA stream (the 8-argument forms use the legacy default stream, 0) and the
 *     function returns without synchronising, except the host entry points,
 *     csr_dict_check_norms and csr_device_status, which synchronise.  A device-pointer
 *     call whose scratch does not have to grow (a repeat of an earlier call's shapes, a
 *     call with its own workspace or dictionary handle, or csr_encode_static) only
 *     launches kernels and may be captured into a CUDA graph and replayed.  A call that
 *     would have to grow the library's scratch while its stream is being captured is
 *     refused with CSR_ERR_WORKSPACE (growing allocates); an outgrown scratch block is
 *     kept until csr_release_workspace, so graphs captured earlier stay valid.
 *   - Library-owned scratch.  Unless a call brings its own memory, it works in ONE
 *     library-owned buffer per device: the fast mode's bf16 copy of D (csr_encode,
 *     csr_encode_ex without `workspace` or `dict`), the few-rows paths' per-row maxima,
 *     the per-atom tables of csr_key_scores / csr_value_mix / csr_decode_attention, the
 *     codes and gradients of csr_dict_train_step, and one status word.  Calls that use it
 *     must therefore be ORDERED on the device (same stream, or events between streams):
 *     two of them running side by side on different streams overwrite each other's
 *     scratch and return wrong results without any error.  Concurrent callers give each
 *     encode its own `workspace` or `dict` and, for the wait status, its own
 *     `dev_status`; such a call touches nothing the library owns.
 *   - Layout.  D is [N][d] row-major fp32: one atom per row, the d channels contiguous
 *     (the paper's d x N matrix of "Sparse representation", stored column by column).
 *     Atoms are assumed unit l2-norm; the encoders do not check this and apply the
 *     formulas as written if they are not (csr_dict_check_norms checks a dictionary once).
 *     The exact mode's promise of fp64-identical picks assumes atom norms of at most
 *     1 + 1e-3: its rounding band scales with the residual's norm only.
 *     X and X_hat are [M][d] row-major.  Codes are
 *     idx [M][s] and coef [M][s] row-major, entry g of a row being iteration g of the
 *     pursuit.
 *   - Limits: d in {64, 128}; 1 <= N <= 65536 (indices are stored as uint16); 1 <= s <= 64;
 *     M >= 0 (M == 0 succeeds and does nothing).  Data pointers must be 16-byte aligned.
 *   - NaN or Inf in X or D: results are unspecified; the call neither crashes nor hangs.
 *   - Device-side waits are bounded.  If one expires the kernel stops early, the outputs
 *     are unspecified and csr_device_status() reports CSR_ERR_TIMEOUT.
 */
#ifndef CSR_H_
#define CSR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CSR_VERSION 120

#define CSR_OK 0
#define CSR_ERR_INVALID_ARG (-1)
#define CSR_ERR_UNSUPPORTED (-2)
#define CSR_ERR_ALIGNMENT (-3)
#define CSR_ERR_CUDA (-4)
#define CSR_ERR_TIMEOUT (-5)
#define CSR_ERR_WORKSPACE (-6)
#define CSR_ERR_BOUNDS (-7)

/* element types of X and X_hat (any of the three) and of coef (F32 or F16) */
#define CSR_DTYPE_F32 0
#define CSR_DTYPE_BF16 1
#define CSR_DTYPE_F16 2

/*
 * Arithmetic mode of the encoder.
 *   CSR_MODE_FP32_EXACT  selects the same atoms as an fp64 evaluation of the pursuit except
 *                        at exact-to-rounding ties; the coefficient and the residual
 *                        update are fp64.  Every correlation of a sweep is computed to
 *                        within a known band, and whenever the largest |correlations| of a
 *                        row are closer than that band the candidates are re-scored in
 *                        fp64.  Three encoders do this, with identical codes:
 *                        (a) sweep on the tcgen05 tensor cores, residual and atoms each
 *                        split into a bf16 high and low part, three bf16 products per
 *                        correlation accumulated in fp32 (band 2^-12 * ||R||): the default
 *                        for 2048 rows or more where the library-owned scratch is in use (no
 *                        caller workspace;
 *                        about 4 * N * d + 2048 * d * min(ceil(M / 256), SMs) bytes of it);
 *                        (b) fp32 operands and fp32 accumulation on the plain ALUs (band
 *                        1.6e-5 * ||R||), one CTA per 64 rows, no scratch: taken when a
 *                        caller workspace is given;
 *                        (c) with few rows (the vectors one decoding step adds: fewer than
 *                        2048) the plain-ALU sweep with the
 *                        dictionary split across the SMs instead of the rows, two launches
 *                        per iteration; library-owned scratch, not taken when a caller
 *                        workspace is given.
 *   CSR_MODE_BF16_FAST   correlations on the tcgen05 tensor cores with bf16 operands
 *                        (residual and atoms rounded to bf16) and fp32 accumulation.
 *                        Near-tied picks may differ from an fp64 evaluation; the mean
 *                        reconstruction error does not, down to a floor of about
 *                        2^-8 * ||x|| (the residual is carried in bf16); use the exact
 *                        mode for errors below 1e-2 * ||x||.  With few rows (at most half
 *                        as many pairs of 128-row tiles as SMs) the dictionary is split
 *                        across the CTAs of thread-block clusters that share the rows,
 *                        still one launch, with identical codes; where clusters cannot be
 *                        launched and the library-owned scratch is in use, across CTAs
 *                        with one sweep and one pick launch per iteration.
 *                        (csr_set_option can force each of these paths.)
 */
#define CSR_MODE_FP32_EXACT 0
#define CSR_MODE_BF16_FAST 1

typedef struct csr_encode_params {
    uint32_t struct_size;   /* sizeof(csr_encode_params_t), for versioning */
    int32_t mode;           /* CSR_MODE_* */
    const void* D;          /* [N][d] fp32 */
    const void* X;          /* [M][d], x_dtype (F32, BF16 or F16; the fast mode rounds to bf16) */
    int32_t x_dtype;
    int32_t coef_dtype;     /* F16 (the paper's stored form) or F32 */
    int64_t M;
    int32_t d, N, s;
    int32_t reserved0;
    uint16_t* out_idx;      /* [M][s] */
    void* out_coef;         /* [M][s], coef_dtype */
    void* stream;           /* cudaStream_t; NULL = legacy default stream */
    void* workspace;        /* scratch of at least csr_encode_workspace_bytes(); NULL = the
                               library keeps one grow-only allocation per device */
    size_t workspace_bytes;
    int64_t ldx;            /* elements between consecutive rows of X; 0 = d (dense) */
    int64_t ld_code;        /* elements between consecutive rows of out_idx and of out_coef;
                               0 = s (dense) */
    const void* dict;       /* csr_dict_t* from csr_dict_create, or NULL (see there) */
    uint32_t* dev_status;   /* fast mode: optional device word (4-byte aligned) that the call zeroes
                               on its stream and a kernel sets non-zero if one of its bounded
                               waits expired; NULL = the library's word, read by
                               csr_device_status.  Ignored by the host entry points. */
} csr_encode_params_t;

typedef struct csr_reconstruct_params {
    uint32_t struct_size;
    int32_t reserved0;
    const void* D;          /* [N][d] fp32 */
    const uint16_t* idx;    /* [M][s] */
    const void* coef;       /* [M][s], coef_dtype */
    int32_t coef_dtype;     /* F16 or F32 */
    int32_t out_dtype;      /* BF16, F16 or F32 */
    int64_t M;
    int32_t d, N, s;
    int32_t reserved1;
    void* X_hat;            /* [M][d], out_dtype */
    void* stream;
    int64_t ld_code;        /* elements between consecutive rows of idx and of coef; 0 = s */
    int64_t ld_xhat;        /* elements between consecutive rows of X_hat; 0 = d */
    const void* dict;       /* csr_dict_t* from csr_dict_create, or NULL: gather the atoms from the
                               handle's fp16 copy of D instead of the fp32 D (see csr_reconstruct) */
} csr_reconstruct_params_t;

/*
 * Matching-pursuit encode ("Sparse representation", Eq. 2-4; "KV Decomposition and
 * Sparse Storage").  For every row x of X: R_0 = x; for g = 0 .. s-1: correlate R_g
 * with all N atoms, i_g = argmax_n |R_g . d_n| (lowest n among equal values),
 * c_g = R_g . d_{i_g} (signed), R_{g+1} = R_g - c_g d_{i_g}.  Atoms are never masked:
 * an atom may be selected more than once.  A zero residual yields (0, 0).
 * Writes out_idx[m][g] = i_g and out_coef[m][g] = c_g in the stored form of "Analysis
 * for CSR": 16-bit index, fp16 coefficient (round to nearest even), 4*s bytes per row.
 *
 * 8-argument form: X is bf16, out_coef is fp16, mode is CSR_MODE_BF16_FAST, stream 0,
 * library-owned workspace.
 */
int csr_encode(const void* D, const void* X, int64_t M, int d, int N, int s, uint16_t* out_idx,
               void* out_coef);
int csr_encode_ex(const csr_encode_params_t* p);

/* Scratch bytes csr_encode_ex needs for the given mode and sizes (0 if none);
 * negative CSR_ERR_* on invalid arguments. */
int64_t csr_encode_workspace_bytes(int mode, int d, int N);

/*
 * De-sparse ("De-Sparse to restore", Eq. 12): X_hat[m,:] = sum_g coef[m][g] * D[idx[m][g]][:],
 * accumulated in fp32 in the order g = 0 .. s-1; repeated indices accumulate.  Every idx
 * must be < N (larger values are clamped to N-1 rather than read out of bounds).
 *
 * With params.dict (a handle of the same D, N, d) the atoms are read from the handle's fp16
 * copy of D, which halves the bytes gathered per row (what bounds this kernel from about
 * s = 4 up) and, with fp16 coefficients, needs no conversion before the multiply.  The result
 * is then Eq. 12 over the atoms rounded to fp16 (11 significant bits): it differs from the
 * fp32-atom result by at most sum_g |coef_g| * (2^-11 * |D[idx_g][k]| + 2^-25) per channel k,
 * well below the rounding of a bf16 or fp16 X_hat.
 *
 * 8-argument form: coef is fp16, X_hat is bf16, stream 0.
 */
int csr_reconstruct(const void* D, const uint16_t* idx, const void* coef, int64_t M, int d, int N,
                    int s, void* X_hat);
int csr_reconstruct_ex(const csr_reconstruct_params_t* p);

/*
 * One decoding step's attention over a cache kept as codes ("De-Sparse to restore" followed by
 * the attention it feeds, with nothing restored): for every stream b and query head h
 *     weights[b][h][:] = softmax_t( scale * Q[b][h] . X~_K[b][t] )          (csr_key_scores + softmax)
 *     out[b][h][:]     = sum_t weights[b][h][t] * X~_V[b][t]                 (csr_value_mix)
 * Keys and values have their own dictionaries (Dk [Nk][d], Dv [Nv][d]) and code arrays
 * ([B][T][sk] and [B][T][sv], one coef_dtype).  `weights` is a caller buffer [B][H][T] fp32 that
 * receives the attention weights; out is [B][H][d] fp32.  T >= 1.  Limits, alignment and
 * reproducibility as for csr_key_scores / csr_value_mix; no causal mask is applied (a
 * decoding step attends to the whole cache).
 */
int csr_decode_attention(const void* Dk, int Nk, const void* Dv, int Nv, int d, const void* Q, int q_dtype, int B, int H,
                         const uint16_t* k_idx, const void* k_coef, int sk, const uint16_t* v_idx, const void* v_coef,
                         int sv, int coef_dtype, int64_t T, float scale, float* weights, float* out, void* stream);

/*
 * Packs fp32 coefficients into the stored form of "Analysis for CSR" (fp16, round to
 * nearest even): for codes that were produced with coef_dtype F32, e.g. by the exact mode
 * for verification, and are now to be kept.  The indices are stored as produced.  n values,
 * dense; both device pointers 16-byte aligned; asynchronous on `stream`.  A pure streaming
 * kernel: 4 bytes read and 2 written per value.
 */
int csr_pack_coefficients(const float* coef32, int64_t n, void* coef16, void* stream);

/*
 * Prepared dictionary.  A handle holds two 16-bit copies of D: bf16 for the fast encoder and
 * fp16 for the de-sparse kernel (params.dict of csr_reconstruct_ex).  The fast mode works on a
 * bf16 copy of D which the encode calls
 * otherwise rebuild in scratch memory on every call (one extra launch of a few
 * microseconds: measured 83 -> 80 us on a 4160-row call, nothing on large ones).  A
 * dictionary is fixed for a layer's lifetime, so the copy can be made once and the encode
 * calls then need no scratch for it: csr_dict_create allocates it (cudaMalloc, N rounded up to 8
 * atoms of d bf16 values), converts D on `stream` and returns a handle; an encode call whose
 * params.dict is that handle uses the copy as it was at creation time (a snapshot: later
 * changes to D do not reach it) and must pass the same D pointer, N and d.  The fp32 D is
 * still read by the exact mode and by every other entry point.  csr_dict_destroy frees the
 * copy after synchronising the device.  A handle belongs to the device that was current
 * when it was created.
 */
typedef struct csr_dict csr_dict_t;
int csr_dict_create(const void* D, int N, int d, void* stream, csr_dict_t** out);
int csr_dict_destroy(csr_dict_t* dict);

/*
 * Row strides ("KV Decomposition and Sparse Storage": a head vector of d_h channels may be
 * split into s_n chunks of d = d_h / s_n channels, each with its own dictionary).  With
 * ldx = d_h and X pointing at channel c*d of row 0, csr_encode_ex encodes chunk c of every
 * head vector in place; with ld_code = s_n*s and out_idx / out_coef pointing at entry c*s,
 * the s codes of chunk c land in columns c*s .. c*s+s-1 of [M][s_n*s] code arrays; the
 * reconstruct strides are the mirror image.  Requirements: ldx >= d, ld_code >= s,
 * ld_xhat >= d; every row of X and of X_hat must start on a 16-byte boundary; out_idx, idx,
 * out_coef and coef need only the alignment of their element type when ld_code is given
 * (dense code arrays must be 16-byte aligned as before).  The host entry points take
 * dense arrays only.
 *
 * Several problems in one call (one dictionary per layer, per K / V, per chunk): the
 * problems are validated first, all of them, and nothing is enqueued if one is invalid;
 * then they are enqueued in order on their streams.  Neighbouring fast-mode problems on
 * the same stream that each bring their own dictionary copy (`dict` or `workspace`) depend
 * on nothing shared and are enqueued side by side: the stream forks into library-owned
 * side streams and joins again before the call returns, so work enqueued afterwards sees
 * all of them (the K rows and the V rows of one decoding step take the time of one).
 * Returns the first failure.
 */
int csr_encode_grouped(const csr_encode_params_t* problems, int count);
int csr_reconstruct_grouped(const csr_reconstruct_params_t* problems, int count);

/*
 * Online part of a dictionary ("Build dictionary": besides the offline atoms a prompt's
 * dictionary holds atoms sampled from the KV cache just computed; atoms are kept at unit
 * l2-norm, the ReNorm step of "NeuralDict").  For i = 0 .. n_rows-1:
 *     D[N_cur + i][:] = X[rows[i]][:] / ||X[rows[i]][:]||_2        (fp32; norm accumulated in fp32)
 * A row whose norm is zero gives a zero atom (which matching pursuit never selects for a
 * non-zero residual).  Which rows are sampled is the caller's choice: `rows` is a DEVICE
 * array of n_rows row numbers in [0, M).  D is the caller's [N_cap][d] fp32 device array of
 * which rows [0, N_cur) are in use; N_cur + n_rows <= N_cap is required.  X is [M][d] with
 * x_dtype F32, BF16 or F16 and row stride ldx (0 = d).  Asynchronous on `stream`.
 */
int csr_dict_append(void* D, int N_cur, int N_cap, int d, const void* X, int x_dtype, int64_t M, int64_t ldx,
                    const int64_t* rows, int n_rows, void* stream);

/*
 * Attention straight from the codes ("De-Sparse to restore": the restored X~ = D r of
 * Eq. 12 is what the attention scores are computed from; both products below are that
 * computation with X~ never written to memory, which is possible because X~ is linear in
 * the atoms).  B code streams (one per sequence and KV head) of T tokens each share the
 * dictionary D; H query heads attend to each stream (H = 1 without grouped queries).
 *
 * csr_key_scores:  scores[b][h][t] = scale * Q[b][h][:] . X~_K[b][t][:]
 *                                  = sum_g coef[b][t][g] * (scale * D[idx[b][t][g]][:] . Q[b][h][:]),
 *     terms added in stored order g = 0 .. s-1 in fp32.  Q is [B][H][d], q_dtype F32, BF16 or F16;
 *     scores is [B][H][T] fp32 (before softmax).
 * csr_value_mix:   out[b][h][:] = sum_t W[b][h][t] * X~_V[b][t][:],
 *     W is [B][H][T] fp32 (attention weights; any finite values, not only softmax rows),
 *     out is [B][H][d] fp32.  The per-atom sums a[n] = sum over (t, g) with idx = n of
 *     W[t] * coef[t][g] are accumulated in 32-bit fixed point scaled to the largest value a
 *     sum can reach (each term is rounded once to fp32 and once to a grid no coarser than
 *     2^-29 of that bound), then out = a D in fp32 in a fixed order: the result is the same
 *     bits on every run.  A NaN or Inf weight or coefficient is carried through fp32 sums
 *     instead and reaches the outputs of its stream.
 *
 * idx and coef are [B][T][s] (coef_dtype F16 or F32); an idx >= N is clamped to N-1.
 * Limits: d in {64, 128}, 1 <= N <= 49152 (one head's N partial products must fit in
 * shared memory), 1 <= s <= 64, 1 <= H <= 64, B, T >= 0.  All pointers are device pointers,
 * 16-byte aligned.  Asynchronous on `stream`.
 */
int csr_key_scores(const void* D, int N, int d, const void* Q, int q_dtype, int B, int H, const uint16_t* idx,
                   const void* coef, int coef_dtype, int64_t T, int s, float scale, float* scores, void* stream);
int csr_value_mix(const void* D, int N, int d, const float* W, int B, int H, const uint16_t* idx, const void* coef,
                  int coef_dtype, int64_t T, int s, float* out, void* stream);

/*
 * One training step of the offline dictionary ("NeuralDict": Algorithm 1, procedure
 * TrainNeurDict, with the MSE loss, the diversity loss, the complete loss and ReNorm).  For
 * the batch X ([M][d], dense):
 *   1. r(x) for every row by matching pursuit with s iterations over the current D (the
 *      encoder of `mode`; its codes are then held fixed: the loss is differentiated with
 *      respect to the atoms only);
 *   2. L_MSE = sum_x ||x - D^T r(x)||^2 and its gradient, which touches only the selected
 *      atoms: -2 * sum_{(x,g): i_g = n} c_g (x - x^);
 *   3. L_div = ||I - D D^T||_F^2 / N^2 and its gradient (4 / N^2) (D D^T - I) D; the N x N
 *      matrix is formed block by block on chip and never stored;
 *   4. D <- ReNorm(D - lr * (grad L_MSE + beta * grad L_div)), every atom back to unit l2-norm.
 * losses (device, two doubles, 8-byte aligned) receives L_MSE and L_div of the dictionary
 * BEFORE the update; the paper's adaptive weight for the next batch is
 * beta = min(0.1 * L_MSE / L_div, 1.0), which the caller forms from them.  The optimiser is
 * a plain gradient step (the paper names none).  D is updated in place and must not be
 * used by other work on the device meanwhile.  Uses the library-owned scratch (order it
 * with the other users of that scratch); asynchronous on `stream`.  Gradient sums use atomic fp32 adds: reproducible to rounding.
 */
typedef struct csr_train_params {
    uint32_t struct_size;   /* sizeof(csr_train_params_t) */
    int32_t mode;           /* CSR_MODE_* of the matching-pursuit forward pass */
    void* D;                /* [N][d] fp32, updated in place */
    const void* X;          /* [M][d], x_dtype (F32, BF16 or F16), dense */
    int32_t x_dtype;
    int32_t d, N, s;
    int64_t M;
    float lr;
    float beta;
    double* losses;         /* device, [2] */
    void* stream;
} csr_train_params_t;
int csr_dict_train_step(const csr_train_params_t* p);

/*
 * Encode with HOST buffers (the same operation as csr_encode_ex; only X, out_idx and
 * out_coef are host pointers, ideally page-locked).  X is copied to the device in
 * chunks that overlap with the encoding of the previous chunk, the codes are copied
 * back, and the function returns after everything has finished.  D stays a device
 * pointer.  Uses library-owned device staging buffers (grow-only, per device) and two
 * library-owned streams, which first wait for everything enqueued so far on params.stream
 * (so a dictionary still being written there is complete before it is read); the fast
 * mode's bf16 copy of D is made once per call; the exact mode's chunk encodes run one after
 * the other (they share the library's scratch) under the copies.  dev_status is ignored.
 */
int csr_encode_host(const csr_encode_params_t* p);

/*
 * De-sparse with HOST buffers (the same operation as csr_reconstruct_ex, Eq. 12; idx, coef
 * and X_hat are host pointers, ideally page-locked): the case of codes kept in host memory
 * and restored on demand.  Codes are copied to the device in chunks, X_hat chunks are
 * copied back while the next chunk is computed, and the function returns after everything
 * has finished.  D stays a device pointer.  Shares the staging buffers of csr_encode_host.
 */
int csr_reconstruct_host(const csr_reconstruct_params_t* p);

/*
 * Fast encode without any allocation (the paper has no counterpart; this entry point
 * exists for the deployment reasons below).  Same operation, layouts and results as the
 * 8-argument csr_encode (bf16 X, fp16 coefficients, fast mode), on the given stream.
 *
 * For whom: callers that may not allocate or free device memory while they run, e.g. an
 * inference server whose device memory is carved up once at start-up, a process whose
 * free device memory is all owned by a framework's caching allocator, or a
 * latency-critical loop that cannot afford the implicit device-wide synchronisation an
 * allocation or a free may cause.  The other encode entry points keep their bf16 copy of
 * the dictionary in a cudaMalloc'ed buffer (or take a caller workspace); this one keeps
 * it in a fixed array inside the library image and calls no cudaMalloc, cudaFree or
 * other allocating routine.
 *
 * Limits and rules
 *   - N8 * d <= CSR_STATIC_MAX_DICT_ELEMS with N8 = N rounded up to a multiple of 8 (8192
 *     atoms of 128 channels, a 2 MiB bf16 copy);
 *     larger dictionaries are rejected with CSR_ERR_UNSUPPORTED.
 *   - The first call on a device looks up the array's device address, once, with that
 *     device current.  That lookup (and the first launch of each kernel) makes the CUDA
 *     runtime load the part of the library image that holds the array, which is when the
 *     2 MiB + 2 KiB are taken from that GPU's memory, to be held until the process exits.
 *     Make one call per device and per shape class (many rows; few rows) at start-up and
 *     before any stream capture begins; later calls take nothing from device memory.
 *   - All calls on a device share the one array, and it keeps what the last call wrote.
 *     Each call rewrites the dictionary copy in full and zeroes its status word before
 *     use, so stale contents never matter; but two calls whose work overlaps on the GPU
 *     (different streams, no ordering between them) race on it.  Order them.
 *   - dev_status: optional device word (4-byte aligned) that is zeroed by the call and
 *     receives a non-zero value if a device-side wait expired; NULL keeps that word
 *     inside the array, where csr_device_status does not look.
 */
#define CSR_STATIC_MAX_DICT_ELEMS (8192 * 128)
int csr_encode_static(const void* D, const void* X, int64_t M, int d, int N, int s, uint16_t* out_idx,
                      void* out_coef, void* stream, uint32_t* dev_status);

/*
 * One-off check of the unit-norm assumption ("Sparse representation": the atoms of D are
 * unit vectors; "NeuralDict": ReNorm restores that after every update).  Computes
 * max_n | ||D[n]||_2 - 1 | in fp32 on `stream`, waits for it, stores it in *max_dev (host
 * pointer, may be NULL) and returns CSR_ERR_INVALID_ARG if it exceeds `tol` (tol < 0: report
 * only).  Not on the hot path: the encoders never call it.  Atoms normalised in fp32 are off
 * by up to about 1e-7.  Uses a word of the library-owned scratch: order it like the
 * other users of that scratch.
 */
int csr_dict_check_norms(const void* D, int N, int d, float tol, void* stream, float* max_dev);

/*
 * Process-wide tuning and diagnostic switches; none is needed in normal use (tests use them
 * to drive every code path, measurements to compare them).  All paths return the same codes.
 *   "fast_group"     0 (default: the library chooses) or 1, 2, 4, 8: atoms per arg-max group
 *                    of the fast encoder's sweep;
 *   "fast_split"     0 (default: few rows split the dictionary across thread-block
 *                    clusters, else across CTAs with a launch pair per iteration),
 *                    1 = always one CTA per pair of row tiles over the whole dictionary,
 *                    2 = no clusters;
 *   "exact_split"    0 (default: the exact mode splits the dictionary for few rows), 1 = never;
 *   "exact_engine"   0 (default: the exact mode's tensor-core encoder unless the rows are few),
 *                    1 = plain-ALU encoders only, 2 = the tensor-core encoder also with few rows;
 *   "wait_limit_ns"  bound of every device-side wait of the tensor-core encoders in nanoseconds
 *                    (default 2e9).  0 lets no wait outlast a single look at its barrier, so
 *                    the first hand-off that is not already complete expires: the call
 *                    returns, its outputs are unspecified and the status word reports
 *                    CSR_ERR_TIMEOUT (how the expiry path is exercised).
 * Takes effect for calls made afterwards; not synchronised with calls in flight on other
 * host threads.  Returns CSR_ERR_INVALID_ARG for an unknown name or value.
 */
int csr_set_option(const char* name, int64_t value);

/*
 * Synchronises the stream and reports whether a kernel of this library has given up on a
 * bounded wait since the last call of this function on the current device: CSR_OK or
 * CSR_ERR_TIMEOUT (or CSR_ERR_CUDA if the stream itself is in error).  A library built with
 * device-side checks (csr_debug_checks() == 1) also reports CSR_ERR_BOUNDS here: an index that a
 * kernel was about to gather with was out of range (an idx >= N given to csr_reconstruct, a
 * candidate atom past the dictionary in the fast encoder); the release build clamps such
 * indices silently, the checked build clamps and records.  Reads the library's
 * status word(s); a call that was given its own dev_status reports there instead.
 */
int csr_device_status(void* stream);

/* Releases the library-owned device buffers of the current device. */
int csr_release_workspace(void);

const char* csr_last_error_string(void);
int csr_version(void);
/* 1 if this library was built with the device-side index checks (build.py --debug), else 0. */
int csr_debug_checks(void);
/*
 * Quantities only a checked build records (CSR_ERR_UNSUPPORTED otherwise); reading one
 * synchronises the device and resets it.
 *   "exact_tensor_error"  the largest | tensor-core correlation - fp64 correlation | / ||R||
 *                         over the picks the exact mode's tensor-core encoder took without
 *                         re-scoring since the last read (must stay below half the band).
 */
int csr_debug_read(const char* name, double* value);

#ifdef __cplusplus
}
#endif
#endif /* CSR_H_ */
