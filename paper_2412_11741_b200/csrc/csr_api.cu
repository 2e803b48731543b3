// C boundary of libcsr: argument checks, workspace management, stream plumbing.
// Every computation is done by the kernels in the other translation units.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "common.cuh"

struct csr_dict {
    uint32_t magic;
    int device;
    const void* D;
    int N, d;
    void* raw;      // cudaMalloc'ed block
    void* bf16;     // 1024-byte aligned bf16 copy inside it (the fast encoder's operand)
    void* f16;      // fp16 copy behind it (the de-sparse kernel's gather source)
};

namespace csr {

static thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

namespace {
std::atomic<int> g_opt_fast_group{0}, g_opt_fast_split{0}, g_opt_exact_split{0}, g_opt_exact_engine{0};
std::atomic<unsigned long long> g_opt_wait_limit_ns{2000000000ull};      // 2 s per wait
}  // namespace

Options options() {
    Options o;
    o.fast_group = g_opt_fast_group.load(std::memory_order_relaxed);
    o.fast_split = g_opt_fast_split.load(std::memory_order_relaxed);
    o.exact_split = g_opt_exact_split.load(std::memory_order_relaxed);
    o.exact_engine = g_opt_exact_engine.load(std::memory_order_relaxed);
    o.wait_limit_ns = g_opt_wait_limit_ns.load(std::memory_order_relaxed);
    return o;
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kStatusBytes = 256;
constexpr int kDiagWord = 2;              // word of the status block a checked build raises (see csr_debug_read)
constexpr uint32_t kDictMagic = 0x43535244u;   // "CSRD"

// Library-owned, grow-only device buffers of one device.
constexpr int kSideStreams = 3;
struct DeviceBuffers {
    void* work = nullptr;      // [status word | encoder scratch]
    size_t work_bytes = 0;
    std::vector<void*> retired;   // outgrown work buffers: kept until csr_release_workspace, because
                                  // kernels already enqueued (or captured into a graph) still use them
    void* stage_x[2] = {nullptr, nullptr};   // host-entry staging: X chunks
    void* stage_idx[2] = {nullptr, nullptr};
    void* stage_coef[2] = {nullptr, nullptr};
    size_t stage_rows = 0;
    size_t stage_x_bytes = 0, stage_code_bytes = 0;
    cudaStream_t copy_streams[2] = {nullptr, nullptr};
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr};
    // grouped calls: problems that may run side by side
    cudaStream_t side[kSideStreams] = {};
    cudaEvent_t side_done[kSideStreams] = {};
    cudaEvent_t fork = nullptr;
};
DeviceBuffers g_dev[kMaxDevices];
std::mutex g_mu;
std::mutex g_group_mu;     // one grouped fork/join at a time: its events are shared

int current_device(int* dev) {
    cudaError_t e = cudaGetDevice(dev);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (*dev < 0 || *dev >= kMaxDevices) return fail(CSR_ERR_UNSUPPORTED, "device ordinal %d not supported", *dev);
    return CSR_OK;
}

// Returns the library's work buffer (status word first), grown to hold `scratch` bytes.
// A buffer that has to grow is replaced, never freed: work already enqueued and captured
// graphs keep the block they were given (csr_release_workspace frees them all).  Growing
// allocates, so it is refused while `stream` is being captured.
int ensure_work(size_t scratch, void** base, cudaStream_t stream) {
    int dev;
    if (int rc = current_device(&dev)) return rc;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceBuffers& b = g_dev[dev];
    const size_t need = kStatusBytes + 1024 + scratch;
    if (b.work_bytes < need) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) {
            cudaGetLastError();
            cap = cudaStreamCaptureStatusNone;
        }
        if (cap != cudaStreamCaptureStatusNone)
            return fail(CSR_ERR_WORKSPACE,
                        "the library scratch would have to grow to %zu bytes during stream capture: make the same "
                        "call once before capturing, or pass a workspace / dictionary handle",
                        need);
        void* fresh = nullptr;
        cudaError_t e = cudaMalloc(&fresh, need);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMalloc(%zu): %s", need, cudaGetErrorString(e));
        e = cudaMemset(fresh, 0, kStatusBytes);
        if (e != cudaSuccess) {
            cudaFree(fresh);
            return fail(CSR_ERR_CUDA, "cudaMemset: %s", cudaGetErrorString(e));
        }
        if (b.work) b.retired.push_back(b.work);
        b.work = fresh;
        b.work_bytes = need;
    }
    *base = b.work;
    return CSR_OK;
}

inline void* align_up(void* p, size_t a) {
    return reinterpret_cast<void*>((reinterpret_cast<uintptr_t>(p) + a - 1) / a * a);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_dims(int d, int N, int s, int64_t M) {
    if (d != 64 && d != 128) return fail(CSR_ERR_UNSUPPORTED, "d = %d: only 64 and 128 are supported", d);
    if (N < 1 || N > 65536) return fail(CSR_ERR_INVALID_ARG, "N = %d outside [1, 65536]", N);
    if (s < 1 || s > 64) return fail(CSR_ERR_INVALID_ARG, "s = %d outside [1, 64]", s);
    if (M < 0) return fail(CSR_ERR_INVALID_ARG, "M = %lld is negative", (long long)M);
    return CSR_OK;
}

int check_encode(const csr_encode_params_t* p, bool host_io) {
    if (!p) return fail(CSR_ERR_INVALID_ARG, "params is NULL");
    if (p->struct_size != sizeof(csr_encode_params_t))
        return fail(CSR_ERR_INVALID_ARG, "struct_size %u != %zu", p->struct_size, sizeof(csr_encode_params_t));
    if (p->mode != CSR_MODE_FP32_EXACT && p->mode != CSR_MODE_BF16_FAST)
        return fail(CSR_ERR_INVALID_ARG, "unknown mode %d", p->mode);
    if (int rc = check_dims(p->d, p->N, p->s, p->M)) return rc;
    if (!valid_x_dtype(p->x_dtype)) return fail(CSR_ERR_INVALID_ARG, "x_dtype must be F32, BF16 or F16");
    if (p->coef_dtype != CSR_DTYPE_F32 && p->coef_dtype != CSR_DTYPE_F16)
        return fail(CSR_ERR_INVALID_ARG, "coef_dtype must be F32 or F16");
    if (!p->D) return fail(CSR_ERR_INVALID_ARG, "D is NULL");
    if (p->M > 0 && (!p->X || !p->out_idx || !p->out_coef))
        return fail(CSR_ERR_INVALID_ARG, "X, out_idx or out_coef is NULL");
    if (p->ldx < 0 || p->ld_code < 0 || (p->ldx && p->ldx < p->d) || (p->ld_code && p->ld_code < p->s))
        return fail(CSR_ERR_INVALID_ARG, "ldx (%lld) must be 0 or >= d, ld_code (%lld) 0 or >= s", (long long)p->ldx,
                    (long long)p->ld_code);
    if (host_io && (p->ldx || p->ld_code)) return fail(CSR_ERR_UNSUPPORTED, "the host entry points take dense arrays");
    if (!aligned16(p->D)) return fail(CSR_ERR_ALIGNMENT, "D must be 16-byte aligned");
    if (!host_io) {
        const size_t xe = dtype_size(p->x_dtype), ce = p->coef_dtype == CSR_DTYPE_F16 ? 2 : 4;
        if (!aligned16(p->X) || (p->ldx && (p->ldx * xe) % 16 != 0))
            return fail(CSR_ERR_ALIGNMENT, "every row of X must start on a 16-byte boundary");
        if (p->ld_code == 0) {
            if (!aligned16(p->out_idx) || !aligned16(p->out_coef))
                return fail(CSR_ERR_ALIGNMENT, "dense out_idx and out_coef must be 16-byte aligned");
        } else if ((reinterpret_cast<uintptr_t>(p->out_idx) % 2) || (reinterpret_cast<uintptr_t>(p->out_coef) % ce)) {
            return fail(CSR_ERR_ALIGNMENT, "out_idx / out_coef are not aligned to their element type");
        }
    }
    if (p->workspace && !aligned16(p->workspace)) return fail(CSR_ERR_ALIGNMENT, "workspace must be 16-byte aligned");
    if (reinterpret_cast<uintptr_t>(p->dev_status) % 4) return fail(CSR_ERR_ALIGNMENT, "dev_status must be 4-byte aligned");
    return CSR_OK;
}

// Chunk of a host-side job: a multiple of 256 rows, about 1/8 of the job, at least 32768 rows.
int64_t host_chunk_rows(int64_t M) {
    int64_t chunk = ((M / 8 + 255) / 256) * 256;
    if (chunk < 32768) chunk = 32768;
    if (chunk > M) chunk = ((M + 255) / 256) * 256;
    return chunk;
}

// Two copy streams with their events and two sets of staging buffers (rows of X or X_hat,
// indices, coefficients), grown on demand.
int ensure_staging(DeviceBuffers& b, size_t need_x, size_t need_c) {
    std::lock_guard<std::mutex> lk(g_mu);
    cudaError_t e = cudaSuccess;
    if (!b.copy_streams[0]) {
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaStreamCreateWithFlags(&b.copy_streams[i], cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b.ev_in[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b.ev_done[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "stream/event creation: %s", cudaGetErrorString(e));
    }
    if (b.stage_x_bytes < need_x || b.stage_code_bytes < need_c) {
        if (need_x < b.stage_x_bytes) need_x = b.stage_x_bytes;
        if (need_c < b.stage_code_bytes) need_c = b.stage_code_bytes;
        cudaDeviceSynchronize();
        for (int i = 0; i < 2; ++i) {
            cudaFree(b.stage_x[i]);
            cudaFree(b.stage_idx[i]);
            cudaFree(b.stage_coef[i]);
            b.stage_x[i] = b.stage_idx[i] = b.stage_coef[i] = nullptr;
        }
        b.stage_x_bytes = b.stage_code_bytes = 0;
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaMalloc(&b.stage_x[i], need_x);
            if (e == cudaSuccess) e = cudaMalloc(&b.stage_idx[i], need_c);
            if (e == cudaSuccess) e = cudaMalloc(&b.stage_coef[i], need_c);
        }
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "staging cudaMalloc: %s", cudaGetErrorString(e));
        b.stage_x_bytes = need_x;
        b.stage_code_bytes = need_c;
    }
    return CSR_OK;
}

int check_reconstruct(const csr_reconstruct_params_t* p, bool host_io) {
    if (!p) return fail(CSR_ERR_INVALID_ARG, "params is NULL");
    if (p->struct_size != sizeof(csr_reconstruct_params_t))
        return fail(CSR_ERR_INVALID_ARG, "struct_size %u != %zu", p->struct_size, sizeof(csr_reconstruct_params_t));
    if (int rc = check_dims(p->d, p->N, p->s, p->M)) return rc;
    if (p->coef_dtype != CSR_DTYPE_F32 && p->coef_dtype != CSR_DTYPE_F16)
        return fail(CSR_ERR_INVALID_ARG, "coef_dtype must be F32 or F16");
    if (!valid_x_dtype(p->out_dtype)) return fail(CSR_ERR_INVALID_ARG, "out_dtype must be F32, BF16 or F16");
    if (!p->D) return fail(CSR_ERR_INVALID_ARG, "D is NULL");
    if (p->M > 0 && (!p->idx || !p->coef || !p->X_hat)) return fail(CSR_ERR_INVALID_ARG, "idx, coef or X_hat is NULL");
    if (p->ld_code < 0 || p->ld_xhat < 0 || (p->ld_code && p->ld_code < p->s) || (p->ld_xhat && p->ld_xhat < p->d))
        return fail(CSR_ERR_INVALID_ARG, "ld_code (%lld) must be 0 or >= s, ld_xhat (%lld) 0 or >= d",
                    (long long)p->ld_code, (long long)p->ld_xhat);
    if (host_io && (p->ld_code || p->ld_xhat)) return fail(CSR_ERR_UNSUPPORTED, "the host entry points take dense arrays");
    if (!aligned16(p->D)) return fail(CSR_ERR_ALIGNMENT, "D must be 16-byte aligned");
    if (p->dict) {
        const csr_dict* dc = static_cast<const csr_dict*>(p->dict);
        int dev = -1;
        if (int rc = current_device(&dev)) return rc;
        if (dc->magic != kDictMagic) return fail(CSR_ERR_INVALID_ARG, "dict is not a live csr_dict_t handle");
        if (dc->device != dev || dc->D != p->D || dc->N != p->N || dc->d != p->d)
            return fail(CSR_ERR_INVALID_ARG, "dict was created for another device, D, N or d");
    }
    if (!host_io) {
        const size_t xe = dtype_size(p->out_dtype), ce = p->coef_dtype == CSR_DTYPE_F16 ? 2 : 4;
        if (!aligned16(p->X_hat) || (p->ld_xhat && (p->ld_xhat * xe) % 16 != 0))
            return fail(CSR_ERR_ALIGNMENT, "every row of X_hat must start on a 16-byte boundary");
        if (p->ld_code == 0) {
            if (!aligned16(p->idx) || !aligned16(p->coef))
                return fail(CSR_ERR_ALIGNMENT, "dense idx and coef must be 16-byte aligned");
        } else if ((reinterpret_cast<uintptr_t>(p->idx) % 2) || (reinterpret_cast<uintptr_t>(p->coef) % ce)) {
            return fail(CSR_ERR_ALIGNMENT, "idx / coef are not aligned to their element type");
        }
    }
    return CSR_OK;
}

ReconstructArgs reconstruct_args(const csr_reconstruct_params_t* p) {
    ReconstructArgs a;
    a.D = static_cast<const float*>(p->D);
    a.dict_f16 = p->dict ? static_cast<const csr_dict*>(p->dict)->f16 : nullptr;
    a.idx = p->idx;
    a.coef = p->coef;
    a.coef_dtype = p->coef_dtype;
    a.out_dtype = p->out_dtype;
    a.M = p->M;
    a.d = p->d;
    a.N = p->N;
    a.s = p->s;
    a.X_hat = p->X_hat;
    a.ld_code = p->ld_code ? p->ld_code : p->s;
    a.ld_xhat = p->ld_xhat ? p->ld_xhat : p->d;
    a.stream = static_cast<cudaStream_t>(p->stream);
    a.status = nullptr;
#ifdef CSR_DEBUG_CHECKS
    void* base = nullptr;                                     // the debug build reports clamped indices in the library's word
    if (ensure_work(0, &base, a.stream) == CSR_OK) a.status = static_cast<uint32_t*>(base);
#endif
    return a;
}

int64_t workspace_bytes(int mode, int d, int N) {
    if (mode == CSR_MODE_FP32_EXACT) return 0;
    return (int64_t)(kStatusBytes + 1024 + encode_fast_workspace_bytes(d, N));
}

// Streams and events of a grouped call, made on first use.
int ensure_side_streams(DeviceBuffers** out) {
    int dev;
    if (int rc = current_device(&dev)) return rc;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceBuffers& b = g_dev[dev];
    if (!b.fork) {
        cudaError_t e = cudaEventCreateWithFlags(&b.fork, cudaEventDisableTiming);
        for (int i = 0; i < kSideStreams && e == cudaSuccess; ++i) {
            e = cudaStreamCreateWithFlags(&b.side[i], cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b.side_done[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "side streams: %s", cudaGetErrorString(e));
    }
    *out = &b;
    return CSR_OK;
}

// Runs one encode on device pointers.  `shared_scratch` = false keeps the call off the parts of
// the library-owned buffer that two encodes in flight would both write.  `prepared` (fast mode
// only) is a bf16 copy of D made by the caller of this function: no conversion is enqueued.
int encode_device(const csr_encode_params_t* p, bool shared_scratch = true, const void* prepared = nullptr) {
    if (p->M == 0) return CSR_OK;
    EncodeArgs a;
    a.D = static_cast<const float*>(p->D);
    a.X = p->X;
    a.x_dtype = p->x_dtype;
    a.coef_dtype = p->coef_dtype;
    a.M = p->M;
    a.d = p->d;
    a.N = p->N;
    a.s = p->s;
    a.out_idx = p->out_idx;
    a.out_coef = p->out_coef;
    a.ldx = p->ldx ? p->ldx : p->d;
    a.ld_code = p->ld_code ? p->ld_code : p->s;
    a.stream = static_cast<cudaStream_t>(p->stream);
    const Options opt = options();
    if (p->mode == CSR_MODE_FP32_EXACT) {
        // Both the few-rows encoder and the tensor-core encoder need scratch, which comes from
        // the library-owned buffer only (a caller workspace is sized for the fast mode, and two
        // encodes in flight must not share it): otherwise the row-tile encoder runs.
        const bool own = shared_scratch && !p->workspace;
        // (measured: the tensor-core encoder takes the same time for any number of rows up to one
        // pair of row tiles per SM and overtakes the split plain-ALU encoder at about 2048 rows)
        const bool split_ok = encode_exact_split_applies(p->M, p->N) && opt.exact_split == 0;
        const bool few = split_ok && p->M < 2048;
        if (own && opt.exact_engine != 1 && (!few || opt.exact_engine == 2)) {
            void* base = nullptr;
            if (int rc = ensure_work(encode_exact_tc_scratch_bytes(p->M, p->d, p->N), &base, a.stream)) return rc;
            uint32_t* words = static_cast<uint32_t*>(base);
            uint32_t* status = p->dev_status ? p->dev_status : words;
            if (p->dev_status) {
                cudaError_t e = cudaMemsetAsync(status, 0, sizeof(uint32_t), a.stream);
                if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
            }
            return launch_encode_exact_tc(a, align_up(static_cast<char*>(base) + kStatusBytes, 1024), status, words + kDiagWord);
        }
        if (own && split_ok) {
            void* base = nullptr;
            if (int rc = ensure_work(encode_exact_split_scratch_bytes(p->M, p->d, p->N), &base, a.stream)) return rc;
            return launch_encode_exact_split(a, align_up(static_cast<char*>(base) + kStatusBytes, 1024));
        }
        return launch_encode_exact(a);
    }

    // The word a kernel raises when one of its waits expires: the caller's, else the library's.
    uint32_t* status = p->dev_status;
    if (status) {
        cudaError_t e = cudaMemsetAsync(status, 0, sizeof(uint32_t), a.stream);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    }
    // few rows: the cluster path needs no scratch; its fallback (a launch pair per iteration)
    // does, and gets it from the library-owned buffer only (a caller workspace is sized for
    // the bf16 copy)
    const bool split = shared_scratch && !p->workspace && !prepared && encode_fast_split_applies(p->M, p->N) &&
                       opt.fast_split != 1;
    const size_t dict_b = (encode_fast_workspace_bytes(p->d, p->N) + 1023) / 1024 * 1024;
    const size_t split_b = split ? encode_fast_split_scratch_bytes(p->M, p->d, p->N) : 0;
    if (p->dict || prepared) {
        const void* copy = prepared;
        if (p->dict) {
            const csr_dict* dc = static_cast<const csr_dict*>(p->dict);
            int dev = -1;
            if (int rc = current_device(&dev)) return rc;
            if (dc->magic != kDictMagic) return fail(CSR_ERR_INVALID_ARG, "dict is not a live csr_dict_t handle");
            if (dc->device != dev || dc->D != p->D || dc->N != p->N || dc->d != p->d)
                return fail(CSR_ERR_INVALID_ARG, "dict was created for another device, D, N or d");
            copy = dc->bf16;
        }
        void* sp = nullptr;
        if (!status || split) {                               // library status word (+ split scratch)
            void* wbase = nullptr;
            if (int rc = ensure_work(split_b, &wbase, a.stream)) return rc;
            if (!status) status = static_cast<uint32_t*>(wbase);
            if (split) sp = align_up(static_cast<char*>(wbase) + kStatusBytes, 1024);
        }
        return launch_encode_fast_prepared(a, copy, status, sp);
    }
    void* base = nullptr;
    if (p->workspace) {
        const int64_t need = workspace_bytes(p->mode, p->d, p->N);
        if ((int64_t)p->workspace_bytes < need)
            return fail(CSR_ERR_WORKSPACE, "workspace of %zu bytes given, %lld needed", p->workspace_bytes,
                        (long long)need);
        base = p->workspace;
        if (!status) {
            cudaError_t e = cudaMemsetAsync(base, 0, kStatusBytes, a.stream);
            if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
        }
    } else {
        if (int rc = ensure_work(dict_b + split_b, &base, a.stream)) return rc;
    }
    if (!status) status = static_cast<uint32_t*>(base);
    char* scratch = static_cast<char*>(align_up(static_cast<char*>(base) + kStatusBytes, 1024));
    if (int rc = prepare_fast_dictionary(a.D, a.N, a.d, scratch, a.stream)) return rc;
    return launch_encode_fast_prepared(a, scratch, status, split ? scratch + dict_b : nullptr);
}

// The host entry points run on two library streams; this makes both wait for whatever the
// caller has enqueued on `user` so far (the dictionary may still be in the making there).
int order_after(DeviceBuffers& b, cudaStream_t user) {
    cudaError_t e = cudaEventRecord(b.ev_in[0], user);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) e = cudaStreamWaitEvent(b.copy_streams[i], b.ev_in[0], 0);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "ordering after the caller's stream: %s", cudaGetErrorString(e));
    return CSR_OK;
}

}  // namespace
}  // namespace csr

using namespace csr;

extern "C" {

int csr_version(void) { return CSR_VERSION; }

int csr_debug_checks(void) {
#ifdef CSR_DEBUG_CHECKS
    return 1;
#else
    return 0;
#endif
}

const char* csr_last_error_string(void) { return g_err; }

int64_t csr_encode_workspace_bytes(int mode, int d, int N) {
    if (mode != CSR_MODE_FP32_EXACT && mode != CSR_MODE_BF16_FAST)
        return fail(CSR_ERR_INVALID_ARG, "unknown mode %d", mode);
    if (int rc = check_dims(d, N, 1, 0)) return rc;
    return workspace_bytes(mode, d, N);
}

int csr_encode_ex(const csr_encode_params_t* p) {
    if (int rc = check_encode(p, false)) return rc;
    return encode_device(p);
}

int csr_encode(const void* D, const void* X, int64_t M, int d, int N, int s, uint16_t* out_idx, void* out_coef) {
    csr_encode_params_t p;
    memset(&p, 0, sizeof(p));
    p.struct_size = sizeof(p);
    p.mode = CSR_MODE_BF16_FAST;
    p.D = D;
    p.X = X;
    p.x_dtype = CSR_DTYPE_BF16;
    p.coef_dtype = CSR_DTYPE_F16;
    p.M = M;
    p.d = d;
    p.N = N;
    p.s = s;
    p.out_idx = out_idx;
    p.out_coef = out_coef;
    return csr_encode_ex(&p);
}

int csr_reconstruct_ex(const csr_reconstruct_params_t* p) {
    if (int rc = check_reconstruct(p, false)) return rc;
    return launch_reconstruct(reconstruct_args(p));
}

int csr_reconstruct(const void* D, const uint16_t* idx, const void* coef, int64_t M, int d, int N, int s,
                    void* X_hat) {
    csr_reconstruct_params_t p;
    memset(&p, 0, sizeof(p));
    p.struct_size = sizeof(p);
    p.D = D;
    p.idx = idx;
    p.coef = coef;
    p.coef_dtype = CSR_DTYPE_F16;
    p.out_dtype = CSR_DTYPE_BF16;
    p.M = M;
    p.d = d;
    p.N = N;
    p.s = s;
    p.X_hat = X_hat;
    return csr_reconstruct_ex(&p);
}

int csr_pack_coefficients(const float* coef32, int64_t n, void* coef16, void* stream) {
    if (n < 0) return fail(CSR_ERR_INVALID_ARG, "n is negative");
    if (n > 0 && (!coef32 || !coef16)) return fail(CSR_ERR_INVALID_ARG, "coef32 or coef16 is NULL");
    if (!aligned16(coef32) || !aligned16(coef16)) return fail(CSR_ERR_ALIGNMENT, "coef32 and coef16 must be 16-byte aligned");
    return launch_pack_coef(coef32, n, coef16, static_cast<cudaStream_t>(stream));
}

int csr_dict_create(const void* D, int N, int d, void* stream, csr_dict_t** out) {
    if (!out) return fail(CSR_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (int rc = check_dims(d, N, 1, 0)) return rc;
    if (!D) return fail(CSR_ERR_INVALID_ARG, "D is NULL");
    if (!aligned16(D)) return fail(CSR_ERR_ALIGNMENT, "D must be 16-byte aligned");
    int dev = -1;
    if (int rc = current_device(&dev)) return rc;
    csr_dict* dc = new (std::nothrow) csr_dict();
    if (!dc) return fail(CSR_ERR_CUDA, "out of host memory");
    const size_t bf16_b = (encode_fast_workspace_bytes(d, N) + 1023) / 1024 * 1024;
    cudaError_t e = cudaMalloc(&dc->raw, 1024 + bf16_b + (size_t)N * d * 2);
    if (e != cudaSuccess) {
        delete dc;
        return fail(CSR_ERR_CUDA, "cudaMalloc: %s", cudaGetErrorString(e));
    }
    dc->bf16 = align_up(dc->raw, 1024);
    dc->f16 = static_cast<char*>(dc->bf16) + bf16_b;
    dc->device = dev;
    dc->D = D;
    dc->N = N;
    dc->d = d;
    int rc = prepare_fast_dictionary(static_cast<const float*>(D), N, d, dc->bf16, static_cast<cudaStream_t>(stream));
    if (rc == CSR_OK) rc = launch_dict_to_f16(static_cast<const float*>(D), N, d, dc->f16, static_cast<cudaStream_t>(stream));
    if (rc != CSR_OK) {
        cudaFree(dc->raw);
        delete dc;
        return rc;
    }
    dc->magic = kDictMagic;
    *out = dc;
    return CSR_OK;
}

int csr_dict_destroy(csr_dict_t* dict) {
    if (!dict) return CSR_OK;
    if (dict->magic != kDictMagic) return fail(CSR_ERR_INVALID_ARG, "dict is not a live csr_dict_t handle");
    dict->magic = 0;
    cudaDeviceSynchronize();
    cudaFree(dict->raw);
    delete dict;
    return CSR_OK;
}

int csr_encode_grouped(const csr_encode_params_t* problems, int count) {
    if (count < 0 || (count > 0 && !problems)) return fail(CSR_ERR_INVALID_ARG, "problems is NULL or count < 0");
    for (int i = 0; i < count; ++i)
        if (int rc = check_encode(&problems[i], false)) return rc;
    // Problems that follow one another on the same stream, in the fast mode, each with its own
    // dictionary copy (a handle or a caller workspace) share nothing the library owns but the
    // status word: they are enqueued side by side (the stream forks into side streams and
    // joins again), which is what the K and V rows of one decoding step want: each fills a
    // fraction of the GPU.  Everything else runs in order.
    auto independent = [](const csr_encode_params_t& q) {
        return q.mode == CSR_MODE_BF16_FAST && (q.dict || q.workspace) && q.M > 0;
    };
    int i = 0;
    while (i < count) {
        int j = i + 1;
        if (independent(problems[i]))
            while (j < count && independent(problems[j]) && problems[j].stream == problems[i].stream) ++j;
        if (j - i < 2) {
            if (int rc = encode_device(&problems[i])) return rc;
            i = j;
            continue;
        }
        DeviceBuffers* b = nullptr;
        if (int rc = ensure_side_streams(&b)) return rc;
        std::lock_guard<std::mutex> group_lock(g_group_mu);
        cudaStream_t main = static_cast<cudaStream_t>(problems[i].stream);
        cudaError_t e = cudaEventRecord(b->fork, main);
        bool used[kSideStreams] = {};
        int rc = CSR_OK;
        for (int k = i + 1; k < j && rc == CSR_OK && e == cudaSuccess; ++k) {
            const int sidx = (k - i - 1) % kSideStreams;
            if (!used[sidx]) e = cudaStreamWaitEvent(b->side[sidx], b->fork, 0);
            used[sidx] = true;
            csr_encode_params_t q = problems[k];
            q.stream = b->side[sidx];
            if (e == cudaSuccess) rc = encode_device(&q, false);
        }
        if (rc == CSR_OK && e == cudaSuccess) rc = encode_device(&problems[i], false);
        // join whatever was forked, also after a failure: the caller's stream must not run ahead
        for (int sidx = 0; sidx < kSideStreams; ++sidx) {
            if (!used[sidx]) continue;
            cudaError_t e2 = cudaEventRecord(b->side_done[sidx], b->side[sidx]);
            if (e2 == cudaSuccess) e2 = cudaStreamWaitEvent(main, b->side_done[sidx], 0);
            if (e == cudaSuccess) e = e2;
        }
        if (rc != CSR_OK) return rc;
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "grouped encode fork/join: %s", cudaGetErrorString(e));
        i = j;
    }
    return CSR_OK;
}

int csr_reconstruct_grouped(const csr_reconstruct_params_t* problems, int count) {
    if (count < 0 || (count > 0 && !problems)) return fail(CSR_ERR_INVALID_ARG, "problems is NULL or count < 0");
    for (int i = 0; i < count; ++i)
        if (int rc = check_reconstruct(&problems[i], false)) return rc;
    for (int i = 0; i < count; ++i)
        if (int rc = launch_reconstruct(reconstruct_args(&problems[i]))) return rc;
    return CSR_OK;
}

int csr_dict_append(void* D, int N_cur, int N_cap, int d, const void* X, int x_dtype, int64_t M, int64_t ldx,
                    const int64_t* rows, int n_rows, void* stream) {
    if (d != 64 && d != 128) return fail(CSR_ERR_UNSUPPORTED, "d = %d: only 64 and 128 are supported", d);
    if (N_cap < 1 || N_cap > 65536 || N_cur < 0 || n_rows < 0 || (int64_t)N_cur + n_rows > N_cap)
        return fail(CSR_ERR_INVALID_ARG, "N_cur = %d, n_rows = %d do not fit N_cap = %d (<= 65536)", N_cur, n_rows, N_cap);
    if (!valid_x_dtype(x_dtype)) return fail(CSR_ERR_INVALID_ARG, "x_dtype must be F32, BF16 or F16");
    if (M < 0 || ldx < 0 || (ldx && ldx < d)) return fail(CSR_ERR_INVALID_ARG, "M < 0 or ldx not 0 or >= d");
    if (n_rows == 0) return CSR_OK;
    if (!D || !X || !rows) return fail(CSR_ERR_INVALID_ARG, "D, X or rows is NULL");
    if (M == 0) return fail(CSR_ERR_INVALID_ARG, "rows given but X is empty");
    const size_t xe = dtype_size(x_dtype);
    if (!aligned16(D) || !aligned16(X) || (ldx && (ldx * xe) % 16 != 0) || (reinterpret_cast<uintptr_t>(rows) % 8))
        return fail(CSR_ERR_ALIGNMENT, "D and every row of X must be 16-byte aligned, rows 8-byte aligned");
    return launch_dict_append(static_cast<float*>(D) + (size_t)N_cur * d, d, X, x_dtype, M, ldx ? ldx : d, rows, n_rows,
                              static_cast<cudaStream_t>(stream));
}

static int check_attn(const void* D, int N, int d, const void* Q, int B, int H, const uint16_t* idx, const void* coef,
                      int coef_dtype, int64_t T, int s, const void* out) {
    if (d != 64 && d != 128) return fail(CSR_ERR_UNSUPPORTED, "d = %d: only 64 and 128 are supported", d);
    if (N < 1 || N > 49152) return fail(CSR_ERR_INVALID_ARG, "N = %d outside [1, 49152]", N);
    if (s < 1 || s > 64) return fail(CSR_ERR_INVALID_ARG, "s = %d outside [1, 64]", s);
    if (H < 1 || H > 64) return fail(CSR_ERR_INVALID_ARG, "H = %d outside [1, 64]", H);
    if (B < 0 || T < 0) return fail(CSR_ERR_INVALID_ARG, "B or T is negative");
    if (coef_dtype != CSR_DTYPE_F32 && coef_dtype != CSR_DTYPE_F16)
        return fail(CSR_ERR_INVALID_ARG, "coef_dtype must be F32 or F16");
    if (!D) return fail(CSR_ERR_INVALID_ARG, "D is NULL");
    if (B > 0 && T > 0 && (!Q || !out || !idx || !coef))
        return fail(CSR_ERR_INVALID_ARG, "a query / weight / code / output pointer is NULL");
    if (!aligned16(D) || !aligned16(Q) || !aligned16(idx) || !aligned16(coef) || !aligned16(out))
        return fail(CSR_ERR_ALIGNMENT, "all pointers must be 16-byte aligned");
    return CSR_OK;
}

int csr_key_scores(const void* D, int N, int d, const void* Q, int q_dtype, int B, int H, const uint16_t* idx,
                   const void* coef, int coef_dtype, int64_t T, int s, float scale, float* scores, void* stream) {
    if (int rc = check_attn(D, N, d, Q, B, H, idx, coef, coef_dtype, T, s, scores)) return rc;
    if (!valid_x_dtype(q_dtype)) return fail(CSR_ERR_INVALID_ARG, "q_dtype must be F32, BF16 or F16");
    AttnArgs a{static_cast<const float*>(D), N, d, Q, q_dtype, B, H, idx, coef, coef_dtype, T, s, scale, scores,
               static_cast<cudaStream_t>(stream)};
    if (B == 0 || T == 0) return CSR_OK;
    void* base = nullptr;
    if (int rc = ensure_work(attn_scratch_bytes(B, H, N, T), &base, a.stream)) return rc;
    return launch_key_scores(a, static_cast<float*>(align_up(static_cast<char*>(base) + kStatusBytes, 1024)));
}

int csr_value_mix(const void* D, int N, int d, const float* W, int B, int H, const uint16_t* idx, const void* coef,
                  int coef_dtype, int64_t T, int s, float* out, void* stream) {
    if (int rc = check_attn(D, N, d, W, B, H, idx, coef, coef_dtype, T, s, out)) return rc;
    if (B > 0 && !out) return fail(CSR_ERR_INVALID_ARG, "out is NULL");     // zeroed even when T == 0
    AttnArgs a{static_cast<const float*>(D), N, d, W, CSR_DTYPE_F32, B, H, idx, coef, coef_dtype, T, s, 1.0f, out,
               static_cast<cudaStream_t>(stream)};
    if (B == 0) return CSR_OK;
    void* base = nullptr;
    if (int rc = ensure_work(attn_scratch_bytes(B, H, N, T), &base, a.stream)) return rc;
    return launch_value_mix(a, static_cast<float*>(align_up(static_cast<char*>(base) + kStatusBytes, 1024)));
}

int csr_decode_attention(const void* Dk, int Nk, const void* Dv, int Nv, int d, const void* Q, int q_dtype, int B, int H,
                         const uint16_t* k_idx, const void* k_coef, int sk, const uint16_t* v_idx, const void* v_coef,
                         int sv, int coef_dtype, int64_t T, float scale, float* weights, float* out, void* stream) {
    if (T == 0 && B > 0) return fail(CSR_ERR_INVALID_ARG, "attention over an empty cache (T = 0) is undefined");
    if (int rc = check_attn(Dv, Nv, d, weights, B, H, v_idx, v_coef, coef_dtype, T, sv, out)) return rc;
    if (int rc = csr_key_scores(Dk, Nk, d, Q, q_dtype, B, H, k_idx, k_coef, coef_dtype, T, sk, scale, weights, stream))
        return rc;
    if (B == 0) return CSR_OK;
    if (int rc = launch_softmax_rows(weights, (int64_t)B * H, T, static_cast<cudaStream_t>(stream))) return rc;
    return csr_value_mix(Dv, Nv, d, weights, B, H, v_idx, v_coef, coef_dtype, T, sv, out, stream);
}

int csr_dict_train_step(const csr_train_params_t* p) {
    if (!p) return fail(CSR_ERR_INVALID_ARG, "params is NULL");
    if (p->struct_size != sizeof(csr_train_params_t))
        return fail(CSR_ERR_INVALID_ARG, "struct_size %u != %zu", p->struct_size, sizeof(csr_train_params_t));
    if (p->mode != CSR_MODE_FP32_EXACT && p->mode != CSR_MODE_BF16_FAST)
        return fail(CSR_ERR_INVALID_ARG, "unknown mode %d", p->mode);
    if (int rc = check_dims(p->d, p->N, p->s, p->M)) return rc;
    if (!valid_x_dtype(p->x_dtype)) return fail(CSR_ERR_INVALID_ARG, "x_dtype must be F32, BF16 or F16");
    if (!p->D || !p->losses || (p->M > 0 && !p->X)) return fail(CSR_ERR_INVALID_ARG, "D, losses or X is NULL");
    if (!aligned16(p->D) || !aligned16(p->X) || (reinterpret_cast<uintptr_t>(p->losses) % 8))
        return fail(CSR_ERR_ALIGNMENT, "D and X must be 16-byte aligned, losses 8-byte aligned");
    if (!(p->lr >= 0.f) || !(p->beta >= 0.f)) return fail(CSR_ERR_INVALID_ARG, "lr and beta must be >= 0");
    // scratch layout: [encoder's own region][idx][coef][grad_mse][grad_div]
    size_t enc = (encode_fast_workspace_bytes(p->d, p->N) + 1023) / 1024 * 1024;
    if (p->M > 0 && encode_fast_split_applies(p->M, p->N)) enc += encode_fast_split_scratch_bytes(p->M, p->d, p->N);
    if (p->M > 0 && encode_exact_split_applies(p->M, p->N)) {
        const size_t sp = encode_exact_split_scratch_bytes(p->M, p->d, p->N);
        if (sp > enc) enc = sp;
    }
    if (p->M > 0 && p->mode == CSR_MODE_FP32_EXACT) {
        const size_t sp = encode_exact_tc_scratch_bytes(p->M, p->d, p->N);
        if (sp > enc) enc = sp;
    }
    enc = (enc + 1023) / 1024 * 1024;
    const size_t idx_b = ((size_t)p->M * p->s * 2 + 255) / 256 * 256;
    const size_t coef_b = ((size_t)p->M * p->s * 4 + 255) / 256 * 256;
    const size_t g_b = ((size_t)p->N * p->d * 4 + 255) / 256 * 256;
    const size_t div_b = div_grad_scratch_bytes(p->N, p->d);
    void* base = nullptr;
    if (int rc = ensure_work(enc + idx_b + coef_b + 2 * g_b + div_b, &base, static_cast<cudaStream_t>(p->stream))) return rc;
    char* q = static_cast<char*>(align_up(static_cast<char*>(base) + kStatusBytes, 1024)) + enc;
    TrainArgs a;
    a.D = static_cast<float*>(p->D);
    a.N = p->N;
    a.d = p->d;
    a.X = p->X;
    a.x_dtype = p->x_dtype;
    a.M = p->M;
    a.s = p->s;
    a.idx = reinterpret_cast<uint16_t*>(q);
    a.coef = reinterpret_cast<float*>(q + idx_b);
    a.grad_mse = reinterpret_cast<float*>(q + idx_b + coef_b);
    a.grad_div = reinterpret_cast<float*>(q + idx_b + coef_b + g_b);
    a.div_scratch = q + idx_b + coef_b + 2 * g_b;
    a.status = static_cast<uint32_t*>(base);
    a.losses = p->losses;
    a.lr = p->lr;
    a.beta = p->beta;
    a.stream = static_cast<cudaStream_t>(p->stream);
    if (p->M > 0) {
        csr_encode_params_t e;
        memset(&e, 0, sizeof(e));
        e.struct_size = sizeof(e);
        e.mode = p->mode;
        e.D = p->D;
        e.X = p->X;
        e.x_dtype = p->x_dtype;
        e.coef_dtype = CSR_DTYPE_F32;
        e.M = p->M;
        e.d = p->d;
        e.N = p->N;
        e.s = p->s;
        e.out_idx = const_cast<uint16_t*>(a.idx);
        e.out_coef = const_cast<float*>(a.coef);
        e.stream = p->stream;
        if (int rc = encode_device(&e)) return rc;      // its ensure_work request is smaller: no regrowth
    }
    return launch_dict_train(a);
}

int csr_encode_host(const csr_encode_params_t* p) {
    if (int rc = check_encode(p, true)) return rc;
    if (p->M == 0) return CSR_OK;
    int dev;
    if (int rc = current_device(&dev)) return rc;
    const size_t xb = dtype_size(p->x_dtype) * (size_t)p->d;
    const size_t cb = (p->coef_dtype == CSR_DTYPE_F16 ? 2 : 4) * (size_t)p->s;
    const size_t ib = 2 * (size_t)p->s;
    const int64_t chunk = host_chunk_rows(p->M);
    DeviceBuffers& b = g_dev[dev];
    if (int rc = ensure_staging(b, (size_t)chunk * xb, (size_t)chunk * (cb > ib ? cb : ib))) return rc;
    if (int rc = order_after(b, static_cast<cudaStream_t>(p->stream))) return rc;
    const int64_t n_chunks = (p->M + chunk - 1) / chunk;
    // Several chunks in the fast mode: the bf16 copy of D is made once, on the first stream, and
    // the second stream waits for it (one conversion per chunk into the one buffer, from two
    // streams, would have each stream rewrite what the other's kernel is reading).
    const void* prepared = nullptr;
    if (p->mode == CSR_MODE_BF16_FAST && !p->dict && n_chunks > 1) {
        void* base = nullptr;
        if (int rc = ensure_work((encode_fast_workspace_bytes(p->d, p->N) + 1023) / 1024 * 1024, &base, b.copy_streams[0]))
            return rc;
        void* copy = align_up(static_cast<char*>(base) + kStatusBytes, 1024);
        if (int rc = prepare_fast_dictionary(static_cast<const float*>(p->D), p->N, p->d, copy, b.copy_streams[0])) return rc;
        cudaError_t e = cudaEventRecord(b.ev_in[1], b.copy_streams[0]);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(b.copy_streams[1], b.ev_in[1], 0);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "dictionary copy hand-over: %s", cudaGetErrorString(e));
        prepared = copy;
    }
    // Chunk j uses slot j % 2 with its own stream for copy-in, encode and copy-out, so the
    // copies of one chunk overlap the kernels of the other.
    int rc = CSR_OK;
    for (int64_t j = 0; j < n_chunks && rc == CSR_OK; ++j) {
        const int slot = (int)(j & 1);
        const int64_t r0 = j * chunk;
        const int64_t rows = (p->M - r0 < chunk) ? (p->M - r0) : chunk;
        cudaStream_t st = b.copy_streams[slot];
        cudaError_t e = cudaMemcpyAsync(b.stage_x[slot], static_cast<const char*>(p->X) + (size_t)r0 * xb,
                                        (size_t)rows * xb, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) {
            rc = fail(CSR_ERR_CUDA, "H2D copy: %s", cudaGetErrorString(e));
            break;
        }
        csr_encode_params_t q = *p;
        q.X = b.stage_x[slot];
        q.M = rows;
        q.out_idx = static_cast<uint16_t*>(b.stage_idx[slot]);
        q.out_coef = b.stage_coef[slot];
        q.stream = st;
        q.workspace = nullptr;
        q.workspace_bytes = 0;
        q.dev_status = nullptr;                           // the chunks run side by side: the library's word collects them
        // The exact mode's encoders keep their scratch in the library-owned buffer: the chunks'
        // kernels then run one after the other (each waits for the one before it, on the other
        // stream; they fill the GPU anyway) while the copies still overlap them.
        const bool chained = p->mode == CSR_MODE_FP32_EXACT && n_chunks > 1;
        if (chained && j > 0) {
            e = cudaStreamWaitEvent(st, b.ev_in[1], 0);
            if (e != cudaSuccess) {
                rc = fail(CSR_ERR_CUDA, "chunk ordering: %s", cudaGetErrorString(e));
                break;
            }
        }
        rc = encode_device(&q, n_chunks == 1 || chained, prepared);
        if (rc != CSR_OK) break;
        if (chained) {
            e = cudaEventRecord(b.ev_in[1], st);
            if (e != cudaSuccess) {
                rc = fail(CSR_ERR_CUDA, "chunk ordering: %s", cudaGetErrorString(e));
                break;
            }
        }
        e = cudaMemcpyAsync(reinterpret_cast<char*>(p->out_idx) + (size_t)r0 * ib, b.stage_idx[slot],
                            (size_t)rows * ib, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(static_cast<char*>(p->out_coef) + (size_t)r0 * cb, b.stage_coef[slot],
                                (size_t)rows * cb, cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) rc = fail(CSR_ERR_CUDA, "D2H copy: %s", cudaGetErrorString(e));
    }
    for (int i = 0; i < 2; ++i) {
        cudaError_t e = cudaStreamSynchronize(b.copy_streams[i]);
        if (e != cudaSuccess && rc == CSR_OK) rc = fail(CSR_ERR_CUDA, "stream sync: %s", cudaGetErrorString(e));
    }
    return rc;
}

int csr_reconstruct_host(const csr_reconstruct_params_t* p) {
    if (int rc = check_reconstruct(p, true)) return rc;
    if (p->M == 0) return CSR_OK;
    int dev;
    if (int rc = current_device(&dev)) return rc;
    const size_t xb = dtype_size(p->out_dtype) * (size_t)p->d;
    const size_t cb = (p->coef_dtype == CSR_DTYPE_F16 ? 2 : 4) * (size_t)p->s;
    const size_t ib = 2 * (size_t)p->s;
    const int64_t chunk = host_chunk_rows(p->M);
    DeviceBuffers& b = g_dev[dev];
    if (int rc = ensure_staging(b, (size_t)chunk * xb, (size_t)chunk * (cb > ib ? cb : ib))) return rc;
    if (int rc = order_after(b, static_cast<cudaStream_t>(p->stream))) return rc;
    // Chunk j uses slot j % 2 with its own stream: the copies of one chunk overlap the kernel
    // of the other.
    const int64_t n_chunks = (p->M + chunk - 1) / chunk;
    int rc = CSR_OK;
    for (int64_t j = 0; j < n_chunks && rc == CSR_OK; ++j) {
        const int slot = (int)(j & 1);
        const int64_t r0 = j * chunk;
        const int64_t rows = (p->M - r0 < chunk) ? (p->M - r0) : chunk;
        cudaStream_t st = b.copy_streams[slot];
        cudaError_t e = cudaMemcpyAsync(b.stage_idx[slot], reinterpret_cast<const char*>(p->idx) + (size_t)r0 * ib,
                                        (size_t)rows * ib, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(b.stage_coef[slot], static_cast<const char*>(p->coef) + (size_t)r0 * cb,
                                (size_t)rows * cb, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) {
            rc = fail(CSR_ERR_CUDA, "H2D copy: %s", cudaGetErrorString(e));
            break;
        }
        csr_reconstruct_params_t q = *p;
        q.idx = static_cast<const uint16_t*>(b.stage_idx[slot]);
        q.coef = b.stage_coef[slot];
        q.X_hat = b.stage_x[slot];
        q.M = rows;
        q.stream = st;
        rc = launch_reconstruct(reconstruct_args(&q));
        if (rc != CSR_OK) break;
        e = cudaMemcpyAsync(static_cast<char*>(p->X_hat) + (size_t)r0 * xb, b.stage_x[slot], (size_t)rows * xb,
                            cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) rc = fail(CSR_ERR_CUDA, "D2H copy: %s", cudaGetErrorString(e));
    }
    for (int i = 0; i < 2; ++i) {
        cudaError_t e = cudaStreamSynchronize(b.copy_streams[i]);
        if (e != cudaSuccess && rc == CSR_OK) rc = fail(CSR_ERR_CUDA, "stream sync: %s", cudaGetErrorString(e));
    }
    return rc;
}

int csr_device_status(void* stream) {
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "stream sync: %s", cudaGetErrorString(e));
    int dev;
    if (int rc = current_device(&dev)) return rc;
    // the current work buffer and the outgrown ones (captured graphs still raise their words)
    std::vector<void*> blocks;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (g_dev[dev].work) blocks.push_back(g_dev[dev].work);
        blocks.insert(blocks.end(), g_dev[dev].retired.begin(), g_dev[dev].retired.end());
    }
    uint32_t seen = 0;
    for (void* work : blocks) {
        uint32_t st = 0;
        e = cudaMemcpy(&st, work, sizeof(st), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "status read: %s", cudaGetErrorString(e));
        if (st != 0) cudaMemset(work, 0, kStatusBytes);
        seen |= st;
    }
    if (seen & kStatusTimeout) return fail(CSR_ERR_TIMEOUT, "a device-side wait expired (status word 0x%x)", seen);
    if (seen & kStatusLayout) return fail(CSR_ERR_CUDA, "a kernel found its shared memory misaligned and did not run");
    if (seen & kStatusBounds)
        return fail(CSR_ERR_BOUNDS, "an index used for a gather was out of range and was clamped (status word 0x%x)", seen);
    if (seen != 0) return fail(CSR_ERR_CUDA, "unknown device status 0x%x", seen);
    return CSR_OK;
}

int csr_release_workspace(void) {
    int dev;
    if (int rc = current_device(&dev)) return rc;
    cudaDeviceSynchronize();
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceBuffers& b = g_dev[dev];
    cudaFree(b.work);
    b.work = nullptr;
    b.work_bytes = 0;
    for (void* old : b.retired) cudaFree(old);
    b.retired.clear();
    for (int i = 0; i < 2; ++i) {
        cudaFree(b.stage_x[i]);
        cudaFree(b.stage_idx[i]);
        cudaFree(b.stage_coef[i]);
        b.stage_x[i] = b.stage_idx[i] = b.stage_coef[i] = nullptr;
    }
    b.stage_x_bytes = b.stage_code_bytes = 0;
    if (b.fork) {
        cudaEventDestroy(b.fork);
        b.fork = nullptr;
        for (int i = 0; i < kSideStreams; ++i) {
            cudaStreamDestroy(b.side[i]);
            cudaEventDestroy(b.side_done[i]);
            b.side[i] = nullptr;
            b.side_done[i] = nullptr;
        }
    }
    return CSR_OK;
}

int csr_set_option(const char* name, int64_t value) {
    if (!name) return fail(CSR_ERR_INVALID_ARG, "name is NULL");
    if (!strcmp(name, "fast_group")) {
        if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8)
            return fail(CSR_ERR_INVALID_ARG, "fast_group must be 0 (library's choice), 1, 2, 4 or 8");
        g_opt_fast_group.store((int)value);
    } else if (!strcmp(name, "fast_split")) {
        if (value < 0 || value > 2) return fail(CSR_ERR_INVALID_ARG, "fast_split must be 0, 1 or 2");
        g_opt_fast_split.store((int)value);
    } else if (!strcmp(name, "exact_split")) {
        if (value < 0 || value > 1) return fail(CSR_ERR_INVALID_ARG, "exact_split must be 0 or 1");
        g_opt_exact_split.store((int)value);
    } else if (!strcmp(name, "exact_engine")) {
        if (value < 0 || value > 2) return fail(CSR_ERR_INVALID_ARG, "exact_engine must be 0, 1 or 2");
        g_opt_exact_engine.store((int)value);
    } else if (!strcmp(name, "wait_limit_ns")) {
        if (value < 0 || value > 60000000000ll) return fail(CSR_ERR_INVALID_ARG, "wait_limit_ns must lie in [0, 6e10]");
        g_opt_wait_limit_ns.store((unsigned long long)value);
    } else {
        return fail(CSR_ERR_INVALID_ARG, "unknown option '%s'", name);
    }
    return CSR_OK;
}

int csr_debug_read(const char* name, double* value) {
    if (!name || !value) return fail(CSR_ERR_INVALID_ARG, "name or value is NULL");
    if (strcmp(name, "exact_tensor_error") != 0) return fail(CSR_ERR_INVALID_ARG, "unknown quantity '%s'", name);
#ifndef CSR_DEBUG_CHECKS
    return fail(CSR_ERR_UNSUPPORTED, "only a library built with CSR_DEBUG_CHECKS records '%s'", name);
#else
    int dev;
    if (int rc = current_device(&dev)) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "device sync: %s", cudaGetErrorString(e));
    void* work = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        work = g_dev[dev].work;
    }
    float v = 0.f;
    if (work) {
        uint32_t* word = static_cast<uint32_t*>(work) + kDiagWord;
        e = cudaMemcpy(&v, word, sizeof(float), cudaMemcpyDeviceToHost);
        if (e == cudaSuccess) e = cudaMemset(word, 0, sizeof(uint32_t));
        if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "diagnostic read: %s", cudaGetErrorString(e));
    }
    *value = static_cast<double>(v);
    return CSR_OK;
#endif
}

int csr_dict_check_norms(const void* D, int N, int d, float tol, void* stream, float* max_dev) {
    if (int rc = check_dims(d, N, 1, 0)) return rc;
    if (!D) return fail(CSR_ERR_INVALID_ARG, "D is NULL");
    if (!aligned16(D)) return fail(CSR_ERR_ALIGNMENT, "D must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    void* base = nullptr;
    if (int rc = ensure_work(0, &base, st)) return rc;
    // a word of the status block that no kernel raises (the first word is the wait status)
    uint32_t* word = static_cast<uint32_t*>(base) + 32;
    cudaError_t e = cudaMemsetAsync(word, 0, sizeof(uint32_t), st);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    if (int rc = launch_dict_norm_deviation(static_cast<const float*>(D), N, d, word, st)) return rc;
    float dev_max = 0.f;
    e = cudaMemcpyAsync(&dev_max, word, sizeof(float), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "norm check: %s", cudaGetErrorString(e));
    if (max_dev) *max_dev = dev_max;
    if (tol >= 0.f && !(dev_max <= tol))
        return fail(CSR_ERR_INVALID_ARG, "an atom's l2-norm is off 1 by %g (tolerance %g)", (double)dev_max, (double)tol);
    return CSR_OK;
}

}  // extern "C"
