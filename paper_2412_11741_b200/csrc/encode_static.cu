// csr_encode_static: the fast encoder for callers that must not allocate.
//
// The fast encoder needs scratch memory: a bf16 copy of the dictionary, which the
// regular entry points keep in a cudaMalloc'ed buffer.  Some users of this library run
// where device allocation is off limits: inside a serving loop whose memory is handed out
// once at start-up and must not move afterwards, under a framework's caching allocator
// that owns all free device memory, or in a latency-critical section where an implicit
// device synchronisation (which cudaMalloc and cudaFree may cause) is not acceptable.
// For them the scratch lives in a file-scope __device__ array that is part of the
// library image, and no call here calls an allocating routine.  The image's device data is
// placed by the CUDA runtime when the module that holds it is first used on a device (with
// lazy module loading: at the first call of this entry point there, which looks the array
// up; the first launch of each kernel loads its code the same way), so the first call on a
// device belongs to start-up; from the second call on nothing is taken from device memory.
// Every GPU that has made that first call holds the bytes until the process exits.
#include <mutex>

#include "common.cuh"

namespace csr {
namespace {

constexpr size_t kStaticMaxDictElems = (size_t)CSR_STATIC_MAX_DICT_ELEMS;   // N * d
constexpr size_t kStaticHeader = 1024;                                      // status word + padding
constexpr size_t kStaticBytes = kStaticHeader + 1024 + kStaticMaxDictElems * 2;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_static_mu;

// Device address of the array on the current device, looked up once per device.
int static_scratch(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(CSR_ERR_UNSUPPORTED, "device ordinal %d not supported", dev);
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p)
            return fail(CSR_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return CSR_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace csr

using namespace csr;

extern "C" int csr_encode_static(const void* D, const void* X, int64_t M, int d, int N, int s, uint16_t* out_idx,
                                 void* out_coef, void* stream, uint32_t* dev_status) {
    if (d != 64 && d != 128) return fail(CSR_ERR_UNSUPPORTED, "d = %d: only 64 and 128 are supported", d);
    if (N < 1 || N > 65536) return fail(CSR_ERR_INVALID_ARG, "N = %d outside [1, 65536]", N);
    if (s < 1 || s > 64) return fail(CSR_ERR_INVALID_ARG, "s = %d outside [1, 64]", s);
    if (M < 0) return fail(CSR_ERR_INVALID_ARG, "M = %lld is negative", (long long)M);
    if (encode_fast_workspace_bytes(d, N) > kStaticMaxDictElems * 2)
        return fail(CSR_ERR_UNSUPPORTED,
                    "dictionary of N*d = %zu elements exceeds the static scratch (CSR_STATIC_MAX_DICT_ELEMS = %zu); "
                    "use csr_encode_ex with a caller workspace",
                    (size_t)N * (size_t)d, kStaticMaxDictElems);
    if (!D) return fail(CSR_ERR_INVALID_ARG, "D is NULL");
    if (M > 0 && (!X || !out_idx || !out_coef)) return fail(CSR_ERR_INVALID_ARG, "X, out_idx or out_coef is NULL");
    if (!aligned16(D) || !aligned16(X) || !aligned16(out_idx) || !aligned16(out_coef))
        return fail(CSR_ERR_ALIGNMENT, "D, X, out_idx and out_coef must be 16-byte aligned");
    if (dev_status && (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return fail(CSR_ERR_ALIGNMENT, "dev_status must be 4-byte aligned");
    if (M == 0) return CSR_OK;

    void* base = nullptr;
    if (int rc = static_scratch(&base)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The status word must start at zero; the dictionary copy is rewritten in full by every call.
    uint32_t* status = dev_status ? dev_status : static_cast<uint32_t*>(base);
    cudaError_t e = cudaMemsetAsync(status, 0, sizeof(uint32_t), st);
    if (e != cudaSuccess) return fail(CSR_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    uintptr_t dict = (reinterpret_cast<uintptr_t>(base) + kStaticHeader + 1023) & ~static_cast<uintptr_t>(1023);

    EncodeArgs a;
    a.D = static_cast<const float*>(D);
    a.X = X;
    a.x_dtype = CSR_DTYPE_BF16;
    a.coef_dtype = CSR_DTYPE_F16;
    a.M = M;
    a.d = d;
    a.N = N;
    a.s = s;
    a.out_idx = out_idx;
    a.out_coef = out_coef;
    a.ldx = d;
    a.ld_code = s;
    a.stream = st;
    return launch_encode_fast(a, reinterpret_cast<void*>(dict), status);
}
