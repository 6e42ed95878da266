// uncomp_gram_static: the Gram stage for callers that cannot hand the library any scratch memory.
//
// Every other entry point works inside a workspace the caller allocates.  Some callers have no way to
// allocate one: a custom-op hook inside a serving framework whose caching allocator owns all device
// memory (a raw cudaMalloc there can fail or fragment the pool), or a latency-critical thread that must
// not pay the device-wide synchronisation cudaMalloc / cudaFree imply.  For them the token-chunk partials
// of the Gram kernels live in a fixed array that is part of the library image: kStaticScratchBytes of
// device memory on every GPU that loads the library, held until the process exits.
#include <mutex>

#include "common.cuh"

namespace uncomp {

constexpr size_t kPartialLen = (size_t)kD * kD + kD;                  // one chunk partial: G (d*d) and s (d)
constexpr size_t kStaticScratchBytes = 32 * kPartialLen * sizeof(double);   // 4,227,072 bytes (4.03 MiB)

// Partials of every (unit, chunk) of the call in progress, then one status word.  Shared by all calls.
static __device__ __align__(256) unsigned char g_gram_scratch[kStaticScratchBytes + 256];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_ptr[kMaxDevices] = {};   // device address of g_gram_scratch per device, resolved once
}  // namespace

// The array's name is only a host-side handle; kernels need the device address, which the runtime
// resolves per device (the device must be current).
static cudaError_t scratch_address(void **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_gram_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace uncomp

using namespace uncomp;

extern "C" int uncomp_gram_static(const uncomp_shape *shape, const void *d_K, uncomp_strides sK, double *d_gram,
                                  void *stream) {
    if (!shape || !d_K || !d_gram) return UNCOMP_E_NULL;
    if (uncomp_workspace_bytes(shape) == 0) return UNCOMP_E_SHAPE;
    if (reinterpret_cast<uintptr_t>(d_K) & 15u) return UNCOMP_E_ALIGN;
    const int64_t eb = shape->dtype == UNCOMP_FP32 ? 4 : 2;
    const int64_t st[4] = {sK.sB, sK.sL, sK.sH, sK.sN};
    for (int i = 0; i < 4; ++i) {
        if (st[i] < 0) return UNCOMP_E_SHAPE;
        if ((st[i] * eb) % 16 != 0) return UNCOMP_E_ALIGN;
    }
    if (sK.sN < shape->d) return UNCOMP_E_SHAPE;
    Plan p = make_plan(*shape);
    const size_t acc = shape->dtype == UNCOMP_FP32 ? sizeof(double) : sizeof(float);
    const size_t slots = kStaticScratchBytes / (kPartialLen * acc);      // partials the array holds: 64 or 32
    if ((size_t)p.units > slots) return UNCOMP_E_LIMIT;                  // not even one partial per unit
    if ((size_t)p.units * p.gram_splits > slots) {
        // fewer, longer token chunks than the workspace entry point would use, so that the partials fit
        const int splits = (int)(slots / p.units);
        const int chunk = ((shape->N + splits - 1) / splits + 127) / 128 * 128;
        p.gram_chunk = chunk;
        p.gram_splits = (shape->N + chunk - 1) / chunk;
    }

    void *scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return UNCOMP_E_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t *d_status = reinterpret_cast<uint32_t *>(static_cast<unsigned char *>(scratch) + kStaticScratchBytes);
    // The array keeps whatever the previous call left.  The partials are fully overwritten by this call's
    // kernels before they are read; only the status word has to start at zero.
    if (cudaMemsetAsync(d_status, 0, sizeof(uint32_t), s) != cudaSuccess) return UNCOMP_E_CUDA;
    const UnitAddr addr = make_addr(*shape, sK);
    cudaError_t e = shape->dtype == UNCOMP_BF16 ? launch_gram_tc(p, d_K, addr, scratch, d_status, s)
                                                : launch_gram_simt(p, d_K, addr, scratch, s);
    if (e != cudaSuccess) return UNCOMP_E_CUDA;
    e = launch_gram_reduce(p, scratch, d_gram, s);
    return e == cudaSuccess ? UNCOMP_OK : UNCOMP_E_CUDA;
}

extern "C" size_t uncomp_gram_static_max_bytes(void) { return kStaticScratchBytes; }
