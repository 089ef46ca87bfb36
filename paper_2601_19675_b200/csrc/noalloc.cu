// lopro_linear_fwd_noalloc: the forward for callers that must not allocate device memory.
// The scratch the forward needs lives in a fixed array inside the library image instead of a
// caller-provided workspace.
#include "common.cuh"
#include "ptx.cuh"

namespace {

// Scratch of the no-allocation entry point.  It is part of the loaded module: every GPU that loads
// the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[LOPRO_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices];  // device address of g_noalloc_scratch, per device (0 = not looked up yet)

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel may
// use; the device address has to be asked for, once per device, with that device current.
lopro_status scratch_address(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LOPRO_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return LOPRO_ERR_UNSUPPORTED;
    void* p = __atomic_load_n(&g_scratch_ptr[dev], __ATOMIC_ACQUIRE);
    if (p == nullptr) {
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) return LOPRO_ERR_CUDA;
        __atomic_store_n(&g_scratch_ptr[dev], p, __ATOMIC_RELEASE);  // two racing threads store the same value
    }
    *out = p;
    return LOPRO_OK;
}

}  // namespace

extern "C" lopro_status lopro_linear_fwd_noalloc(const lopro_desc* desc, const void* packed, const uint16_t* x_bf16,
                                                 int64_t ldx, void* y, int64_t ldy, int32_t out_dtype, int32_t T,
                                                 void* stream) {
    if (!desc) return LOPRO_ERR_INVALID_ARG;
    if (T < 0) return LOPRO_ERR_INVALID_ARG;
    const size_t need = lopro_workspace_bytes(desc, T);
    if (need == 0) return lopro_check_desc(desc) != LOPRO_OK ? lopro_check_desc(desc) : LOPRO_ERR_INVALID_ARG;
    if (need > (size_t)LOPRO_NOALLOC_SCRATCH_BYTES) return LOPRO_ERR_BUFFER_TOO_SMALL;  // layer x tokens too large
    if (T == 0) return LOPRO_OK;
    void* scratch = nullptr;
    lopro_status st = scratch_address(&scratch);
    if (st != LOPRO_OK) return st;
    // Nothing in the scratch has to start at zero: the first kernel of the forward rewrites the status
    // word and every other region is written before it is read.
    return lopro_linear_fwd(desc, packed, x_bf16, ldx, y, ldy, out_dtype, T, scratch, (size_t)LOPRO_NOALLOC_SCRATCH_BYTES,
                            stream);
}

namespace {

// One block, one thread: a barrier that expects bytes nobody sends, the library's bounded wait, the time-out path.
__global__ void selftest_wait_kernel(int* status) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x != 0) return;
    *status = (int)LOPRO_OK;
    const uint32_t b = lopro::smem_u32(&bar);
    lopro::mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    lopro::mbar_expect_tx(b, 16);                    // one arrival, 16 bytes announced; no copy is ever issued
    if (!lopro::mbar_wait(b, 0, 1u << 12)) atomicExch(status, (int)LOPRO_ERR_TIMEOUT);
}

}  // namespace

extern "C" lopro_status lopro_selftest_wait(void* status_word, void* stream) {
    if (!status_word || ((uintptr_t)status_word % 4) != 0) return LOPRO_ERR_INVALID_ARG;
    selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((int*)status_word);
    return cudaGetLastError() == cudaSuccess ? LOPRO_OK : LOPRO_ERR_CUDA;
}
