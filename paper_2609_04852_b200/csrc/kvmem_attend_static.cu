// kvmem_view_attend_static: decode attention over the view for callers that cannot allocate.
//
// Some hosts of this library have no way to obtain device memory once they are running: an
// inference server that hands every free byte of HBM to its KV pool at start-up and runs with its
// allocator frozen, a plug-in that is only given the buffers of one request (query, view, output),
// or code on a latency path where a cudaMalloc (which synchronises the device) is not acceptable.
// kvmem_view_attend needs a split-K workspace from the caller; this variant instead keeps that
// workspace in a fixed array that is part of the library image.  The paper has no counterpart.
//
// The array is a file-scope __device__ object: every GPU that loads the library carries it
// (kStaticAttendBytes, about 4 MiB) until the process exits.  In host code its name is only a
// stand-in, not a device address, so the address is looked up once per device with
// cudaGetSymbolAddress while that device is current, and that pointer is what the kernels receive.
#include <mutex>

#include "kvmem_internal.cuh"

namespace kvmem {

constexpr int kStaticAttendMaxHeads = 8;                       // n_sessions * n_layers * n_kv_heads
// split-K partials for 8 heads: 64 splits x 16 rows x (128 fp32 outputs + one (max, sum) pair)
constexpr size_t kStaticAttendBytes = (size_t)kStaticAttendMaxHeads * 64 * 16 * 128 * sizeof(float) +
                                      (size_t)kStaticAttendMaxHeads * 64 * 16 * sizeof(float2);

static __device__ __align__(256) unsigned char g_attend_scratch[kStaticAttendBytes];

static void* g_scratch_ptr[kMaxDevices] = {};
static std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device (looked up on first use).
static cudaError_t scratch_for_current_device(int device, void** out) {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_attend_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[device] = p;
    }
    *out = g_scratch_ptr[device];
    return cudaSuccess;
}

}  // namespace kvmem

using namespace kvmem;

extern "C" int kvmem_view_attend_static(kvmem_pool_t* pool, int32_t n_sessions, const void* q, int32_t n_q_tokens,
                                        const void* view_k, const void* view_v, int32_t view_cap_tokens,
                                        const int32_t* n_sel, float scale, float* out, float* lse, void* stream) {
    if (!pool || pool->magic != kMagic) { set_error("pool handle is null or stale"); return KVMEM_E_STATE; }
    if (n_sessions < 1) { set_error("n_sessions must be positive"); return KVMEM_E_INVALID; }
    const long long heads = (long long)n_sessions * pool->cfg.n_layers * pool->cfg.n_kv_heads;
    if (heads > kStaticAttendMaxHeads) {
        set_error("kvmem_view_attend_static handles at most %d (session, layer, KV head) triples per call, got %lld; "
                  "use kvmem_view_attend with a caller workspace for more",
                  kStaticAttendMaxHeads, heads);
        return KVMEM_E_CAPACITY;
    }
    size_t need = kvmem_attend_workspace_bytes(&pool->cfg, n_sessions, n_q_tokens > 0 ? n_q_tokens : 1);
    if (need == 0 || need > kStaticAttendBytes) {
        set_error("built-in scratch holds %zu bytes, this call needs %zu", kStaticAttendBytes, need);
        return KVMEM_E_CAPACITY;
    }
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) { set_error("cudaGetDevice: %s", cudaGetErrorString(e)); return KVMEM_E_CUDA; }
    if (device != pool->cfg.device || device < 0 || device >= kMaxDevices) {
        set_error("the pool lives on device %d but device %d is current", pool->cfg.device, device);
        return KVMEM_E_STATE;
    }
    void* scratch = nullptr;
    e = scratch_for_current_device(device, &scratch);
    if (e != cudaSuccess) { set_error("cudaGetSymbolAddress: %s", cudaGetErrorString(e)); return KVMEM_E_CUDA; }
    // Nothing in the scratch has to start at zero: the split kernel overwrites every slot that the
    // merge kernel reads, so whatever the previous call left behind is never observed.
    return kvmem_view_attend(pool, n_sessions, q, n_q_tokens, view_k, view_v, view_cap_tokens, n_sel, scale, out, lse,
                             scratch, kStaticAttendBytes, stream);
}
