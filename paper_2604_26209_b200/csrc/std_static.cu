// std_attn_decode_static: std_attn_decode for callers that must not allocate device memory.
//
// The split-KV partials that std_attn_decode keeps in a caller-provided workspace live here in a
// fixed array inside the library's device image, so a caller that has no allocator at hand (code
// running inside a memory-pool callback, a plugin of a host application that owns all device memory,
// a process whose device heap is already committed to KV caches) can still run the comparison kernel.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kScratchBytes = 16u << 20;          // 16 MiB, held by every device that loads the library
constexpr int kMaxDevices = 64;

// File-scope device array.  In host code this name is only a handle for cudaGetSymbolAddress; the
// kernels receive the device address obtained below.
static __device__ __align__(256) unsigned char g_std_scratch[kScratchBytes];

std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the current device, looked up once per device.
int scratch_for_current_device(void** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { hpd::set_last_cuda_error(e); return HPD_E_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return HPD_E_CAPACITY;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_std_scratch);
        if (e != cudaSuccess || !p) {
            hpd::set_last_cuda_error(e);
            return HPD_E_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return HPD_OK;
}

}  // namespace

extern "C" {

size_t std_attn_decode_static_max_bytes(void) { return kScratchBytes; }

int std_attn_decode_static(const hpd_geom* geom, int max_rows, int max_seq_len, long long total_tokens, const int32_t* n_active,
                           const void* q, const void* dup_k, const void* dup_v,
                           const int64_t* seq_start, const int32_t* seq_len,
                           void* o, float* lse, void* stream)
{
    int rc = hpd::geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (max_rows < 0 || max_seq_len < 0) return HPD_E_ARG;
    if (max_rows == 0) return HPD_OK;
    const size_t need = std_workspace_bytes(geom, max_rows, max_seq_len);
    if (need > kScratchBytes) return HPD_E_WORKSPACE;      // beyond the built-in scratch: use std_attn_decode
    void* scratch = nullptr;
    rc = scratch_for_current_device(&scratch);
    if (rc != HPD_OK) return rc;
    // Every partial that the merge reads is written by the same call first, so nothing has to be cleared.
    return std_attn_decode(geom, max_rows, max_seq_len, total_tokens, n_active, q, dup_k, dup_v, seq_start, seq_len, o, lse,
                           scratch, kScratchBytes, stream);
}

}  // extern "C"
