// gka_fwd_chunked_noalloc: the chunked forward for callers that cannot hand over scratch memory.
//
// gka_fwd_chunked needs a caller-provided workspace for the cross-chunk state scan.  Some callers
// have no way to get one at the time of the call: code running inside a stream-ordered region where
// cudaMalloc is forbidden or would synchronise the device, plugins of serving runtimes that own all
// device memory and pre-plan it, interrupt-style or real-time host threads that must not enter the
// allocator, and embedders that link this library into a process without any tensor framework.
// For them this entry point keeps the scratch in a fixed array that is part of the library image.
//
// The array lives in every CUDA context that loads the library, for the life of that context, so
// it is kept small; problems whose scan needs more are rejected.  All calls on a device share the
// array: two calls must not overlap on the GPU (not even on different streams), or they race.
// Nothing in the scratch has to start at zero: every word that is read was written earlier in the
// same call, so stale contents of an earlier call are harmless.
#include <stdio.h>

#include "gka_common.cuh"

namespace {

constexpr size_t kScratchBytes = GKA_NOALLOC_SCRATCH_BYTES;

// File-scope device array.  In host code this name is only a handle for cudaGetSymbolAddress, never a
// device address: the address is looked up once per device and that pointer is what the kernels get.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_ptr[kMaxDevices] = {nullptr};

}  // namespace

extern "C" {

size_t gka_noalloc_scratch_bytes(void) { return kScratchBytes; }

gka_status gka_fwd_chunked_noalloc(const gka_desc *desc, const void *q, const void *k, const void *v,
                                   const float *gate, const float *lam, int n_iter, int chunk, void *out,
                                   float *state_out) {
    if (!desc) return GKA_ERR_NULL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GKA_ERR_CUDA;
    if (!g_scratch_ptr[dev]) {
        // First call on this device (with this device current): resolve the array's device address.
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return GKA_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    gka_desc d = *desc;
    d.workspace = g_scratch_ptr[dev];
    d.workspace_bytes = kScratchBytes;
    // gka_fwd_chunked validates every argument and returns GKA_ERR_WORKSPACE, before launching anything,
    // when gka_fwd_workspace_bytes() of this problem exceeds the built-in scratch
    return gka_fwd_chunked(&d, q, k, v, gate, lam, n_iter, chunk, out, state_out);
}

}  // extern "C"
