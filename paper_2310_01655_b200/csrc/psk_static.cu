// psk_causal_attn_fwd_static: the forward pass for callers that are not allowed to
// allocate device memory.  Its scratch is a fixed array inside the library image, so the
// call needs no workspace argument and performs no allocation of any kind.
#include "psk_internal.cuh"

#include <mutex>

using namespace psk;

#ifndef PSK_STATIC_SCRATCH_BYTES
#define PSK_STATIC_SCRATCH_BYTES (16u << 20)   /* 16 MiB, resident on every GPU that loads the library */
#endif

// File-scope scratch.  On the host this name is only a handle for the runtime's symbol
// table, never a device address: host code must go through cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[PSK_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
char* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device, resolved once per device and kept for
// the life of the process (it does not survive a cudaDeviceReset of that device).
int scratch_for_current_device(char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSK_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || p == nullptr) return PSK_ERR_CUDA;
        g_scratch_ptr[dev] = static_cast<char*>(p);
    }
    *out = g_scratch_ptr[dev];
    return PSK_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

size_t psk_static_scratch_bytes(void) { return (size_t)PSK_STATIC_SCRATCH_BYTES; }

int psk_causal_attn_fwd_static(const psk_shape* shape, const void* Q, const void* K, const void* V,
                               const void* G1, const void* G2, void* O, float* denom, void* stream) {
    if (shape == nullptr) return PSK_ERR_INVALID_ARG;
    // Same validation as the workspace-taking call, forced onto the CUDA-core kernels.
    psk_shape sh = *shape;
    sh.path = PSK_PATH_CUDA_CORES;
    const size_t need = psk_workspace_bytes(&sh, 0);
    if (need == 0) {
        // Invalid shape: let the regular entry point name the reason (it fails before any launch).
        return psk_causal_attn_fwd(&sh, Q, K, V, G1, G2, O, denom, nullptr, 0, stream);
    }
    if (!Q || !K || !V || !O || (sh.p != 2 && (!G1 || !G2))) return PSK_ERR_INVALID_ARG;   // p = 2 reads no G
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(G1) || !aligned16(G2) ||
        !aligned16(O) || !aligned16(denom))
        return PSK_ERR_ALIGN;
    if (need > (size_t)PSK_STATIC_SCRATCH_BYTES) return PSK_ERR_WORKSPACE;   // problem too large for the array
    char* scratch = nullptr;
    const int st = scratch_for_current_device(&scratch);
    if (st != PSK_OK) return st;
    // The array keeps whatever the previous call left.  Only the status word must start at
    // zero; every other region is fully written by this call's kernels before it is read.
    return psk_causal_attn_fwd(&sh, Q, K, V, G1, G2, O, denom, scratch, (size_t)PSK_STATIC_SCRATCH_BYTES, stream);
}

}  // extern "C"
