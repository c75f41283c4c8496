// Internal declarations shared by the translation units of libpsk (not installed).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "psk.h"

namespace psk {

// Validated problem description handed to the launchers.
struct Dims {
    int B, H, n, h, r, b, t;          // t = n / b blocks per head (Section 3.1)
    int p;                            // degree: 4, or 2 (no sketch: the half sketch is the row itself, r = h)
    int64_t sb, sh, sn;               // element strides of the [B,H,n,h] tensors
    int g_heads;                      // 1 or H
    bool bf16;                        // storage type
    bool keep_states;                 // PSK_FLAG_KEEP_STATES
    bool local;                       // PSK_FLAG_LOCAL_EXACT
    bool noncausal;                   // PSK_FLAG_NONCAUSAL: no lt(), one global state per head
    int seq_segments;                 // runs a head's sequence is cut into for the state scan; 0 = library's choice
    // tensor-core kernels: the tensors they "sketch" already hold the half sketch (tc_common.cuh,
    // read_half_sketch); `xsb, xsh, xsn` are the strides of those tensors and of their gradients
    bool sketch_linear = false;
    int64_t xsb = 0, xsh = 0, xsn = 0;
    // given half sketches WITH exact same-block weights: the raw rows (strides sb, sh, sn) next to
    // the half sketches, and where the same-block part of their gradients goes (contiguous
    // [B,H,n,64] bf16); the sketch part of the gradient goes to the tensors "dQ", "dK" as always
    const void* rawQ = nullptr;
    const void* rawK = nullptr;
    void* rawdQ = nullptr;
    void* rawdK = nullptr;
    // learnable sketch (Algorithm 2): the half sketch comes from two dense networks instead of G1, G2
    bool learned = false;
    const float* lparams = nullptr;   // packed parameters of both networks (psk_learned.cu)
    float* dlparams = nullptr;        // their gradients (backward only)
    int BH() const { return B * H; }
};

constexpr size_t kAlign = 256;
constexpr size_t kStatusBytes = 256;  // first bytes of every workspace: device status word(s)

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Scratch layout of the CUDA-core path (all fp32).
struct CcWorkspace {
    size_t status, Mq, Mk, Vt, Zst, E, Rst, dMq, dMk, dXq, dXk, total;
};
CcWorkspace cc_workspace(const Dims& d, bool backward);

// CUDA-core (fp32 arithmetic) launchers.  Each returns a cudaError_t from the launches
// and adds the number of kernels it enqueued to *launches.
cudaError_t cc_sketch(const Dims& d, const void* X, const void* G1, const void* G2,
                      float* M_out, float* Phi_out, cudaStream_t s, int* launches);
cudaError_t cc_fwd(const Dims& d, const void* Q, const void* K, const void* V,
                   const void* G1, const void* G2, void* O, float* denom,
                   char* ws, cudaStream_t s, int* launches);
cudaError_t cc_bwd(const Dims& d, const void* Q, const void* K, const void* V,
                   const void* G1, const void* G2, const void* O, const float* denom,
                   const void* dO, void* dQ, void* dK, void* dV,
                   char* ws, cudaStream_t s, int* launches);

// Learnable sketch (CUDA cores): M = sqrt(r) tanh(f1(x) * f2(x) / sqrt(r)) and its backward
// (dX = chain rule + `add`; parameter gradients are added to d.dlparams).
size_t learned_param_count(int h, int r);
cudaError_t learned_sketch(const Dims& d, const void* X, float* M, float* Phi, cudaStream_t s, int* launches);
cudaError_t learned_sketch_bwd(const Dims& d, const void* X, const float* dM, const float* add, void* dX,
                               cudaStream_t s, int* launches);

cudaError_t cc_sketch_bwd(const Dims& d, const void* X, const void* G1, const void* G2, const float* dM,
                          const float* add, void* dX, cudaStream_t s, int* launches);

// Degree 8 and the learnable sketch on the tensor cores: half sketches by their own tensor-core
// sketch kernels, attention on them by the tensor-core kernels in linear sketch mode (psk_given.cu).
bool given_supported(const Dims& d);
size_t given_workspace_bytes(const Dims& d, bool backward);
cudaError_t given_fwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                      void* O, float* denom, char* ws, cudaStream_t s, int* launches);
cudaError_t given_bwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                      const void* O, const float* denom, const void* dO, void* dQ, void* dK, void* dV, char* ws,
                      cudaStream_t s, int* launches);

// The learnable sketch's networks on the tensor cores (psk_learned_tc.cu): bf16, r <= 32.
// `prepare` once per call, `sketch` / `sketch_bwd` per tensor (they write the [hi | lo] rows the
// attention kernels read, and take their gradient), `finish` once after the last sketch_bwd.
bool learned_tc_supported(const Dims& d);
size_t learned_tc_workspace_bytes(const Dims& d, bool backward);
cudaError_t learned_tc_prepare(const Dims& d, bool backward, char* ws, cudaStream_t s, int* launches);
cudaError_t learned_tc_sketch(const Dims& d, const void* X, void* S, char* ws, int* status, cudaStream_t s, int* launches);
cudaError_t learned_tc_sketch_bwd(const Dims& d, const void* X, const void* dS, const void* add, void* dX, char* ws,
                                  int* status, cudaStream_t s, int* launches);
cudaError_t learned_tc_finish(const Dims& d, char* ws, cudaStream_t s, int* launches);

// Degree 8's half sketch on the tensor cores (psk_sketch8_tc.cu): bf16, r <= 32.  `prepare` once per
// call; `fwd` writes the [hi | lo] rows the attention kernels read, `bwd` takes their gradient.
bool sketch8_tc_supported(const Dims& d);
size_t sketch8_tc_bank_bytes(const Dims& d);
cudaError_t sketch8_tc_prepare(const Dims& d, const void* G1, const void* G2, char* bank, cudaStream_t s, int* launches);
cudaError_t sketch8_tc_fwd(const Dims& d, const void* X, void* S, char* bank, int* status, cudaStream_t s, int* launches);
cudaError_t sketch8_tc_bwd(const Dims& d, const void* X, const void* dS, void* dX, char* bank, int* status, cudaStream_t s,
                           int* launches);

// Tensor-core (bf16 operands, fp32 accumulation) launchers.
size_t tc_workspace_bytes(const Dims& d, bool backward);
bool tc_supported(const Dims& d, bool backward);
cudaError_t tc_fwd(const Dims& d, const void* Q, const void* K, const void* V,
                   const void* G1, const void* G2, void* O, float* denom,
                   char* ws, cudaStream_t s, int* launches);
cudaError_t tc_bwd(const Dims& d, const void* Q, const void* K, const void* V,
                   const void* G1, const void* G2, const void* O, const float* denom,
                   const void* dO, void* dQ, void* dK, void* dV,
                   char* ws, cudaStream_t s, int* launches);

// Optional per-kernel timing (psk_profile_*): when enabled, each launch is bracketed by
// CUDA events on its own stream; disabled, these are no-ops.
void prof_begin(const char* name, cudaStream_t s);
void prof_end(cudaStream_t s);

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

}  // namespace psk
