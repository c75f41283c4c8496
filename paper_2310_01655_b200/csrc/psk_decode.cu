// Recurrent form of causal Polysketch attention: one new token per (batch, head) per call.
// lt(phi'(Q) phi'(K)^T) [V | 1] row by row is a running state (the "linear transformer" view
// the paper's Section 3 starts from; Section 3.1's Z_l is this state at block boundaries):
//   S_t = S_{t-1} + phi'(k_t) [v_t | 1]^T          (r^2 x 65, fp32, kept by the caller)
//   N_t = phi'(q_t)^T S_t,   d_t = 1 + N_t[64],   o_t = N_t[:64] / d_t
// so inference costs O(r^2 h) per token whatever the context length.  The step is bound by
// reading and writing the state once: one CTA per head streams it with coalesced rows.
#include "psk_internal.cuh"

namespace psk {
namespace {

constexpr int kCols = 65;            // [v | 1]
constexpr int kSplit = 8;            // feature rows are dealt to eight thread groups
constexpr int kBatch = 8;            // state rows a thread has in flight at once
constexpr int kThreads = kCols * kSplit;

template <typename T, int R>
__global__ void __launch_bounds__(kThreads)
decode_step_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                   const T* __restrict__ G1, const T* __restrict__ G2, int g_heads, int H,
                   float* __restrict__ state, T* __restrict__ o, float* __restrict__ denom) {
    __shared__ float sx[2][64], sm[2][R], sv[kCols];
    __shared__ double part[kSplit][kCols];
    const int bh = blockIdx.x, tid = threadIdx.x;
    const int g = g_heads == 1 ? 0 : bh % H;
    if (tid < 64) {
        sx[0][tid] = ldf(q + (size_t)bh * 64 + tid);
        sx[1][tid] = ldf(k + (size_t)bh * 64 + tid);
        sv[tid] = ldf(v + (size_t)bh * 64 + tid);
    }
    if (tid == 64) sv[64] = 1.f;
    __syncthreads();
    // half sketches m(q_t), m(k_t) (Algorithm 1, degree-2 level)
    if (tid < 2 * R) {
        const int w = tid / R, c = tid % R;
        const T* g1 = G1 + (size_t)g * 64 * R;
        const T* g2 = G2 + (size_t)g * 64 * R;
        float a1 = 0.f, a2 = 0.f;
        for (int t = 0; t < 64; ++t) {
            a1 = fmaf(sx[w][t], ldf(g1 + t * R + c), a1);
            a2 = fmaf(sx[w][t], ldf(g2 + t * R + c), a2);
        }
        sm[w][c] = a1 * a2 * rsqrtf((float)R);
    }
    __syncthreads();
    // state rows f = a r + b (the Kronecker order of Section 1.2); thread = (column, row group)
    const int c = tid % kCols, fy = tid / kCols;
    float* S = state + (size_t)bh * R * R * kCols;
    const float vc = sv[c];
    // (the sum over the r^2 features cancels heavily -- it equals a square of a short sum -- and
    // the kernel is bound by the state's bytes, so the few accumulations run in double)
    double acc = 0.0;
    static_assert((R * R) % (kSplit * kBatch) == 0, "whole batches of state rows per thread");
    for (int f0 = fy; f0 < R * R; f0 += kSplit * kBatch) {
        float s[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) s[j] = S[(size_t)(f0 + j * kSplit) * kCols + c];     // all loads first
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int f = f0 + j * kSplit, a = f / R, b = f % R;
            s[j] = fmaf(sm[1][a] * sm[1][b], vc, s[j]);
            S[(size_t)f * kCols + c] = s[j];
            acc += (double)(sm[0][a] * sm[0][b]) * (double)s[j];
        }
    }
    part[fy][c] = acc;
    __syncthreads();
    if (tid < kCols) {
        double nsum = 0.0;
#pragma unroll
        for (int i = 0; i < kSplit; ++i) nsum += part[i][tid];
        part[0][tid] = nsum;
    }
    __syncthreads();
    const float d = 1.f + (float)part[0][64];
    if (tid < 64) stf(o + (size_t)bh * 64 + tid, (float)part[0][tid] / d);
    if (tid == 64 && denom != nullptr) denom[bh] = d;
}

bool decode_shape_ok(const psk_shape* sh) {
    return sh != nullptr && (sh->dtype == PSK_F32 || sh->dtype == PSK_BF16) && sh->B > 0 && sh->H > 0 &&
           (int64_t)sh->B * sh->H < ((int64_t)1 << 31) && (sh->g_heads == 1 || sh->g_heads == sh->H);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
cudaError_t launch(const psk_shape* sh, const void* q, const void* k, const void* v, const void* G1, const void* G2,
                   float* state, void* o, float* denom, cudaStream_t s) {
    const int bh = sh->B * sh->H;
#define PSK_DEC(R)                                                                                              \
    decode_step_kernel<T, R><<<bh, kThreads, 0, s>>>((const T*)q, (const T*)k, (const T*)v, (const T*)G1,     \
                                                    (const T*)G2, sh->g_heads, sh->H, state, (T*)o, denom)
    prof_begin("decode_step_kernel", s);
    switch (sh->r) {
        case 16: PSK_DEC(16); break;
        case 32: PSK_DEC(32); break;
        default: PSK_DEC(64); break;
    }
    prof_end(s);
#undef PSK_DEC
    return cudaGetLastError();
}

}  // namespace
}  // namespace psk

using namespace psk;

extern "C" {

size_t psk_decode_state_bytes(const psk_shape* shape) {
    if (!decode_shape_ok(shape) || (shape->r != 16 && shape->r != 32 && shape->r != 64)) return 0;
    return (size_t)shape->B * shape->H * shape->r * shape->r * kCols * sizeof(float);
}

int psk_decode_step(const psk_shape* shape, const void* q, const void* k, const void* v, const void* G1,
                    const void* G2, float* state, void* o, float* denom, void* stream) {
    if (shape == nullptr) return PSK_ERR_INVALID_ARG;
    if (shape->dtype != PSK_F32 && shape->dtype != PSK_BF16) return PSK_ERR_INVALID_ARG;
    if (!decode_shape_ok(shape)) return PSK_ERR_SHAPE;
    if (shape->p != 4 || shape->h != 64 || (shape->r != 16 && shape->r != 32 && shape->r != 64) || shape->flags != 0)
        return PSK_ERR_UNSUPPORTED;
    if (!q || !k || !v || !G1 || !G2 || !state || !o) return PSK_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(G1) || !aligned16(G2) || !aligned16(state) ||
        !aligned16(o))
        return PSK_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    const cudaError_t e = shape->dtype == PSK_BF16
                              ? launch<__nv_bfloat16>(shape, q, k, v, G1, G2, state, o, denom, s)
                              : launch<float>(shape, q, k, v, G1, G2, state, o, denom, s);
    return e == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

}  // extern "C"
