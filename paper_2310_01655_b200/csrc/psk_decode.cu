// Recurrent form of causal Polysketch attention: one new token per (batch, head) per call.
// lt(phi'(Q) phi'(K)^T) [V | 1] row by row is a running state (the "linear transformer" view
// the paper's Section 3 starts from; Section 3.1's Z_l is this state at block boundaries):
//   S_t = S_{t-1} + phi'(k_t) [v_t | 1]^T          (r^2 x 65, fp32, kept by the caller)
//   N_t = phi'(q_t)^T S_t,   d_t = 1 + N_t[64],   o_t = N_t[:64] / d_t
// so inference costs O(r^2 h) per token whatever the context length.  The step is bound by
// reading and writing the state once.  A cluster of four CTAs per head streams a quarter of the
// state rows each (coalesced, eight rows in flight per thread) and the partial sums of
// phi'(q_t)^T S_t meet in the first CTA's shared memory: four times as many CTAs as heads, so
// that a few hundred heads still fill 148 SMs evenly.
#include "psk_internal.cuh"

#include <cooperative_groups.h>

namespace psk {
namespace {

constexpr int kCols = 65;            // [v | 1]
constexpr int kSplit = 4;            // a CTA's feature rows are dealt to four thread groups
constexpr int kBatch = 8;            // state rows a thread has in flight at once
constexpr int kCluster = 4;          // CTAs per head
constexpr int kThreads = kCols * kSplit;

template <typename T, int R>
__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads)
decode_step_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                   const T* __restrict__ G1, const T* __restrict__ G2, int g_heads, int H,
                   float* __restrict__ state, T* __restrict__ o, float* __restrict__ denom) {
    constexpr int kRowsPerCta = R * R / kCluster, kStep = kSplit * kBatch;
    static_assert(kRowsPerCta % kStep == 0, "whole batches of state rows per thread");
    __shared__ float sx[2][64], sm[2][R], sv[kCols], sphi[2][kRowsPerCta];
    __shared__ double part[kSplit][kCols];
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int cr = (int)cluster.block_rank();
    const int bh = blockIdx.x / kCluster, tid = threadIdx.x;
    const int g = g_heads == 1 ? 0 : bh % H;
    // state rows f = a r + b (the Kronecker order of Section 1.2); thread = (column, row group).
    // The first batch of rows is requested before anything else: it is in flight while the half
    // sketches are computed.
    const int c = tid % kCols, fy = tid / kCols;
    float* S = state + ((size_t)bh * R * R + (size_t)cr * kRowsPerCta) * kCols;      // this CTA's rows
    float cur[kBatch];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) cur[j] = S[(size_t)(fy + j * kSplit) * kCols + c];
    if (tid < 64) {
        sx[0][tid] = ldf(q + (size_t)bh * 64 + tid);
        sx[1][tid] = ldf(k + (size_t)bh * 64 + tid);
        sv[tid] = ldf(v + (size_t)bh * 64 + tid);
    }
    if (tid == 64) sv[64] = 1.f;
    __syncthreads();
    // half sketches m(q_t), m(k_t) (Algorithm 1, degree-2 level): four threads per entry, 16 of the
    // 64 terms each, so that no warp waits long at the barrier behind a few busy ones
    if (tid < 256) {                                  // (whole warps: the shuffles below need their four lanes)
        const T* g1 = G1 + (size_t)g * 64 * R;
        const T* g2 = G2 + (size_t)g * 64 * R;
        for (int base = tid; base < 8 * R; base += 256) {
            const int e = base / 4, sub = base % 4, w = e / R, cc = e % R;
            float a1 = 0.f, a2 = 0.f;
#pragma unroll 4
            for (int t = sub * 16; t < sub * 16 + 16; ++t) {
                a1 = fmaf(sx[w][t], ldf(g1 + t * R + cc), a1);
                a2 = fmaf(sx[w][t], ldf(g2 + t * R + cc), a2);
            }
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a2 += __shfl_xor_sync(0xffffffffu, a2, 1);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 2); a2 += __shfl_xor_sync(0xffffffffu, a2, 2);
            if (sub == 0) sm[w][cc] = a1 * a2 * rsqrtf((float)R);
        }
    }
    __syncthreads();
    // features of this CTA's rows, once: phi'(q_t)[f] and phi'(k_t)[f]
    for (int i = tid; i < kRowsPerCta; i += kThreads) {
        const int f = cr * kRowsPerCta + i, a = f / R, b = f % R;
        sphi[0][i] = sm[0][a] * sm[0][b];
        sphi[1][i] = sm[1][a] * sm[1][b];
    }
    __syncthreads();
    const float vc = sv[c];
    // (the sum over the r^2 features cancels heavily -- it equals a square of a short sum -- so the
    // products, rounded once to fp32, are added up in double)
    double acc = 0.0;
    for (int i0 = fy; i0 < kRowsPerCta; i0 += kStep) {
        float nxt[kBatch];
        if (i0 + kStep < kRowsPerCta) {               // next batch: requested before this one is used
#pragma unroll
            for (int j = 0; j < kBatch; ++j) nxt[j] = S[(size_t)(i0 + kStep + j * kSplit) * kCols + c];
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int i = i0 + j * kSplit;
            const float sn = fmaf(sphi[1][i], vc, cur[j]);
            S[(size_t)i * kCols + c] = sn;
            acc += (double)(sphi[0][i] * sn);
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) cur[j] = nxt[j];
    }
    part[fy][c] = acc;
    __syncthreads();
    if (tid < kCols) {
        double nsum = 0.0;
#pragma unroll
        for (int i = 0; i < kSplit; ++i) nsum += part[i][tid];
        part[0][tid] = nsum;
    }
    cluster.sync();                                   // every CTA's partial sums are in place
    if (cr == 0) {
        if (tid < kCols) {
            double nsum = part[0][tid];
            for (int rk = 1; rk < kCluster; ++rk) nsum += cluster.map_shared_rank(&part[0][0], rk)[tid];
            part[1][tid] = nsum;
        }
        __syncthreads();
        const float d = 1.f + (float)part[1][64];
        if (tid < 64) stf(o + (size_t)bh * 64 + tid, (float)part[1][tid] / d);
        if (tid == 64 && denom != nullptr) denom[bh] = d;
    }
    cluster.sync();                                   // ... and stay until the first CTA has read them
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
    decode_step_kernel<T, R><<<bh * kCluster, kThreads, 0, s>>>((const T*)q, (const T*)k, (const T*)v, (const T*)G1,     \
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
