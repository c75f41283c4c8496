// Attention on GIVEN half sketches, on the tensor cores: degree 8 (one more level of Algorithm 1)
// and the learnable sketch (Algorithm 2) only change how the half sketch m(x) is formed; features
// m (x) m, block states and row kernels are the ones of degree 4.  So sketch kernels of their own
// (psk_sketch8_tc.cu, psk_learned_tc.cu) form m for Q and K as two bf16 terms side by side,
// [hi | lo] (64 columns, zero-padded), and the tensor-core kernels run in their "linear" sketch mode
// on those arrays in place of Q and K: their sketch GEMM against [I; I] adds the two terms back
// together in fp32 (tc_common.cuh, read_half_sketch).  Backward: the kernels return the gradient
// with respect to the [hi | lo] columns, whose first r columns are dL/dm; the existing
// sketch-backward kernels take it from there.  r <= 32 (both terms fit the 64 columns), bf16 storage.
// Exact same-block weights (learnable sketch only): the kernels also get the raw rows, for the
// same-block scores, and return those rows' same-block gradient next to the half sketch's.
#include "tc_common.cuh"

namespace psk {

namespace {

struct GivenWs { size_t tc, Mq, Mk, Sq, Sk, dSq, dSk, dXq, dXk, ltc, sk8, total; };

Dims linear_dims(const Dims& d) {
    Dims l = d;
    l.p = 4; l.learned = false; l.lparams = nullptr; l.dlparams = nullptr;
    l.local = d.local && d.learned;         // exact same-block weights: the kernels also get the raw rows
    l.sketch_linear = true;
    l.g_heads = 1;
    l.xsn = 64; l.xsh = (int64_t)d.n * 64; l.xsb = (int64_t)d.H * d.n * 64;      // [B, H, n, 64] contiguous
    return l;
}

GivenWs given_ws(const Dims& d, bool backward) {
    GivenWs w{};
    const size_t rows = (size_t)d.BH() * d.n;
    size_t off = 0;
    w.tc = off; off += align_up(tc_workspace_bytes(linear_dims(d), backward));     // first: its status word is the call's
    if (sketch8_tc_supported(d)) {                                                  // degree 8: the sketch kernels write [hi | lo] themselves
        w.sk8 = off; off += sketch8_tc_bank_bytes(d);
    } else {
        w.Mq = off; off += align_up(rows * d.r * sizeof(float));                    // m, later dL/dm (fp32)
        w.Mk = off; off += align_up(rows * d.r * sizeof(float));
    }
    w.Sq = off; off += align_up(rows * 64 * sizeof(bf16));                          // [hi | lo]
    w.Sk = off; off += align_up(rows * 64 * sizeof(bf16));
    if (backward) {
        w.dSq = off; off += align_up(rows * 64 * sizeof(bf16));                     // gradient of the [hi | lo] columns
        w.dSk = off; off += align_up(rows * 64 * sizeof(bf16));
        if (d.local) {                                                              // same-block gradients of the raw rows
            w.dXq = off; off += align_up(rows * 64 * sizeof(bf16));
            w.dXk = off; off += align_up(rows * 64 * sizeof(bf16));
        }
    }
    if (d.learned && learned_tc_supported(d)) { w.ltc = off; off += align_up(learned_tc_workspace_bytes(d, backward)); }
    w.total = off;
    return w;
}

// one thread = 8 consecutive columns of a row of the [rows, 64] bf16 array
__global__ void __launch_bounds__(256)
split_kernel(const float* __restrict__ M, int r, size_t rows, bf16* __restrict__ S) {
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= rows * 8) return;
    const size_t row = e / 8;
    const int c0 = (int)(e % 8) * 8;
    uint32_t pk[4];
#pragma unroll
    for (int j = 0; j < 8; j += 2) {
        float x[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int c = c0 + j + q;
            float v = 0.f;
            if (c < 2 * r) {
                const float m = M[row * r + (c % r)];
                const float hi = __bfloat162float(__float2bfloat16_rn(m));
                v = c < r ? hi : m - hi;
            }
            x[q] = v;
        }
        pk[j / 2] = tc::pack_bf16(x[0], x[1]);
    }
    *reinterpret_cast<uint4*>(S + row * 64 + c0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

// dL/dm = the first r columns of the gradient of the [hi | lo] columns (m = hi + lo)
__global__ void __launch_bounds__(256)
unsplit_kernel(const bf16* __restrict__ dS, int r, size_t rows, float* __restrict__ dM) {
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= rows * r) return;
    dM[e] = __bfloat162float(dS[(e / r) * 64 + (e % r)]);
}

cudaError_t half_sketches(const Dims& d, const void* Q, const void* K, const void* G1, const void* G2, char* ws,
                          const GivenWs& w, bool backward, cudaStream_t s, int* launches) {
    const size_t rows = (size_t)d.BH() * d.n;
    const void* X[2] = {Q, K};
    const size_t mo[2] = {w.Mq, w.Mk}, so[2] = {w.Sq, w.Sk};
    const bool nets_on_tc = d.learned && learned_tc_supported(d);
    if (nets_on_tc) PSK_TRY(learned_tc_prepare(d, backward, ws + w.ltc, s, launches));
    if (sketch8_tc_supported(d)) {
        PSK_TRY(sketch8_tc_prepare(d, G1, G2, ws + w.sk8, s, launches));
        for (int i = 0; i < 2; ++i)
            PSK_TRY(sketch8_tc_fwd(d, X[i], ws + so[i], ws + w.sk8, reinterpret_cast<int*>(ws + w.tc), s, launches));
        return cudaSuccess;
    }
    for (int i = 0; i < 2; ++i) {
        float* M = reinterpret_cast<float*>(ws + mo[i]);
        if (nets_on_tc) PSK_TRY(learned_tc_sketch(d, X[i], M, ws + w.ltc, reinterpret_cast<int*>(ws + w.tc), s, launches));
        else PSK_TRY(cc_sketch(d, X[i], G1, G2, M, nullptr, s, launches));
        prof_begin("split_kernel", s);
        split_kernel<<<(unsigned)((rows * 8 + 255) / 256), 256, 0, s>>>(M, d.r, rows, reinterpret_cast<bf16*>(ws + so[i]));
        prof_end(s);
        ++*launches;
        PSK_TRY(cudaGetLastError());
    }
    return cudaSuccess;
}

}  // namespace

bool given_supported(const Dims& d) {
    // exact same-block weights: only with the learnable sketch on the tensor-core networks (the
    // same-block gradient of the raw rows joins the networks' gradient there)
    return d.bf16 && (d.p == 8 || d.learned) && d.r <= 32 && !d.noncausal &&
           (!d.local || (d.learned && learned_tc_supported(d))) && tc_supported(linear_dims(d), false);
}

size_t given_workspace_bytes(const Dims& d, bool backward) { return given_ws(d, backward || d.keep_states).total; }

cudaError_t given_fwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                      void* O, float* denom, char* ws, cudaStream_t s, int* launches) {
    const GivenWs w = given_ws(d, d.keep_states);
    PSK_TRY(half_sketches(d, Q, K, G1, G2, ws, w, false, s, launches));
    Dims l = linear_dims(d);
    l.rawQ = Q; l.rawK = K;
    return tc_fwd(l, ws + w.Sq, ws + w.Sk, V, nullptr, nullptr, O, denom, ws + w.tc, s, launches);
}

cudaError_t given_bwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                      const void* O, const float* denom, const void* dO, void* dQ, void* dK, void* dV, char* ws,
                      cudaStream_t s, int* launches) {
    const GivenWs w = given_ws(d, true);
    const size_t rows = (size_t)d.BH() * d.n;
    PSK_TRY(half_sketches(d, Q, K, G1, G2, ws, w, true, s, launches));
    Dims l = linear_dims(d);
    l.rawQ = Q; l.rawK = K;
    if (l.local) { l.rawdQ = ws + w.dXq; l.rawdK = ws + w.dXk; }
    PSK_TRY(tc_bwd(l, ws + w.Sq, ws + w.Sk, V, nullptr, nullptr, O, denom, dO, ws + w.dSq, ws + w.dSk, dV, ws + w.tc, s, launches));
    const void* X[2] = {Q, K};
    void* dX[2] = {dQ, dK};
    const size_t mo[2] = {w.Mq, w.Mk}, go[2] = {w.dSq, w.dSk}, xo[2] = {w.dXq, w.dXk};
    const bool nets_on_tc = d.learned && learned_tc_supported(d);
    if (sketch8_tc_supported(d)) {
        for (int i = 0; i < 2; ++i)
            PSK_TRY(sketch8_tc_bwd(d, X[i], ws + go[i], dX[i], ws + w.sk8, reinterpret_cast<int*>(ws + w.tc), s, launches));
        return cudaSuccess;
    }
    for (int i = 0; i < 2; ++i) {
        float* dM = reinterpret_cast<float*>(ws + mo[i]);       // m itself is no longer needed
        prof_begin("unsplit_kernel", s);
        unsplit_kernel<<<(unsigned)((rows * d.r + 255) / 256), 256, 0, s>>>(reinterpret_cast<const bf16*>(ws + go[i]), d.r, rows, dM);
        prof_end(s);
        ++*launches;
        PSK_TRY(cudaGetLastError());
        if (nets_on_tc)
            PSK_TRY(learned_tc_sketch_bwd(d, X[i], dM, l.local ? ws + xo[i] : nullptr, dX[i], ws + w.ltc, reinterpret_cast<int*>(ws + w.tc), s, launches));
        else PSK_TRY(cc_sketch_bwd(d, X[i], G1, G2, dM, nullptr, dX[i], s, launches));
    }
    if (nets_on_tc) PSK_TRY(learned_tc_finish(d, ws + w.ltc, s, launches));
    return cudaSuccess;
}

}  // namespace psk
