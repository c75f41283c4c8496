// Attention on GIVEN half sketches, on the tensor cores: degree 8 (one more level of Algorithm 1)
// and the learnable sketch (Algorithm 2) only change how the half sketch m(x) is formed; features
// m (x) m, block states and row kernels are the ones of degree 4.  So sketch kernels of their own
// (psk_sketch8_tc.cu, psk_learned_tc.cu) form m for Q and K as two bf16 terms side by side,
// [hi | lo] (64 columns, zero-padded), and the tensor-core kernels run in their "linear" sketch mode
// on those arrays in place of Q and K: their sketch GEMM against [I; I] adds the two terms back
// together in fp32 (tc_common.cuh, read_half_sketch).  Backward: the kernels return the gradient
// with respect to the [hi | lo] columns, whose first r columns are dL/dm; the sketch kernels'
// backward takes it from there.  r <= 32 (both terms fit the 64 columns), bf16 storage.
// Exact same-block weights (learnable sketch only): the kernels also get the raw rows, for the
// same-block scores, and return those rows' same-block gradient next to the half sketch's.
#include "tc_common.cuh"

namespace psk {

namespace {

struct GivenWs { size_t tc, Sq, Sk, dSq, dSk, dXq, dXk, sketch, total; };

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
    // the sketch kernels' own scratch: operand banks, and for the networks one pass's activations
    w.sketch = off;
    off += d.learned ? align_up(learned_tc_workspace_bytes(d, backward)) : sketch8_tc_bank_bytes(d);
    w.total = off;
    return w;
}

// the sketch kernels' operand banks, then (unless `kept`: the forward left them in this workspace)
// the [hi | lo] rows of both tensors' half sketches
cudaError_t half_sketches(const Dims& d, const void* Q, const void* K, const void* G1, const void* G2, char* ws,
                          const GivenWs& w, bool backward, bool kept, cudaStream_t s, int* launches) {
    const void* X[2] = {Q, K};
    const size_t so[2] = {w.Sq, w.Sk};
    int* status = reinterpret_cast<int*>(ws + w.tc);
    if (d.learned) PSK_TRY(learned_tc_prepare(d, backward, ws + w.sketch, s, launches));
    else PSK_TRY(sketch8_tc_prepare(d, G1, G2, ws + w.sketch, s, launches));
    if (kept) return cudaSuccess;
    for (int i = 0; i < 2; ++i) {
        if (d.learned) PSK_TRY(learned_tc_sketch(d, X[i], ws + so[i], ws + w.sketch, status, s, launches));
        else PSK_TRY(sketch8_tc_fwd(d, X[i], ws + so[i], ws + w.sketch, status, s, launches));
    }
    return cudaSuccess;
}

}  // namespace

bool given_supported(const Dims& d) {
    // exact same-block weights: only with the learnable sketch (the same-block gradient of the raw
    // rows joins the networks' gradient there)
    if (!d.bf16 || d.noncausal || !tc_supported(linear_dims(d), false)) return false;
    return d.learned ? learned_tc_supported(d) : (sketch8_tc_supported(d) && !d.local);
}

size_t given_workspace_bytes(const Dims& d, bool backward) { return given_ws(d, backward || d.keep_states).total; }

cudaError_t given_fwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                      void* O, float* denom, char* ws, cudaStream_t s, int* launches) {
    const GivenWs w = given_ws(d, d.keep_states);
    PSK_TRY(half_sketches(d, Q, K, G1, G2, ws, w, false, false, s, launches));
    Dims l = linear_dims(d);
    l.rawQ = Q; l.rawK = K;
    return tc_fwd(l, ws + w.Sq, ws + w.Sk, V, nullptr, nullptr, O, denom, ws + w.tc, s, launches);
}

cudaError_t given_bwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                      const void* O, const float* denom, const void* dO, void* dQ, void* dK, void* dV, char* ws,
                      cudaStream_t s, int* launches) {
    const GivenWs w = given_ws(d, true);
    // PSK_FLAG_KEEP_STATES: the half sketches are part of what the forward left in the workspace
    PSK_TRY(half_sketches(d, Q, K, G1, G2, ws, w, true, d.keep_states, s, launches));
    Dims l = linear_dims(d);
    l.rawQ = Q; l.rawK = K;
    if (l.local) { l.rawdQ = ws + w.dXq; l.rawdK = ws + w.dXk; }
    PSK_TRY(tc_bwd(l, ws + w.Sq, ws + w.Sk, V, nullptr, nullptr, O, denom, dO, ws + w.dSq, ws + w.dSk, dV, ws + w.tc, s, launches));
    const void* X[2] = {Q, K};
    void* dX[2] = {dQ, dK};
    const size_t go[2] = {w.dSq, w.dSk}, xo[2] = {w.dXq, w.dXk};
    int* status = reinterpret_cast<int*>(ws + w.tc);
    for (int i = 0; i < 2; ++i) {
        if (d.learned)
            PSK_TRY(learned_tc_sketch_bwd(d, X[i], ws + go[i], l.local ? ws + xo[i] : nullptr, dX[i], ws + w.sketch, status, s, launches));
        else
            PSK_TRY(sketch8_tc_bwd(d, X[i], ws + go[i], dX[i], ws + w.sketch, status, s, launches));
    }
    if (d.learned) PSK_TRY(learned_tc_finish(d, ws + w.sketch, s, launches));
    return cudaSuccess;
}

}  // namespace psk
