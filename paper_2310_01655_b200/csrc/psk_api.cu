// C ABI of libpsk: argument validation and dispatch.  See include/psk.h for the contract.
#include "psk_internal.cuh"
#include "tc_features.cuh"

#include <string.h>
#include <string>
#include <vector>

using namespace psk;

namespace psk {
namespace {
struct ProfRec { const char* name; cudaEvent_t a, b; };
bool g_prof_on = false;
std::vector<ProfRec> g_prof;
}  // namespace
void prof_begin(const char* name, cudaStream_t s) {
    if (!g_prof_on) return;
    ProfRec r{name, nullptr, nullptr};
    if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
    cudaEventRecord(r.a, s);
    g_prof.push_back(r);
}
void prof_end(cudaStream_t s) {
    if (!g_prof_on || g_prof.empty()) return;
    cudaEventRecord(g_prof.back().b, s);
}
}  // namespace psk

namespace {

thread_local int g_last_launches = 0;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates a shape and fills Dims.  Returns PSK_OK or the error the header documents.
int make_dims(const psk_shape* sh, Dims* d) {
    if (sh == nullptr) return PSK_ERR_INVALID_ARG;
    if (sh->dtype != PSK_F32 && sh->dtype != PSK_BF16) return PSK_ERR_INVALID_ARG;
    if (sh->path < PSK_PATH_AUTO || sh->path > PSK_PATH_TENSOR_CORES) return PSK_ERR_INVALID_ARG;
    if (sh->flags & ~(int32_t)(PSK_FLAG_KEEP_STATES | PSK_FLAG_LOCAL_EXACT | PSK_FLAG_NONCAUSAL)) return PSK_ERR_INVALID_ARG;
    if (sh->B <= 0 || sh->H <= 0 || sh->n <= 0 || sh->b <= 0) return PSK_ERR_SHAPE;
    if ((sh->p != 4 && sh->p != 2 && sh->p != 8) || sh->h != 64) return PSK_ERR_UNSUPPORTED;
    // exact same-block weights are built for degree 4 (and are what degree 2 computes anyway)
    if (sh->p == 8 && (sh->flags & PSK_FLAG_LOCAL_EXACT)) return PSK_ERR_UNSUPPORTED;
    if (sh->r != 16 && sh->r != 32 && sh->r != 64) return PSK_ERR_UNSUPPORTED;
    if (sh->p == 2 && sh->r != sh->h) return PSK_ERR_UNSUPPORTED;      // p = 2: M = X, so r is h
    if (sh->b % 128 != 0 || sh->n % sh->b != 0) return PSK_ERR_SHAPE;
    if (sh->g_heads != 1 && sh->g_heads != sh->H) return PSK_ERR_SHAPE;
    if (sh->stride_n < sh->h || sh->stride_h <= 0 || sh->stride_b <= 0) return PSK_ERR_SHAPE;
    if ((int64_t)sh->B * sh->H * sh->n >= (int64_t)1 << 31) return PSK_ERR_SHAPE;
    const int esz = sh->dtype == PSK_BF16 ? 2 : 4;
    if ((sh->stride_n * esz) % 16 || (sh->stride_h * esz) % 16 || (sh->stride_b * esz) % 16)
        return PSK_ERR_ALIGN;
    d->B = sh->B; d->H = sh->H; d->n = sh->n; d->h = sh->h; d->r = sh->r; d->b = sh->b;
    d->t = sh->n / sh->b;
    d->sb = sh->stride_b; d->sh = sh->stride_h; d->sn = sh->stride_n;
    d->xsb = d->sb; d->xsh = d->sh; d->xsn = d->sn;
    d->sketch_linear = sh->p == 2;          // degree 2: the rows are their own half sketch
    d->g_heads = sh->g_heads;
    d->bf16 = sh->dtype == PSK_BF16;
    d->keep_states = (sh->flags & PSK_FLAG_KEEP_STATES) != 0;
    d->p = sh->p;
    // p = 2 has no sketch error: the exact same-block weights are what it computes anyway
    d->local = (sh->flags & PSK_FLAG_LOCAL_EXACT) != 0 && sh->p == 4;
    d->noncausal = (sh->flags & PSK_FLAG_NONCAUSAL) != 0;
    // without the mask there are no blocks to treat exactly, and only the degree-4 tensor-core kernels serve it
    if (d->noncausal && ((sh->flags & PSK_FLAG_LOCAL_EXACT) || sh->p != 4 || sh->dtype != PSK_BF16 ||
                         sh->path == PSK_PATH_CUDA_CORES))
        return PSK_ERR_UNSUPPORTED;
    if (sh->seq_segments < 0) return PSK_ERR_INVALID_ARG;
    // runs start at block boundaries (at 128-row tiles when there is no mask and hence no block)
    if (sh->seq_segments > 1 && (d->noncausal ? sh->n / 128 : d->t) % sh->seq_segments != 0) return PSK_ERR_SHAPE;
    d->seq_segments = sh->seq_segments;
    return PSK_OK;
}

// 0 = CUDA cores, 1 = tensor cores, 2 = tensor cores on half sketches formed by sketch kernels of
// their own (degree 8, learnable sketch: psk_given.cu), <0 = error
int pick_path(const psk_shape* sh, const Dims& d, bool backward) {
    if (sh->path == PSK_PATH_CUDA_CORES) return 0;
    if (given_supported(d)) return 2;
    if (d.p == 8 || d.learned) return sh->path == PSK_PATH_TENSOR_CORES ? PSK_ERR_UNSUPPORTED : 0;
    if (sh->path == PSK_PATH_TENSOR_CORES) return (d.bf16 && tc_supported(d, backward)) ? 1 : PSK_ERR_UNSUPPORTED;
    return (d.bf16 && tc_supported(d, backward)) ? 1 : 0;
}

size_t path_workspace(int path, const Dims& d, bool backward) {
    return path == 2 ? given_workspace_bytes(d, backward)
                     : (path == 1 ? tc_workspace_bytes(d, backward) : cc_workspace(d, backward).total);
}

}  // namespace

extern "C" {

int psk_version(void) { return 200; }

const char* psk_status_string(int status) {
    switch (status) {
        case PSK_OK: return "ok";
        case PSK_ERR_INVALID_ARG: return "invalid argument (null pointer or bad enum)";
        case PSK_ERR_UNSUPPORTED: return "unsupported configuration (need p=4, p=8 or p=2 with r=h; h=64; r in {16,32,64})";
        case PSK_ERR_SHAPE: return "bad shape (need b % 128 == 0, n % b == 0, positive extents)";
        case PSK_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
        case PSK_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case PSK_ERR_CUDA: return "CUDA runtime error";
        case PSK_ERR_TIMEOUT: return "device-side bounded wait gave up";
        default: return "unknown status";
    }
}

size_t psk_workspace_bytes(const psk_shape* shape, int for_backward) {
    Dims d;
    if (make_dims(shape, &d) != PSK_OK) return 0;
    const int path = pick_path(shape, d, for_backward != 0);
    if (path < 0) return 0;
    return path_workspace(path, d, for_backward != 0);
}

int psk_sketch(const psk_shape* shape, const void* X, const void* G1, const void* G2,
               float* M_out, float* Phi_out, void* stream) {
    Dims d;
    const int st = make_dims(shape, &d);
    if (st != PSK_OK) return st;
    if (!X || !M_out || (d.p != 2 && (!G1 || !G2))) return PSK_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(G1) || !aligned16(G2) || !aligned16(M_out) || !aligned16(Phi_out))
        return PSK_ERR_ALIGN;
    int launches = 0;
    const cudaError_t e = cc_sketch(d, X, G1, G2, M_out, Phi_out, (cudaStream_t)stream, &launches);
    g_last_launches = launches;
    return e == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

int psk_causal_attn_fwd(const psk_shape* shape, const void* Q, const void* K, const void* V,
                        const void* G1, const void* G2, void* O, float* denom,
                        void* workspace, size_t workspace_bytes, void* stream) {
    Dims d;
    const int st = make_dims(shape, &d);
    if (st != PSK_OK) return st;
    if (!Q || !K || !V || !O || (d.p != 2 && (!G1 || !G2))) return PSK_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(G1) || !aligned16(G2) ||
        !aligned16(O) || !aligned16(denom))
        return PSK_ERR_ALIGN;
    const int path = pick_path(shape, d, false);
    if (path < 0) return path;
    const size_t need = psk_workspace_bytes(shape, 0);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) % kAlign))
        return PSK_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    int launches = 0;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, s);
    if (e == cudaSuccess)
        e = path == 2 ? given_fwd(d, Q, K, V, G1, G2, O, denom, (char*)workspace, s, &launches)
            : path == 1 ? tc_fwd(d, Q, K, V, G1, G2, O, denom, (char*)workspace, s, &launches)
                        : cc_fwd(d, Q, K, V, G1, G2, O, denom, (char*)workspace, s, &launches);
    g_last_launches = launches;
    return e == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

int psk_causal_attn_bwd(const psk_shape* shape, const void* Q, const void* K, const void* V,
                        const void* G1, const void* G2, const void* O, const float* denom,
                        const void* dO, void* dQ, void* dK, void* dV,
                        void* workspace, size_t workspace_bytes, void* stream) {
    Dims d;
    const int st = make_dims(shape, &d);
    if (st != PSK_OK) return st;
    if (!Q || !K || !V || !O || !denom || !dO || !dQ || !dK || !dV || (d.p != 2 && (!G1 || !G2)))
        return PSK_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(G1) || !aligned16(G2) ||
        !aligned16(O) || !aligned16(denom) || !aligned16(dO) || !aligned16(dQ) || !aligned16(dK) ||
        !aligned16(dV))
        return PSK_ERR_ALIGN;
    const int path = pick_path(shape, d, true);
    if (path < 0) return path;
    const size_t need = psk_workspace_bytes(shape, 1);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) % kAlign))
        return PSK_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    int launches = 0;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, s);
    if (e == cudaSuccess)
        e = path == 2 ? given_bwd(d, Q, K, V, G1, G2, O, denom, dO, dQ, dK, dV, (char*)workspace, s, &launches)
            : path == 1 ? tc_bwd(d, Q, K, V, G1, G2, O, denom, dO, dQ, dK, dV, (char*)workspace, s, &launches)
                        : cc_bwd(d, Q, K, V, G1, G2, O, denom, dO, dQ, dK, dV, (char*)workspace, s, &launches);
    g_last_launches = launches;
    return e == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

// ---- learnable sketch (Algorithm 2): the same calls with network parameters in place of G1, G2 ----
static int learned_dims(const psk_shape* shape, psk_shape* sh, Dims* d) {
    if (shape == nullptr) return PSK_ERR_INVALID_ARG;
    *sh = *shape;
    sh->g_heads = 1;
    if (sh->p != 4) return PSK_ERR_UNSUPPORTED;
    // (validated as a CUDA-core call; the tensor-core route below adds its own conditions)
    const int32_t want = sh->path;
    sh->path = PSK_PATH_CUDA_CORES;
    const int st = make_dims(sh, d);
    if (st != PSK_OK) return st;
    d->learned = true;
    sh->path = want;
    if (want == PSK_PATH_TENSOR_CORES && !given_supported(*d)) return PSK_ERR_UNSUPPORTED;
    return PSK_OK;
}
static bool learned_on_tc(const psk_shape& sh, const Dims& d) { return sh.path != PSK_PATH_CUDA_CORES && given_supported(d); }

size_t psk_learned_param_count(int h, int r) {
    if (h != 64 || (r != 16 && r != 32 && r != 64)) return 0;
    return learned_param_count(h, r);
}

size_t psk_learned_workspace_bytes(const psk_shape* shape, int for_backward) {
    psk_shape sh; Dims d;
    if (learned_dims(shape, &sh, &d) != PSK_OK) return 0;
    return learned_on_tc(sh, d) ? given_workspace_bytes(d, for_backward != 0) : cc_workspace(d, for_backward != 0).total;
}

int psk_learned_sketch(const psk_shape* shape, const void* X, const float* params, float* M_out, float* Phi_out,
                       void* stream) {
    psk_shape sh; Dims d;
    const int st = learned_dims(shape, &sh, &d);
    if (st != PSK_OK) return st;
    if (!X || !params || !M_out) return PSK_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(params) || !aligned16(M_out) || !aligned16(Phi_out)) return PSK_ERR_ALIGN;
    d.lparams = params;
    int launches = 0;
    const cudaError_t e = cc_sketch(d, X, nullptr, nullptr, M_out, Phi_out, (cudaStream_t)stream, &launches);
    g_last_launches = launches;
    return e == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

int psk_learned_attn_fwd(const psk_shape* shape, const void* Q, const void* K, const void* V, const float* params,
                         void* O, float* denom, void* workspace, size_t workspace_bytes, void* stream) {
    psk_shape sh; Dims d;
    const int st = learned_dims(shape, &sh, &d);
    if (st != PSK_OK) return st;
    if (!Q || !K || !V || !O || !params) return PSK_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(params) || !aligned16(O) || !aligned16(denom))
        return PSK_ERR_ALIGN;
    const bool tcp = learned_on_tc(sh, d);
    const size_t need = tcp ? given_workspace_bytes(d, false) : cc_workspace(d, false).total;
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) % kAlign)) return PSK_ERR_WORKSPACE;
    d.lparams = params;
    cudaStream_t s = (cudaStream_t)stream;
    int launches = 0;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, s);
    if (e == cudaSuccess)
        e = tcp ? given_fwd(d, Q, K, V, nullptr, nullptr, O, denom, (char*)workspace, s, &launches)
                : cc_fwd(d, Q, K, V, nullptr, nullptr, O, denom, (char*)workspace, s, &launches);
    g_last_launches = launches;
    return e == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

int psk_learned_attn_bwd(const psk_shape* shape, const void* Q, const void* K, const void* V, const float* params,
                         const void* O, const float* denom, const void* dO, void* dQ, void* dK, void* dV,
                         float* dparams, void* workspace, size_t workspace_bytes, void* stream) {
    psk_shape sh; Dims d;
    const int st = learned_dims(shape, &sh, &d);
    if (st != PSK_OK) return st;
    if (!Q || !K || !V || !O || !denom || !dO || !dQ || !dK || !dV || !params || !dparams) return PSK_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(params) || !aligned16(O) || !aligned16(denom) ||
        !aligned16(dO) || !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) || !aligned16(dparams))
        return PSK_ERR_ALIGN;
    const bool tcp = learned_on_tc(sh, d);
    const size_t need = tcp ? given_workspace_bytes(d, true) : cc_workspace(d, true).total;
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) % kAlign)) return PSK_ERR_WORKSPACE;
    d.lparams = params;
    d.dlparams = dparams;
    cudaStream_t s = (cudaStream_t)stream;
    int launches = 0;
    cudaError_t e = cudaMemsetAsync(workspace, 0, kStatusBytes, s);
    // the kernels add into the gradient array: it starts at zero
    if (e == cudaSuccess) e = cudaMemsetAsync(dparams, 0, 2 * learned_param_count(d.h, d.r) * sizeof(float), s);
    if (e == cudaSuccess)
        e = tcp ? given_bwd(d, Q, K, V, nullptr, nullptr, O, denom, dO, dQ, dK, dV, (char*)workspace, s, &launches)
                : cc_bwd(d, Q, K, V, nullptr, nullptr, O, denom, dO, dQ, dK, dV, (char*)workspace, s, &launches);
    g_last_launches = launches;
    return e == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

int psk_check(const void* workspace, void* stream) {
    if (!workspace) return PSK_ERR_INVALID_ARG;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return PSK_ERR_CUDA;
    int word = 0;
    if (cudaMemcpy(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return PSK_ERR_CUDA;
    return word == 0 ? PSK_OK : PSK_ERR_TIMEOUT;
}

int psk_last_launch_count(void) { return g_last_launches; }

int psk_profile_enable(int enable) {
    for (auto& r : g_prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    g_prof.clear();
    g_prof_on = enable != 0;
    return PSK_OK;
}

int psk_profile_count(void) { return (int)g_prof.size(); }

int psk_profile_get(int index, char* name, size_t name_cap, float* ms) {
    if (index < 0 || index >= (int)g_prof.size() || !ms) return PSK_ERR_INVALID_ARG;
    const ProfRec& r = g_prof[index];
    if (cudaEventSynchronize(r.b) != cudaSuccess) return PSK_ERR_CUDA;
    if (cudaEventElapsedTime(ms, r.a, r.b) != cudaSuccess) return PSK_ERR_CUDA;
    if (name && name_cap) { strncpy(name, r.name, name_cap - 1); name[name_cap - 1] = 0; }
    return PSK_OK;
}

}  // extern "C"

namespace {
template <int R>
int feature_table(int* a, int* b, float* w, int cap) {
    using F = psk::tc::Feat<R>;
    if (cap < F::F) return PSK_ERR_WORKSPACE;
    for (int f = 0; f < F::F; ++f) {
        if (F::kCirc) {
            const int s = 2 * (f / (2 * R)) + ((f / R) & 1);
            a[f] = f % R;
            b[f] = (a[f] + s) % R;
        } else {
            a[f] = F::a(f);
            b[f] = F::b(f);
        }
        w[f] = F::weight(f);
    }
    return F::F;
}
}  // namespace

extern "C" int psk_feature_table(int r, int* a, int* b, float* w, int cap) {
    if (!a || !b || !w) return PSK_ERR_INVALID_ARG;
    switch (r) {
        case 16: return feature_table<16>(a, b, w, cap);
        case 32: return feature_table<32>(a, b, w, cap);
        case 64: return feature_table<64>(a, b, w, cap);
    }
    return PSK_ERR_UNSUPPORTED;
}
