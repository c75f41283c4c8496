// Learnable sketch (Algorithm 2 of the paper's appendix, "Replacing Random Projections with
// Learnable Transformations") on the CUDA cores, fp32 arithmetic.
//
//   M = sqrt(r) tanh( sqrt(1/r) [ f_1(x) * f_2(x) ] )          (degree-2 level; p = 4 attention)
// with two dense networks of equal structure and separate parameters.  Each network: layer
// normalisation of the input, dense h -> 8r, gelu, layer normalisation, dense 8r -> r, dense r -> 8r,
// gelu, dense 8r -> r.  Readings where the appendix is silent: the dense layers carry biases, each
// normalisation a learnable gain and bias with eps = 1e-6 inside the square root, gelu is
// x Phi(x), and one pair of networks serves every head (the paper shares it within a layer).
// Only the half sketch changes: features M (x) M, block states and the row kernels are the ones of
// the random sketch, so these kernels sit where sketch_kernel / sketch_bwd_kernel sit.
//
// Packed parameters of one network (fp32), in this order:
//   g0[h] c0[h] | W1[h][8r] b1[8r] | g1[8r] c1[8r] | W2[8r][r] b2[r] | W3[r][8r] b3[8r] | W4[8r][r] b4[r]
// (gain and bias of a normalisation, then row-major weight and bias of each dense layer);
// the two networks follow one another.  Parameter gradients use the same layout and are ADDED to
// (fp32 atomics, so their last bits depend on the order of arrival).
#include "psk_internal.cuh"

#define PSK_TRY_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return e_; } while (0)

namespace psk {

namespace {

constexpr int kRows = 16;                 // rows of X per CTA
constexpr int kThreads = 256;
constexpr float kLnEps = 1e-6f;

struct NetLayout {
    int h, r, m;                          // m = 8r
    int g0, c0, W1, b1, g1, c1, W2, b2, W3, b3, W4, b4, count;
    __host__ __device__ NetLayout(int h_, int r_) : h(h_), r(r_), m(8 * r_) {
        int o = 0;
        g0 = o; o += h; c0 = o; o += h;
        W1 = o; o += h * m; b1 = o; o += m;
        g1 = o; o += m; c1 = o; o += m;
        W2 = o; o += m * r; b2 = o; o += r;
        W3 = o; o += r * m; b3 = o; o += m;
        W4 = o; o += m * r; b4 = o; o += r;
        count = o;
    }
};

struct Slice {
    int H; int64_t sb, sh, sn;
    __device__ int64_t row(int bh, int i) const {
        return (int64_t)(bh / H) * sb + (int64_t)(bh % H) * sh + (int64_t)i * sn;
    }
};

__device__ __forceinline__ float gelu_f(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_grad_f(float x) {
    return 0.5f * (1.f + erff(x * 0.70710678118654752f)) + x * __expf(-0.5f * x * x) * 0.3989422804014327f;
}

// out[row][j] = sum_k in[row][k] W[k][j] + b[j]   (W row-major [K][N] in global memory)
__device__ void dense(float* out, int po, const float* in, int pi, const float* __restrict__ W,
                      const float* __restrict__ b, int K, int N) {
    for (int e = threadIdx.x; e < kRows * N; e += kThreads) {
        const int row = e / N, j = e % N;
        float acc = b[j];
        for (int k = 0; k < K; ++k) acc = fmaf(in[row * pi + k], W[(size_t)k * N + j], acc);
        out[row * po + j] = acc;
    }
}
// out[row][k] = sum_j in[row][j] W[k][j]           (back through a dense layer)
__device__ void dense_t(float* out, int po, const float* in, int pi, const float* __restrict__ W, int K, int N) {
    for (int e = threadIdx.x; e < kRows * K; e += kThreads) {
        const int row = e / K, k = e % K;
        float acc = 0.f;
        for (int j = 0; j < N; ++j) acc = fmaf(in[row * pi + j], W[(size_t)k * N + j], acc);
        out[row * po + k] = acc;
    }
}
// dW[k][j] += sum_row a[row][k] d[row][j],  db[j] += sum_row d[row][j]
__device__ void accum_dense(float* __restrict__ dW, float* __restrict__ db, const float* a, int pa, const float* d,
                            int pd, int K, int N) {
    for (int e = threadIdx.x; e < K * N; e += kThreads) {
        const int k = e / N, j = e % N;
        float acc = 0.f;
#pragma unroll
        for (int row = 0; row < kRows; ++row) acc = fmaf(a[row * pa + k], d[row * pd + j], acc);
        atomicAdd(dW + (size_t)k * N + j, acc);
    }
    for (int j = threadIdx.x; j < N; j += kThreads) {
        float acc = 0.f;
#pragma unroll
        for (int row = 0; row < kRows; ++row) acc += d[row * pd + j];
        atomicAdd(db + j, acc);
    }
}
// Layer normalisation of every row (one warp per two rows): nrm = (x - mean) / sqrt(var + eps) and
// 1 / sqrt(var + eps); z = nrm * gain + bias is formed by the users.
__device__ void layer_norm_rows(float* nrm, int pn, const float* x, int px, int N, float* rsig) {
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    for (int row = warp; row < kRows; row += kThreads / 32) {
        float s = 0.f;
        for (int j = lane; j < N; j += 32) s += x[row * px + j];
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float mu = s / (float)N;
        float v = 0.f;
        for (int j = lane; j < N; j += 32) { const float t = x[row * px + j] - mu; v = fmaf(t, t, v); }
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        const float rs = rsqrtf(v / (float)N + kLnEps);
        for (int j = lane; j < N; j += 32) nrm[row * pn + j] = (x[row * px + j] - mu) * rs;
        if (lane == 0) rsig[row] = rs;
    }
}
// Back through z = nrm * gain + bias: dx = rsig (dn - mean(dn) - nrm mean(dn nrm)), dn = dz gain;
// dgain += sum_rows dz nrm, dbias += sum_rows dz.  `d` holds dz on entry and dx on return.
__device__ void layer_norm_back(float* d, int pd, const float* nrm, int pn, const float* __restrict__ gain, int N,
                                const float* rsig, float* __restrict__ dgain, float* __restrict__ dbias) {
    for (int j = threadIdx.x; j < N; j += kThreads) {
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int row = 0; row < kRows; ++row) { a = fmaf(d[row * pd + j], nrm[row * pn + j], a); b += d[row * pd + j]; }
        atomicAdd(dgain + j, a);
        atomicAdd(dbias + j, b);
    }
    __syncthreads();
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    for (int row = warp; row < kRows; row += kThreads / 32) {
        float s1 = 0.f, s2 = 0.f;
        for (int j = lane; j < N; j += 32) {
            const float dn = d[row * pd + j] * gain[j];
            s1 += dn; s2 = fmaf(dn, nrm[row * pn + j], s2);
        }
        for (int o = 16; o > 0; o >>= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); }
        const float m1 = s1 / (float)N, m2 = s2 / (float)N, rs = rsig[row];
        for (int j = lane; j < N; j += 32)
            d[row * pd + j] = rs * (d[row * pd + j] * gain[j] - m1 - nrm[row * pn + j] * m2);
    }
}

// Shared-memory plan of one CTA (floats); pitches are odd so that column walks do not collide.
struct Plan {
    int h, r, m, ph, pr, pm;
    int X, N0, P1, N1, A2, P3, F1, F2, D8, Dr, Dh, RS0, RS1, total;
    __host__ __device__ Plan(int h_, int r_) : h(h_), r(r_), m(8 * r_), ph(h_ + 1), pr(r_ + 1), pm(8 * r_ + 1) {
        int o = 0;
        X = o; o += kRows * ph;        // input rows
        N0 = o; o += kRows * ph;       // normalised input (before gain and bias)
        P1 = o; o += kRows * pm;       // first pre-activation
        N1 = o; o += kRows * pm;       // normalised gelu(P1)
        A2 = o; o += kRows * pr;       // second hidden layer
        P3 = o; o += kRows * pm;       // third pre-activation
        F1 = o; o += kRows * pr;       // outputs of the two networks
        F2 = o; o += kRows * pr;
        D8 = o; o += kRows * pm;       // a delta of width 8r / a scratch row of that width
        Dr = o; o += kRows * pr;       // a delta of width r
        Dh = o; o += kRows * ph;       // dX accumulated over the two networks
        RS0 = o; o += kRows; RS1 = o; o += kRows;
        total = o;
    }
};

// Forward of one network on the CTA's rows: leaves N0, P1, N1, A2, P3 and writes f into `F`.
__device__ void net_forward(float* sm, const Plan& pl, const NetLayout& nl, const float* __restrict__ P, float* F) {
    layer_norm_rows(sm + pl.N0, pl.ph, sm + pl.X, pl.ph, pl.h, sm + pl.RS0);
    __syncthreads();
    // z0 = N0 * g0 + c0 goes through D8's first columns (h <= 8r)
    for (int e = threadIdx.x; e < kRows * pl.h; e += kThreads) {
        const int row = e / pl.h, k = e % pl.h;
        sm[pl.D8 + row * pl.pm + k] = fmaf(sm[pl.N0 + row * pl.ph + k], P[nl.g0 + k], P[nl.c0 + k]);
    }
    __syncthreads();
    dense(sm + pl.P1, pl.pm, sm + pl.D8, pl.pm, P + nl.W1, P + nl.b1, pl.h, pl.m);
    __syncthreads();
    for (int e = threadIdx.x; e < kRows * pl.m; e += kThreads) {
        const int row = e / pl.m, j = e % pl.m;
        sm[pl.D8 + row * pl.pm + j] = gelu_f(sm[pl.P1 + row * pl.pm + j]);
    }
    __syncthreads();
    layer_norm_rows(sm + pl.N1, pl.pm, sm + pl.D8, pl.pm, pl.m, sm + pl.RS1);
    __syncthreads();
    for (int e = threadIdx.x; e < kRows * pl.m; e += kThreads) {
        const int row = e / pl.m, j = e % pl.m;
        sm[pl.D8 + row * pl.pm + j] = fmaf(sm[pl.N1 + row * pl.pm + j], P[nl.g1 + j], P[nl.c1 + j]);      // z1
    }
    __syncthreads();
    dense(sm + pl.A2, pl.pr, sm + pl.D8, pl.pm, P + nl.W2, P + nl.b2, pl.m, pl.r);
    __syncthreads();
    dense(sm + pl.P3, pl.pm, sm + pl.A2, pl.pr, P + nl.W3, P + nl.b3, pl.r, pl.m);
    __syncthreads();
    for (int e = threadIdx.x; e < kRows * pl.m; e += kThreads) {
        const int row = e / pl.m, j = e % pl.m;
        sm[pl.D8 + row * pl.pm + j] = gelu_f(sm[pl.P3 + row * pl.pm + j]);                                 // a3
    }
    __syncthreads();
    dense(F, pl.pr, sm + pl.D8, pl.pm, P + nl.W4, P + nl.b4, pl.m, pl.r);
    __syncthreads();
}

template <typename T>
__device__ void load_rows(float* sm, const Plan& pl, Slice sl, const T* __restrict__ X, int bh, int i0) {
    for (int e = threadIdx.x; e < kRows * pl.h; e += kThreads) {
        const int row = e / pl.h, c = e % pl.h;
        sm[pl.X + row * pl.ph + c] = ldf(X + sl.row(bh, i0 + row) + c);
    }
    __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
learned_sketch_kernel(Slice sl, int n, int h, int r, const T* __restrict__ X, const float* __restrict__ params,
                      float* __restrict__ M_out, float* __restrict__ Phi_out) {
    extern __shared__ float sm[];
    const Plan pl(h, r);
    const NetLayout nl(h, r);
    const int bh = blockIdx.y, i0 = blockIdx.x * kRows;
    load_rows(sm, pl, sl, X, bh, i0);
    net_forward(sm, pl, nl, params, sm + pl.F1);
    net_forward(sm, pl, nl, params + nl.count, sm + pl.F2);
    const float sr = sqrtf((float)r), isr = rsqrtf((float)r);
    for (int e = threadIdx.x; e < kRows * r; e += kThreads) {
        const int row = e / r, j = e % r;
        const float m = sr * tanhf(sm[pl.F1 + row * pl.pr + j] * sm[pl.F2 + row * pl.pr + j] * isr);
        sm[pl.Dr + row * pl.pr + j] = m;
        M_out[((size_t)bh * n + i0 + row) * r + j] = m;
    }
    if (Phi_out != nullptr) {           // phi'(x)[a*r+b] = m_a m_b (Kronecker order of Section 1.2)
        __syncthreads();
        for (int e = threadIdx.x; e < kRows * r * r; e += kThreads) {
            const int row = e / (r * r), f = e % (r * r);
            Phi_out[((size_t)bh * n + i0 + row) * r * r + f] = sm[pl.Dr + row * pl.pr + f / r] * sm[pl.Dr + row * pl.pr + f % r];
        }
    }
}

// Back through one network: `sm + pl.Dr` holds df on entry; dX is ADDED into Dh; parameter
// gradients are added to dP.  Forward intermediates of this network must be in place (net_forward).
__device__ void net_backward(float* sm, const Plan& pl, const NetLayout& nl, const float* __restrict__ P,
                             float* __restrict__ dP) {
    // a3 = gelu(P3) into D8; dW4 += a3^T df, db4 += sum df
    for (int e = threadIdx.x; e < kRows * pl.m; e += kThreads) {
        const int row = e / pl.m, j = e % pl.m;
        sm[pl.D8 + row * pl.pm + j] = gelu_f(sm[pl.P3 + row * pl.pm + j]);
    }
    __syncthreads();
    accum_dense(dP + nl.W4, dP + nl.b4, sm + pl.D8, pl.pm, sm + pl.Dr, pl.pr, pl.m, pl.r);
    __syncthreads();
    // dp3 = (df W4^T) * gelu'(p3)
    dense_t(sm + pl.D8, pl.pm, sm + pl.Dr, pl.pr, P + nl.W4, pl.m, pl.r);
    __syncthreads();
    for (int e = threadIdx.x; e < kRows * pl.m; e += kThreads) {
        const int row = e / pl.m, j = e % pl.m;
        sm[pl.D8 + row * pl.pm + j] *= gelu_grad_f(sm[pl.P3 + row * pl.pm + j]);
    }
    __syncthreads();
    accum_dense(dP + nl.W3, dP + nl.b3, sm + pl.A2, pl.pr, sm + pl.D8, pl.pm, pl.r, pl.m);
    // da2 = dp3 W3^T (into Dr: df is no longer needed)
    dense_t(sm + pl.Dr, pl.pr, sm + pl.D8, pl.pm, P + nl.W3, pl.r, pl.m);
    __syncthreads();
    // z1 = N1 * g1 + c1 into D8 (dp3 is consumed); dW2 += z1^T da2, db2 += sum da2
    for (int e = threadIdx.x; e < kRows * pl.m; e += kThreads) {
        const int row = e / pl.m, j = e % pl.m;
        sm[pl.D8 + row * pl.pm + j] = fmaf(sm[pl.N1 + row * pl.pm + j], P[nl.g1 + j], P[nl.c1 + j]);
    }
    __syncthreads();
    accum_dense(dP + nl.W2, dP + nl.b2, sm + pl.D8, pl.pm, sm + pl.Dr, pl.pr, pl.m, pl.r);
    __syncthreads();
    // dz1 = da2 W2^T into D8, back through the second normalisation, times gelu'(p1)
    dense_t(sm + pl.D8, pl.pm, sm + pl.Dr, pl.pr, P + nl.W2, pl.m, pl.r);
    __syncthreads();
    layer_norm_back(sm + pl.D8, pl.pm, sm + pl.N1, pl.pm, P + nl.g1, pl.m, sm + pl.RS1, dP + nl.g1, dP + nl.c1);
    __syncthreads();
    for (int e = threadIdx.x; e < kRows * pl.m; e += kThreads) {
        const int row = e / pl.m, j = e % pl.m;
        sm[pl.D8 + row * pl.pm + j] *= gelu_grad_f(sm[pl.P1 + row * pl.pm + j]);
    }
    __syncthreads();
    // z0 = N0 * g0 + c0 into P3's first columns (P3 is consumed); dW1 += z0^T dp1, db1 += sum dp1
    for (int e = threadIdx.x; e < kRows * pl.h; e += kThreads) {
        const int row = e / pl.h, k = e % pl.h;
        sm[pl.P3 + row * pl.pm + k] = fmaf(sm[pl.N0 + row * pl.ph + k], P[nl.g0 + k], P[nl.c0 + k]);
    }
    __syncthreads();
    accum_dense(dP + nl.W1, dP + nl.b1, sm + pl.P3, pl.pm, sm + pl.D8, pl.pm, pl.h, pl.m);
    __syncthreads();
    // dz0 = dp1 W1^T into P3's first columns, back through the first normalisation, added to dX
    dense_t(sm + pl.P3, pl.pm, sm + pl.D8, pl.pm, P + nl.W1, pl.h, pl.m);
    __syncthreads();
    layer_norm_back(sm + pl.P3, pl.pm, sm + pl.N0, pl.ph, P + nl.g0, pl.h, sm + pl.RS0, dP + nl.g0, dP + nl.c0);
    __syncthreads();
    for (int e = threadIdx.x; e < kRows * pl.h; e += kThreads) {
        const int row = e / pl.h, k = e % pl.h;
        sm[pl.Dh + row * pl.ph + k] += sm[pl.P3 + row * pl.pm + k];
    }
    __syncthreads();
}

// dX = chain rule of sum(dM * M) through both networks (+ `add`, the part of the gradient that
// reached X directly), parameter gradients added to dparams.
template <typename T>
__global__ void __launch_bounds__(kThreads)
learned_sketch_bwd_kernel(Slice sl, int n, int h, int r, const T* __restrict__ X, const float* __restrict__ params,
                          const float* __restrict__ dM, const float* __restrict__ add, T* __restrict__ dX,
                          float* __restrict__ dparams) {
    extern __shared__ float sm[];
    const Plan pl(h, r);
    const NetLayout nl(h, r);
    const int bh = blockIdx.y, i0 = blockIdx.x * kRows;
    load_rows(sm, pl, sl, X, bh, i0);
    for (int e = threadIdx.x; e < kRows * pl.ph; e += kThreads) sm[pl.Dh + e] = 0.f;
    net_forward(sm, pl, nl, params, sm + pl.F1);
    net_forward(sm, pl, nl, params + nl.count, sm + pl.F2);
    const float isr = rsqrtf((float)r);
    // network 2's intermediates are in place: its df = dM (1 - t^2) f1
    for (int net = 1; net >= 0; --net) {
        if (net == 0) net_forward(sm, pl, nl, params, sm + pl.Dr);      // intermediates of network 1 again (f1 itself is kept in F1)
        for (int e = threadIdx.x; e < kRows * r; e += kThreads) {
            const int row = e / r, j = e % r;
            const float f1 = sm[pl.F1 + row * pl.pr + j], f2 = sm[pl.F2 + row * pl.pr + j];
            const float t = tanhf(f1 * f2 * isr);
            const float du = dM[((size_t)bh * n + i0 + row) * r + j] * (1.f - t * t);
            sm[pl.Dr + row * pl.pr + j] = du * (net == 1 ? f1 : f2);
        }
        __syncthreads();
        net_backward(sm, pl, nl, params + net * nl.count, dparams + net * nl.count);
    }
    for (int e = threadIdx.x; e < kRows * h; e += kThreads) {
        const int row = e / h, c = e % h;
        float v = sm[pl.Dh + row * pl.ph + c];
        if (add != nullptr) v += add[((size_t)bh * n + i0 + row) * h + c];
        stf(dX + sl.row(bh, i0 + row) + c, v);
    }
}

}  // namespace

size_t learned_param_count(int h, int r) { return (size_t)NetLayout(h, r).count; }

template <typename T>
static cudaError_t sketch_t(const Dims& d, const T* X, float* M, float* Phi, cudaStream_t s, int* launches) {
    const size_t smem = (size_t)Plan(d.h, d.r).total * sizeof(float);
    PSK_TRY_CUDA(cudaFuncSetAttribute(learned_sketch_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    prof_begin("learned_sketch_kernel", s);
    learned_sketch_kernel<T><<<dim3(d.n / kRows, d.BH()), kThreads, smem, s>>>(
        Slice{d.H, d.sb, d.sh, d.sn}, d.n, d.h, d.r, X, d.lparams, M, Phi);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <typename T>
static cudaError_t sketch_bwd_t(const Dims& d, const T* X, const float* dM, const float* add, T* dX, cudaStream_t s,
                                int* launches) {
    const size_t smem = (size_t)Plan(d.h, d.r).total * sizeof(float);
    PSK_TRY_CUDA(cudaFuncSetAttribute(learned_sketch_bwd_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    prof_begin("learned_sketch_bwd_kernel", s);
    learned_sketch_bwd_kernel<T><<<dim3(d.n / kRows, d.BH()), kThreads, smem, s>>>(
        Slice{d.H, d.sb, d.sh, d.sn}, d.n, d.h, d.r, X, d.lparams, dM, add, dX, d.dlparams);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t learned_sketch(const Dims& d, const void* X, float* M, float* Phi, cudaStream_t s, int* launches) {
    return d.bf16 ? sketch_t(d, (const __nv_bfloat16*)X, M, Phi, s, launches) : sketch_t(d, (const float*)X, M, Phi, s, launches);
}

cudaError_t learned_sketch_bwd(const Dims& d, const void* X, const float* dM, const float* add, void* dX, cudaStream_t s,
                               int* launches) {
    return d.bf16 ? sketch_bwd_t(d, (const __nv_bfloat16*)X, dM, add, (__nv_bfloat16*)dX, s, launches)
                  : sketch_bwd_t(d, (const float*)X, dM, add, (float*)dX, s, launches);
}

}  // namespace psk
