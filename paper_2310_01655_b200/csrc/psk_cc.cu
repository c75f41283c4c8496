// CUDA-core path: causal Polysketch attention in fp32 arithmetic, the steps of
// Section 3.1 as separate kernels (half sketch -> per-block states H_l -> prefix scan
// Z_l -> output rows P_l + phi'(Q_l) Z_l -> division by D~).  Serves fp32 storage (the
// tensor cores' tf32 rounding cannot hold 1e-4 through a degree-4 polynomial) and
// cross-checks the tensor-core path on bf16 storage.
#include "psk_internal.cuh"

namespace psk {

CcWorkspace cc_workspace(const Dims& d, bool backward) {
    CcWorkspace w{};
    const size_t rows = (size_t)d.BH() * d.n;
    const size_t st = (size_t)d.BH() * d.t * d.r * d.r * 65 * sizeof(float);
    size_t off = 0;
    w.status = off; off += kStatusBytes;
    w.Mq = off;  off += align_up(rows * d.r * sizeof(float));
    w.Mk = off;  off += align_up(rows * d.r * sizeof(float));
    w.Vt = off;  off += align_up(rows * 65 * sizeof(float));
    w.Zst = off; off += align_up(st);
    if (backward) {
        w.E = off;   off += align_up(rows * 65 * sizeof(float));
        w.Rst = off; off += align_up(st);
        w.dMq = off; off += align_up(rows * d.r * sizeof(float));
        w.dMk = off; off += align_up(rows * d.r * sizeof(float));
        if (d.local) {     // gradients that reach Q and K directly, through the exact same-block weights
            w.dXq = off; off += align_up(rows * 64 * sizeof(float));
            w.dXk = off; off += align_up(rows * 64 * sizeof(float));
        }
    }
    w.total = off;
    return w;
}

namespace {

constexpr int H64 = 64;     // head dimension (only value supported)
constexpr int YC = 65;      // columns of [V | 1] and of E
constexpr int YS = 68;      // padded shared-memory row stride for 65-column rows

struct Slice {              // addressing of one [B,H,n,h] tensor
    int H; int64_t sb, sh, sn;
    __device__ int64_t row(int bh, int i) const {
        return (int64_t)(bh / H) * sb + (int64_t)(bh % H) * sh + (int64_t)i * sn;
    }
};

// ---------------------------------------------------------------------------
// Half sketch m(x) = (x G1)*(x G2)/sqrt(r)  (Algorithm 1, degree-2 level), 64 rows per CTA
// ---------------------------------------------------------------------------
template <typename T, int R>
__global__ void __launch_bounds__(256)
sketch_kernel(Slice sl, const T* __restrict__ X, const T* __restrict__ G1, const T* __restrict__ G2,
              int g_heads, int n, float* __restrict__ M_out, float* __restrict__ Phi_out) {
    extern __shared__ float smem[];
    float* sG1 = smem;                  // [64][R]
    float* sG2 = sG1 + H64 * R;         // [64][R]
    float* sX = sG2 + H64 * R;          // [64][65]
    float* sM = sX + 64 * 65;           // [64][R+1]
    const int bh = blockIdx.y, i0 = blockIdx.x * 64, tid = threadIdx.x;
    const int g = (g_heads == 1) ? 0 : (bh % sl.H);
    for (int e = tid; e < H64 * R; e += 256) {
        sG1[e] = ldf(G1 + (size_t)g * H64 * R + e);
        sG2[e] = ldf(G2 + (size_t)g * H64 * R + e);
    }
    for (int e = tid; e < 64 * H64; e += 256) {
        const int rr = e / H64, c = e % H64;
        sX[rr * 65 + c] = ldf(X + sl.row(bh, i0 + rr) + c);
    }
    __syncthreads();
    const float rs = rsqrtf((float)R);
    const int c = tid % R;
    for (int rr = tid / R; rr < 64; rr += 256 / R) {
        float a1 = 0.f, a2 = 0.f;
#pragma unroll 16
        for (int t = 0; t < H64; ++t) {
            const float x = sX[rr * 65 + t];
            a1 = fmaf(x, sG1[t * R + c], a1);
            a2 = fmaf(x, sG2[t * R + c], a2);
        }
        const float m = a1 * a2 * rs;
        sM[rr * (R + 1) + c] = m;
        M_out[((size_t)bh * n + i0 + rr) * R + c] = m;
    }
    if (Phi_out != nullptr) {           // phi'(x)[a*R+b] = m_a m_b (Section 1.2 ordering)
        __syncthreads();
        for (int e = tid; e < 64 * R * R; e += 256) {
            const int rr = e / (R * R), f = e % (R * R);
            Phi_out[((size_t)bh * n + i0 + rr) * R * R + f] =
                sM[rr * (R + 1) + f / R] * sM[rr * (R + 1) + f % R];
        }
    }
}

// ---------------------------------------------------------------------------
// Degree p = 2 (Algorithm 1 with p/2 = 1): the "half sketch" is the row itself, M = X, and
// phi'(x) = x (x) x has h^2 entries: exact degree-2 polynomial attention, no Gaussians.
// Forward copy M = X (optionally Phi = X (x) X); backward dX = dM (+ add).  One warp per row.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
identity_sketch_kernel(Slice sl, int n, int total_rows, const T* __restrict__ X, float* __restrict__ M,
                       float* __restrict__ Phi) {
    const int row = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
    if (row >= total_rows) return;
    const int64_t base = sl.row(row / n, row % n);
    const float x0 = ldf(X + base + lane), x1 = ldf(X + base + lane + 32);
    M[(size_t)row * 64 + lane] = x0;
    M[(size_t)row * 64 + lane + 32] = x1;
    if (Phi != nullptr) {
        for (int a = 0; a < 64; ++a) {
            const float xa = __shfl_sync(0xffffffffu, a < 32 ? x0 : x1, a % 32);
            Phi[((size_t)row * 64 + a) * 64 + lane] = xa * x0;
            Phi[((size_t)row * 64 + a) * 64 + lane + 32] = xa * x1;
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
identity_sketch_bwd_kernel(Slice sl, int n, int total_rows, const float* __restrict__ dM,
                           const float* __restrict__ add, T* __restrict__ dX) {
    const int row = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
    if (row >= total_rows) return;
    const int64_t base = sl.row(row / n, row % n);
#pragma unroll
    for (int c = lane; c < 64; c += 32) {
        float v = dM[(size_t)row * 64 + c];
        if (add != nullptr) v += add[(size_t)row * 64 + c];
        stf(dX + base + c, v);
    }
}

// ---------------------------------------------------------------------------
// Degree p = 8: one more level of Algorithm 1's recursion.  Two independent degree-2 sketches
//   M1 = (X Ga1)*(X Ga2)/sqrt(r),  M2 = (X Gb1)*(X Gb2)/sqrt(r)
// are combined through r x r Gaussians,  M = (M1 Gc1)*(M2 Gc2)/sqrt(r); phi' = M (x) M as before.
// G1 holds [Ga1; Gb1; Gc1] and G2 holds [Ga2; Gb2; Gc2], each (2h + r) x r row-major per head.
// 32 rows per CTA; the Gaussians are read from global memory (they stay in cache).
// ---------------------------------------------------------------------------
template <int R> struct Sk8 {
    static constexpr int kRows = 32, kLd = R + 1;
    static constexpr int kGRows = 2 * H64 + R;             // rows of one packed Gaussian set
    static constexpr int X = 0;                            // [32][65]
    static constexpr int A1 = X + kRows * 65, A2 = A1 + kRows * kLd, B1 = A2 + kRows * kLd, B2 = B1 + kRows * kLd;
    static constexpr int M1 = B2 + kRows * kLd, M2 = M1 + kRows * kLd, C1 = M2 + kRows * kLd, C2 = C1 + kRows * kLd;
    static constexpr int total = C2 + kRows * kLd;
    static constexpr size_t bytes = (size_t)total * sizeof(float);
};

// shared by the forward and the backward: X tile -> A1, A2, B1, B2, M1, M2, C1 = M1 Gc1, C2 = M2 Gc2
template <typename T, int R>
__device__ __forceinline__ void sketch8_forward_tile(float* smem, Slice sl, const T* __restrict__ X,
                                                     const T* __restrict__ g1, const T* __restrict__ g2,
                                                     int bh, int i0, int tid) {
    using L = Sk8<R>;
    for (int e = tid; e < L::kRows * H64; e += 256) {
        const int rr = e / H64, c = e % H64;
        smem[L::X + rr * 65 + c] = ldf(X + sl.row(bh, i0 + rr) + c);
    }
    __syncthreads();
    const float rs = rsqrtf((float)R);
    for (int e = tid; e < L::kRows * R; e += 256) {
        const int rr = e / R, c = e % R;
        float a1 = 0.f, a2 = 0.f, b1 = 0.f, b2 = 0.f;
        for (int t = 0; t < H64; ++t) {
            const float x = smem[L::X + rr * 65 + t];
            a1 = fmaf(x, ldf(g1 + t * R + c), a1);
            a2 = fmaf(x, ldf(g2 + t * R + c), a2);
            b1 = fmaf(x, ldf(g1 + (H64 + t) * R + c), b1);
            b2 = fmaf(x, ldf(g2 + (H64 + t) * R + c), b2);
        }
        const int o = rr * L::kLd + c;
        smem[L::A1 + o] = a1; smem[L::A2 + o] = a2; smem[L::B1 + o] = b1; smem[L::B2 + o] = b2;
        smem[L::M1 + o] = a1 * a2 * rs;
        smem[L::M2 + o] = b1 * b2 * rs;
    }
    __syncthreads();
    for (int e = tid; e < L::kRows * R; e += 256) {
        const int rr = e / R, c = e % R;
        float c1 = 0.f, c2 = 0.f;
        for (int k = 0; k < R; ++k) {
            c1 = fmaf(smem[L::M1 + rr * L::kLd + k], ldf(g1 + (2 * H64 + k) * R + c), c1);
            c2 = fmaf(smem[L::M2 + rr * L::kLd + k], ldf(g2 + (2 * H64 + k) * R + c), c2);
        }
        smem[L::C1 + rr * L::kLd + c] = c1;
        smem[L::C2 + rr * L::kLd + c] = c2;
    }
    __syncthreads();
}

template <typename T, int R>
__global__ void __launch_bounds__(256)
sketch8_kernel(Slice sl, const T* __restrict__ X, const T* __restrict__ G1, const T* __restrict__ G2,
               int g_heads, int n, float* __restrict__ M_out, float* __restrict__ Phi_out) {
    extern __shared__ float smem[];
    using L = Sk8<R>;
    const int bh = blockIdx.y, i0 = blockIdx.x * L::kRows, tid = threadIdx.x;
    const int g = (g_heads == 1) ? 0 : (bh % sl.H);
    const T* g1 = G1 + (size_t)g * L::kGRows * R;
    const T* g2 = G2 + (size_t)g * L::kGRows * R;
    sketch8_forward_tile<T, R>(smem, sl, X, g1, g2, bh, i0, tid);
    const float rs = rsqrtf((float)R);
    for (int e = tid; e < L::kRows * R; e += 256) {
        const int rr = e / R, c = e % R;
        const float m = smem[L::C1 + rr * L::kLd + c] * smem[L::C2 + rr * L::kLd + c] * rs;
        smem[L::M1 + rr * L::kLd + c] = m;                 // (M1 is dead: keep M for Phi)
        M_out[((size_t)bh * n + i0 + rr) * R + c] = m;
    }
    if (Phi_out != nullptr) {
        __syncthreads();
        for (int e = tid; e < L::kRows * R * R; e += 256) {
            const int rr = e / (R * R), f = e % (R * R);
            Phi_out[((size_t)bh * n + i0 + rr) * R * R + f] =
                smem[L::M1 + rr * L::kLd + f / R] * smem[L::M1 + rr * L::kLd + f % R];
        }
    }
}

// Chain rule through the degree-8 half sketch (forward values recomputed):
//   dC1 = dM*C2/sqrt(r), dC2 = dM*C1/sqrt(r);  dM1 = dC1 Gc1^T, dM2 = dC2 Gc2^T;
//   dA1 = dM1*A2/sqrt(r), dA2 = dM1*A1/sqrt(r), dB1 = dM2*B2/sqrt(r), dB2 = dM2*B1/sqrt(r);
//   dX = dA1 Ga1^T + dA2 Ga2^T + dB1 Gb1^T + dB2 Gb2^T.
template <typename T, int R>
__global__ void __launch_bounds__(256)
sketch8_bwd_kernel(Slice sl, const T* __restrict__ X, const T* __restrict__ G1, const T* __restrict__ G2,
                   int g_heads, int n, const float* __restrict__ dM, T* __restrict__ dX) {
    extern __shared__ float smem[];
    using L = Sk8<R>;
    const int bh = blockIdx.y, i0 = blockIdx.x * L::kRows, tid = threadIdx.x;
    const int g = (g_heads == 1) ? 0 : (bh % sl.H);
    const T* g1 = G1 + (size_t)g * L::kGRows * R;
    const T* g2 = G2 + (size_t)g * L::kGRows * R;
    sketch8_forward_tile<T, R>(smem, sl, X, g1, g2, bh, i0, tid);
    const float rs = rsqrtf((float)R);
    // dC1, dC2 over C1, C2 (each entry is read and written by one thread)
    for (int e = tid; e < L::kRows * R; e += 256) {
        const int rr = e / R, c = e % R, o = rr * L::kLd + c;
        const float gm = dM[((size_t)bh * n + i0 + rr) * R + c] * rs;
        const float c1 = smem[L::C1 + o], c2 = smem[L::C2 + o];
        smem[L::C1 + o] = gm * c2;
        smem[L::C2 + o] = gm * c1;
    }
    __syncthreads();
    // dM1, dM2 over M1, M2 (M1, M2 themselves are no longer needed)
    for (int e = tid; e < L::kRows * R; e += 256) {
        const int rr = e / R, k = e % R;
        float d1 = 0.f, d2 = 0.f;
        for (int c = 0; c < R; ++c) {
            d1 = fmaf(smem[L::C1 + rr * L::kLd + c], ldf(g1 + (2 * H64 + k) * R + c), d1);
            d2 = fmaf(smem[L::C2 + rr * L::kLd + c], ldf(g2 + (2 * H64 + k) * R + c), d2);
        }
        smem[L::M1 + rr * L::kLd + k] = d1;
        smem[L::M2 + rr * L::kLd + k] = d2;
    }
    __syncthreads();
    // dA1, dA2, dB1, dB2 over A1, A2, B1, B2
    for (int e = tid; e < L::kRows * R; e += 256) {
        const int rr = e / R, c = e % R, o = rr * L::kLd + c;
        const float d1 = smem[L::M1 + o] * rs, d2 = smem[L::M2 + o] * rs;
        const float a1 = smem[L::A1 + o], a2 = smem[L::A2 + o], b1 = smem[L::B1 + o], b2 = smem[L::B2 + o];
        smem[L::A1 + o] = d1 * a2; smem[L::A2 + o] = d1 * a1;
        smem[L::B1 + o] = d2 * b2; smem[L::B2 + o] = d2 * b1;
    }
    __syncthreads();
    for (int e = tid; e < L::kRows * H64; e += 256) {
        const int rr = e / H64, t = e % H64;
        float dx = 0.f;
        for (int c = 0; c < R; ++c) {
            const int o = rr * L::kLd + c;
            dx = fmaf(smem[L::A1 + o], ldf(g1 + t * R + c), dx);
            dx = fmaf(smem[L::A2 + o], ldf(g2 + t * R + c), dx);
            dx = fmaf(smem[L::B1 + o], ldf(g1 + (H64 + t) * R + c), dx);
            dx = fmaf(smem[L::B2 + o], ldf(g2 + (H64 + t) * R + c), dx);
        }
        stf(dX + sl.row(bh, i0 + rr) + t, dx);
    }
}

// ---------------------------------------------------------------------------
// Row preparation: mode 0 writes V~ = [V | 1]; mode 1 writes E = [dO/d | -(dO.O)/d]
// One warp per row.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
rows_prep_kernel(Slice sl, int n, int total_rows, int mode, const T* __restrict__ V,
                 const T* __restrict__ O, const float* __restrict__ denom,
                 const T* __restrict__ dO, float* __restrict__ out) {
    const int row = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
    if (row >= total_rows) return;
    const int bh = row / n, i = row % n;
    const int64_t base = sl.row(bh, i);
    float* o = out + (size_t)row * YC;
    if (mode == 0) {
        o[lane] = ldf(V + base + lane);
        o[lane + 32] = ldf(V + base + lane + 32);
        if (lane == 0) o[64] = 1.f;
    } else {
        const float g0 = ldf(dO + base + lane), g1 = ldf(dO + base + lane + 32);
        float dot = g0 * ldf(O + base + lane) + g1 * ldf(O + base + lane + 32);
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
        const float inv = 1.f / denom[row];
        o[lane] = g0 * inv;
        o[lane + 32] = g1 * inv;
        if (lane == 0) o[64] = -dot * inv;
    }
}

// ---------------------------------------------------------------------------
// Per-block state H_l = phi'(M_l)^T Y_l  (Section 3.1), M the half sketches of the
// block's rows, Y its [b,65] right-hand side.  One thread per feature (a,b).
// ---------------------------------------------------------------------------
template <int R>
__global__ void __launch_bounds__(128)
state_kernel(const float* __restrict__ M, const float* __restrict__ Y, int n, int b, int t,
             float* __restrict__ S) {
    __shared__ float sM[32][R];
    __shared__ __align__(16) float sY[32][YS];
    const int tid = threadIdx.x, l = blockIdx.y, bh = blockIdx.z;
    const int f = blockIdx.x * 128 + tid, fa = f / R, fb = f % R;
    float acc[YC];
#pragma unroll
    for (int c = 0; c < YC; ++c) acc[c] = 0.f;
    const size_t row0 = (size_t)bh * n + (size_t)l * b;
    for (int j0 = 0; j0 < b; j0 += 32) {
        __syncthreads();
        for (int e = tid; e < 32 * R; e += 128) sM[e / R][e % R] = M[(row0 + j0) * R + e];
        for (int e = tid; e < 32 * YC; e += 128) sY[e / YC][e % YC] = Y[(row0 + j0) * YC + e];
        __syncthreads();
        if (f < R * R) {
#pragma unroll 4
            for (int j = 0; j < 32; ++j) {
                const float phi = sM[j][fa] * sM[j][fb];
#pragma unroll
                for (int c = 0; c < 64; c += 4) {
                    const float4 y = *reinterpret_cast<const float4*>(&sY[j][c]);
                    acc[c] = fmaf(phi, y.x, acc[c]);
                    acc[c + 1] = fmaf(phi, y.y, acc[c + 1]);
                    acc[c + 2] = fmaf(phi, y.z, acc[c + 2]);
                    acc[c + 3] = fmaf(phi, y.w, acc[c + 3]);
                }
                acc[64] = fmaf(phi, sY[j][64], acc[64]);
            }
        }
    }
    if (f < R * R) {
        float* o = S + (((size_t)bh * t + l) * R * R + f) * YC;
#pragma unroll
        for (int c = 0; c < YC; ++c) o[c] = acc[c];
    }
}

// Exclusive prefix (reverse = 0: Z_l = sum_{j<l} H_j, Section 3.1) or exclusive suffix
// (reverse = 1: sum_{j>l} H_j) over the t states of each head, in place, sequential in l.
__global__ void __launch_bounds__(256)
scan_kernel(float* __restrict__ S, size_t elems, int t, int reverse) {
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= elems) return;
    float* p = S + (size_t)blockIdx.y * t * elems + e;
    float run = 0.f;
    if (!reverse) {
        for (int l = 0; l < t; ++l) { const float v = p[(size_t)l * elems]; p[(size_t)l * elems] = run; run += v; }
    } else {
        for (int l = t - 1; l >= 0; --l) { const float v = p[(size_t)l * elems]; p[(size_t)l * elems] = run; run += v; }
    }
}

// acc[0..64] += coef * row[0..64]   (row in shared memory, 16-byte aligned, stride YS)
__device__ __forceinline__ void axpy65(float (&acc)[YC], float coef, const float* row) {
#pragma unroll
    for (int c = 0; c < 64; c += 4) {
        const float4 z = *reinterpret_cast<const float4*>(row + c);
        acc[c] = fmaf(coef, z.x, acc[c]);
        acc[c + 1] = fmaf(coef, z.y, acc[c + 1]);
        acc[c + 2] = fmaf(coef, z.z, acc[c + 2]);
        acc[c + 3] = fmaf(coef, z.w, acc[c + 3]);
    }
    acc[64] = fmaf(coef, row[64], acc[64]);
}
// row[0..64] . y[0..64]
__device__ __forceinline__ float dot65(const float* row, const float (&y)[YC]) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int c = 0; c < 64; c += 4) {
        const float4 z = *reinterpret_cast<const float4*>(row + c);
        s0 = fmaf(z.x, y[c], s0);
        s1 = fmaf(z.y, y[c + 1], s1);
        s2 = fmaf(z.z, y[c + 2], s2);
        s3 = fmaf(z.w, y[c + 3], s3);
    }
    return (s0 + s1) + (s2 + s3) + row[64] * y[64];
}

// Shared-memory carve-up of the three row kernels (one thread per row, 128 rows per CTA):
//   sS   [R][YS]        slice a of the block's prefix/suffix state: rows (a, 0..R-1)
//   sOwn [128][R+1]     this tile's own half sketches (runtime-indexed access by a)
//   sOut [128][R+1]     per-row results indexed by a
//   sM2  [32][R]        chunk of the other side's half sketches (diagonal tile)
//   sY2  [32][YS]       chunk of the other side's 65-column rows (diagonal tile)
// and, with exact same-block weights (Section 3.2):
//   sXo  [128][65]      this tile's own raw rows (q or k), each read by its own thread only
//   sX2  [32][64]       chunk of the other side's raw rows
template <int R> struct RowSmem {
    static constexpr int S = 0;
    static constexpr int Own = S + R * YS;
    static constexpr int Out = Own + 128 * (R + 1);
    static constexpr int M2 = Out + 128 * (R + 1);
    static constexpr int Y2 = M2 + 32 * R;
    static constexpr int total = Y2 + 32 * YS;
    static constexpr size_t bytes = (size_t)total * sizeof(float);
    static constexpr int Xo = total;
    static constexpr int X2 = Xo + 128 * 65;
    static constexpr size_t bytes_local = (size_t)(X2 + 32 * 64) * sizeof(float);
};

// <own raw row (shared memory, stride 65), row jj of the other side's chunk>
__device__ __forceinline__ float dot64_raw(const float* own, const float* other) {
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < 64; ++c) s = fmaf(own[c], other[c], s);
    return s;
}

// ---------------------------------------------------------------------------
// Forward output rows (Section 3.1): row i of block l = P_l row + phi'(q_i)^T Z_l, with
// P_l = lt((L R^T)^2) [V_l | 1]; then d_i = 1 + last column, O_i = first 64 / d_i.
// LOCAL: P_l = lt((Q_l K_l^T)^4) [V_l | 1] instead, from the block's raw queries and keys
// (Section 3.2).
// ---------------------------------------------------------------------------
template <typename T, int R, bool LOCAL>
__global__ void __launch_bounds__(128)
fwd_out_kernel(Slice sl, int n, int b, int t, const float* __restrict__ Mq, const float* __restrict__ Mk,
               const float* __restrict__ Vt, const float* __restrict__ Z,
               const T* __restrict__ Qraw, const T* __restrict__ Kraw,
               T* __restrict__ O, float* __restrict__ denom) {
    extern __shared__ __align__(16) float smem[];
    float* sS = smem + RowSmem<R>::S;
    float* sOwn = smem + RowSmem<R>::Own;
    float* sM2 = smem + RowSmem<R>::M2;
    float* sY2 = smem + RowSmem<R>::Y2;
    const int tid = threadIdx.x, tile = blockIdx.x, l = blockIdx.y, bh = blockIdx.z;
    const int i_blk = tile * 128 + tid;                 // row within the block
    const size_t blk0 = (size_t)bh * n + (size_t)l * b;  // first row of the block
    const size_t row = blk0 + i_blk;
    float mq[R], acc[YC];
#pragma unroll
    for (int c = 0; c < R; ++c) { mq[c] = Mq[row * R + c]; sOwn[tid * (R + 1) + c] = mq[c]; }
#pragma unroll
    for (int c = 0; c < YC; ++c) acc[c] = 0.f;
    float* sXo = smem + RowSmem<R>::Xo + tid * 65;
    float* sX2 = smem + RowSmem<R>::X2;
    if constexpr (LOCAL) {
        const int64_t o = sl.row(bh, l * b + i_blk);
        for (int c = 0; c < 64; ++c) sXo[c] = ldf(Qraw + o + c);
    }
    // earlier blocks through the prefix state
    const float* Zl = Z + ((size_t)bh * t + l) * R * R * YC;
    if (l > 0) {
        for (int a = 0; a < R; ++a) {
            __syncthreads();
            for (int e = tid; e < R * YC; e += 128) sS[(e / YC) * YS + e % YC] = Zl[(size_t)a * R * YC + e];
            __syncthreads();
            const float ma = sOwn[tid * (R + 1) + a];
#pragma unroll
            for (int bb = 0; bb < R; ++bb) axpy65(acc, ma * mq[bb], sS + bb * YS);
        }
    }
    // same block: j <= i through the b x b tile of squared half-sketch scores
    const int jend = tile * 128 + 128;                  // keys needed by this row tile
    const int warp_imax = tile * 128 + (tid | 31);
    for (int j0 = 0; j0 < jend; j0 += 32) {
        __syncthreads();
        if constexpr (LOCAL) {
            for (int e = tid; e < 32 * 64; e += 128) sX2[e] = ldf(Kraw + sl.row(bh, l * b + j0 + e / 64) + e % 64);
        } else {
            for (int e = tid; e < 32 * R; e += 128) sM2[e] = Mk[(blk0 + j0) * R + e];
        }
        for (int e = tid; e < 32 * YC; e += 128) sY2[(e / YC) * YS + e % YC] = Vt[(blk0 + j0) * YC + e];
        __syncthreads();
        if (j0 > warp_imax) continue;
        for (int jj = 0; jj < 32; ++jj) {
            if (j0 + jj > i_blk) break;
            float s = 0.f;
            if constexpr (LOCAL) {
                const float x = dot64_raw(sXo, sX2 + jj * 64);
                s = x * x;                                  // weight s^2 = (q . k)^4
            } else {
#pragma unroll
                for (int c = 0; c < R; ++c) s = fmaf(mq[c], sM2[jj * R + c], s);
            }
            axpy65(acc, s * s, sY2 + jj * YS);
        }
    }
    const float d = 1.f + acc[64];
    const float inv = 1.f / d;
    const int64_t o = sl.row(bh, l * b + i_blk);
#pragma unroll
    for (int c = 0; c < 64; ++c) stf(O + o + c, acc[c] * inv);
    if (denom != nullptr) denom[row] = d;
}

// ---------------------------------------------------------------------------
// Backward, query side.  d m(q_i) = 2 mat(Z_l E_i) m(q_i)  +  sum_{j<=i, same block}
// 2 s_ij (E_i . v~_j) m(k_j).
// LOCAL (Section 3.2): the same-block pairs carry W_ij = x_ij^4, x_ij = q_i . k_j, whose gradient
// reaches q_i directly:  dXl_i = sum_{j<=i, same block} 4 x_ij^3 (E_i . v~_j) k_j.
// ---------------------------------------------------------------------------
template <typename T, int R, bool LOCAL>
__global__ void __launch_bounds__(128)
bwd_q_kernel(Slice sl, int n, int b, int t, const float* __restrict__ Mq, const float* __restrict__ Mk,
             const float* __restrict__ Vt, const float* __restrict__ E, const float* __restrict__ Z,
             const T* __restrict__ Qraw, const T* __restrict__ Kraw,
             float* __restrict__ dMq, float* __restrict__ dXl) {
    extern __shared__ __align__(16) float smem[];
    float* sS = smem + RowSmem<R>::S;
    float* sOut = smem + RowSmem<R>::Out;
    float* sM2 = smem + RowSmem<R>::M2;
    float* sY2 = smem + RowSmem<R>::Y2;
    const int tid = threadIdx.x, tile = blockIdx.x, l = blockIdx.y, bh = blockIdx.z;
    const int i_blk = tile * 128 + tid;
    const size_t blk0 = (size_t)bh * n + (size_t)l * b;
    const size_t row = blk0 + i_blk;
    float mq[R], dm[R], e[YC];
#pragma unroll
    for (int c = 0; c < R; ++c) { mq[c] = Mq[row * R + c]; dm[c] = 0.f; sOut[tid * (R + 1) + c] = 0.f; }
#pragma unroll
    for (int c = 0; c < YC; ++c) e[c] = E[row * YC + c];
    const float* Zl = Z + ((size_t)bh * t + l) * R * R * YC;
    if (l > 0) {
        for (int a = 0; a < R; ++a) {
            __syncthreads();
            for (int x = tid; x < R * YC; x += 128) sS[(x / YC) * YS + x % YC] = Zl[(size_t)a * R * YC + x];
            __syncthreads();
            float ta = 0.f;
#pragma unroll
            for (int bb = 0; bb < R; ++bb) ta = fmaf(dot65(sS + bb * YS, e), mq[bb], ta);
            sOut[tid * (R + 1) + a] = 2.f * ta;
        }
    }
    const int jend = tile * 128 + 128;
    const int warp_imax = tile * 128 + (tid | 31);
    float* sXo = smem + RowSmem<R>::Xo + tid * 65;
    float* sX2 = smem + RowSmem<R>::X2;
    float dxl[LOCAL ? 64 : 1];
    if constexpr (LOCAL) {
        const int64_t o = sl.row(bh, l * b + i_blk);
        for (int c = 0; c < 64; ++c) sXo[c] = ldf(Qraw + o + c);
#pragma unroll
        for (int c = 0; c < 64; ++c) dxl[c] = 0.f;
    }
    for (int j0 = 0; j0 < jend; j0 += 32) {
        __syncthreads();
        if constexpr (LOCAL) {
            for (int x = tid; x < 32 * 64; x += 128) sX2[x] = ldf(Kraw + sl.row(bh, l * b + j0 + x / 64) + x % 64);
        } else {
            for (int x = tid; x < 32 * R; x += 128) sM2[x] = Mk[(blk0 + j0) * R + x];
        }
        for (int x = tid; x < 32 * YC; x += 128) sY2[(x / YC) * YS + x % YC] = Vt[(blk0 + j0) * YC + x];
        __syncthreads();
        if (j0 > warp_imax) continue;
        for (int jj = 0; jj < 32; ++jj) {
            if (j0 + jj > i_blk) break;
            if constexpr (LOCAL) {
                const float x = dot64_raw(sXo, sX2 + jj * 64);
                const float dx = 4.f * x * x * x * dot65(sY2 + jj * YS, e);
#pragma unroll
                for (int c = 0; c < 64; ++c) dxl[c] = fmaf(dx, sX2[jj * 64 + c], dxl[c]);
            } else {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < R; ++c) s = fmaf(mq[c], sM2[jj * R + c], s);
                const float ds = 2.f * s * dot65(sY2 + jj * YS, e);
#pragma unroll
                for (int c = 0; c < R; ++c) dm[c] = fmaf(ds, sM2[jj * R + c], dm[c]);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < R; ++c) dMq[row * R + c] = dm[c] + sOut[tid * (R + 1) + c];
    if constexpr (LOCAL) {
#pragma unroll
        for (int c = 0; c < 64; ++c) dXl[row * 64 + c] = dxl[c];
    }
}

// ---------------------------------------------------------------------------
// Backward, key/value side.  With R_l the suffix state sum_{blocks>l} phi'(Q)^T E:
//   d m(k_j) = 2 mat(R_l v~_j) m(k_j) + sum_{i>=j, same block} 2 s_ij (E_i . v~_j) m(q_i)
//   dV_j     = (R_l^T phi'(k_j))[:h]  + sum_{i>=j, same block} s_ij^2 E_i[:h]
// LOCAL (Section 3.2): same-block weights x_ij^4, x_ij = q_i . k_j:
//   dXl_j = sum_{i>=j, same block} 4 x_ij^3 (E_i . v~_j) q_i,   dV_j += sum x_ij^4 E_i[:h]
// ---------------------------------------------------------------------------
template <typename T, int R, bool LOCAL>
__global__ void __launch_bounds__(128)
bwd_k_kernel(Slice sl, int n, int b, int t, const float* __restrict__ Mq, const float* __restrict__ Mk,
             const float* __restrict__ Vt, const float* __restrict__ E, const float* __restrict__ Rs,
             const T* __restrict__ Qraw, const T* __restrict__ Kraw,
             float* __restrict__ dMk, float* __restrict__ dXl, T* __restrict__ dV) {
    extern __shared__ __align__(16) float smem[];
    float* sS = smem + RowSmem<R>::S;
    float* sOwn = smem + RowSmem<R>::Own;
    float* sOut = smem + RowSmem<R>::Out;
    float* sM2 = smem + RowSmem<R>::M2;
    float* sY2 = smem + RowSmem<R>::Y2;
    const int tid = threadIdx.x, tile = blockIdx.x, l = blockIdx.y, bh = blockIdx.z;
    const int j_blk = tile * 128 + tid;
    const size_t blk0 = (size_t)bh * n + (size_t)l * b;
    const size_t row = blk0 + j_blk;
    float mk[R], dm[R], v[YC], dv[YC];
#pragma unroll
    for (int c = 0; c < R; ++c) {
        mk[c] = Mk[row * R + c]; dm[c] = 0.f;
        sOwn[tid * (R + 1) + c] = mk[c]; sOut[tid * (R + 1) + c] = 0.f;
    }
#pragma unroll
    for (int c = 0; c < YC; ++c) { v[c] = Vt[row * YC + c]; dv[c] = 0.f; }
    const float* Rl = Rs + ((size_t)bh * t + l) * R * R * YC;
    if (l < t - 1) {
        for (int a = 0; a < R; ++a) {
            __syncthreads();
            for (int x = tid; x < R * YC; x += 128) sS[(x / YC) * YS + x % YC] = Rl[(size_t)a * R * YC + x];
            __syncthreads();
            const float ma = sOwn[tid * (R + 1) + a];
            float ta = 0.f;
#pragma unroll
            for (int bb = 0; bb < R; ++bb) {
                ta = fmaf(dot65(sS + bb * YS, v), mk[bb], ta);
                axpy65(dv, ma * mk[bb], sS + bb * YS);
            }
            sOut[tid * (R + 1) + a] = 2.f * ta;
        }
    }
    // same block: queries i >= j
    const int i_begin = tile * 128;                     // first query row any thread here needs
    const int warp_jmin = tile * 128 + (tid & ~31);
    float* sXo = smem + RowSmem<R>::Xo + tid * 65;
    float* sX2 = smem + RowSmem<R>::X2;
    float dxl[LOCAL ? 64 : 1];
    if constexpr (LOCAL) {
        const int64_t o = sl.row(bh, l * b + j_blk);
        for (int c = 0; c < 64; ++c) sXo[c] = ldf(Kraw + o + c);
#pragma unroll
        for (int c = 0; c < 64; ++c) dxl[c] = 0.f;
    }
    for (int i0 = i_begin; i0 < b; i0 += 32) {
        __syncthreads();
        if constexpr (LOCAL) {
            for (int x = tid; x < 32 * 64; x += 128) sX2[x] = ldf(Qraw + sl.row(bh, l * b + i0 + x / 64) + x % 64);
        } else {
            for (int x = tid; x < 32 * R; x += 128) sM2[x] = Mq[(blk0 + i0) * R + x];
        }
        for (int x = tid; x < 32 * YC; x += 128) sY2[(x / YC) * YS + x % YC] = E[(blk0 + i0) * YC + x];
        __syncthreads();
        if (i0 + 31 < warp_jmin) continue;
        for (int ii = 0; ii < 32; ++ii) {
            if (i0 + ii < j_blk) continue;
            if constexpr (LOCAL) {
                const float x = dot64_raw(sXo, sX2 + ii * 64);
                const float x2 = x * x;
                const float dx = 4.f * x2 * x * dot65(sY2 + ii * YS, v);
#pragma unroll
                for (int c = 0; c < 64; ++c) dxl[c] = fmaf(dx, sX2[ii * 64 + c], dxl[c]);
                axpy65(dv, x2 * x2, sY2 + ii * YS);
            } else {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < R; ++c) s = fmaf(mk[c], sM2[ii * R + c], s);
                const float ds = 2.f * s * dot65(sY2 + ii * YS, v);
#pragma unroll
                for (int c = 0; c < R; ++c) dm[c] = fmaf(ds, sM2[ii * R + c], dm[c]);
                axpy65(dv, s * s, sY2 + ii * YS);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < R; ++c) dMk[row * R + c] = dm[c] + sOut[tid * (R + 1) + c];
    if constexpr (LOCAL) {
#pragma unroll
        for (int c = 0; c < 64; ++c) dXl[row * 64 + c] = dxl[c];
    }
    const int64_t o = sl.row(bh, l * b + j_blk);
#pragma unroll
    for (int c = 0; c < 64; ++c) stf(dV + o + c, dv[c]);
}

// ---------------------------------------------------------------------------
// Chain rule through the half sketch: dX = ((dM*A2) G1^T + (dM*A1) G2^T)/sqrt(r),
// A1 = X G1, A2 = X G2 recomputed.  64 rows per CTA.  `add` (optional, [rows][64]): gradient
// that reached X without passing through the sketch, added before the result is rounded.
// ---------------------------------------------------------------------------
template <typename T, int R>
__global__ void __launch_bounds__(256)
sketch_bwd_kernel(Slice sl, const T* __restrict__ X, const T* __restrict__ G1, const T* __restrict__ G2,
                  int g_heads, int n, const float* __restrict__ dM, const float* __restrict__ add,
                  T* __restrict__ dX) {
    extern __shared__ float smem[];
    float* sG1 = smem;                      // [64][R+1]
    float* sG2 = sG1 + H64 * (R + 1);       // [64][R+1]
    float* sX = sG2 + H64 * (R + 1);        // [64][65]
    float* sU1 = sX + 64 * 65;              // [64][R+1]
    float* sU2 = sU1 + 64 * (R + 1);        // [64][R+1]
    const int bh = blockIdx.y, i0 = blockIdx.x * 64, tid = threadIdx.x;
    const int g = (g_heads == 1) ? 0 : (bh % sl.H);
    for (int e = tid; e < H64 * R; e += 256) {
        sG1[(e / R) * (R + 1) + e % R] = ldf(G1 + (size_t)g * H64 * R + e);
        sG2[(e / R) * (R + 1) + e % R] = ldf(G2 + (size_t)g * H64 * R + e);
    }
    for (int e = tid; e < 64 * H64; e += 256) {
        const int rr = e / H64, c = e % H64;
        sX[rr * 65 + c] = ldf(X + sl.row(bh, i0 + rr) + c);
    }
    __syncthreads();
    const float rs = rsqrtf((float)R);
    {
        const int c = tid % R;
        for (int rr = tid / R; rr < 64; rr += 256 / R) {
            float a1 = 0.f, a2 = 0.f;
#pragma unroll 16
            for (int t = 0; t < H64; ++t) {
                const float x = sX[rr * 65 + t];
                a1 = fmaf(x, sG1[t * (R + 1) + c], a1);
                a2 = fmaf(x, sG2[t * (R + 1) + c], a2);
            }
            const float g_m = dM[((size_t)bh * n + i0 + rr) * R + c] * rs;
            sU1[rr * (R + 1) + c] = g_m * a2;
            sU2[rr * (R + 1) + c] = g_m * a1;
        }
    }
    __syncthreads();
    {
        const int t = tid % 64;
        for (int rr = tid / 64; rr < 64; rr += 4) {
            float dx = add != nullptr ? add[((size_t)bh * n + i0 + rr) * 64 + t] : 0.f;
#pragma unroll 16
            for (int c = 0; c < R; ++c) {
                dx = fmaf(sU1[rr * (R + 1) + c], sG1[t * (R + 1) + c], dx);
                dx = fmaf(sU2[rr * (R + 1) + c], sG2[t * (R + 1) + c], dx);
            }
            stf(dX + sl.row(bh, i0 + rr) + t, dx);
        }
    }
}

// ---------------------------------------------------------------------------
// host-side launch helpers
// ---------------------------------------------------------------------------
#define PSK_TRY(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return e_; } while (0)

template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

template <typename T, int R>
cudaError_t launch_sketch(const Dims& d, const T* X, const T* G1, const T* G2, float* M, float* Phi,
                          cudaStream_t s, int* launches) {
    if (d.learned) return learned_sketch(d, X, M, Phi, s, launches);      // Algorithm 2: two dense networks
    if (d.p == 2) {           // M = X (R = 64 = h)
        const int rows = d.BH() * d.n;
        prof_begin("identity_sketch_kernel", s);
        identity_sketch_kernel<T><<<(rows + 7) / 8, 256, 0, s>>>(Slice{d.H, d.sb, d.sh, d.sn}, d.n, rows, X, M, Phi);
        prof_end(s);
        ++*launches;
        return cudaGetLastError();
    }
    if (d.p == 8) {           // one more recursion level: packed Gaussians [Ga; Gb; Gc]
        PSK_TRY((allow_smem(sketch8_kernel<T, R>, Sk8<R>::bytes)));
        prof_begin("sketch8_kernel", s);
        sketch8_kernel<T, R><<<dim3(d.n / Sk8<R>::kRows, d.BH()), 256, Sk8<R>::bytes, s>>>(
            Slice{d.H, d.sb, d.sh, d.sn}, X, G1, G2, d.g_heads, d.n, M, Phi);
        prof_end(s);
        ++*launches;
        return cudaGetLastError();
    }
    const size_t smem = (size_t)(2 * H64 * R + 64 * 65 + 64 * (R + 1)) * sizeof(float);
    PSK_TRY(allow_smem(sketch_kernel<T, R>, smem));
    Slice sl{d.H, d.sb, d.sh, d.sn};
    prof_begin("sketch_kernel", s);
    sketch_kernel<T, R><<<dim3(d.n / 64, d.BH()), 256, smem, s>>>(sl, X, G1, G2, d.g_heads, d.n, M, Phi);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <int R>
cudaError_t launch_states(const Dims& d, const float* M, const float* Y, float* S, bool reverse,
                          cudaStream_t s, int* launches) {
    prof_begin("state_kernel", s);
    state_kernel<R><<<dim3((R * R + 127) / 128, d.t, d.BH()), 128, 0, s>>>(M, Y, d.n, d.b, d.t, S);
    prof_end(s);
    ++*launches;
    PSK_TRY(cudaGetLastError());
    const size_t elems = (size_t)R * R * YC;
    prof_begin("scan_kernel", s);
    scan_kernel<<<dim3((unsigned)((elems + 255) / 256), d.BH()), 256, 0, s>>>(S, elems, d.t, reverse ? 1 : 0);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <typename T, int R>
cudaError_t fwd_impl(const Dims& d, const T* Q, const T* K, const T* V, const T* G1, const T* G2,
                     T* O, float* denom, char* ws, cudaStream_t s, int* launches) {
    const CcWorkspace w = cc_workspace(d, false);
    float* Mq = (float*)(ws + w.Mq); float* Mk = (float*)(ws + w.Mk);
    float* Vt = (float*)(ws + w.Vt); float* Z = (float*)(ws + w.Zst);
    Slice sl{d.H, d.sb, d.sh, d.sn};
    const int rows = d.BH() * d.n;
    PSK_TRY((launch_sketch<T, R>(d, Q, G1, G2, Mq, nullptr, s, launches)));
    PSK_TRY((launch_sketch<T, R>(d, K, G1, G2, Mk, nullptr, s, launches)));
    prof_begin("rows_prep_kernel", s);
    rows_prep_kernel<T><<<(rows + 7) / 8, 256, 0, s>>>(sl, d.n, rows, 0, V, nullptr, nullptr, nullptr, Vt);
    prof_end(s);
    ++*launches;
    PSK_TRY(cudaGetLastError());
    PSK_TRY((launch_states<R>(d, Mk, Vt, Z, false, s, launches)));
    prof_begin("fwd_out_kernel", s);
    if (d.local) {
        PSK_TRY((allow_smem(fwd_out_kernel<T, R, true>, RowSmem<R>::bytes_local)));
        fwd_out_kernel<T, R, true><<<dim3(d.b / 128, d.t, d.BH()), 128, RowSmem<R>::bytes_local, s>>>(
            sl, d.n, d.b, d.t, Mq, Mk, Vt, Z, Q, K, O, denom);
    } else {
        PSK_TRY((allow_smem(fwd_out_kernel<T, R, false>, RowSmem<R>::bytes)));
        fwd_out_kernel<T, R, false><<<dim3(d.b / 128, d.t, d.BH()), 128, RowSmem<R>::bytes, s>>>(
            sl, d.n, d.b, d.t, Mq, Mk, Vt, Z, Q, K, O, denom);
    }
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

// Chain rule through the half sketch of one tensor: dX from dM (+ `add`, the part of the gradient
// that reached X directly through exact same-block weights).
template <typename T, int R>
cudaError_t launch_sketch_bwd(const Dims& d, const T* X, const T* G1, const T* G2, const float* dM, const float* add,
                              T* dX, cudaStream_t s, int* launches) {
    Slice sl{d.H, d.sb, d.sh, d.sn};
    const int rows = d.BH() * d.n;
    if (d.learned) return learned_sketch_bwd(d, X, dM, add, dX, s, launches);     // two networks; gradients add up
    if (d.p == 2) {           // dX = dM (+ add)
        prof_begin("identity_sketch_bwd_kernel", s);
        identity_sketch_bwd_kernel<T><<<(rows + 7) / 8, 256, 0, s>>>(sl, d.n, rows, dM, add, dX);
        prof_end(s);
        ++*launches;
        return cudaGetLastError();
    }
    if (d.p == 8) {
        PSK_TRY((allow_smem(sketch8_bwd_kernel<T, R>, Sk8<R>::bytes)));
        prof_begin("sketch8_bwd_kernel", s);
        sketch8_bwd_kernel<T, R><<<dim3(d.n / Sk8<R>::kRows, d.BH()), 256, Sk8<R>::bytes, s>>>(sl, X, G1, G2, d.g_heads, d.n, dM, dX);
        prof_end(s);
        ++*launches;
        return cudaGetLastError();
    }
    const size_t smem = (size_t)(2 * H64 * (R + 1) + 64 * 65 + 2 * 64 * (R + 1)) * sizeof(float);
    PSK_TRY(allow_smem(sketch_bwd_kernel<T, R>, smem));
    prof_begin("sketch_bwd_kernel", s);
    sketch_bwd_kernel<T, R><<<dim3(d.n / 64, d.BH()), 256, smem, s>>>(sl, X, G1, G2, d.g_heads, d.n, dM, add, dX);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <typename T, int R>
cudaError_t bwd_impl(const Dims& d, const T* Q, const T* K, const T* V, const T* G1, const T* G2,
                     const T* O, const float* denom, const T* dO, T* dQ, T* dK, T* dV,
                     char* ws, cudaStream_t s, int* launches) {
    const CcWorkspace w = cc_workspace(d, true);
    float* Mq = (float*)(ws + w.Mq); float* Mk = (float*)(ws + w.Mk);
    float* Vt = (float*)(ws + w.Vt); float* Z = (float*)(ws + w.Zst);
    float* E = (float*)(ws + w.E); float* Rs = (float*)(ws + w.Rst);
    float* dMq = (float*)(ws + w.dMq); float* dMk = (float*)(ws + w.dMk);
    Slice sl{d.H, d.sb, d.sh, d.sn};
    const int rows = d.BH() * d.n;
    PSK_TRY((launch_sketch<T, R>(d, Q, G1, G2, Mq, nullptr, s, launches)));
    PSK_TRY((launch_sketch<T, R>(d, K, G1, G2, Mk, nullptr, s, launches)));
    prof_begin("rows_prep_kernel", s);
    rows_prep_kernel<T><<<(rows + 7) / 8, 256, 0, s>>>(sl, d.n, rows, 0, V, nullptr, nullptr, nullptr, Vt);
    prof_end(s);
    prof_begin("rows_prep_kernel", s);
    rows_prep_kernel<T><<<(rows + 7) / 8, 256, 0, s>>>(sl, d.n, rows, 1, nullptr, O, denom, dO, E);
    prof_end(s);
    *launches += 2;
    PSK_TRY(cudaGetLastError());
    PSK_TRY((launch_states<R>(d, Mk, Vt, Z, false, s, launches)));
    PSK_TRY((launch_states<R>(d, Mq, E, Rs, true, s, launches)));
    const dim3 grid(d.b / 128, d.t, d.BH());
    float* dXq = d.local ? (float*)(ws + w.dXq) : nullptr;
    float* dXk = d.local ? (float*)(ws + w.dXk) : nullptr;
    if (d.local) {
        PSK_TRY((allow_smem(bwd_q_kernel<T, R, true>, RowSmem<R>::bytes_local)));
        PSK_TRY((allow_smem(bwd_k_kernel<T, R, true>, RowSmem<R>::bytes_local)));
        prof_begin("bwd_q_kernel", s);
        bwd_q_kernel<T, R, true><<<grid, 128, RowSmem<R>::bytes_local, s>>>(sl, d.n, d.b, d.t, Mq, Mk, Vt, E, Z, Q, K, dMq, dXq);
        prof_end(s);
        prof_begin("bwd_k_kernel", s);
        bwd_k_kernel<T, R, true><<<grid, 128, RowSmem<R>::bytes_local, s>>>(sl, d.n, d.b, d.t, Mq, Mk, Vt, E, Rs, Q, K, dMk, dXk, dV);
        prof_end(s);
    } else {
        PSK_TRY((allow_smem(bwd_q_kernel<T, R, false>, RowSmem<R>::bytes)));
        PSK_TRY((allow_smem(bwd_k_kernel<T, R, false>, RowSmem<R>::bytes)));
        prof_begin("bwd_q_kernel", s);
        bwd_q_kernel<T, R, false><<<grid, 128, RowSmem<R>::bytes, s>>>(sl, d.n, d.b, d.t, Mq, Mk, Vt, E, Z, Q, K, dMq, nullptr);
        prof_end(s);
        prof_begin("bwd_k_kernel", s);
        bwd_k_kernel<T, R, false><<<grid, 128, RowSmem<R>::bytes, s>>>(sl, d.n, d.b, d.t, Mq, Mk, Vt, E, Rs, Q, K, dMk, nullptr, dV);
        prof_end(s);
    }
    *launches += 2;
    PSK_TRY(cudaGetLastError());
    PSK_TRY((launch_sketch_bwd<T, R>(d, Q, G1, G2, dMq, dXq, dQ, s, launches)));
    return launch_sketch_bwd<T, R>(d, K, G1, G2, dMk, dXk, dK, s, launches);
}

#define PSK_DISPATCH(CALL_F32, CALL_BF16)                                   \
    if (d.bf16) {                                                           \
        typedef __nv_bfloat16 T;                                            \
        switch (d.r) { case 16: { constexpr int R = 16; return CALL_BF16; } \
                       case 32: { constexpr int R = 32; return CALL_BF16; } \
                       case 64: { constexpr int R = 64; return CALL_BF16; } } \
    } else {                                                                \
        typedef float T;                                                    \
        switch (d.r) { case 16: { constexpr int R = 16; return CALL_F32; }  \
                       case 32: { constexpr int R = 32; return CALL_F32; }  \
                       case 64: { constexpr int R = 64; return CALL_F32; } } \
    }                                                                       \
    return cudaErrorInvalidValue;

}  // namespace

cudaError_t cc_sketch(const Dims& d, const void* X, const void* G1, const void* G2,
                      float* M_out, float* Phi_out, cudaStream_t s, int* launches) {
#define C_ (launch_sketch<T, R>(d, (const T*)X, (const T*)G1, (const T*)G2, M_out, Phi_out, s, launches))
    PSK_DISPATCH(C_, C_)
#undef C_
}

cudaError_t cc_sketch_bwd(const Dims& d, const void* X, const void* G1, const void* G2, const float* dM,
                          const float* add, void* dX, cudaStream_t s, int* launches) {
#define C_ (launch_sketch_bwd<T, R>(d, (const T*)X, (const T*)G1, (const T*)G2, dM, add, (T*)dX, s, launches))
    PSK_DISPATCH(C_, C_)
#undef C_
}

cudaError_t cc_fwd(const Dims& d, const void* Q, const void* K, const void* V,
                   const void* G1, const void* G2, void* O, float* denom,
                   char* ws, cudaStream_t s, int* launches) {
#define C_ (fwd_impl<T, R>(d, (const T*)Q, (const T*)K, (const T*)V, (const T*)G1, (const T*)G2, \
                           (T*)O, denom, ws, s, launches))
    PSK_DISPATCH(C_, C_)
#undef C_
}

cudaError_t cc_bwd(const Dims& d, const void* Q, const void* K, const void* V,
                   const void* G1, const void* G2, const void* O, const float* denom,
                   const void* dO, void* dQ, void* dK, void* dV,
                   char* ws, cudaStream_t s, int* launches) {
#define C_ (bwd_impl<T, R>(d, (const T*)Q, (const T*)K, (const T*)V, (const T*)G1, (const T*)G2, \
                           (const T*)O, denom, (const T*)dO, (T*)dQ, (T*)dK, (T*)dV, ws, s, launches))
    PSK_DISPATCH(C_, C_)
#undef C_
}

}  // namespace psk
