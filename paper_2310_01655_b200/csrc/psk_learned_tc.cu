// Learnable sketch (Algorithm 2 of the paper's appendix) with its dense layers on the tensor
// cores: bf16 operands, fp32 accumulation in tensor memory, r <= 32 (8r <= 256), h = 64.
//
//   f(x) = W4^T gelu(W3^T (W2^T LN1(gelu(W1^T LN0(x) + b1)) + b2) + b3) + b4      (two such networks)
//   M    = sqrt(r) tanh(f_1(x) * f_2(x) / sqrt(r))
//
// Rows are processed in chunks; inside a chunk every layer is one launch (ltc_wide_kernel,
// ltc_narrow_kernel, ltc_dense_kernel; 128 rows per tile: activations by TMA, the layer's weights
// as the MN-major B operand, the accumulator read back by thread = row, where bias, gelu and the
// layer normalisations are plain per-thread loops), with the activations the backward needs
// kept in the workspace as bf16.
// The gains of the normalisations are folded into the following layer's weights
// (z W = n (diag(g) W) + c W), so the normalised activations n are the GEMM operands and
// their gradients come out of the GEMM with the gain already applied.  Weight gradients are
// sums over ALL rows of outer products: ltc_wgrad_kernel accumulates P^T S over a slab of rows in
// tensor memory and adds the result to an fp32 accumulator once per slab, and sums the delta
// operand's columns from the same tiles; gains, biases and the folded terms are taken from those
// accumulators and sums by a last small kernel.
// Every r-wide array is padded to 64 columns and every 8r-wide one to 256 (zeros), so two GEMM
// shapes, 64 -> 256 and 256 -> 64, serve all sixteen layer passes.
#include "tc_common.cuh"

#include <cstdlib>

namespace psk {

namespace {

using namespace tc;

constexpr float kLnEps = 1e-6f;
constexpr size_t kChunkRows = (size_t)1 << 20;        // rows per pass over the layers
constexpr int kMat = 64 * 256;                        // elements of one operand matrix
constexpr int kBank = 12;                             // operand matrices per network
constexpr int kVec = 256 + 64 + 256 + 64;             // folded biases of one network: b1' | b2' | b3 | b4
constexpr int kSums = 256 + 64 + 256 + 64;            // column sums of one network: dp1 | da2 | dp3 | df

// gelu(x) = x Phi(x) and its derivative Phi(x) + x phi(x).  erfc(z), z = |x| / sqrt(2), by the
// five-term rational approximation in t = 1 / (1 + 0.3275911 z) (absolute error 1.5e-7); its
// exponential exp(-z^2) = exp(-x^2 / 2) is the normal density's too.  With E = erfc(z):
//   gelu(x) = max(x, 0) - |x| E / 2,     Phi(x) = 1/2 + copysign(1/2 - E/2, x).
__device__ __forceinline__ float rcp_approx(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float ex2_approx(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
// half of erfc(|x| / sqrt(2)) and exp(-x^2 / 2)
__device__ __forceinline__ float half_erfc(float ax, float& e) {
    const float z = ax * 0.70710678118654752f;
    const float t = rcp_approx(fmaf(0.3275911f, z, 1.f));
    e = ex2_approx(z * z * -1.4426950408889634f);
    float poly = fmaf(0.5f * 1.061405429f, t, 0.5f * -1.453152027f);
    poly = fmaf(poly, t, 0.5f * 1.421413741f);
    poly = fmaf(poly, t, 0.5f * -0.284496736f);
    poly = fmaf(poly, t, 0.5f * 0.254829592f);
    return poly * t * e;
}
__device__ __forceinline__ float gelu_f(float x) {
    float e;
    const float ax = fabsf(x);
    return fmaf(-ax, half_erfc(ax, e), fmaxf(x, 0.f));
}
__device__ __forceinline__ float gelu_grad_f(float x) {
    float e;
    const float q = half_erfc(fabsf(x), e);
    return fmaf(x, 0.3989422804014327f * e, 0.5f + copysignf(0.5f - q, x));
}

struct NetLayout {
    int h, r, m;
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

// ---------------------------------------------------------------------------
// operand bank: per network eight bf16 matrices and the folded biases
//   0: diag(g0) W1  [64][256]     4: W4^T           [64][256]
//   1: diag(g1) W2  [256][64]     5: W3^T           [256][64]
//   2: W3           [64][256]     6: (diag(g1) W2)^T [64][256]
//   3: W4           [256][64]     7: (diag(g0) W1)^T [256][64]
//   8..11: what rounding 0..3 to bf16 left over (the forward multiplies by hi + lo)
// (rows / columns beyond r or 8r are zero)
// ---------------------------------------------------------------------------
__device__ float bank_entry(const NetLayout& nl, const float* P, int which, int row, int col) {
    const int r = nl.r, m = nl.m;
    switch (which) {
        case 0: return col < m ? P[nl.g0 + row] * P[nl.W1 + row * m + col] : 0.f;                  // [k][j]
        case 1: return (row < m && col < r) ? P[nl.g1 + row] * P[nl.W2 + row * r + col] : 0.f;      // [j][c]
        case 2: return (row < r && col < m) ? P[nl.W3 + row * m + col] : 0.f;                       // [c][j]
        case 3: return (row < m && col < r) ? P[nl.W4 + row * r + col] : 0.f;                       // [j][c]
        case 4: return (col < m && row < r) ? P[nl.W4 + col * r + row] : 0.f;                       // [c][j]
        case 5: return (row < m && col < r) ? P[nl.W3 + col * m + row] : 0.f;                       // [j][c]
        case 6: return (col < m && row < r) ? P[nl.g1 + col] * P[nl.W2 + col * r + row] : 0.f;      // [c][j]
        default: return row < m ? P[nl.g0 + col] * P[nl.W1 + col * m + row] : 0.f;                  // [j][k]
    }
}

__global__ void __launch_bounds__(256)
ltc_bank_kernel(int h, int r, const float* __restrict__ params, bf16* __restrict__ bank, float* __restrict__ vec) {
    const NetLayout nl(h, r);
    const int net = blockIdx.y;
    const float* P = params + (size_t)net * nl.count;
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e < 8 * kMat) {
        const int which = e / kMat, idx = e % kMat;
        const int cols = (which % 2 == 0) ? 256 : 64;
        const float v = bank_entry(nl, P, which, idx / cols, idx % cols);
        const bf16 hi = __float2bfloat16_rn(v);
        bank[(size_t)net * kBank * kMat + e] = hi;
        if (which < 4) bank[(size_t)net * kBank * kMat + 8 * kMat + e] = __float2bfloat16_rn(v - __bfloat162float(hi));
    } else if (e < 8 * kMat + kVec) {
        const int v = e - 8 * kMat;
        float out = 0.f;
        if (v < 256) {                                   // b1' = c0 W1 + b1
            if (v < nl.m) { out = P[nl.b1 + v]; for (int k = 0; k < h; ++k) out = fmaf(P[nl.c0 + k], P[nl.W1 + k * nl.m + v], out); }
        } else if (v < 320) {                            // b2' = c1 W2 + b2
            const int c = v - 256;
            if (c < r) { out = P[nl.b2 + c]; for (int j = 0; j < nl.m; ++j) out = fmaf(P[nl.c1 + j], P[nl.W2 + j * r + c], out); }
        } else if (v < 576) {
            if (v - 320 < nl.m) out = P[nl.b3 + v - 320];
        } else {
            if (v - 576 < r) out = P[nl.b4 + v - 576];
        }
        vec[(size_t)net * kVec + v] = out;
    }
}

// ---------------------------------------------------------------------------
// dense layer: Out[128 rows x ND] = epilogue(A[128 x KD] B[KD x ND])
// ---------------------------------------------------------------------------
enum { EPI_LN = 0, EPI_B64 = 1, EPI_GELU = 2, EPI_F32 = 3, EPI_DGELU = 4, EPI_LNBWD = 5 };

struct DenseArgs {
    const float* bias;      // [64] or null
    bf16* out0;             // EPI_B64: [rows][64] bf16 (the forward's narrow layers: the hi terms)
    bf16* out1;             //          the lo terms (forward only)
    float* outf;            // EPI_F32: [rows][ncols]
    int ncols;              // EPI_F32: columns stored
    int accumulate;         // EPI_F32: add to what is there (backward only)
};

__device__ __forceinline__ void store8(bf16* dst, const float* v) {
    *reinterpret_cast<uint4*>(dst) = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
// v = hi + lo as two bf16 terms
__device__ __forceinline__ void store8_split(bf16* hi, bf16* lo, const float* v) {
    float h[8], l[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { h[i] = __bfloat162float(__float2bfloat16_rn(v[i])); l[i] = v[i] - h[i]; }
    store8(hi, h);
    store8(lo, l);
}
// (The forward's layers multiply hi + lo pairs of bf16 arrays for both activations and weights,
// A_hi B_hi + A_lo B_hi + A_hi B_lo: a half sketch feeds fourth powers of cancelling sums, and
// single bf16 operands, 2^-9 per entry and four layers deep, would leave percents of error on the
// attention's output; the pairs leave 2^-17.  The backward's deltas are single bf16.)
//
// Narrow layers of the backward (256 -> 64, single operands): one tile per CTA, 128 threads.
constexpr int kDenseSmem = 128 * 256 * 2 + 256 * 64 * 2 + 1024;

template <int EPI>
__global__ void __launch_bounds__(128)
ltc_dense_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mB, DenseArgs a, int* status) {
    static_assert(EPI == EPI_B64 || EPI == EPI_F32, "the 256 -> 64 layers");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sA = align1024(smem_raw);
    uint8_t* sB = sA + 65536;
    __shared__ uint64_t bar_ld, bar_mma;
    __shared__ uint32_t tm_slot;
    __shared__ float s_bias[64];
    const int tid = threadIdx.x, warp = tid / 32;
    const int tile = blockIdx.x;
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_ld, 1); mbar_init(&bar_mma, 1);
        mbar_fence_init();
    }
    if (warp == 0) { tmem_alloc(&tm_slot, 64); tmem_relinquish(); }
    if (tid < 64) s_bias[tid] = a.bias != nullptr ? a.bias[tid] : 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot;
    if (tid == 0) {
        mbar_expect_tx(&bar_ld, 65536 + 32768);
#pragma unroll
        for (int s = 0; s < 4; ++s) tma_load_2d(sA + s * 16384, &mA, s * 64, tile * 128, &bar_ld);
        tma_load_2d(sB, &mB, 0, 0, &bar_ld);
        if (mbar_wait(&bar_ld, 0, status, kErrTma)) {
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
            const uint64_t ad = smem_desc(smem_u32(sA), 0, 1024, kSwz128);
            const uint64_t bd = smem_desc(smem_u32(sB), 0, 1024, kSwz128);
#pragma unroll
            for (int k = 0; k < 16; ++k)
                umma_ss(tm, desc_off(ad, (k / 4) * 16384 + (k % 4) * 32), desc_off(bd, k * 2048), idesc, k > 0);
            umma_commit(&bar_mma);
        }
    }
    const bool ok = mbar_wait(&bar_mma, 0, status, kErrMma);
    tc_fence_after();
    const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
    const size_t row = (size_t)tile * 128 + tid;
    if (ok) {
        if constexpr (EPI == EPI_B64) {
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t u[32];
                tmem_ld32(lane_tm + c0, u);
                tmem_ld_wait();
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(u[j]) + s_bias[c0 + j];
#pragma unroll
                for (int j = 0; j < 32; j += 8) store8(a.out0 + row * 64 + c0 + j, v + j);
            }
        } else {
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                if (c0 < a.ncols) {
                    uint32_t u[32];
                    tmem_ld32(lane_tm + c0, u);
                    tmem_ld_wait();
                    float* dst = a.outf + row * a.ncols + c0;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        if (c0 + j < a.ncols) {
                            float4 o = make_float4(__uint_as_float(u[j]) + s_bias[c0 + j], __uint_as_float(u[j + 1]) + s_bias[c0 + j + 1],
                                                   __uint_as_float(u[j + 2]) + s_bias[c0 + j + 2], __uint_as_float(u[j + 3]) + s_bias[c0 + j + 3]);
                            if (a.accumulate) {
                                const float4 p = *reinterpret_cast<const float4*>(dst + j);
                                o.x += p.x; o.y += p.y; o.z += p.z; o.w += p.w;
                            }
                            *reinterpret_cast<float4*>(dst + j) = o;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 64);
}

// ---------------------------------------------------------------------------
// narrow layers of the forward (256 -> 64, hi + lo pairs): persistent, one CTA per SM.  The layer's
// weights stay in shared memory; the activation tiles stream through a four-stage ring of
// 64-column chunks (hi and lo, 32 KB a stage) that the producer thread keeps full across tile
// boundaries; the accumulator is double-buffered in tensor memory, so the rows' epilogue of one
// tile runs under the loads and MMAs of the next.  Warps 0-3: epilogue (thread = row); warp 4: TMA
// producer; warp 5: MMA issuer.
// ---------------------------------------------------------------------------
constexpr int kNrStages = 4, kNrStage = 32768;
constexpr int kNrSmem = 65536 + kNrStages * kNrStage + 1024;

template <int EPI>
__global__ void __launch_bounds__(192, 1)
ltc_narrow_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mA2,
                  const __grid_constant__ CUtensorMap mB, const __grid_constant__ CUtensorMap mB2, DenseArgs a, int tiles,
                  int* status) {
    static_assert(EPI == EPI_B64 || EPI == EPI_F32, "the 256 -> 64 layers");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sB = align1024(smem_raw);
    uint8_t* sR = sB + 65536;
    __shared__ uint64_t bar_b, bar_full[kNrStages], bar_empty[kNrStages], bar_accfull[2], bar_accfree[2];
    __shared__ uint32_t tm_slot;
    __shared__ float s_bias[64];
    const int tid = threadIdx.x, warp = tid / 32;
    const int ntl = (tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_b, 1);
        for (int s = 0; s < kNrStages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(&bar_accfull[0], 1); mbar_init(&bar_accfull[1], 1);
        mbar_init(&bar_accfree[0], 128); mbar_init(&bar_accfree[1], 128);
        mbar_fence_init();
    }
    if (warp == 0) { tmem_alloc(&tm_slot, 128); tmem_relinquish(); }
    if (tid < 64) s_bias[tid] = a.bias != nullptr ? a.bias[tid] : 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot;
    if (tid == 128) {
        // ---- producer ----
        mbar_expect_tx(&bar_b, 65536);
        tma_load_2d(sB, &mB, 0, 0, &bar_b);
        tma_load_2d(sB + 32768, &mB2, 0, 0, &bar_b);
        bool ok = true;
        int it = 0;
        for (int i = 0; i < ntl && ok; ++i) {
            const int tile = blockIdx.x + i * gridDim.x;
            for (int c = 0; c < 4 && ok; ++c, ++it) {
                const int s = it % kNrStages;
                if (it >= kNrStages) ok = mbar_spin(&bar_empty[s], ((it / kNrStages) - 1) & 1, status, kErrMma);
                if (!ok) break;
                mbar_expect_tx(&bar_full[s], kNrStage);
                tma_load_2d(sR + s * kNrStage, &mA, c * 64, tile * 128, &bar_full[s]);
                tma_load_2d(sR + s * kNrStage + 16384, &mA2, c * 64, tile * 128, &bar_full[s]);
            }
        }
    } else if (tid == 160) {
        // ---- MMA issuer ----
        constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
        bool ok = mbar_spin(&bar_b, 0, status, kErrTma);
        const uint64_t bhi = smem_desc(smem_u32(sB), 0, 1024, kSwz128);
        const uint64_t blo = smem_desc(smem_u32(sB) + 32768, 0, 1024, kSwz128);
        int it = 0;
        for (int i = 0; i < ntl && ok; ++i) {
            const int buf = i & 1;
            if (i >= 2) ok = mbar_spin(&bar_accfree[buf], ((i / 2) - 1) & 1, status, kErrMma);
            for (int c = 0; c < 4 && ok; ++c, ++it) {
                const int s = it % kNrStages;
                ok = mbar_spin(&bar_full[s], (it / kNrStages) & 1, status, kErrTma);
                if (!ok) break;
                tc_fence_after();
                const uint64_t ahi = smem_desc(smem_u32(sR) + s * kNrStage, 0, 1024, kSwz128);
                const uint64_t alo = smem_desc(smem_u32(sR) + s * kNrStage + 16384, 0, 1024, kSwz128);
#pragma unroll
                for (int part = 0; part < 3; ++part) {
                    const uint64_t ad = part == 1 ? alo : ahi;
                    const uint64_t bd = part == 2 ? blo : bhi;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_ss(tm + buf * 64, desc_off(ad, k * 32), desc_off(bd, c * 8192 + k * 2048), idesc,
                                (c > 0 || part > 0 || k > 0) ? 1u : 0u);
                }
                umma_commit(&bar_empty[s]);
            }
            if (ok) umma_commit(&bar_accfull[buf]);
        }
    } else if (warp < 4) {
        // ---- epilogue ----
        const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
        for (int i = 0; i < ntl && ok; ++i) {
            const int buf = i & 1;
            const size_t row = (size_t)(blockIdx.x + i * gridDim.x) * 128 + tid;
            ok = mbar_wait(&bar_accfull[buf], (i / 2) & 1, status, kErrMma);
            if (!ok) break;
            tc_fence_after();
            if constexpr (EPI == EPI_B64) {
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t u[32];
                    tmem_ld32(lane_tm + buf * 64 + c0, u);
                    tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(u[j]) + s_bias[c0 + j];
#pragma unroll
                    for (int j = 0; j < 32; j += 8) store8_split(a.out0 + row * 64 + c0 + j, a.out1 + row * 64 + c0 + j, v + j);
                }
            } else {
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    if (c0 < a.ncols) {
                        uint32_t u[32];
                        tmem_ld32(lane_tm + buf * 64 + c0, u);
                        tmem_ld_wait();
                        float* dst = a.outf + row * a.ncols + c0;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (c0 + j < a.ncols)
                                *reinterpret_cast<float4*>(dst + j) =
                                    make_float4(__uint_as_float(u[j]) + s_bias[c0 + j], __uint_as_float(u[j + 1]) + s_bias[c0 + j + 1],
                                                __uint_as_float(u[j + 2]) + s_bias[c0 + j + 2], __uint_as_float(u[j + 3]) + s_bias[c0 + j + 3]);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&bar_accfree[buf]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 128);
}

// ---------------------------------------------------------------------------
// wide layer: Out[128 rows x 256] = epilogue(A[128 x 64] B[64 x 256]).  256 threads: the two
// warpgroups share the rows (thread = row) and take two 64-column groups each; every output
// leaves as TMA stores of [128 x 64] tiles staged in shared memory.  SPLIT (forward): hi + lo
// operand pairs, the staging tiles lie over the operands (dead once the MMAs have completed).
// Backward: single operands, side tiles (the forward's activations) by TMA, the output written
// in place over the side tile it consumed.
// ---------------------------------------------------------------------------
struct WideArgs {
    const float* bias;      // [256] or null
    float* rs_out;          // EPI_LN: 1 / sigma of every row
    const float* rs_in;     // EPI_LNBWD
    int ncols;              // live columns (8r)
    int keep_pre;           // EPI_LN, EPI_GELU: also store the pre-activation (output 0), which only the backward reads
};

template <int EPI, bool SPLIT>
struct WideSmem {
    static constexpr int kA1 = 16384, kB1 = 32768;
    static constexpr int kA = kA1 * (SPLIT ? 2 : 1), kB = kB1 * (SPLIT ? 2 : 1);
    static constexpr int kSides = EPI == EPI_DGELU ? 1 : (EPI == EPI_LNBWD ? 2 : 0);
    static constexpr int bytes = kA + kB + kSides * 65536 + 1024;
    static_assert(!SPLIT || kA + kB == 2 * 3 * 16384, "three staging tiles per warpgroup over the operands");
    static_assert(SPLIT == (kSides == 0), "forward: pairs and no side tiles; backward: the reverse");
};

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, const void* src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(src)), "r"(c0), "r"(c1)
                 : "memory");
}
// 8 consecutive columns of a row of a 128-byte-swizzled [128 x 64] bf16 tile
__device__ __forceinline__ void tile_put8(uint8_t* tile, int row, int chunk, const float* v) {
    *reinterpret_cast<uint4*>(tile + swz128_offset(row, chunk)) =
        make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
// v = hi + lo: one packed conversion gives two hi terms, whose float values are the halves of that word
__device__ __forceinline__ void tile_put8_split(uint8_t* hi_tile, uint8_t* lo_tile, int row, int chunk, const float* v) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        h[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
        l[i] = pack_bf16(v[2 * i] - __uint_as_float(h[i] << 16), v[2 * i + 1] - __uint_as_float(h[i] & 0xffff0000u));
    }
    const uint32_t o = swz128_offset(row, chunk);
    *reinterpret_cast<uint4*>(hi_tile + o) = make_uint4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<uint4*>(lo_tile + o) = make_uint4(l[0], l[1], l[2], l[3]);
}
__device__ __forceinline__ void tile_get8(const uint8_t* tile, int row, int chunk, float* v) {
    const uint4 q = *reinterpret_cast<const uint4*>(tile + swz128_offset(row, chunk));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// FULL: all 256 columns are live (8r = 256), no masks
template <int EPI, bool SPLIT, bool FULL>
__global__ void __launch_bounds__(256)
ltc_wide_kernel(const __grid_constant__ CUtensorMap mA, const __grid_constant__ CUtensorMap mA2,
                const __grid_constant__ CUtensorMap mB, const __grid_constant__ CUtensorMap mB2,
                const __grid_constant__ CUtensorMap mS0, const __grid_constant__ CUtensorMap mS1,
                const __grid_constant__ CUtensorMap mO0, const __grid_constant__ CUtensorMap mO1,
                const __grid_constant__ CUtensorMap mO2, WideArgs a, int* status) {
    using L = WideSmem<EPI, SPLIT>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sA = align1024(smem_raw);
    uint8_t* sB = sA + L::kA;
    uint8_t* sS = sB + L::kB;
    __shared__ uint64_t bar_ld, bar_side, bar_mma;
    __shared__ uint32_t tm_slot;
    __shared__ __align__(16) float s_bias[256];
    __shared__ float2 s_part[2][128];
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int wg = warp / 4, rowt = (warp % 4) * 32 + lane;
    const int tile = blockIdx.x;
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_ld, 1); mbar_init(&bar_side, 1); mbar_init(&bar_mma, 1);
        mbar_fence_init();
    }
    if (warp == 0) { tmem_alloc(&tm_slot, 256); tmem_relinquish(); }
    s_bias[tid] = a.bias != nullptr ? a.bias[tid] : 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot;
    if (tid == 0) {
        mbar_expect_tx(&bar_ld, L::kA + L::kB);
        tma_load_2d(sA, &mA, 0, tile * 128, &bar_ld);
#pragma unroll
        for (int g = 0; g < 4; ++g) tma_load_2d(sB + g * 8192, &mB, g * 64, 0, &bar_ld);
        if constexpr (SPLIT) {
            tma_load_2d(sA + L::kA1, &mA2, 0, tile * 128, &bar_ld);
#pragma unroll
            for (int g = 0; g < 4; ++g) tma_load_2d(sB + L::kB1 + g * 8192, &mB2, g * 64, 0, &bar_ld);
        }
        if constexpr (L::kSides > 0) {
            mbar_expect_tx(&bar_side, L::kSides * 65536);
#pragma unroll
            for (int g = 0; g < 4; ++g) tma_load_2d(sS + g * 16384, &mS0, g * 64, tile * 128, &bar_side);
            if constexpr (L::kSides > 1) {
#pragma unroll
                for (int g = 0; g < 4; ++g) tma_load_2d(sS + 65536 + g * 16384, &mS1, g * 64, tile * 128, &bar_side);
            }
        }
        if (mbar_wait(&bar_ld, 0, status, kErrTma)) {
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16(128, 256, false, true);
#pragma unroll
            for (int part = 0; part < (SPLIT ? 3 : 1); ++part) {
                const uint64_t ad = smem_desc(smem_u32(sA) + (part == 1 ? L::kA1 : 0), 0, 1024, kSwz128);
                const uint64_t bd = smem_desc(smem_u32(sB) + (part == 2 ? L::kB1 : 0), 8192, 1024, kSwz128);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_ss(tm, desc_off(ad, k * 32), desc_off(bd, k * 2048), idesc, (part > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(&bar_mma);
        }
    }
    bool ok = mbar_wait(&bar_mma, 0, status, kErrMma);
    if constexpr (L::kSides > 0) ok = ok && mbar_wait(&bar_side, 0, status, kErrTma);
    ok = __syncthreads_and(ok) != 0;             // one decision for the whole CTA: the epilogue has barriers
    tc_fence_after();
    const uint32_t lane_tm = tm + ((uint32_t)((warp % 4) * 32) << 16);
    const size_t row = (size_t)tile * 128 + rowt;
    const bool elected = (tid % 128) == 0;
    auto wg_sync = [&]() {
        if (wg == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
        else asm volatile("bar.sync 2, 128;" ::: "memory");
    };
    if (ok) {
        if constexpr (EPI == EPI_GELU) {
            uint8_t* stg = sA + wg * 3 * 16384;
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                const int cg = wg * 2 + i;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int c0 = cg * 64 + half * 32;
                    uint32_t u[32];
                    tmem_ld32(lane_tm + c0, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        float pv[8], g[8];
                        const float4 b0 = *reinterpret_cast<const float4*>(s_bias + c0 + j), b1 = *reinterpret_cast<const float4*>(s_bias + c0 + j + 4);
                        const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            pv[q] = __uint_as_float(u[j + q]) + bv[q];
                            g[q] = (FULL || c0 + j + q < a.ncols) ? gelu_f(pv[q]) : 0.f;
                        }
                        if (a.keep_pre) tile_put8(stg, rowt, half * 4 + j / 8, pv);
                        tile_put8_split(stg + 16384, stg + 32768, rowt, half * 4 + j / 8, g);
                    }
                }
                fence_proxy_async_smem();
                wg_sync();
                if (elected) {
                    if (a.keep_pre) tma_store_2d(&mO0, stg, cg * 64, tile * 128);
                    tma_store_2d(&mO1, stg + 16384, cg * 64, tile * 128);
                    tma_store_2d(&mO2, stg + 32768, cg * 64, tile * 128);
                    bulk_commit();
                    bulk_wait_read();
                }
                wg_sync();
            }
        } else if constexpr (EPI == EPI_LN) {
            uint8_t* stg = sA + wg * 3 * 16384;
            float s = 0.f, ss = 0.f;
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                const int cg = wg * 2 + i;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int c0 = cg * 64 + half * 32;
                    uint32_t u[32];
                    tmem_ld32(lane_tm + c0, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        float pv[8];
                        const float4 b0 = *reinterpret_cast<const float4*>(s_bias + c0 + j), b1 = *reinterpret_cast<const float4*>(s_bias + c0 + j + 4);
                        const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            pv[q] = __uint_as_float(u[j + q]) + bv[q];
                            const float g = (FULL || c0 + j + q < a.ncols) ? gelu_f(pv[q]) : 0.f;
                            s += g; ss = fmaf(g, g, ss);
                            u[j + q] = __float_as_uint(g);
                        }
                        if (a.keep_pre) tile_put8(stg, rowt, half * 4 + j / 8, pv);
                    }
                    tmem_st32(lane_tm + c0, u);
                }
                if (a.keep_pre) {
                    fence_proxy_async_smem();
                    wg_sync();
                    if (elected) {
                        tma_store_2d(&mO0, stg, cg * 64, tile * 128);
                        bulk_commit();
                        bulk_wait_read();
                    }
                    wg_sync();
                }
            }
            tmem_st_wait();
            s_part[wg][rowt] = make_float2(s, ss);
            __syncthreads();
            const float2 p0 = s_part[0][rowt], p1 = s_part[1][rowt];
            const float inv = 1.f / (float)a.ncols;
            const float mu = (p0.x + p1.x) * inv;
            const float rs = rsqrtf(fmaxf((p0.y + p1.y) * inv - mu * mu, 0.f) + kLnEps);
            if (wg == 0) a.rs_out[row] = rs;
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                const int cg = wg * 2 + i;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int c0 = cg * 64 + half * 32;
                    uint32_t u[32];
                    tmem_ld32(lane_tm + c0, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        float nrm[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) nrm[q] = (FULL || c0 + j + q < a.ncols) ? (__uint_as_float(u[j + q]) - mu) * rs : 0.f;
                        tile_put8_split(stg + 16384, stg + 32768, rowt, half * 4 + j / 8, nrm);
                    }
                }
                fence_proxy_async_smem();
                wg_sync();
                if (elected) {
                    tma_store_2d(&mO1, stg + 16384, cg * 64, tile * 128);
                    tma_store_2d(&mO2, stg + 32768, cg * 64, tile * 128);
                    bulk_commit();
                    bulk_wait_read();
                }
                wg_sync();
            }
        } else if constexpr (EPI == EPI_DGELU) {
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                const int cg = wg * 2 + i;
                uint8_t* side = sS + cg * 16384;          // p3's tile, overwritten by dp3
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int c0 = cg * 64 + half * 32;
                    uint32_t u[32];
                    tmem_ld32(lane_tm + c0, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        float pv[8], o[8];
                        tile_get8(side, rowt, half * 4 + j / 8, pv);
#pragma unroll
                        for (int q = 0; q < 8; ++q) o[q] = (FULL || c0 + j + q < a.ncols) ? __uint_as_float(u[j + q]) * gelu_grad_f(pv[q]) : 0.f;
                        tile_put8(side, rowt, half * 4 + j / 8, o);
                    }
                }
                fence_proxy_async_smem();
                wg_sync();
                if (elected) { tma_store_2d(&mO0, side, cg * 64, tile * 128); bulk_commit(); }
            }
            if (elected) bulk_wait_read();
        } else {   // EPI_LNBWD: back through n = (g - mu) / sigma and g = gelu(p)
            float s1 = 0.f, s2 = 0.f;
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                const int cg = wg * 2 + i;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t u[32];
                    tmem_ld32(lane_tm + cg * 64 + half * 32, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        float nrm[8];
                        tile_get8(sS + cg * 16384, rowt, half * 4 + j / 8, nrm);
#pragma unroll
                        for (int q = 0; q < 8; ++q) { const float dn = __uint_as_float(u[j + q]); s1 += dn; s2 = fmaf(dn, nrm[q], s2); }
                    }
                }
            }
            s_part[wg][rowt] = make_float2(s1, s2);
            __syncthreads();
            const float2 p0 = s_part[0][rowt], p1 = s_part[1][rowt];
            const float inv = 1.f / (float)a.ncols;
            const float m1 = (p0.x + p1.x) * inv, m2 = (p0.y + p1.y) * inv, rs = a.rs_in[row];
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                const int cg = wg * 2 + i;
                uint8_t* side = sS + 65536 + cg * 16384;  // p1's tile, overwritten by dp1
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int c0 = cg * 64 + half * 32;
                    uint32_t u[32];
                    tmem_ld32(lane_tm + c0, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        float nrm[8], pv[8], o[8];
                        tile_get8(sS + cg * 16384, rowt, half * 4 + j / 8, nrm);
                        tile_get8(side, rowt, half * 4 + j / 8, pv);
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            o[q] = (FULL || c0 + j + q < a.ncols) ? rs * (__uint_as_float(u[j + q]) - m1 - nrm[q] * m2) * gelu_grad_f(pv[q]) : 0.f;
                        tile_put8(side, rowt, half * 4 + j / 8, o);
                    }
                }
                fence_proxy_async_smem();
                wg_sync();
                if (elected) { tma_store_2d(&mO0, side, cg * 64, tile * 128); bulk_commit(); }
            }
            if (elected) bulk_wait_read();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 256);
}

// ---------------------------------------------------------------------------
// weight gradients: Gt[256][64] += sum over a slab of rows of P[row][:]^T S[row][:]
// (P: [rows][256] bf16, S: [rows][64] bf16; both tiles go to the tensor cores as TMA left them:
// P^T is an MN-major A operand, S an MN-major B operand, the contraction runs over the rows)
// ---------------------------------------------------------------------------
constexpr int kWgStage = 65536 + 16384;
constexpr int kWgSmem = 2 * kWgStage + 1024;

__global__ void __launch_bounds__(160)
ltc_wgrad_kernel(const __grid_constant__ CUtensorMap mP, const __grid_constant__ CUtensorMap mS, float* __restrict__ Gt,
                 float* __restrict__ colsum, int sum_wide, int ntiles, int tiles_per_cta, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_full[2], bar_free[2], bar_done;
    __shared__ uint32_t tm_slot;
    const int tid = threadIdx.x, warp = tid / 32;
    const int t0 = blockIdx.x * tiles_per_cta;
    const int T = min(tiles_per_cta, ntiles - t0);
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_full[0], 1); mbar_init(&bar_full[1], 1);
        mbar_init(&bar_free[0], 5); mbar_init(&bar_free[1], 5);        // the tile's MMAs and the four summing warps
        mbar_init(&bar_done, 1);
        mbar_fence_init();
    }
    if (warp == 0) { tmem_alloc(&tm_slot, 128); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot;
    if (tid == 0) {
        auto load = [&](int j) {
            const int s = j & 1;
            uint8_t* sP = smem + s * kWgStage;
            mbar_expect_tx(&bar_full[s], kWgStage);
#pragma unroll
            for (int g = 0; g < 4; ++g) tma_load_2d(sP + g * 16384, &mP, g * 64, (t0 + j) * 128, &bar_full[s]);
            tma_load_2d(sP + 65536, &mS, 0, (t0 + j) * 128, &bar_full[s]);
        };
        load(0);
        if (T > 1) load(1);
        constexpr uint32_t idesc = idesc_bf16(128, 64, true, true);
        bool ok = true;
        for (int j = 0; j < T && ok; ++j) {
            const int s = j & 1;
            ok = mbar_spin(&bar_full[s], (j >> 1) & 1, status, kErrTma);
            if (!ok) break;
            tc_fence_after();
            const uint32_t base = smem_u32(smem + s * kWgStage);
            const uint64_t sd = smem_desc(base + 65536, 0, 1024, kSwz128);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const uint64_t pd = smem_desc(base + half * 32768, 16384, 1024, kSwz128);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_ss(tm + half * 64, desc_off(pd, k * 2048), desc_off(sd, k * 2048), idesc, (j > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(&bar_free[s]);
            if (j + 2 < T) {
                ok = mbar_spin(&bar_free[s], (j >> 1) & 1, status, kErrMma);
                if (ok) load(j + 2);
            }
        }
        if (ok) umma_commit(&bar_done);
    } else if (warp >= 1) {
        // Warps 1-4: column sums of the delta operand (the wide one's 256 columns, two per thread,
        // or the narrow one's 64) from the tiles while they sit in shared memory: the bias
        // gradients, and what the folded normalisation gains need.
        const int j0 = tid - 32;
        float acc0 = 0.f, acc1 = 0.f;
        bool ok = true;
        for (int j = 0; j < T; ++j) {
            const int s = j & 1;
            if (ok) ok = mbar_wait(&bar_full[s], (j >> 1) & 1, status, kErrTma);
            if (ok) {
                const uint8_t* st = smem + s * kWgStage;
                if (sum_wide) {
                    const uint8_t* c0p = st + (j0 / 64) * 16384 + (j0 % 8) * 2;
                    const uint8_t* c1p = c0p + 32768;
                    const uint32_t ch = (j0 % 64) / 8;
#pragma unroll 8
                    for (int row = 0; row < 128; ++row) {
                        const uint32_t o = swz128_offset(row, ch);
                        acc0 += __bfloat162float(*reinterpret_cast<const bf16*>(c0p + o));
                        acc1 += __bfloat162float(*reinterpret_cast<const bf16*>(c1p + o));
                    }
                } else if (j0 < 64) {
                    const uint8_t* cp = st + 65536 + (j0 % 8) * 2;
                    const uint32_t ch = j0 / 8;
#pragma unroll 8
                    for (int row = 0; row < 128; ++row) acc0 += __bfloat162float(*reinterpret_cast<const bf16*>(cp + swz128_offset(row, ch)));
                }
            }
            __syncwarp();
            if (tid % 32 == 0) mbar_arrive(&bar_free[s]);      // (also after a failed wait: the issuer must not be left waiting)
        }
        if (ok && colsum != nullptr) {
            if (sum_wide) { atomicAdd(colsum + j0, acc0); atomicAdd(colsum + j0 + 128, acc1); }
            else if (j0 < 64) atomicAdd(colsum + j0, acc0);
        }
    }
    const bool ok = mbar_wait(&bar_done, 0, status, kErrMma);
    tc_fence_after();
    if (ok && warp < 4) {
        const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t u[32];
                tmem_ld32(lane_tm + half * 64 + c0, u);
                tmem_ld_wait();
                float* dst = Gt + (size_t)(half * 128 + tid) * 64 + c0;
#pragma unroll
                for (int j = 0; j < 32; ++j) atomicAdd(dst + j, __uint_as_float(u[j]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 128);
}

// ---------------------------------------------------------------------------
// CUDA-core helpers around the layers
// ---------------------------------------------------------------------------
struct Slice {
    int H, n; int64_t sb, sh, sn;
    __device__ int64_t row(size_t R) const {
        const int bh = (int)(R / n), i = (int)(R % n);
        return (int64_t)(bh / H) * sb + (int64_t)(bh % H) * sh + (int64_t)i * sn;
    }
};

// n0 = (x - mean) / sigma of every row as hi + lo, 1 / sigma kept.  One warp per row, two columns
// per lane, eight rows per warp with their loads issued together.
constexpr int kLnRowsPerWarp = 8;
__global__ void __launch_bounds__(256)
ltc_ln0_kernel(Slice sl, const bf16* __restrict__ X, size_t row0, int rows, bf16* __restrict__ n0, bf16* __restrict__ n0_lo,
               float* __restrict__ rs0) {
    const int lane = threadIdx.x % 32;
    const int i0 = (blockIdx.x * 8 + threadIdx.x / 32) * kLnRowsPerWarp;
    __nv_bfloat162 x2[kLnRowsPerWarp];
#pragma unroll
    for (int q = 0; q < kLnRowsPerWarp; ++q)
        if (i0 + q < rows) x2[q] = *reinterpret_cast<const __nv_bfloat162*>(X + sl.row(row0 + i0 + q) + 2 * lane);
#pragma unroll
    for (int q = 0; q < kLnRowsPerWarp; ++q) {
        const int i = i0 + q;
        if (i >= rows) break;
        const float a = __low2float(x2[q]), b = __high2float(x2[q]);
        float s = a + b;
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        const float mu = s * (1.f / 64.f);
        float v = (a - mu) * (a - mu) + (b - mu) * (b - mu);
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        const float rs = rsqrtf(v * (1.f / 64.f) + kLnEps);
        const float na = (a - mu) * rs, nb = (b - mu) * rs;
        const uint32_t h = pack_bf16(na, nb);
        *reinterpret_cast<uint32_t*>(n0 + (size_t)i * 64 + 2 * lane) = h;
        *reinterpret_cast<uint32_t*>(n0_lo + (size_t)i * 64 + 2 * lane) =
            pack_bf16(na - __uint_as_float(h << 16), nb - __uint_as_float(h & 0xffff0000u));
        if (lane == 0) rs0[i] = rs;
    }
}

// dX = back through the first normalisation of the summed gradient of n0 (+ add)
__global__ void __launch_bounds__(256)
ltc_ln0_bwd_kernel(Slice sl, size_t row0, int rows, const float* __restrict__ dn0, const bf16* __restrict__ n0,
                   const float* __restrict__ rs0, const bf16* __restrict__ add, bf16* __restrict__ dX) {
    const int lane = threadIdx.x % 32;
    const int i = blockIdx.x * 8 + threadIdx.x / 32;
    if (i >= rows) return;
    const float2 d = *reinterpret_cast<const float2*>(dn0 + (size_t)i * 64 + 2 * lane);
    const __nv_bfloat162 n2 = *reinterpret_cast<const __nv_bfloat162*>(n0 + (size_t)i * 64 + 2 * lane);
    const float na = __low2float(n2), nb = __high2float(n2);
    float s1 = d.x + d.y, s2 = d.x * na + d.y * nb;
    for (int o = 16; o > 0; o >>= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); }
    const float m1 = s1 * (1.f / 64.f), m2 = s2 * (1.f / 64.f), rs = rs0[i];
    float oa = rs * (d.x - m1 - na * m2), ob = rs * (d.y - m1 - nb * m2);
    if (add != nullptr) {
        const __nv_bfloat162 q = *reinterpret_cast<const __nv_bfloat162*>(add + (row0 + i) * 64 + 2 * lane);
        oa += __low2float(q); ob += __high2float(q);
    }
    *reinterpret_cast<uint32_t*>(dX + sl.row(row0 + i) + 2 * lane) = pack_bf16(oa, ob);
}

// M = sqrt(r) tanh(f1 f2 / sqrt(r)), written as the [hi | lo] rows (64 bf16 columns, zero beyond 2r) the
// attention kernels read in their linear sketch mode; one thread = 8 consecutive columns of a row
__global__ void __launch_bounds__(256)
ltc_combine_kernel(const float* __restrict__ f1, const float* __restrict__ f2, int r, size_t rows, bf16* __restrict__ S) {
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= rows * 8) return;
    const size_t row = e / 8;
    const int c0 = (int)(e % 8) * 8;
    const float sr = sqrtf((float)r), isr = rsqrtf((float)r);
    uint32_t pk[4];
#pragma unroll
    for (int j = 0; j < 8; j += 2) {
        float x[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int c = c0 + j + q;
            float v = 0.f;
            if (c < 2 * r) {
                const size_t o = row * r + (c % r);
                const float m = sr * tanhf(f1[o] * f2[o] * isr);
                const float hi = __bfloat162float(__float2bfloat16_rn(m));
                v = c < r ? hi : m - hi;
            }
            x[q] = v;
        }
        pk[j / 2] = pack_bf16(x[0], x[1]);
    }
    *reinterpret_cast<uint4*>(S + row * 64 + c0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

// df1 = dM (1 - t^2) f2, df2 = dM (1 - t^2) f1 as bf16 rows of 64 columns (zero beyond r); dM = the
// first r columns of dS, the gradient of the [hi | lo] rows (M = hi + lo)
__global__ void __launch_bounds__(256)
ltc_combine_bwd_kernel(const float* __restrict__ f1, const float* __restrict__ f2, const bf16* __restrict__ dS, int r,
                       size_t rows, bf16* __restrict__ df1, bf16* __restrict__ df2) {
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= rows * 64) return;
    const size_t row = e / 64;
    const int c = (int)(e % 64);
    float o1 = 0.f, o2 = 0.f;
    if (c < r) {
        const float a = f1[row * r + c], b = f2[row * r + c];
        const float t = tanhf(a * b * rsqrtf((float)r));
        const float du = __bfloat162float(dS[e]) * (1.f - t * t);
        o1 = du * b; o2 = du * a;
    }
    df1[e] = __float2bfloat16_rn(o1);
    df2[e] = __float2bfloat16_rn(o2);
}

// parameter gradients of one network from the four accumulators and the column sums
//   G1t = dp1^T n0, G2 = n1^T da2, G3t = dp3^T a2, G4 = a3^T df   (each [256][64])
__global__ void __launch_bounds__(256)
ltc_finish_kernel(int h, int r, const float* __restrict__ params, const float* __restrict__ G, const float* __restrict__ sums,
                  float* __restrict__ dparams) {
    const NetLayout nl(h, r);
    const int net = blockIdx.y, m = nl.m;
    const float* P = params + (size_t)net * nl.count;
    float* dP = dparams + (size_t)net * nl.count;
    const float* G1t = G + (size_t)net * 4 * kMat;
    const float* G2 = G1t + kMat;
    const float* G3t = G2 + kMat;
    const float* G4 = G3t + kMat;
    const float* s_dp1 = sums + (size_t)net * kSums;
    const float* s_da2 = s_dp1 + 256;
    const float* s_dp3 = s_da2 + 64;
    const float* s_df = s_dp3 + 256;
    const int e = blockIdx.x * 256 + threadIdx.x;
    if (e >= nl.count) return;
    float g = 0.f;
    if (e < nl.c0) {                                           // dg0[k] = sum_j W1[k][j] G1t[j][k]
        const int k = e - nl.g0;
        for (int j = 0; j < m; ++j) g = fmaf(P[nl.W1 + k * m + j], G1t[j * 64 + k], g);
    } else if (e < nl.W1) {                                    // dc0[k] = sum_j W1[k][j] s_dp1[j]
        const int k = e - nl.c0;
        for (int j = 0; j < m; ++j) g = fmaf(P[nl.W1 + k * m + j], s_dp1[j], g);
    } else if (e < nl.b1) {                                    // dW1[k][j] = g0[k] G1t[j][k] + c0[k] s_dp1[j]
        const int k = (e - nl.W1) / m, j = (e - nl.W1) % m;
        g = P[nl.g0 + k] * G1t[j * 64 + k] + P[nl.c0 + k] * s_dp1[j];
    } else if (e < nl.g1) {
        g = s_dp1[e - nl.b1];
    } else if (e < nl.c1) {                                    // dg1[j] = sum_c W2[j][c] G2[j][c]
        const int j = e - nl.g1;
        for (int c = 0; c < r; ++c) g = fmaf(P[nl.W2 + j * r + c], G2[j * 64 + c], g);
    } else if (e < nl.W2) {                                    // dc1[j] = sum_c W2[j][c] s_da2[c]
        const int j = e - nl.c1;
        for (int c = 0; c < r; ++c) g = fmaf(P[nl.W2 + j * r + c], s_da2[c], g);
    } else if (e < nl.b2) {                                    // dW2[j][c] = g1[j] G2[j][c] + c1[j] s_da2[c]
        const int j = (e - nl.W2) / r, c = (e - nl.W2) % r;
        g = P[nl.g1 + j] * G2[j * 64 + c] + P[nl.c1 + j] * s_da2[c];
    } else if (e < nl.W3) {
        g = s_da2[e - nl.b2];
    } else if (e < nl.b3) {                                    // dW3[c][j] = G3t[j][c]
        const int c = (e - nl.W3) / m, j = (e - nl.W3) % m;
        g = G3t[j * 64 + c];
    } else if (e < nl.W4) {
        g = s_dp3[e - nl.b3];
    } else if (e < nl.b4) {                                    // dW4[j][c] = G4[j][c]
        const int j = (e - nl.W4) / r, c = (e - nl.W4) % r;
        g = G4[j * 64 + c];
    } else {
        g = s_df[e - nl.b4];
    }
    dP[e] += g;
}

// ---------------------------------------------------------------------------
// host
// ---------------------------------------------------------------------------
struct NetBuf { size_t p1, n1, n1_lo, p3, a3, a3_lo, a2, a2_lo, rs1, f; };
struct LtcWs {
    size_t bank, vec, G, sums, n0, n0_lo, rs0, df[2], dp3, da2, dp1, dn0, total;
    NetBuf net[2];
    size_t C;
};

// Rows per pass.  PSK_LEARNED_CHUNK_ROWS in the environment overrides the default (a multiple of
// 128; read at every call, so that workspace queries and calls of one process agree as long as
// it is not changed between them): for tests of the chunk loop on small inputs, and for tuning.
size_t chunk_rows() {
    const char* e = std::getenv("PSK_LEARNED_CHUNK_ROWS");
    if (e != nullptr) {
        const long long v = std::atoll(e);
        if (v >= 128 && v % 128 == 0) return (size_t)v;
    }
    return kChunkRows;
}

LtcWs ltc_ws(const Dims& d, bool backward) {
    LtcWs w{};
    const size_t rows = (size_t)d.BH() * d.n;
    const size_t chunk = chunk_rows();
    w.C = rows < chunk ? rows : chunk;
    const size_t C = w.C;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes); return o; };
    w.bank = take((size_t)2 * kBank * kMat * sizeof(bf16));
    w.vec = take((size_t)2 * kVec * sizeof(float));
    w.G = take((size_t)2 * 4 * kMat * sizeof(float));       // G and sums are zeroed together
    w.sums = take((size_t)2 * kSums * sizeof(float));
    w.n0 = take(C * 64 * sizeof(bf16));
    w.n0_lo = take(C * 64 * sizeof(bf16));
    w.rs0 = take(C * sizeof(float));
    for (int t = 0; t < 2; ++t) {
        w.net[t].p1 = take(C * 256 * sizeof(bf16));
        w.net[t].n1 = take(C * 256 * sizeof(bf16));
        w.net[t].n1_lo = take(C * 256 * sizeof(bf16));
        w.net[t].p3 = take(C * 256 * sizeof(bf16));
        w.net[t].a3 = take(C * 256 * sizeof(bf16));
        w.net[t].a3_lo = take(C * 256 * sizeof(bf16));
        w.net[t].a2 = take(C * 64 * sizeof(bf16));
        w.net[t].a2_lo = take(C * 64 * sizeof(bf16));
        w.net[t].rs1 = take(C * sizeof(float));
        w.net[t].f = take(C * d.r * sizeof(float));
    }
    if (backward) {
        w.df[0] = take(C * 64 * sizeof(bf16));
        w.df[1] = take(C * 64 * sizeof(bf16));
        w.dp3 = take(C * 256 * sizeof(bf16));
        w.da2 = take(C * 64 * sizeof(bf16));
        w.dp1 = take(C * 256 * sizeof(bf16));
        w.dn0 = take(C * 64 * sizeof(float));
    }
    w.total = off;
    return w;
}

struct Maps {                       // tensor maps over the chunk buffers (built once per call)
    CUtensorMap bank[2][kBank];
    CUtensorMap n0, n0_lo, df[2], dp3, da2, dp1;
    CUtensorMap p1[2], n1[2], n1_lo[2], p3[2], a3[2], a3_lo[2], a2[2], a2_lo[2];
};

bool build_maps(const LtcWs& w, char* ws, bool backward, Maps* M) {
    const int64_t C = (int64_t)w.C;
    bool ok = true;
    for (int t = 0; t < 2; ++t) {
        for (int i = 0; i < kBank; ++i) {
            const bf16* base = reinterpret_cast<const bf16*>(ws + w.bank) + ((size_t)t * kBank + i) * kMat;
            ok = ok && ((i % 2 == 0) ? tc_map_2d(&M->bank[t][i], base, 256, 64, 64) : tc_map_2d(&M->bank[t][i], base, 64, 256, 256));
        }
        ok = ok && tc_map_2d(&M->p1[t], ws + w.net[t].p1, 256, C, 128) && tc_map_2d(&M->n1[t], ws + w.net[t].n1, 256, C, 128) &&
             tc_map_2d(&M->p3[t], ws + w.net[t].p3, 256, C, 128) && tc_map_2d(&M->a3[t], ws + w.net[t].a3, 256, C, 128) &&
             tc_map_2d(&M->a2[t], ws + w.net[t].a2, 64, C, 128) && tc_map_2d(&M->n1_lo[t], ws + w.net[t].n1_lo, 256, C, 128) &&
             tc_map_2d(&M->a3_lo[t], ws + w.net[t].a3_lo, 256, C, 128) && tc_map_2d(&M->a2_lo[t], ws + w.net[t].a2_lo, 64, C, 128);
    }
    ok = ok && tc_map_2d(&M->n0, ws + w.n0, 64, C, 128) && tc_map_2d(&M->n0_lo, ws + w.n0_lo, 64, C, 128);
    if (backward)
        ok = ok && tc_map_2d(&M->df[0], ws + w.df[0], 64, C, 128) && tc_map_2d(&M->df[1], ws + w.df[1], 64, C, 128) &&
             tc_map_2d(&M->dp3, ws + w.dp3, 256, C, 128) && tc_map_2d(&M->da2, ws + w.da2, 64, C, 128) &&
             tc_map_2d(&M->dp1, ws + w.dp1, 256, C, 128);
    return ok;
}

// names under which the instances appear in the per-kernel timing records
const char* const kDenseName[6] = {"", "ltc_dense_bwd_mid_kernel", "", "ltc_dense_bwd_in_kernel", "ltc_dense_bwd_gelu_kernel",
                                   "ltc_dense_bwd_norm_kernel"};
const char* const kDenseSplitName[6] = {"ltc_dense_norm_kernel", "ltc_dense_mid_kernel", "ltc_dense_gelu_kernel",
                                        "ltc_dense_out_kernel", "", ""};

// wide layers (64 -> 256)
template <int EPI, bool SPLIT>
cudaError_t wide(const CUtensorMap& mA, const CUtensorMap& mA2, const CUtensorMap& mB, const CUtensorMap& mB2,
                 const CUtensorMap& mS0, const CUtensorMap& mS1, const CUtensorMap& mO0, const CUtensorMap& mO1,
                 const CUtensorMap& mO2, const WideArgs& a, int tiles, int* status, cudaStream_t s, int* launches) {
    constexpr int smem = WideSmem<EPI, SPLIT>::bytes;
    PSK_TRY(set_smem(ltc_wide_kernel<EPI, SPLIT, true>, smem));
    PSK_TRY(set_smem(ltc_wide_kernel<EPI, SPLIT, false>, smem));
    prof_begin(SPLIT ? kDenseSplitName[EPI] : kDenseName[EPI], s);
    if (a.ncols == 256) ltc_wide_kernel<EPI, SPLIT, true><<<tiles, 256, smem, s>>>(mA, mA2, mB, mB2, mS0, mS1, mO0, mO1, mO2, a, status);
    else ltc_wide_kernel<EPI, SPLIT, false><<<tiles, 256, smem, s>>>(mA, mA2, mB, mB2, mS0, mS1, mO0, mO1, mO2, a, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}
// narrow layers (256 -> 64) of the backward: single bf16 operands
template <int EPI>
cudaError_t dense(const CUtensorMap& mA, const CUtensorMap& mB, const DenseArgs& a, int tiles, int* status, cudaStream_t s,
                  int* launches) {
    PSK_TRY(set_smem(ltc_dense_kernel<EPI>, kDenseSmem));
    prof_begin(kDenseName[EPI], s);
    ltc_dense_kernel<EPI><<<tiles, 128, kDenseSmem, s>>>(mA, mB, a, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}
// narrow layers of the forward: hi + lo operand pairs, persistent kernel
template <int EPI>
cudaError_t narrow(const CUtensorMap& mA, const CUtensorMap& mA2, const CUtensorMap& mB, const CUtensorMap& mB2,
                   const DenseArgs& a, int tiles, int* status, cudaStream_t s, int* launches) {
    PSK_TRY(set_smem(ltc_narrow_kernel<EPI>, kNrSmem));
    static int sms = 0;
    if (sms == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
    }
    prof_begin(kDenseSplitName[EPI], s);
    ltc_narrow_kernel<EPI><<<tiles < sms ? tiles : sms, 192, kNrSmem, s>>>(mA, mA2, mB, mB2, a, tiles, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

// (colsum: where the column sums of the delta operand are added; wide = that operand is P)
cudaError_t wgrad(const CUtensorMap& mP, const CUtensorMap& mS, float* Gt, float* colsum, bool wide, int tiles, int* status,
                  cudaStream_t s, int* launches) {
    PSK_TRY(set_smem(ltc_wgrad_kernel, kWgSmem));
    int per = (tiles + 295) / 296;            // about two CTAs per SM, but at least four tiles per result added
    if (per < 4) per = tiles < 4 ? tiles : 4;
    const int grid = (tiles + per - 1) / per;
    prof_begin("ltc_wgrad_kernel", s);
    ltc_wgrad_kernel<<<grid, 160, kWgSmem, s>>>(mP, mS, Gt, colsum, wide ? 1 : 0, tiles, per, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

// forward of both networks on `c` rows starting at row0: activations and f into the chunk buffers
// (keep_pre: also the pre-activations p1, p3, which only the backward reads)
cudaError_t forward_chunk(const Dims& d, const LtcWs& w, const Maps& M, const void* X, size_t row0, int c, bool keep_pre, char* ws,
                          int* status, cudaStream_t s, int* launches) {
    const Slice sl{d.H, d.n, d.sb, d.sh, d.sn};
    const int tiles = c / 128, m = 8 * d.r;
    prof_begin("ltc_ln0_kernel", s);
    ltc_ln0_kernel<<<(c + 8 * kLnRowsPerWarp - 1) / (8 * kLnRowsPerWarp), 256, 0, s>>>(sl, (const bf16*)X, row0, c, (bf16*)(ws + w.n0), (bf16*)(ws + w.n0_lo), (float*)(ws + w.rs0));
    prof_end(s);
    ++*launches;
    PSK_TRY(cudaGetLastError());
    for (int t = 0; t < 2; ++t) {
        const NetBuf& nb = w.net[t];
        const float* vec = (const float*)(ws + w.vec) + (size_t)t * kVec;
        PSK_TRY((wide<EPI_LN, true>(M.n0, M.n0_lo, M.bank[t][0], M.bank[t][8], M.n0, M.n0, M.p1[t], M.n1[t], M.n1_lo[t],
                                    WideArgs{vec, (float*)(ws + nb.rs1), nullptr, m, keep_pre ? 1 : 0}, tiles, status, s, launches)));
        PSK_TRY(narrow<EPI_B64>(M.n1[t], M.n1_lo[t], M.bank[t][1], M.bank[t][9],
                                DenseArgs{vec + 256, (bf16*)(ws + nb.a2), (bf16*)(ws + nb.a2_lo), nullptr, 0, 0}, tiles, status, s, launches));
        PSK_TRY((wide<EPI_GELU, true>(M.a2[t], M.a2_lo[t], M.bank[t][2], M.bank[t][10], M.n0, M.n0, M.p3[t], M.a3[t], M.a3_lo[t],
                                      WideArgs{vec + 320, nullptr, nullptr, m, keep_pre ? 1 : 0}, tiles, status, s, launches)));
        PSK_TRY(narrow<EPI_F32>(M.a3[t], M.a3_lo[t], M.bank[t][3], M.bank[t][11],
                                DenseArgs{vec + 576, nullptr, nullptr, (float*)(ws + nb.f), d.r, 0}, tiles, status, s, launches));
    }
    return cudaSuccess;
}

}  // namespace

bool learned_tc_supported(const Dims& d) { return d.bf16 && d.learned && d.h == 64 && d.r <= 32 && d.r % 4 == 0; }

size_t learned_tc_workspace_bytes(const Dims& d, bool backward) { return ltc_ws(d, backward).total; }

// operand bank of both networks; backward: also clears the gradient accumulators
cudaError_t learned_tc_prepare(const Dims& d, bool backward, char* ws, cudaStream_t s, int* launches) {
    const LtcWs w = ltc_ws(d, backward);
    prof_begin("ltc_bank_kernel", s);
    ltc_bank_kernel<<<dim3((8 * kMat + kVec + 255) / 256, 2), 256, 0, s>>>(d.h, d.r, d.lparams, (bf16*)(ws + w.bank), (float*)(ws + w.vec));
    prof_end(s);
    ++*launches;
    PSK_TRY(cudaGetLastError());
    if (backward) PSK_TRY(cudaMemsetAsync(ws + w.G, 0, (w.sums - w.G) + (size_t)2 * kSums * sizeof(float), s));
    return cudaSuccess;
}

// S = the [hi | lo] rows of the half sketch of X (contiguous [rows][64] bf16)
cudaError_t learned_tc_sketch(const Dims& d, const void* X, void* S, char* ws, int* status, cudaStream_t s, int* launches) {
    const LtcWs w = ltc_ws(d, false);            // the forward's buffers come first in either layout
    Maps M;
    if (!build_maps(w, ws, false, &M)) return cudaErrorInvalidValue;
    const size_t rows = (size_t)d.BH() * d.n;
    for (size_t row0 = 0; row0 < rows; row0 += w.C) {
        const int c = (int)(rows - row0 < w.C ? rows - row0 : w.C);
        PSK_TRY(forward_chunk(d, w, M, X, row0, c, false, ws, status, s, launches));
        prof_begin("ltc_combine_kernel", s);
        ltc_combine_kernel<<<(unsigned)(((size_t)c * 8 + 255) / 256), 256, 0, s>>>((const float*)(ws + w.net[0].f), (const float*)(ws + w.net[1].f),
                                                                              d.r, (size_t)c, (bf16*)S + row0 * 64);
        prof_end(s);
        ++*launches;
        PSK_TRY(cudaGetLastError());
    }
    return cudaSuccess;
}

// dX = chain rule through both networks of the gradient dS of the [hi | lo] rows (+ add, a contiguous [rows][64] bf16 array
// or null: the part of the gradient that reached X directly); the weight-gradient
// accumulators in the workspace grow by this tensor's share (learned_tc_finish turns them into
// parameter gradients)
cudaError_t learned_tc_sketch_bwd(const Dims& d, const void* X, const void* dS, const void* add, void* dX, char* ws,
                                  int* status, cudaStream_t s, int* launches) {
    const LtcWs w = ltc_ws(d, true);
    Maps M;
    if (!build_maps(w, ws, true, &M)) return cudaErrorInvalidValue;
    const Slice sl{d.H, d.n, d.sb, d.sh, d.sn};
    const size_t rows = (size_t)d.BH() * d.n;
    const int m = 8 * d.r;
    for (size_t row0 = 0; row0 < rows; row0 += w.C) {
        const int c = (int)(rows - row0 < w.C ? rows - row0 : w.C);
        const int tiles = c / 128;
        PSK_TRY(forward_chunk(d, w, M, X, row0, c, true, ws, status, s, launches));
        prof_begin("ltc_combine_bwd_kernel", s);
        ltc_combine_bwd_kernel<<<(unsigned)(((size_t)c * 64 + 255) / 256), 256, 0, s>>>(
            (const float*)(ws + w.net[0].f), (const float*)(ws + w.net[1].f), (const bf16*)dS + row0 * 64, d.r, (size_t)c,
            (bf16*)(ws + w.df[0]), (bf16*)(ws + w.df[1]));
        prof_end(s);
        ++*launches;
        PSK_TRY(cudaGetLastError());
        for (int t = 0; t < 2; ++t) {
            const NetBuf& nb = w.net[t];
            float* G = (float*)(ws + w.G) + (size_t)t * 4 * kMat;
            float* sums = (float*)(ws + w.sums) + (size_t)t * kSums;
            // dp3 = (df W4^T) * gelu'(p3);  dW4 ~ a3^T df
            PSK_TRY((wide<EPI_DGELU, false>(M.df[t], M.df[t], M.bank[t][4], M.bank[t][4], M.p3[t], M.p3[t], M.dp3, M.dp3, M.dp3,
                                            WideArgs{nullptr, nullptr, nullptr, m, 0}, tiles, status, s, launches)));
            PSK_TRY(wgrad(M.a3[t], M.df[t], G + 3 * kMat, sums + 576, false, tiles, status, s, launches));
            // da2 = dp3 W3^T;  dW3 ~ dp3^T a2
            PSK_TRY(wgrad(M.dp3, M.a2[t], G + 2 * kMat, sums + 320, true, tiles, status, s, launches));
            PSK_TRY(dense<EPI_B64>(M.dp3, M.bank[t][5], DenseArgs{nullptr, (bf16*)(ws + w.da2), nullptr, nullptr, 0, 0}, tiles, status, s, launches));
            // dp1 = LN1 backward(da2 (g1 W2)^T) * gelu'(p1);  dW2 ~ n1^T da2
            PSK_TRY(wgrad(M.n1[t], M.da2, G + 1 * kMat, sums + 256, false, tiles, status, s, launches));
            PSK_TRY((wide<EPI_LNBWD, false>(M.da2, M.da2, M.bank[t][6], M.bank[t][6], M.n1[t], M.p1[t], M.dp1, M.dp1, M.dp1,
                                            WideArgs{nullptr, nullptr, (const float*)(ws + nb.rs1), m, 0}, tiles, status, s, launches)));
            // dn0 (+)= dp1 (g0 W1)^T;  dW1 ~ dp1^T n0
            PSK_TRY(wgrad(M.dp1, M.n0, G + 0 * kMat, sums + 0, true, tiles, status, s, launches));
            PSK_TRY(dense<EPI_F32>(M.dp1, M.bank[t][7], DenseArgs{nullptr, nullptr, nullptr, (float*)(ws + w.dn0), 64, t}, tiles, status, s, launches));
        }
        prof_begin("ltc_ln0_bwd_kernel", s);
        ltc_ln0_bwd_kernel<<<(c + 7) / 8, 256, 0, s>>>(sl, row0, c, (const float*)(ws + w.dn0), (const bf16*)(ws + w.n0),
                                                      (const float*)(ws + w.rs0), (const bf16*)add, (bf16*)dX);
        prof_end(s);
        ++*launches;
        PSK_TRY(cudaGetLastError());
    }
    return cudaSuccess;
}

// parameter gradients (added to d.dlparams) from everything learned_tc_sketch_bwd accumulated
cudaError_t learned_tc_finish(const Dims& d, char* ws, cudaStream_t s, int* launches) {
    const LtcWs w = ltc_ws(d, true);
    const int count = NetLayout(d.h, d.r).count;
    prof_begin("ltc_finish_kernel", s);
    ltc_finish_kernel<<<dim3((count + 255) / 256, 2), 256, 0, s>>>(d.h, d.r, d.lparams, (const float*)(ws + w.G),
                                                                   (const float*)(ws + w.sums), d.dlparams);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace psk
