// Degree 8: the deeper half sketch (one more level of Algorithm 1's recursion) on the tensor cores,
// bf16 storage, r <= 32.
//   M1 = (X Ga1)*(X Ga2)/sqrt(r),  M2 = (X Gb1)*(X Gb2)/sqrt(r),  M = (M1 Gc1)*(M2 Gc2)/sqrt(r)
// One CTA per 128-row tile, thread = row.  Forward: X [Ga1 | Ga2 | Gb1 | Gb2] in one GEMM, the
// products M1, M2 split into hi + lo bf16 terms (they feed another cancelling sum), [M1 | M2] against
// the block-diagonal of Gc1, Gc2 in a second GEMM, and M written straight as the [hi | lo] rows the
// attention kernels read in their linear sketch mode.  Backward: the same two GEMMs again, then
// dC -> dM1, dM2 and dA, dB -> dX through the transposes, which are the same shared-memory tiles
// read K-major instead of MN-major.
#include "tc_common.cuh"

namespace psk {
namespace {

using namespace tc;

constexpr int kW1 = 64 * 128, kW2 = 64 * 64;      // elements per head: [64][128] and [64][64]

// W1[g][k][n] = [Ga1 | Ga2 | Gb1 | Gb2][k][n] (zero beyond 4r), W2[g] = blockdiag(Gc1, Gc2) (zero elsewhere)
__global__ void __launch_bounds__(256)
sk8_bank_kernel(const bf16* __restrict__ G1, const bf16* __restrict__ G2, int r, bf16* __restrict__ W1, bf16* __restrict__ W2) {
    const int g = blockIdx.y, e = blockIdx.x * 256 + threadIdx.x;
    const size_t gbase = (size_t)g * (128 + r) * r;
    const bf16 zero = __float2bfloat16_rn(0.f);
    if (e < kW1) {
        const int k = e / 128, n = e % 128;
        bf16 v = zero;
        if (n < 4 * r) {
            const int which = n / r, c = n % r;            // 0: Ga1, 1: Ga2, 2: Gb1, 3: Gb2
            const bf16* G = (which & 1) ? G2 : G1;
            v = G[gbase + (size_t)((which >> 1) * 64 + k) * r + c];
        }
        W1[(size_t)g * kW1 + e] = v;
    } else if (e < kW1 + kW2) {
        const int k = (e - kW1) / 64, n = (e - kW1) % 64;
        bf16 v = zero;
        if (k < r && n < r) v = G1[gbase + (size_t)(128 + k) * r + n];
        else if (k >= r && k < 2 * r && n >= r && n < 2 * r) v = G2[gbase + (size_t)(128 + k - r) * r + (n - r)];
        W2[(size_t)g * kW2 + (e - kW1)] = v;
    }
}

__device__ __forceinline__ void put8(uint8_t* tile, int row, int chunk, const float* v) {
    *reinterpret_cast<uint4*>(tile + swz128_offset(row, chunk)) =
        make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
__device__ __forceinline__ void tma_store_tile(const CUtensorMap* m, const void* src, int c1, int c2, int c3) {
    tma_store_4d(m, src, 0, c1, c2, c3);
}

struct Sk8Smem {      // bytes; every tile 1024-byte aligned
    static constexpr uint32_t X = 0, D = 16384, W1 = 32768, W2 = 49152, HL = 57344, total = HL + 32768;
};

// ---- GEMM 1 and 2 of both passes (one thread issues; the callers wait on `bar`) ----
template <int R>
__device__ __forceinline__ void issue_first(uint32_t tm, const uint8_t* smem) {       // D1 = X W1, N = 4R
    constexpr uint32_t idesc = idesc_bf16(128, 4 * R, false, true);
    const uint64_t ad = smem_desc(smem_u32(smem + Sk8Smem::X), 0, 1024, kSwz128);
    const uint64_t bd = smem_desc(smem_u32(smem + Sk8Smem::W1), 8192, 1024, kSwz128);
#pragma unroll
    for (int k = 0; k < 4; ++k) umma_ss(tm, desc_off(ad, k * 32), desc_off(bd, k * 2048), idesc, k > 0);
}
template <int R>
__device__ __forceinline__ void issue_second(uint32_t tm_d2, const uint8_t* smem) {   // D2 = [M1 | M2] W2, hi then lo
    constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
    const uint64_t bd = smem_desc(smem_u32(smem + Sk8Smem::W2), 0, 1024, kSwz128);
#pragma unroll
    for (int part = 0; part < 2; ++part) {
        const uint64_t ad = smem_desc(smem_u32(smem + Sk8Smem::HL) + part * 16384, 0, 1024, kSwz128);
#pragma unroll
        for (int k = 0; k < 2 * R / 16; ++k) umma_ss(tm_d2, desc_off(ad, k * 32), desc_off(bd, k * 2048), idesc, (part > 0 || k > 0) ? 1u : 0u);
    }
}
// this thread's row of [M1 | M2] from D1, as hi and lo tiles (columns beyond 2R stay zero from the start)
template <int R>
__device__ __forceinline__ void stage_m12(uint32_t lane_tm, uint8_t* smem, int row) {
    const float rs = rsqrtf((float)R);
#pragma unroll
    for (int half = 0; half < 2; ++half) {              // M1 from columns [0, 2R), M2 from [2R, 4R)
#pragma unroll
        for (int c0 = 0; c0 < R; c0 += 16) {
            uint32_t u1[16], u2[16];
            tmem_ld16(lane_tm + half * 2 * R + c0, u1);
            tmem_ld16(lane_tm + half * 2 * R + R + c0, u2);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
                float hi[8], lo[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const float m = __uint_as_float(u1[j + q]) * __uint_as_float(u2[j + q]) * rs;
                    hi[q] = __bfloat162float(__float2bfloat16_rn(m));
                    lo[q] = m - hi[q];
                }
                const int chunk = (half * R + c0 + j) / 8;
                put8(smem + Sk8Smem::HL, row, chunk, hi);
                put8(smem + Sk8Smem::HL + 16384, row, chunk, lo);
            }
        }
    }
}

template <int R>
__global__ void __launch_bounds__(128)
sk8_tc_fwd_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW1,
                  const __grid_constant__ CUtensorMap mapW2, const __grid_constant__ CUtensorMap mapS, int g_heads, int H,
                  int* status) {
    using L = Sk8Smem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_ld, bar_mma;
    __shared__ uint32_t tm_slot;
    const int tid = threadIdx.x, warp = tid / 32;
    const int i0 = blockIdx.x * 128, bh = blockIdx.y, hi_ = bh % H, bi = bh / H;
    const int g = g_heads == 1 ? 0 : hi_;
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_ld, 1); mbar_init(&bar_mma, 1);
        mbar_fence_init();
        mbar_expect_tx(&bar_ld, 16384 + (4 * R / 64) * 8192 + 8192);
        tma_load_4d(smem + L::X, &mapX, 0, i0, hi_, bi, &bar_ld);
#pragma unroll
        for (int q = 0; q < 4 * R / 64; ++q) tma_load_3d(smem + L::W1 + q * 8192, &mapW1, q * 64, 0, g, &bar_ld);
        tma_load_3d(smem + L::W2, &mapW2, 0, 0, g, &bar_ld);
    }
    if (warp == 0) { tmem_alloc(&tm_slot, 256); tmem_relinquish(); }
    // columns of the [M1 | M2] tiles beyond 2R are never written: clear this row of both tiles
    for (int ch = 2 * R / 8; ch < 8; ++ch) {
        *reinterpret_cast<uint4*>(smem + L::HL + swz128_offset(tid, ch)) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(smem + L::HL + 16384 + swz128_offset(tid, ch)) = make_uint4(0, 0, 0, 0);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot, lane_tm = tm + ((uint32_t)(warp * 32) << 16);
    bool ok = mbar_wait(&bar_ld, 0, status, kErrTma);
    if (tid == 0 && ok) { tc_fence_after(); issue_first<R>(tm, smem); umma_commit(&bar_mma); }
    ok = ok && mbar_wait(&bar_mma, 0, status, kErrMma);
    tc_fence_after();
    if (ok) stage_m12<R>(lane_tm, smem, tid);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) { tc_fence_after(); issue_second<R>(tm + 128, smem); umma_commit(&bar_mma); }
    ok = ok && mbar_wait(&bar_mma, 1, status, kErrMma);
    tc_fence_after();
    if (ok) {
        // M = C1 * C2 / sqrt(R), written as the row [hi | lo | 0] over the X tile (dead since GEMM 1)
        const float rs = rsqrtf((float)R);
        float m[R];
#pragma unroll
        for (int c0 = 0; c0 < R; c0 += 16) {
            uint32_t u1[16], u2[16];
            tmem_ld16(lane_tm + 128 + c0, u1);
            tmem_ld16(lane_tm + 128 + R + c0, u2);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) m[c0 + j] = __uint_as_float(u1[j]) * __uint_as_float(u2[j]) * rs;
        }
        store_hilo_tiles<R>(smem + L::X, m, tid);
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) {
        tma_store_tile(&mapS, smem + L::X, i0, hi_, bi);
        bulk_commit();
        bulk_wait_read();
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 256);
}

// dX from the gradient of the [hi | lo] rows (its first R columns are dL/dM)
template <int R>
__global__ void __launch_bounds__(128)
sk8_tc_bwd_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW1,
                  const __grid_constant__ CUtensorMap mapW2, const __grid_constant__ CUtensorMap mapDS,
                  const __grid_constant__ CUtensorMap mapDX, int g_heads, int H, int* status) {
    using L = Sk8Smem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_ld, bar_mma;
    __shared__ uint32_t tm_slot;
    const int tid = threadIdx.x, warp = tid / 32;
    const int i0 = blockIdx.x * 128, bh = blockIdx.y, hi_ = bh % H, bi = bh / H;
    const int g = g_heads == 1 ? 0 : hi_;
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_ld, 1); mbar_init(&bar_mma, 1);
        mbar_fence_init();
        mbar_expect_tx(&bar_ld, 32768 + (4 * R / 64) * 8192 + 8192);
        tma_load_4d(smem + L::X, &mapX, 0, i0, hi_, bi, &bar_ld);
        tma_load_4d(smem + L::D, &mapDS, 0, i0, hi_, bi, &bar_ld);
#pragma unroll
        for (int q = 0; q < 4 * R / 64; ++q) tma_load_3d(smem + L::W1 + q * 8192, &mapW1, q * 64, 0, g, &bar_ld);
        tma_load_3d(smem + L::W2, &mapW2, 0, 0, g, &bar_ld);
    }
    if (warp == 0) { tmem_alloc(&tm_slot, 256); tmem_relinquish(); }
    for (int ch = 2 * R / 8; ch < 8; ++ch) {
        *reinterpret_cast<uint4*>(smem + L::HL + swz128_offset(tid, ch)) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(smem + L::HL + 16384 + swz128_offset(tid, ch)) = make_uint4(0, 0, 0, 0);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot, lane_tm = tm + ((uint32_t)(warp * 32) << 16);
    constexpr uint32_t cD1 = 0, cD2 = 128, cD4 = 192;       // D3 reuses D2's columns
    const float rs = rsqrtf((float)R);
    uint32_t uses = 0;
    bool ok = mbar_wait(&bar_ld, 0, status, kErrTma);
    if (tid == 0 && ok) { tc_fence_after(); issue_first<R>(tm + cD1, smem); umma_commit(&bar_mma); }
    ok = ok && mbar_wait(&bar_mma, uses++ & 1, status, kErrMma);
    tc_fence_after();
    if (ok) stage_m12<R>(lane_tm + cD1, smem, tid);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) { tc_fence_after(); issue_second<R>(tm + cD2, smem); umma_commit(&bar_mma); }
    ok = ok && mbar_wait(&bar_mma, uses++ & 1, status, kErrMma);
    tc_fence_after();
    if (ok) {
        // [dC1 | dC2] = [dM * C2 | dM * C1] / sqrt(R), written over this thread's row of the dS tile
        float dmv[R];
#pragma unroll
        for (int ch = 0; ch < R / 8; ++ch) {
            const uint4 q = *reinterpret_cast<const uint4*>(smem + L::D + swz128_offset(tid, ch));
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                dmv[ch * 8 + 2 * i] = __uint_as_float(w[i] << 16) * rs;
                dmv[ch * 8 + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u) * rs;
            }
        }
#pragma unroll
        for (int c0 = 0; c0 < R; c0 += 16) {
            uint32_t u1[16], u2[16];
            tmem_ld16(lane_tm + cD2 + c0, u1);
            tmem_ld16(lane_tm + cD2 + R + c0, u2);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
                float d1[8], d2[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    d1[q] = dmv[c0 + j + q] * __uint_as_float(u2[j + q]);
                    d2[q] = dmv[c0 + j + q] * __uint_as_float(u1[j + q]);
                }
                put8(smem + L::D, tid, (c0 + j) / 8, d1);
                put8(smem + L::D, tid, (R + c0 + j) / 8, d2);
            }
        }
        for (int ch = 2 * R / 8; ch < 8; ++ch)
            *reinterpret_cast<uint4*>(smem + L::D + swz128_offset(tid, ch)) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) {
        // [dM1 | dM2] = [dC1 | dC2] W2^T: W2's tile read K-major (its columns are this GEMM's contraction)
        tc_fence_after();
        constexpr uint32_t idesc = idesc_bf16(128, 64, false, false);
        const uint64_t ad = smem_desc(smem_u32(smem + L::D), 0, 1024, kSwz128);
        const uint64_t bd = smem_desc(smem_u32(smem + L::W2), 0, 1024, kSwz128);
#pragma unroll
        for (int k = 0; k < 2 * R / 16; ++k) umma_ss(tm + cD2, desc_off(ad, k * 32), desc_off(bd, k * 32), idesc, k > 0);
        umma_commit(&bar_mma);
    }
    ok = ok && mbar_wait(&bar_mma, uses++ & 1, status, kErrMma);
    tc_fence_after();
    if (ok) {
        // [dA1 | dA2 | dB1 | dB2] = [dM1*A2 | dM1*A1 | dM2*B2 | dM2*B1] / sqrt(R) over the hi/lo tiles (dead since GEMM 2)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int c0 = 0; c0 < R; c0 += 16) {
                uint32_t dmu[16], u1[16], u2[16];
                tmem_ld16(lane_tm + cD2 + half * R + c0, dmu);
                tmem_ld16(lane_tm + cD1 + half * 2 * R + c0, u1);
                tmem_ld16(lane_tm + cD1 + half * 2 * R + R + c0, u2);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; j += 8) {
                    float e1[8], e2[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float dmq = __uint_as_float(dmu[j + q]) * rs;
                        e1[q] = dmq * __uint_as_float(u2[j + q]);
                        e2[q] = dmq * __uint_as_float(u1[j + q]);
                    }
                    const int col1 = half * 2 * R + c0 + j, col2 = col1 + R;      // columns of the [128 x 4R] operand
                    put8(smem + L::HL + (col1 / 64) * 16384, tid, (col1 % 64) / 8, e1);
                    put8(smem + L::HL + (col2 / 64) * 16384, tid, (col2 % 64) / 8, e2);
                }
            }
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) {
        // dX = [dA1 | dA2 | dB1 | dB2] W1^T: W1's two column groups read K-major
        tc_fence_after();
        constexpr uint32_t idesc = idesc_bf16(128, 64, false, false);
#pragma unroll
        for (int k = 0; k < 4 * R / 16; ++k) {
            const uint64_t ad = smem_desc(smem_u32(smem + L::HL) + (k / 4) * 16384, 0, 1024, kSwz128);
            const uint64_t bd = smem_desc(smem_u32(smem + L::W1) + (k / 4) * 8192, 0, 1024, kSwz128);
            umma_ss(tm + cD4, desc_off(ad, (k % 4) * 32), desc_off(bd, (k % 4) * 32), idesc, k > 0);
        }
        umma_commit(&bar_mma);
    }
    ok = ok && mbar_wait(&bar_mma, uses++ & 1, status, kErrMma);
    tc_fence_after();
    if (ok) {
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(lane_tm + cD4 + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
                float o[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) o[q] = __uint_as_float(v[j + q]);
                put8(smem + L::X, tid, (c0 + j) / 8, o);
            }
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) {
        tma_store_tile(&mapDX, smem + L::X, i0, hi_, bi);
        bulk_commit();
        bulk_wait_read();
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 256);
}

struct Sk8Maps { CUtensorMap W1, W2; };

bool sk8_maps(const Dims& d, char* bank, Sk8Maps* m) {
    bf16* W1 = reinterpret_cast<bf16*>(bank);
    bf16* W2 = W1 + (size_t)d.g_heads * kW1;
    return tc_map_3d(&m->W1, W1, 128, 64, d.g_heads, 64, 64) && tc_map_3d(&m->W2, W2, 64, 64, d.g_heads, 64, 64);
}

template <int R>
cudaError_t fwd_t(const Dims& d, const void* X, void* S, char* bank, int* status, cudaStream_t s, int* launches) {
    Sk8Maps wm;
    CUtensorMap mX, mS;
    const int64_t hs = (int64_t)d.n * 64, bs = (int64_t)d.H * hs;
    if (!sk8_maps(d, bank, &wm) || !tc_map_rows(&mX, X, d.B, d.H, d.n, d.sb, d.sh, d.sn) || !tc_map_rows(&mS, S, d.B, d.H, d.n, bs, hs, 64))
        return cudaErrorInvalidValue;
    constexpr size_t smem = Sk8Smem::total + 1024;
    PSK_TRY(set_smem(sk8_tc_fwd_kernel<R>, smem));
    prof_begin("sk8_tc_fwd_kernel", s);
    sk8_tc_fwd_kernel<R><<<dim3(d.n / 128, d.BH()), 128, smem, s>>>(mX, wm.W1, wm.W2, mS, d.g_heads, d.H, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <int R>
cudaError_t bwd_t(const Dims& d, const void* X, const void* dS, void* dX, char* bank, int* status, cudaStream_t s, int* launches) {
    Sk8Maps wm;
    CUtensorMap mX, mDS, mDX;
    const int64_t hs = (int64_t)d.n * 64, bs = (int64_t)d.H * hs;
    if (!sk8_maps(d, bank, &wm) || !tc_map_rows(&mX, X, d.B, d.H, d.n, d.sb, d.sh, d.sn) || !tc_map_rows(&mDS, dS, d.B, d.H, d.n, bs, hs, 64) ||
        !tc_map_rows(&mDX, dX, d.B, d.H, d.n, d.sb, d.sh, d.sn))
        return cudaErrorInvalidValue;
    constexpr size_t smem = Sk8Smem::total + 1024;
    PSK_TRY(set_smem(sk8_tc_bwd_kernel<R>, smem));
    prof_begin("sk8_tc_bwd_kernel", s);
    sk8_tc_bwd_kernel<R><<<dim3(d.n / 128, d.BH()), 128, smem, s>>>(mX, wm.W1, wm.W2, mDS, mDX, d.g_heads, d.H, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace

bool sketch8_tc_supported(const Dims& d) { return d.bf16 && d.p == 8 && !d.learned && d.h == 64 && (d.r == 16 || d.r == 32); }

size_t sketch8_tc_bank_bytes(const Dims& d) { return align_up((size_t)d.g_heads * (kW1 + kW2) * sizeof(bf16)); }

cudaError_t sketch8_tc_prepare(const Dims& d, const void* G1, const void* G2, char* bank, cudaStream_t s, int* launches) {
    bf16* W1 = reinterpret_cast<bf16*>(bank);
    bf16* W2 = W1 + (size_t)d.g_heads * kW1;
    prof_begin("sk8_bank_kernel", s);
    sk8_bank_kernel<<<dim3((kW1 + kW2 + 255) / 256, d.g_heads), 256, 0, s>>>((const bf16*)G1, (const bf16*)G2, d.r, W1, W2);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

// S = the [hi | lo] rows of the degree-8 half sketch of X (contiguous [B,H,n,64] bf16)
cudaError_t sketch8_tc_fwd(const Dims& d, const void* X, void* S, char* bank, int* status, cudaStream_t s, int* launches) {
    return d.r == 16 ? fwd_t<16>(d, X, S, bank, status, s, launches) : fwd_t<32>(d, X, S, bank, status, s, launches);
}

// dX (strides of X) from dS, the gradient of those rows (only its first r columns matter)
cudaError_t sketch8_tc_bwd(const Dims& d, const void* X, const void* dS, void* dX, char* bank, int* status, cudaStream_t s,
                           int* launches) {
    return d.r == 16 ? bwd_t<16>(d, X, dS, dX, bank, status, s, launches) : bwd_t<32>(d, X, dS, dX, bank, status, s, launches);
}

}  // namespace psk
