// lt(A B^T) C for given bf16 feature matrices on the tensor cores: Section 3.1's block algorithm,
//   H_l = B_l^T C_l,  Z_l = sum_{j<l} H_j,  rows of block l = lt(A_l B_l^T) C_l + A_l Z_l,
// with fp32 accumulation in tensor memory.  A, B: [batch, n, m] bf16 (m a multiple of 64),
// C: [batch, n, 64] bf16, Out: [batch, n, 64] fp32, blocks of b = 128 or 256 rows.
// Every operand goes to the tensor cores as TMA left it in shared memory: B_l^T C_l contracts over
// the rows (both tiles MN-major), A_l Z_l and A_l B_l^T over the features (A, B K-major, Z MN-major).
#include "tc_common.cuh"

namespace psk {

namespace {

using namespace tc;

// ---------------------------------------------------------------------------
// prefix states, bf16 [batch][t][m][64] (entry l: the sum over the blocks before l; l = 0 unused).
// grid (ceil(m/128), batch), 128 threads: a CTA walks the whole sequence for 128 features, the
// running sum stays in tensor memory and is copied out at every block boundary.
// ---------------------------------------------------------------------------
constexpr int kStStage = 32768 + 16384;     // two 64-feature groups of the B tile, the C tile
constexpr int kStSmem = 2 * kStStage + 1024;

__global__ void __launch_bounds__(128)
lt_tc_state_kernel(const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapC, bf16* __restrict__ Z,
                   int m, int t, int tpb, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_full[2], bar_free[2], bar_acc;
    __shared__ uint32_t tm_slot;
    const int tid = threadIdx.x, warp = tid / 32;
    const int f0 = blockIdx.x * 128, bt = blockIdx.y;
    const int NT = (t - 1) * tpb;               // the last block's state is never used
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_full[0], 1); mbar_init(&bar_full[1], 1);
        mbar_init(&bar_free[0], 1); mbar_init(&bar_free[1], 1);
        mbar_init(&bar_acc, 1);
        mbar_fence_init();
    }
    if (warp == 0) { tmem_alloc(&tm_slot, 64); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot;
    auto load = [&](int j) {
        const int s = j & 1;
        uint8_t* st = smem + s * kStStage;
        mbar_expect_tx(&bar_full[s], kStStage);
        tma_load_3d(st, &mapB, f0, j * 128, bt, &bar_full[s]);
        tma_load_3d(st + 16384, &mapB, f0 + 64, j * 128, bt, &bar_full[s]);     // beyond m: zeros
        tma_load_3d(st + 32768, &mapC, 0, j * 128, bt, &bar_full[s]);
    };
    if (tid == 0 && NT > 0) { load(0); if (NT > 1) load(1); }
    bool ok = true;
    for (int l = 0; l + 1 < t; ++l) {
        if (tid == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, 64, true, true);
            for (int tt = 0; tt < tpb && ok; ++tt) {
                const int j = l * tpb + tt, s = j & 1;
                ok = mbar_spin(&bar_full[s], (j >> 1) & 1, status, kErrTma);
                if (!ok) break;
                tc_fence_after();
                const uint32_t base = smem_u32(smem + s * kStStage);
                const uint64_t ad = smem_desc(base, 16384, 1024, kSwz128);
                const uint64_t bd = smem_desc(base + 32768, 0, 1024, kSwz128);
#pragma unroll
                for (int k = 0; k < 8; ++k) umma_ss(tm, desc_off(ad, k * 2048), desc_off(bd, k * 2048), idesc, (j > 0 || k > 0) ? 1u : 0u);
                umma_commit(&bar_free[s]);
                if (j + 2 < NT) {
                    ok = mbar_spin(&bar_free[s], (j >> 1) & 1, status, kErrMma);
                    if (ok) load(j + 2);
                }
            }
            if (ok) umma_commit(&bar_acc);
        }
        ok = mbar_wait(&bar_acc, l & 1, status, kErrMma) && ok;
        tc_fence_after();
        if (ok && f0 + tid < m) {
            bf16* dst = Z + (((size_t)bt * t + l + 1) * m + f0 + tid) * 64;
            const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t u[32];
                tmem_ld32(lane_tm + c0, u);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 8)
                    *reinterpret_cast<uint4*>(dst + c0 + j) =
                        make_uint4(pack_bf16(__uint_as_float(u[j]), __uint_as_float(u[j + 1])), pack_bf16(__uint_as_float(u[j + 2]), __uint_as_float(u[j + 3])),
                                   pack_bf16(__uint_as_float(u[j + 4]), __uint_as_float(u[j + 5])), pack_bf16(__uint_as_float(u[j + 6]), __uint_as_float(u[j + 7])));
            }
        }
        // the next block's MMAs add to the accumulator only after everyone has read it
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 64);
}

// ---------------------------------------------------------------------------
// rows: grid (b/128, t, batch), 160 threads.  Warps 0-3: thread = row (masking, epilogue); warp 4:
// one thread issues every TMA load and every MMA.  The features are walked once in chunks of 64:
// each chunk of the own rows multiplies the prefix state's chunk (into O) and the same chunk of
// every row tile of the block up to the own one (into that tile's scores S); the masked scores then
// multiply the tiles of C from tensor memory.
// ---------------------------------------------------------------------------
constexpr int kRwStage = 16384 + 8192 + 2 * 16384;
constexpr int kRwSmem = 2 * kRwStage + 2 * 16384 + 1024;
constexpr uint32_t cO = 0, cS = 128;

__global__ void __launch_bounds__(160)
lt_tc_rows_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                  const __grid_constant__ CUtensorMap mapC, const __grid_constant__ CUtensorMap mapZ,
                  float* __restrict__ Out, int n, int m, int b, int t, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    uint8_t* sC = smem + 2 * kRwStage;
    __shared__ uint64_t bar_full[2], bar_free[2], bar_c, bar_s, bar_p, bar_o;
    __shared__ uint32_t tm_slot;
    const int tid = threadIdx.x, warp = tid / 32;
    const int tau = blockIdx.x, l = blockIdx.y, bt = blockIdx.z;
    const int row0 = l * b + tau * 128, nch = m / 64, ntl = tau + 1;
    if (tid == 0) {
        cta_giveup_init();
        mbar_init(&bar_full[0], 1); mbar_init(&bar_full[1], 1);
        mbar_init(&bar_free[0], 1); mbar_init(&bar_free[1], 1);
        mbar_init(&bar_c, 1); mbar_init(&bar_s, 1); mbar_init(&bar_o, 1);
        mbar_init(&bar_p, 128);
        mbar_fence_init();
    }
    if (warp == 4) { tmem_alloc(&tm_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tm_slot;
    if (tid == 128) {
        mbar_expect_tx(&bar_c, ntl * 16384);
        for (int tp = 0; tp < ntl; ++tp) tma_load_3d(sC + tp * 16384, &mapC, 0, l * b + tp * 128, bt, &bar_c);
        auto load = [&](int c) {
            const int s = c & 1;
            uint8_t* st = smem + s * kRwStage;
            mbar_expect_tx(&bar_full[s], 16384 + (l > 0 ? 8192 : 0) + ntl * 16384);
            tma_load_3d(st, &mapA, c * 64, row0, bt, &bar_full[s]);
            if (l > 0) tma_load_3d(st + 16384, &mapZ, 0, c * 64, bt * t + l, &bar_full[s]);
            for (int tp = 0; tp < ntl; ++tp) tma_load_3d(st + 24576 + tp * 16384, &mapB, c * 64, l * b + tp * 128, bt, &bar_full[s]);
        };
        load(0);
        if (nch > 1) load(1);
        constexpr uint32_t idesc_z = idesc_bf16(128, 64, false, true);
        constexpr uint32_t idesc_s = idesc_bf16(128, 128, false, false);
        bool ok = true;
        for (int c = 0; c < nch && ok; ++c) {
            const int s = c & 1;
            ok = mbar_spin(&bar_full[s], (c >> 1) & 1, status, kErrTma);
            if (!ok) break;
            tc_fence_after();
            const uint32_t base = smem_u32(smem + s * kRwStage);
            const uint64_t ad = smem_desc(base, 0, 1024, kSwz128);
            if (l > 0) {
                const uint64_t zd = smem_desc(base + 16384, 0, 1024, kSwz128);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_ss(tm + cO, desc_off(ad, k * 32), desc_off(zd, k * 2048), idesc_z, (c > 0 || k > 0) ? 1u : 0u);
            }
            for (int tp = 0; tp < ntl; ++tp) {
                const uint64_t bd = smem_desc(base + 24576 + tp * 16384, 0, 1024, kSwz128);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_ss(tm + cS + tp * 128, desc_off(ad, k * 32), desc_off(bd, k * 32), idesc_s, (c > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(&bar_free[s]);
            if (c + 2 < nch) {
                ok = mbar_spin(&bar_free[s], (c >> 1) & 1, status, kErrMma);
                if (ok) load(c + 2);
            }
        }
        if (ok) {
            umma_commit(&bar_s);
            ok = mbar_spin(&bar_c, 0, status, kErrTma) && mbar_spin(&bar_p, 0, status, kErrMma);
        }
        if (ok) {
            tc_fence_after();
            for (int tp = 0; tp < ntl; ++tp) {
                const uint64_t cd = smem_desc(smem_u32(sC + tp * 16384), 0, 1024, kSwz128);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_ts(tm + cO, tm + cS + tp * 128 + k * 8, desc_off(cd, k * 2048), idesc_z, (l > 0 || tp > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(&bar_o);
        }
    } else if (warp < 4) {
        const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
        bool ok = mbar_wait(&bar_s, 0, status, kErrMma);
        tc_fence_after();
        if (ok) {
            for (int tp = 0; tp < ntl; ++tp) {
                const bool diag = tp == tau;
#pragma unroll
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t u[32], pk[16];
                    tmem_ld32(lane_tm + cS + tp * 128 + c0, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const float x = (diag && c0 + j > tid) ? 0.f : __uint_as_float(u[j]);
                        const float y = (diag && c0 + j + 1 > tid) ? 0.f : __uint_as_float(u[j + 1]);
                        pk[j / 2] = pack_bf16(x, y);
                    }
                    // the masked scores as the bf16 A operand of the last GEMM, over the columns just read
                    tmem_st16(lane_tm + cS + tp * 128 + c0 / 2, pk);
                }
            }
            tmem_st_wait();
        }
        tc_fence_before();
        mbar_arrive(&bar_p);
        ok = ok && mbar_wait(&bar_o, 0, status, kErrMma);
        tc_fence_after();
        if (ok) {
            float* dst = Out + ((size_t)bt * n + row0 + tid) * 64;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t u[32];
                tmem_ld32(lane_tm + cO + c0, u);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(dst + c0 + j) = make_float4(__uint_as_float(u[j]), __uint_as_float(u[j + 1]),
                                                                           __uint_as_float(u[j + 2]), __uint_as_float(u[j + 3]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tm, 512);
}

bool lt_tc_args_ok(int batch, int n, int m, int k, int b) {
    return batch > 0 && n > 0 && m > 0 && m % 64 == 0 && k == 64 && (b == 128 || b == 256) && n % b == 0 &&
           (int64_t)batch * n < ((int64_t)1 << 31);
}

}  // namespace
}  // namespace psk

using namespace psk;

extern "C" {

size_t psk_lt_multiply_bf16_workspace_bytes(int batch, int n, int m, int k, int b) {
    if (!lt_tc_args_ok(batch, n, m, k, b)) return 0;
    return kStatusBytes + align_up((size_t)batch * (n / b) * m * 64 * sizeof(bf16));
}

int psk_lt_multiply_bf16(int batch, int n, int m, int k, int b, const void* A, const void* B, const void* C, float* Out,
                         void* workspace, size_t workspace_bytes, void* stream) {
    if (!lt_tc_args_ok(batch, n, m, k, b)) return PSK_ERR_SHAPE;
    if (!A || !B || !C || !Out) return PSK_ERR_INVALID_ARG;
    for (const void* p : {A, B, C, (const void*)Out, (const void*)workspace})
        if (reinterpret_cast<uintptr_t>(p) & 15u) return PSK_ERR_ALIGN;
    const size_t need = psk_lt_multiply_bf16_workspace_bytes(batch, n, m, k, b);
    if (!workspace || workspace_bytes < need) return PSK_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    int* status = static_cast<int*>(workspace);
    bf16* Z = reinterpret_cast<bf16*>(static_cast<char*>(workspace) + kStatusBytes);
    const int t = n / b, tpb = b / 128;
    if (cudaMemsetAsync(workspace, 0, kStatusBytes, s) != cudaSuccess) return PSK_ERR_CUDA;
    CUtensorMap mA, mB, mC, mZ;
    if (!tc_map_3d(&mA, A, m, n, batch, 64, 128) || !tc_map_3d(&mB, B, m, n, batch, 64, 128) ||
        !tc_map_3d(&mC, C, 64, n, batch, 64, 128) || !tc_map_3d(&mZ, Z, 64, m, (int64_t)batch * t, 64, 64))
        return PSK_ERR_CUDA;
    if (cudaFuncSetAttribute(lt_tc_state_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStSmem) != cudaSuccess ||
        cudaFuncSetAttribute(lt_tc_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRwSmem) != cudaSuccess)
        return PSK_ERR_CUDA;
    if (t > 1) {
        prof_begin("lt_tc_state_kernel", s);
        lt_tc_state_kernel<<<dim3((m + 127) / 128, batch), 128, kStSmem, s>>>(mB, mC, Z, m, t, tpb, status);
        prof_end(s);
    }
    prof_begin("lt_tc_rows_kernel", s);
    lt_tc_rows_kernel<<<dim3(tpb, t, batch), 160, kRwSmem, s>>>(mA, mB, mC, mZ, Out, n, m, b, t, status);
    prof_end(s);
    return cudaGetLastError() == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

}  // extern "C"
