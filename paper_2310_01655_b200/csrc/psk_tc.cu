// Tensor-core path (bf16 operands, fp32 accumulation in tensor memory) of causal Polysketch
// attention.  Same steps as Section 3.1 -- per-block states, prefix scan, output rows -- with
// the r(r+1)/2 distinct features of the self-tensored sketch (tc_features.cuh) generated in
// registers and handed to tcgen05.mma without ever touching HBM.
//
// State storage (HBM scratch): S[BH][t][80][FP] bf16, "transposed + extended": row c < 64 is
// column c of H_l / Z_l (features contiguous), row 64 is the normaliser column (the "| 1" of
// [V | 1], or the last column of E in the backward), rows 65..79 are zero.  One TMA box of
// [80 rows x 64 features] serves as a K-major B operand with N = 80 (contract over features)
// or as an MN-major B operand with K = 80 (contract over the 65 columns).
#include "psk_internal.cuh"
#include "tc_features.cuh"
#include "tc_common.cuh"

#include <mutex>
#include <type_traits>

namespace psk {

using namespace tc;
typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------------------
// host: tensor maps
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeFn encoder() {
    static EncodeFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
    });
    return fn;
}

// [B,H,n,64] bf16 tensor with element strides; box = 128 rows x 64 columns, 128-byte swizzle.
bool tc_map_rows(CUtensorMap* m, const void* base, int B, int H, int n, int64_t sb, int64_t sh, int64_t sn) {
    EncodeFn enc = encoder();
    if (!enc) return false;
    cuuint64_t dims[4] = {64, (cuuint64_t)n, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)sn * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
    cuuint32_t box[4] = {64, 128, 1, 1}, es[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// States S[nblk][80][FP] bf16; box = 80 rows x 64 features.
bool tc_map_states(CUtensorMap* m, const void* base, int FP, int64_t nblk) {
    EncodeFn enc = encoder();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)FP, 80, (cuuint64_t)nblk};
    cuuint64_t strides[2] = {(cuuint64_t)FP * 2, (cuuint64_t)FP * 160};
    cuuint32_t box[3] = {64, 80, 1}, es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

// ---------------------------------------------------------------------------
// Per-block state  H_l = phi(X_l)^T [Y_l | y65]   (Section 3.1), feature tiles [T0, T0+TN)
//   X: tensor that is sketched (K for the forward state, Q for the backward's reverse state)
//   Y: [V] or [E(:, :64)];  y65: last column (nullptr = all ones)
// grid (t, BH), 128 threads: thread = token for the sketch and the feature generator,
// thread = feature row for the epilogue.
// ---------------------------------------------------------------------------
template <int R>
struct StateSmem {
    static constexpr uint32_t X = 0, Y = 16384, Ext = 32768, G = 49152;
    static constexpr uint32_t A0 = G + (2 * R * 128 < 1024 ? 1024 : 2 * R * 128);
    static constexpr uint32_t A1 = A0 + 32768, total = A1 + 32768;
};

template <int R, int T0, int TN>
__global__ void __launch_bounds__(128)
tc_state_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                const bf16* __restrict__ G1, const bf16* __restrict__ G2, int g_heads, int H, int n, int b, int t,
                const float* __restrict__ y65, const float* __restrict__ cmean, int center_mode,
                bf16* __restrict__ S, int* status) {
    using F = Feat<R>;
    using L = StateSmem<R>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_load, bar_sketch, bar_a[2];
    __shared__ uint32_t tmem_slot;
    __shared__ float cm[64];
    const int tid = threadIdx.x, warp = tid / 32, l = blockIdx.x, bh = blockIdx.y;
    const int hi = bh % H, bi = bh / H;
    const int g = g_heads == 1 ? 0 : hi;

    if (tid == 0) {
        mbar_init(&bar_load, 1); mbar_init(&bar_sketch, 1); mbar_init(&bar_a[0], 1); mbar_init(&bar_a[1], 1);
        mbar_fence_init();
        tma_prefetch_desc(&mapX); tma_prefetch_desc(&mapY);
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    build_g_tile<R>(smem + L::G, G1 + (size_t)g * 64 * R, G2 + (size_t)g * 64 * R, tid);
    if (cmean != nullptr && tid < 64) cm[tid] = cmean[(size_t)bh * 64 + tid];
    for (int e = tid; e < 16384 / 16; e += 128) reinterpret_cast<uint4*>(smem + L::Ext)[e] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_slot;
    const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
    constexpr uint32_t kAcc = 2 * R;               // accumulators start after the sketch columns
    constexpr uint32_t idesc_state = idesc_bf16(128, 80, true, true);

    uint32_t a_use0 = 0, a_use1 = 0;
    bool ok = true;
    const int ntt = b / 128;
    for (int tt = 0; tt < ntt && ok; ++tt) {
        const int row0 = l * b + tt * 128;
        if (tid == 0) {
            mbar_expect_tx(&bar_load, 32768);
            tma_load_4d(smem + L::X, &mapX, 0, row0, hi, bi, &bar_load);
            tma_load_4d(smem + L::Y, &mapY, 0, row0, hi, bi, &bar_load);
        }
        {   // last column of this token's right-hand side row
            const float y = y65 ? y65[(size_t)bh * n + row0 + tid] : 1.f;
            *reinterpret_cast<bf16*>(smem + L::Ext + swz128_offset(tid, 0)) = __float2bfloat16_rn(y);
        }
        ok = mbar_wait(&bar_load, tt & 1, status, kErrTma);
        if (tid == 0) {
            tc_fence_after();
            issue_sketch<R>(tm, smem + L::X, smem + L::G);
            umma_commit(&bar_sketch);
        }
        ok = ok && mbar_wait(&bar_sketch, tt & 1, status, kErrMma);
        tc_fence_after();
        float m[R];
        read_half_sketch<R>(lane_tm, m);
        static_for<0, TN>([&](auto ic) {
            constexpr int I = decltype(ic)::value;
            const int it = tt * TN + I, buf = it & 1;
            const uint32_t used = buf ? a_use1 : a_use0;
            if (used > 0) ok = ok && mbar_wait(&bar_a[buf], (used - 1) & 1, status, kErrMma);
            uint8_t* sA = smem + (buf ? L::A1 : L::A0);
            static_for<0, 16>([&](auto cc) {
                constexpr int C = decltype(cc)::value;
                uint32_t pk[4];
                gen_features<R, (T0 + I) * 128 + C * 8, false, 4>(m, pk);
                *reinterpret_cast<uint4*>(sA + (C / 8) * 16384 + swz128_offset(tid, C % 8)) =
                    make_uint4(pk[0], pk[1], pk[2], pk[3]);
            });
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_ss(tm + kAcc + 80 * I, smem_desc(smem_u32(sA) + k * 2048, 16384, 1024, kSwz128),
                            smem_desc(smem_u32(smem + L::Y) + k * 2048, 16384, 1024, kSwz128), idesc_state,
                            (tt > 0 || k > 0) ? 1u : 0u);
                umma_commit(&bar_a[buf]);
            }
            if (buf) ++a_use1; else ++a_use0;
        });
        // the next token tile overwrites Y / Ext (and the sketch columns): drain the state MMAs
        if (a_use0 > 0) ok = ok && mbar_wait(&bar_a[0], (a_use0 - 1) & 1, status, kErrMma);
        if (a_use1 > 0) ok = ok && mbar_wait(&bar_a[1], (a_use1 - 1) & 1, status, kErrMma);
        tc_fence_after();
        __syncthreads();
    }
    // epilogue: lane = feature row; store transposed (+ extended) as bf16
    if (ok) {
        const size_t blk = (size_t)bh * t + l;
        static_for<0, TN>([&](auto ic) {
            constexpr int I = decltype(ic)::value;
            const int f = (T0 + I) * 128 + tid;
            bf16* dst = S + blk * 80 * F::FP + f;
            float last;                         // column 64 of this feature row
            {
                uint32_t v[16];
                tmem_ld16(lane_tm + kAcc + 80 * I + 64, v);
                tmem_ld_wait();
                last = __uint_as_float(v[0]);
            }
            float corr = 0.f;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_tm + kAcc + 80 * I + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    float x = __uint_as_float(v[j]);
                    // centred values without touching the operands (all in fp32):
                    //   mode 1: sum phi (y - c)^T = H[:, :64] - H[:, 64] c^T
                    //   mode 2: last column becomes H[:, 64] - H[:, :64] c
                    if (center_mode == 1) x = fmaf(-cm[c0 + j], last, x);
                    if (center_mode == 2) corr = fmaf(cm[c0 + j], x, corr);
                    dst[(size_t)(c0 + j) * F::FP] = __float2bfloat16_rn(x);
                }
            }
            dst[(size_t)64 * F::FP] = __float2bfloat16_rn(last - corr);
#pragma unroll
            for (int j = 1; j < 16; ++j) dst[(size_t)(64 + j) * F::FP] = __float2bfloat16_rn(0.f);
        });
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

// Exclusive prefix (or suffix) over the t block states of each head, in place: fp32 running sum,
// bf16 storage.  Each thread owns 8 consecutive elements.
__global__ void __launch_bounds__(256)
tc_scan_kernel(bf16* __restrict__ S, size_t elems8, int t, int reverse) {
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= elems8) return;
    uint4* p = reinterpret_cast<uint4*>(S) + (size_t)blockIdx.y * t * elems8 + e;
    float run[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) run[j] = 0.f;
    constexpr int U = 8;                       // loads in flight per thread
    for (int s0 = 0; s0 < t; s0 += U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int s = s0 + u;
            if (s < t) v[u] = p[(size_t)(reverse ? (t - 1 - s) : s) * elems8];
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int s = s0 + u;
            if (s < t) {
                const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    o[j] = pack_bf16(run[2 * j], run[2 * j + 1]);
                    run[2 * j] += __uint_as_float(w[j] << 16);
                    run[2 * j + 1] += __uint_as_float(w[j] & 0xFFFF0000u);
                }
                p[(size_t)(reverse ? (t - 1 - s) : s) * elems8] = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Forward output rows (Section 3.1): for a 128-row tile of block l,
//   N = phi_w(Q) Z_l  (tensor memory A operand x TMA-fed Z chunks, N = 80: column 64 = normaliser)
//     + sum over key tiles of the same block  lt((M_q M_k^T)^2) V
//   d = 1 + rowsum(diagonal weights) + N[:, 64];  O = N[:, :64] / d
// grid (b/128, t, BH), 128 threads (thread = query row).
// ---------------------------------------------------------------------------
constexpr int kZStages = 4;
constexpr uint32_t kZStageBytes = 80 * 128;     // one [80 rows x 64 features] box

template <int R>
struct OutSmem {
    static constexpr uint32_t Q = 0, K = 16384, V = 32768, G = 49152;
    static constexpr uint32_t Mq = G + (2 * R * 128 < 1024 ? 1024 : 2 * R * 128);
    static constexpr uint32_t Mk = Mq + 128 * 3 * R * 2;      // split operands: 3R columns
    static constexpr uint32_t Z = (Mk + 128 * 3 * R * 2 + 1023) / 1024 * 1024;
    static constexpr uint32_t total = Z + kZStages * kZStageBytes;
};

// MODE 0: forward (writes O, denom).  MODE 1: the backward's recomputation of the row numerators
// against centred prefix states; writes E = dO/d (bf16), e65 = -(dO.(O - c))/d and
// e65h = e65 - E.c (fp32), with O - c = (N' - c)/d taken from the fp32 accumulators rather than
// from the rounded O the caller holds.
template <int R, int MODE>
__global__ void __launch_bounds__(128)
tc_fwd_out_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                  const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapZ,
                  const bf16* __restrict__ G1, const bf16* __restrict__ G2, int g_heads, int H, int n, int b, int t,
                  const float* __restrict__ cmean, bf16* __restrict__ O, int64_t sb, int64_t sh, int64_t sn,
                  float* __restrict__ denom, const bf16* __restrict__ dO, bf16* __restrict__ E,
                  float* __restrict__ e65, float* __restrict__ e65h, int* status) {
    using F = Feat<R>;
    using L = OutSmem<R>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_q, bar_kv, bar_mma, bar_a[2], bar_z[kZStages];
    __shared__ uint32_t tmem_slot;
    __shared__ float cm[64];
    const int tid = threadIdx.x, warp = tid / 32, tau = blockIdx.x, l = blockIdx.y, bh = blockIdx.z;
    const int hi = bh % H, bi = bh / H;
    const int g = g_heads == 1 ? 0 : hi;
    const int row0 = l * b + tau * 128;
    const int blk = bh * t + l;

    if (tid == 0) {
        mbar_init(&bar_q, 1); mbar_init(&bar_kv, 1); mbar_init(&bar_mma, 1);
        mbar_init(&bar_a[0], 1); mbar_init(&bar_a[1], 1);
        for (int s = 0; s < kZStages; ++s) mbar_init(&bar_z[s], 1);
        mbar_fence_init();
        tma_prefetch_desc(&mapQ); tma_prefetch_desc(&mapK); tma_prefetch_desc(&mapV); tma_prefetch_desc(&mapZ);
        mbar_expect_tx(&bar_q, 16384);
        tma_load_4d(smem + L::Q, &mapQ, 0, row0, hi, bi, &bar_q);
        if (l > 0) {
            for (int c = 0; c < kZStages && c < F::NC; ++c) {
                mbar_expect_tx(&bar_z[c], kZStageBytes);
                tma_load_3d(smem + L::Z + c * kZStageBytes, &mapZ, c * 64, 0, blk, &bar_z[c]);
            }
        }
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    build_g_tile<R>(smem + L::G, G1 + (size_t)g * 64 * R, G2 + (size_t)g * 64 * R, tid);
    if (MODE == 1 && tid < 64) cm[tid] = cmean[(size_t)bh * 64 + tid];
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_slot;
    const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
    // tensor-memory columns
    constexpr uint32_t cSk = 0, cS = 128, cW = 256, cA = 320, cO = 384;
    uint32_t mma_uses = 0;
    bool ok = true;

    // ---- half sketch of the query rows ----
    ok = mbar_wait(&bar_q, 0, status, kErrTma);
    if (tid == 0) {
        tc_fence_after();
        issue_sketch<R>(tm + cSk, smem + L::Q, smem + L::G);
        umma_commit(&bar_mma);
    }
    ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
    ++mma_uses;
    tc_fence_after();
    float mq[R];
    read_half_sketch<R>(lane_tm + cSk, mq);
    store_split_rows<R, true>(smem + L::Mq, mq, tid);

    // ---- earlier blocks: weighted features (tensor memory) x prefix state ----
    if (l > 0) {
        uint32_t a_uses[2] = {0, 0};
        static_for<0, F::NC>([&](auto cc) {
            constexpr int C = decltype(cc)::value;
            constexpr int buf = C & 1, stage = C % kZStages;
            constexpr int ksteps = (F::FK - C * 64) >= 64 ? 4 : (F::FK - C * 64) / 16;
            if (a_uses[buf] > 0) {
                ok = ok && mbar_wait(&bar_a[buf], (a_uses[buf] - 1) & 1, status, kErrMma);
                // chunk C-2 is done with its stage: refill it with chunk C-2+kZStages
                if (tid == 0 && C - 2 + kZStages < F::NC) {
                    constexpr int s2 = (C - 2 + 2 * kZStages) % kZStages;
                    mbar_expect_tx(&bar_z[s2], kZStageBytes);
                    tma_load_3d(smem + L::Z + s2 * kZStageBytes, &mapZ, (C - 2 + kZStages) * 64, 0, blk, &bar_z[s2]);
                }
            }
            tc_fence_after();
            uint32_t pk[16];
            gen_features<R, C * 64, true, 16>(mq, pk);
            tmem_st16(lane_tm + cA + buf * 32, pk);
            gen_features<R, C * 64 + 32, true, 16>(mq, pk);
            tmem_st16(lane_tm + cA + buf * 32 + 16, pk);
            tmem_st_wait();
            ok = ok && mbar_wait(&bar_z[stage], (C / kZStages) & 1, status, kErrTma);
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                constexpr uint32_t idesc = idesc_bf16(128, 80, false, false);
                const uint32_t zb = smem_u32(smem + L::Z + stage * kZStageBytes);
#pragma unroll
                for (int k = 0; k < ksteps; ++k)
                    umma_ts(tm + cO, tm + cA + buf * 32 + k * 8, smem_desc(zb + k * 32, 0, 1024, kSwz128), idesc,
                            (C > 0 || k > 0) ? 1u : 0u);
                umma_commit(&bar_a[buf]);
            }
            ++a_uses[buf];
        });
    }

    // ---- same block: key tiles tp <= tau through squared half-sketch scores ----
    float rowsum = 0.f;
    for (int tp = 0; tp <= tau && ok; ++tp) {
        if (tid == 0) {
            // previous users of sK / sV / cW (sketch, P) have completed: bar_mma was waited on below
            mbar_expect_tx(&bar_kv, 32768);
            tma_load_4d(smem + L::K, &mapK, 0, l * b + tp * 128, hi, bi, &bar_kv);
            tma_load_4d(smem + L::V, &mapV, 0, l * b + tp * 128, hi, bi, &bar_kv);
        }
        ok = mbar_wait(&bar_kv, tp & 1, status, kErrTma);
        if (tid == 0) {
            tc_fence_after();
            issue_sketch<R>(tm + cSk, smem + L::K, smem + L::G);
            umma_commit(&bar_mma);
        }
        ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
        ++mma_uses;
        tc_fence_after();
        {
            float mk[R];
            read_half_sketch<R>(lane_tm + cSk, mk);
            store_split_rows<R, false>(smem + L::Mk, mk, tid);
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16(128, 128, false, false);
#pragma unroll
            for (int k = 0; k < 3 * R / 16; ++k)
                umma_ss(tm + cS, smem_desc(smem_u32(smem + L::Mq) + k * 4096, 2048, 128, kSwzNone),
                        smem_desc(smem_u32(smem + L::Mk) + k * 4096, 2048, 128, kSwzNone), idesc, k > 0);
            umma_commit(&bar_mma);
        }
        ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
        ++mma_uses;
        tc_fence_after();
        const bool diag = (tp == tau);
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
            uint32_t v[32], pk[16];
            tmem_ld32(lane_tm + cS + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                float w0 = __uint_as_float(v[j]), w1 = __uint_as_float(v[j + 1]);
                w0 = (diag && c0 + j > tid) ? 0.f : w0 * w0;
                w1 = (diag && c0 + j + 1 > tid) ? 0.f : w1 * w1;
                rowsum += w0 + w1;
                pk[j / 2] = pack_bf16(w0, w1);
            }
            tmem_st16(lane_tm + cW + c0 / 2, pk);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
#pragma unroll
            for (int k = 0; k < 8; ++k)
                umma_ts(tm + cO, tm + cW + k * 8, smem_desc(smem_u32(smem + L::V) + k * 2048, 0, 1024, kSwz128), idesc,
                        (l > 0 || tp > 0 || k > 0) ? 1u : 0u);
            umma_commit(&bar_mma);
        }
        ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
        ++mma_uses;
        tc_fence_after();
    }

    // ---- epilogue ----
    if (ok) {
        float acc[64];
        float d = 1.f + rowsum;
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(lane_tm + cO + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) acc[c0 + j] = __uint_as_float(v[j]);
        }
        if (l > 0) {
            uint32_t v[16];
            tmem_ld16(lane_tm + cO + 64, v);
            tmem_ld_wait();
            d += __uint_as_float(v[0]);
        }
        if constexpr (MODE == 0) {
            const float inv = 1.f / d;
            bf16* o = O + (int64_t)bi * sb + (int64_t)hi * sh + (int64_t)(row0 + tid) * sn;
#pragma unroll
            for (int c = 0; c < 64; c += 8) {
                uint4 v;
                v.x = pack_bf16(acc[c] * inv, acc[c + 1] * inv);
                v.y = pack_bf16(acc[c + 2] * inv, acc[c + 3] * inv);
                v.z = pack_bf16(acc[c + 4] * inv, acc[c + 5] * inv);
                v.w = pack_bf16(acc[c + 6] * inv, acc[c + 7] * inv);
                *reinterpret_cast<uint4*>(o + c) = v;
            }
            if (denom != nullptr) denom[(size_t)bh * n + row0 + tid] = d;
        } else {
            // acc = phi Z' + W V with Z' built from centred values and V raw:
            // N' = acc - rowsum(W) c is the numerator of centred values, O - c = (N' - c) / d.
            const size_t row = (size_t)bh * n + row0 + tid;
            const float dd = denom[row];              // the forward's normaliser (fp32 input)
            const float inv = 1.f / dd;
            const bf16* gp = dO + (int64_t)bi * sb + (int64_t)hi * sh + (int64_t)(row0 + tid) * sn;
            float dot = 0.f, ec = 0.f;
#pragma unroll
            for (int c = 0; c < 64; c += 8) {
                const uint4 gv = *reinterpret_cast<const uint4*>(gp + c);
                const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
                uint32_t ew[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float g0 = __uint_as_float(gw[j] << 16), g1 = __uint_as_float(gw[j] & 0xFFFF0000u);
                    const float c0 = cm[c + 2 * j], c1 = cm[c + 2 * j + 1];
                    dot = fmaf(g0, acc[c + 2 * j] - (rowsum + 1.f) * c0, dot);
                    dot = fmaf(g1, acc[c + 2 * j + 1] - (rowsum + 1.f) * c1, dot);
                    ec = fmaf(g0 * inv, c0, ec);
                    ec = fmaf(g1 * inv, c1, ec);
                    ew[j] = pack_bf16(g0 * inv, g1 * inv);
                }
                *reinterpret_cast<uint4*>(E + row * 64 + c) = make_uint4(ew[0], ew[1], ew[2], ew[3]);
            }
            const float e = -dot * inv * inv;
            e65[row] = e;
            e65h[row] = e - ec;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

// Column means of V per head: cmean[bh][c] = (1/n) sum_i V[bh][i][c].  The kernels work with
// v - cmean (and add cmean back times the row's weight sum): an exact identity that keeps the
// bf16 states free of the common component of the values, which otherwise cancels only after
// rounding in the backward.  One CTA per head, fixed summation order.
__global__ void __launch_bounds__(256)
tc_vmean_kernel(const bf16* __restrict__ V, int H, int n, int64_t sb, int64_t sh, int64_t sn,
                float* __restrict__ cmean) {
    __shared__ float part[8][64];
    const int bh = blockIdx.x, tid = threadIdx.x, lane = tid % 32, rg = tid / 32;
    const bf16* base = V + (int64_t)(bh / H) * sb + (int64_t)(bh % H) * sh + 2 * lane;
    float s0 = 0.f, s1 = 0.f;
    for (int i = rg; i < n; i += 8) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(base + (int64_t)i * sn);
        s0 += __low2float(v);
        s1 += __high2float(v);
    }
    part[rg][2 * lane] = s0;
    part[rg][2 * lane + 1] = s1;
    __syncthreads();
    if (tid < 64) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < 8; ++r) s += part[r][tid];
        cmean[(size_t)bh * 64 + tid] = s / (float)n;
    }
}

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------

// States of every block + scan.  X is sketched, Y is the right-hand side.
template <int R, int T0, int TN>
cudaError_t launch_state_group(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const bf16* G1,
                               const bf16* G2, const float* y65, const float* cmean, int center_mode, bf16* S, int* status,
                               cudaStream_t s, int* launches) {
    constexpr size_t smem = StateSmem<R>::total + 1024;
    PSK_TRY(set_smem(tc_state_kernel<R, T0, TN>, smem));
    prof_begin("tc_state_kernel", s);
    tc_state_kernel<R, T0, TN><<<dim3(d.t, d.BH()), 128, smem, s>>>(mX, mY, G1, G2, d.g_heads, d.H, d.n, d.b, d.t,
                                                                   y65, cmean, center_mode, S, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <int R>
cudaError_t launch_states(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const bf16* G1, const bf16* G2,
                          const float* y65, const float* cmean, int center_mode, bf16* S, bool reverse, int* status,
                          cudaStream_t s, int* launches) {
    if constexpr (R == 16) {
        PSK_TRY((launch_state_group<16, 0, 2>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, status, s, launches)));
    } else if constexpr (R == 32) {
        PSK_TRY((launch_state_group<32, 0, 5>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, status, s, launches)));
    } else {
        PSK_TRY((launch_state_group<64, 0, 4>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, status, s, launches)));
        PSK_TRY((launch_state_group<64, 4, 4>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, status, s, launches)));
        PSK_TRY((launch_state_group<64, 8, 3>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, status, s, launches)));
        PSK_TRY((launch_state_group<64, 11, 3>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, status, s, launches)));
        PSK_TRY((launch_state_group<64, 14, 3>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, status, s, launches)));
    }
    const size_t elems8 = (size_t)80 * Feat<R>::FP / 8;
    prof_begin("tc_scan_kernel", s);
    tc_scan_kernel<<<dim3((unsigned)((elems8 + 255) / 256), d.BH()), 256, 0, s>>>(S, elems8, d.t, reverse ? 1 : 0);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <int R>
cudaError_t fwd_impl(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                     void* O, float* denom, char* ws, cudaStream_t s, int* launches) {
    const TcWorkspace w = tc_ws<R>(d, false);
    int* status = reinterpret_cast<int*>(ws + w.status);
    bf16* Z = reinterpret_cast<bf16*>(ws + w.Z);
    CUtensorMap mQ, mK, mV, mZ;
    if (!tc_map_rows(&mQ, Q, d.B, d.H, d.n, d.sb, d.sh, d.sn) || !tc_map_rows(&mK, K, d.B, d.H, d.n, d.sb, d.sh, d.sn) ||
        !tc_map_rows(&mV, V, d.B, d.H, d.n, d.sb, d.sh, d.sn) || !tc_map_states(&mZ, Z, Feat<R>::FP, (int64_t)d.BH() * d.t))
        return cudaErrorInvalidValue;
    PSK_TRY((launch_states<R>(d, mK, mV, (const bf16*)G1, (const bf16*)G2, nullptr, nullptr, 0, Z, false, status, s,
                              launches)));
    constexpr size_t smem = OutSmem<R>::total + 1024;
    PSK_TRY(set_smem(tc_fwd_out_kernel<R, 0>, smem));
    prof_begin("tc_fwd_out_kernel", s);
    tc_fwd_out_kernel<R, 0><<<dim3(d.b / 128, d.t, d.BH()), 128, smem, s>>>(
        mQ, mK, mV, mZ, (const bf16*)G1, (const bf16*)G2, d.g_heads, d.H, d.n, d.b, d.t, nullptr, (bf16*)O, d.sb, d.sh, d.sn,
        denom, nullptr, nullptr, nullptr, nullptr, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace

bool tc_supported(const Dims& d, bool backward) {
    (void)backward;
    return d.bf16 && encoder() != nullptr;
}

size_t tc_workspace_bytes(const Dims& d, bool backward) {
    switch (d.r) {
        case 16: return tc_ws<16>(d, backward).total;
        case 32: return tc_ws<32>(d, backward).total;
        default: return tc_ws<64>(d, backward).total;
    }
}

cudaError_t tc_fwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                   void* O, float* denom, char* ws, cudaStream_t s, int* launches) {
    switch (d.r) {
        case 16: return fwd_impl<16>(d, Q, K, V, G1, G2, O, denom, ws, s, launches);
        case 32: return fwd_impl<32>(d, Q, K, V, G1, G2, O, denom, ws, s, launches);
        case 64: return fwd_impl<64>(d, Q, K, V, G1, G2, O, denom, ws, s, launches);
    }
    return cudaErrorInvalidValue;
}

template <int R>
static cudaError_t recompute_impl(const Dims& d, const CUtensorMap& mQ, const CUtensorMap& mK, const CUtensorMap& mV,
                                  const CUtensorMap& mZ, const bf16* G1, const bf16* G2, const float* cmean,
                                  const float* denom, const bf16* dO, bf16* E, float* e65, float* e65h, int* status,
                                  cudaStream_t s, int* launches) {
    constexpr size_t smem = OutSmem<R>::total + 1024;
    PSK_TRY(set_smem(tc_fwd_out_kernel<R, 1>, smem));
    prof_begin("tc_bwd_recompute_kernel", s);
    tc_fwd_out_kernel<R, 1><<<dim3(d.b / 128, d.t, d.BH()), 128, smem, s>>>(
        mQ, mK, mV, mZ, G1, G2, d.g_heads, d.H, d.n, d.b, d.t, cmean, nullptr, d.sb, d.sh, d.sn,
        const_cast<float*>(denom), dO, E, e65, e65h, status);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tc_recompute(const Dims& d, const CUtensorMap& mQ, const CUtensorMap& mK, const CUtensorMap& mV,
                         const CUtensorMap& mZ, const bf16* G1, const bf16* G2, const float* cmean, const float* denom,
                         const bf16* dO, bf16* E, float* e65, float* e65h, int* status, cudaStream_t s, int* launches) {
    switch (d.r) {
        case 16: return recompute_impl<16>(d, mQ, mK, mV, mZ, G1, G2, cmean, denom, dO, E, e65, e65h, status, s, launches);
        case 32: return recompute_impl<32>(d, mQ, mK, mV, mZ, G1, G2, cmean, denom, dO, E, e65, e65h, status, s, launches);
        case 64: return recompute_impl<64>(d, mQ, mK, mV, mZ, G1, G2, cmean, denom, dO, E, e65, e65h, status, s, launches);
    }
    return cudaErrorInvalidValue;
}

cudaError_t tc_vmean(const Dims& d, const void* V, float* cmean, cudaStream_t s, int* launches) {
    prof_begin("tc_vmean_kernel", s);
    tc_vmean_kernel<<<d.BH(), 256, 0, s>>>((const bf16*)V, d.H, d.n, d.sb, d.sh, d.sn, cmean);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tc_states(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const bf16* G1, const bf16* G2,
                      const float* y65, const float* cmean, int center_mode, bf16* S, bool reverse, int* status,
                          cudaStream_t s, int* launches) {
    switch (d.r) {
        case 16: return launch_states<16>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, reverse, status, s, launches);
        case 32: return launch_states<32>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, reverse, status, s, launches);
        case 64: return launch_states<64>(d, mX, mY, G1, G2, y65, cmean, center_mode, S, reverse, status, s, launches);
    }
    return cudaErrorInvalidValue;
}

}  // namespace psk
