// Tensor-core path (bf16 operands, fp32 accumulation in tensor memory) of causal Polysketch
// attention.  Same steps as Section 3.1 -- per-block states, prefix scan, output rows -- with
// the r(r+1)/2 distinct features of the self-tensored sketch (tc_features.cuh) generated in
// registers and handed to tcgen05.mma without ever touching HBM.
//
// State storage (HBM scratch): S[BH][t][FP][80] bf16, one 160-byte row per feature: the 64
// columns of H_l / Z_l, then the normaliser column (the "| 1" of [V | 1], or the last column of E
// in the backward), then zeros.  A stage of a consumer is two TMA boxes of [64 features x 128 B]:
// columns 0..63 and columns 64..79 (+ zero fill).  Together they are an MN-major B operand with
// N = 80 (contract over features) or a K-major B operand with K = 64 + 16 (contract over the
// state's columns).
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
// Row-major [rows][cols] bf16 matrix (cols a multiple of 64); box = box_rows rows x 64 columns,
// 128-byte swizzle.
bool tc_map_2d(CUtensorMap* m, const void* base, int cols, int64_t rows, int box_rows) {
    EncodeFn enc = encoder();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows}, es[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// [outer][rows][cols] bf16, contiguous; box = box_rows rows x box_cols columns of one outer index.
bool tc_map_3d(CUtensorMap* m, const void* base, int cols, int64_t rows, int64_t outer, int box_cols, int box_rows) {
    EncodeFn enc = encoder();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)outer};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)rows * cols * 2};
    cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1}, es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// States S[nblk][FP][80] bf16 (feature-major rows: 64 state columns, the last column, 15 zeros).
// Box = 64 features x 64 columns; a second box at column 64 brings the last column (columns
// beyond 80 lie outside the tensor and arrive as zeros).
bool tc_map_states(CUtensorMap* m, const void* base, int FP, int64_t nblk) {
    EncodeFn enc = encoder();
    if (!enc) return false;
    cuuint64_t dims[3] = {80, (cuuint64_t)FP, (cuuint64_t)nblk};
    cuuint64_t strides[2] = {160, (cuuint64_t)FP * 160};
    cuuint32_t box[3] = {64, 64, 1}, es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


namespace {

// ---------------------------------------------------------------------------
// Forward output rows (Section 3.1): for a 128-row tile of block l,
//   N = phi_w(Q) Z_l  (tensor memory A operand x TMA-fed Z chunks, N = 80: column 64 = normaliser)
//     + sum over key tiles of the same block  lt((M_q M_k^T)^2) [V | 1]
//   d = 1 + normaliser;  O = N[:, :64] / d
// grid (b/128, t, BH), 160 threads.  Warps 0-3: thread = query row (half sketches, features,
// weights, epilogue).  Warp 4: one thread issues every TMA load and every MMA; the two sides meet
// only at mbarriers, so the rows never wait for an issue sequence and the tensor pipe runs ahead.
// ---------------------------------------------------------------------------
#ifdef PSK_FWD_TRACE
// scratch builds only: clock stamps of one CTA, one slot per (event, index)
__device__ long long g_ftr[64 * 16];
#define FTR(ev, idx) do { if (blockIdx.x == 1 && blockIdx.y == 5 && blockIdx.z == 3) g_ftr[(ev) * 16 + (idx)] = clock64(); } while (0)
#else
#define FTR(ev, idx)
#endif

// Warps 0-3: rows.  Warp 4: one thread issues every TMA load and every MMA.  (A second issuing
// thread in a sixth warp for the odd state chunks was measured: 1 % faster, and the two threads'
// MMAs reach the accumulator in an order that changes from run to run, so results were no longer
// bitwise reproducible.  Not kept.)
constexpr int kOutThreads = 160;
#define PSK_OUT_ISSUERS 1
constexpr int kZStages = 4;                     // three in the shared region + the query tile's buffer
constexpr uint32_t kZStageBytes = 16384;        // two [64 features x 128 B] boxes: columns 0..63, 64..79
constexpr int kFeatBufs = kZStages;             // feature staging buffers in tensor memory, 32 columns each:
                                                // chunk C uses buffer and stage C % 4, both freed by its MMAs

template <int R, bool LOCAL = false>
struct OutSmem {
    // The prefix-state stages (first phase), the key/value tiles with the keys' split half
    // sketches (second phase) and the output staging tiles (epilogue) share one region; small
    // enough for two CTAs per SM when R <= 32.
    static constexpr uint32_t Q = 0, G = 16384;
    static constexpr uint32_t Ones = G + GImage<R>::bytes;           // 4 KB of bf16 1.0: B operand of the row sums
    static constexpr uint32_t Mq = Ones + 4096;
    // split operand: 3R columns.  (LOCAL: no split operands; the region holds the ring's last
    // stage and then the value tile, because the query tile stays alive for the exact scores.)
    static constexpr uint32_t kMqBytes = LOCAL ? 16384 : 128 * 3 * R * 2;
    static constexpr uint32_t U = (Mq + kMqBytes + 1023) / 1024 * 1024;
    static constexpr uint32_t Z = U;
    // key tile in ring stage 1, value tile in the query tile's buffer (ring stage 3), split key
    // sketches over stage 2: the stages the last chunks free first, so the first key/value tile is
    // fetched while the last chunks are still being multiplied
    static constexpr uint32_t Z3 = LOCAL ? Mq : Q;                   // ring stage 3
    static constexpr uint32_t K = U + 16384, V = Z3, Mk = U + 32768;
    static constexpr int kStageK = 1, kStageV = kZStages - 1;
    // last chunk that uses ring stage s (-1: none)
    __host__ __device__ static constexpr int last_chunk(int nc, int s) { return nc > s ? s + (nc - 1 - s) / kZStages * kZStages : -1; }
    static constexpr uint32_t So = U, Soc = U + 16384;               // O tile, O - c tile (bf16 each)
    static constexpr uint32_t kPhase1 = (kZStages - 1) * kZStageBytes, kPhase2 = 32768 + (LOCAL ? 0 : 128 * 3 * R * 2), kEpi = 32768;
    static constexpr uint32_t kMax12 = kPhase1 > kPhase2 ? kPhase1 : kPhase2;
    static constexpr uint32_t total = U + (kMax12 > kEpi ? kMax12 : kEpi);
    // stage s of the prefix-state ring; the last one is the query tile's buffer, dead after the sketch
    __device__ static uint32_t zstage(int s) { return s < kZStages - 1 ? Z + s * kZStageBytes : Z3; }
};


// MODE 0: forward (writes O, denom, optionally O - c in fp32).  MODE 1: the backward's
// recomputation of the row numerators against centred prefix states; writes y65 = -(dO.(O - c))
// and e65h = -(dO.O)/d (fp32), with O - c = (N' - c)/d taken from the fp32 accumulators rather
// than from the rounded O the caller holds.
// LOCAL (Section 3.2): the same-block scores are (q_i . k_j)^2 from the raw query and key tiles
// (bf16 operands, exact products, fp32 sums) in place of m(q_i) . m(k_j); squared like those,
// they give the exact weights (q_i . k_j)^4.  No key sketches, no split operands.
// LIN: the rows hold a given half sketch (tc_common.cuh, read_half_sketch).
// LIN and LOCAL: mapQ is the given half sketch, mapQraw the raw query rows (fetched into the query
// tile's buffer once the sketch GEMM has read it), mapK the raw key rows.
template <int R, int MODE, bool LOCAL, bool LIN>
__global__ void __launch_bounds__(kOutThreads, ((R <= 32 || LOCAL) ? 2 : 1))
tc_fwd_out_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapQraw,
                  const __grid_constant__ CUtensorMap mapK,
                  const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapZ,
                  const __grid_constant__ CUtensorMap mapO, const __grid_constant__ CUtensorMap mapOc,
                  const uint8_t* __restrict__ gimg, int g_heads, int H, int n, int b, int t,
                  const float* __restrict__ cmean, int64_t sb, int64_t sh, int64_t sn,
                  float* __restrict__ denom, const bf16* __restrict__ dO,
                  float* __restrict__ y65, float* __restrict__ e65h, int keep_oc, int noncausal, int* status) {
    constexpr bool lin = LIN;
    using F = Feat<R>;
    using L = OutSmem<R, LOCAL>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_q, bar_kv, bar_sk, bar_go, bar_mk, bar_s, bar_p, bar_pv;
    __shared__ uint64_t bar_z[kZStages], bar_feat[kFeatBufs], bar_a[kFeatBufs];
    __shared__ uint32_t tmem_slot;
    __shared__ float cm[64];
    const int tid = threadIdx.x, warp = tid / 32, tau = blockIdx.x, l = blockIdx.y, bh = blockIdx.z;
    const int hi = bh % H, bi = bh / H;
    const int g = g_heads == 1 ? 0 : hi;
    FTR(0, 0);
    const int row0 = l * b + tau * 128;
    // Non-causal (Section 3, first formula): one state per head, the sum over the whole sequence,
    // multiplies every row tile, and there are no same-block tiles.
    const int blk = noncausal ? bh : bh * t + l;
    const bool has_prefix = noncausal || l > 0;

    if (tid == 0) {
        // the query tile is what everything waits for: its request goes out before anything else
        mbar_init(&bar_q, 1);
        mbar_fence_init();
        mbar_expect_tx(&bar_q, 16384 + GImage<R>::bytes);
        tma_load_4d(smem + L::Q, &mapQ, 0, row0, hi, bi, &bar_q);
        bulk_load(smem + L::G, gimg + (size_t)g * GImage<R>::bytes, GImage<R>::bytes, &bar_q);
        mbar_init(&bar_kv, 1); mbar_init(&bar_sk, 1); mbar_init(&bar_s, 1); mbar_init(&bar_pv, 1);
        mbar_init(&bar_mk, 128); mbar_init(&bar_p, 128); mbar_init(&bar_go, 128);
        for (int s = 0; s < kZStages; ++s) mbar_init(&bar_z[s], 1);
        for (int s = 0; s < kFeatBufs; ++s) { mbar_init(&bar_feat[s], 128); mbar_init(&bar_a[s], 1); }
        cta_giveup_init();
        mbar_fence_init();
        tma_prefetch_desc(&mapK); tma_prefetch_desc(&mapV); tma_prefetch_desc(&mapZ);
    }
    // The same-block key/value tiles are loaded late (their buffers hold state chunks first, and a
    // tile's buffers are free only when the previous tile's MMAs are done): ask for them in L2 now,
    // so that those loads pay the L2 latency and not HBM's.  (Forward rows 4.48 -> 4.40 ms at
    // configuration 2; the same in the backward's row kernels made them 2 % slower and is not there.)
    if (tid == 32 && !noncausal) {
        for (int tp = 0; tp <= tau; ++tp) {
            tma_prefetch_4d(&mapK, 0, l * b + tp * 128, hi, bi);
            tma_prefetch_4d(&mapV, 0, l * b + tp * 128, hi, bi);
        }
    }
    if (warp == 4) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    for (int e = tid; e < 256; e += kOutThreads)
        reinterpret_cast<uint4*>(smem + L::Ones)[e] = make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
    if (tid < 64) cm[tid] = cmean != nullptr ? cmean[(size_t)bh * 64 + tid] : 0.f;
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_slot;
    if (tid == 0) FTR(1, 0);
    // tensor-memory columns: sketch accumulators, feature staging buffers, scores and packed
    // weights all live in [0, 128), each consumed before the next is produced; then the output
    // accumulator (64 + the prefix normaliser's 16) and the same-block row sums (16)
    constexpr uint32_t cSk = 0, cS = 0, cW = 0, cA = 0, cO = 128, cN = cO + 80;
    bool ok = true;

    // First phase, issuing side: the chunks `first`, `first + step`, ... of the prefix state.
    // B = the chunk's 64 feature rows x 80 columns, MN-major: 16 features per K step, the second
    // 64-column group (columns 64..79) 8192 B further on.  Everything the loop needs is in registers
    // before it waits: between "features staged" and "MMAs issued" lie the four MMA instructions
    // and nothing else.  (The stages are refilled by the rows' side, which learns first that a
    // buffer is free.)
    auto issue_chunks = [&](int first, int step) {
        constexpr uint32_t idesc = idesc_bf16(128, 80, false, true);
        const uint64_t zd0 = smem_desc(smem_u32(smem + L::Z), 8192, 1024, kSwz128);
        const uint64_t zdq = smem_desc(smem_u32(smem + L::Z3), 8192, 1024, kSwz128);
#pragma unroll 1
        for (int C = first; C < F::NC && ok; C += step) {
            const int s = C % kZStages;
            const uint32_t par = (C / kZStages) & 1;
            const int ksteps = (F::FK - C * 64) >= 64 ? 4 : (F::FK - C * 64) / 16;
            const uint64_t zd = s == kZStages - 1 ? zdq : desc_off(zd0, s * kZStageBytes);
            const uint32_t at = tm + cA + s * 32;
            ok = mbar_spin(&bar_z[s], par, status, kErrTma);
            FTR(4, C);
            ok = ok && mbar_spin(&bar_feat[s], par, status, kErrMma);
            FTR(5, C);
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < ksteps) umma_ts(tm + cO, at + k * 8, desc_off(zd, k * 2048), idesc, (C > 0 || k > 0) ? 1u : 0u);
            umma_commit(&bar_a[s]);
            FTR(6, C);
        }
    };

    if (warp == 4) {
        // ================================ issuer ================================
        if (tid == 128) {
            // (the first state chunks are requested here, not by the thread that sets the barriers
            // up: everyone waits for that thread, only this one waits for the query tile anyway)
            if (has_prefix) {
                for (int c = 0; c < kZStages - 1 && c < F::NC; ++c) {
                    mbar_expect_tx(&bar_z[c], kZStageBytes);
                    tma_load_3d(smem + L::zstage(c), &mapZ, 0, c * 64, blk, &bar_z[c]);
                    tma_load_3d(smem + L::zstage(c) + 8192, &mapZ, 64, c * 64, blk, &bar_z[c]);
                }
            }
            ok = mbar_spin(&bar_q, 0, status, kErrTma);
            FTR(2, 0);
            tc_fence_after();
            issue_sketch<R>(tm + cSk, smem + L::Q, smem + L::G);
            umma_commit(&bar_sk);
            FTR(3, 0);
            if constexpr (LIN && LOCAL) {
                ok = ok && mbar_spin(&bar_sk, 0, status, kErrMma);
                mbar_expect_tx(&bar_q, 16384);
                tma_load_4d(smem + L::Q, &mapQraw, 0, row0, hi, bi, &bar_q);
            }
            if (has_prefix && kZStages - 1 < F::NC) {
                // the query tile has been consumed: its buffer becomes the ring's last stage
                ok = ok && mbar_spin(&bar_sk, 0, status, kErrMma);
                mbar_expect_tx(&bar_z[kZStages - 1], kZStageBytes);
                tma_load_3d(smem + L::zstage(kZStages - 1), &mapZ, 0, (kZStages - 1) * 64, blk, &bar_z[kZStages - 1]);
                tma_load_3d(smem + L::zstage(kZStages - 1) + 8192, &mapZ, 64, (kZStages - 1) * 64, blk, &bar_z[kZStages - 1]);
            }
            if (has_prefix) issue_chunks(0, PSK_OUT_ISSUERS);     // earlier blocks: features x prefix state chunks
            if (has_prefix && !noncausal) {
                // first key/value tile of the same block, each into its stage as soon as the last
                // chunk that used it has been multiplied
                constexpr int cK = L::last_chunk(F::NC, L::kStageK), cV = L::last_chunk(F::NC, L::kStageV);
                mbar_expect_tx(&bar_kv, 32768);
                if (cK >= 0) ok = ok && mbar_spin(&bar_a[L::kStageK], (cK / kZStages) & 1, status, kErrMma);
                tma_load_4d(smem + L::K, &mapK, 0, l * b, hi, bi, &bar_kv);
                if (cV >= 0) ok = ok && mbar_spin(&bar_a[L::kStageV], (cV / kZStages) & 1, status, kErrMma);
                else ok = ok && mbar_spin(&bar_sk, 0, status, kErrMma);     // no chunk used it: the query sketch did
                tma_load_4d(smem + L::V, &mapV, 0, l * b, hi, bi, &bar_kv);
                // the sketch reuses the staging columns and the split key sketches the remaining
                // stage: every MMA of the first phase must have completed
                ok = ok && mbar_spin(&bar_a[(F::NC - 1) % kFeatBufs], ((F::NC - 1) / kFeatBufs) & 1, status, kErrMma);
            }
            // same block: key tiles tp <= tau through squared half-sketch scores; descriptors and
            // addresses are loop invariants, so every issue sequence below is MMA instructions only
            const uint64_t qd = smem_desc(smem_u32(smem + L::Mq), 2048, 128, kSwzNone);
            const uint64_t kd = smem_desc(smem_u32(smem + L::Mk), 2048, 128, kSwzNone);
            const uint64_t vd = smem_desc(smem_u32(smem + L::V), 0, 1024, kSwz128);
            const uint64_t od = smem_desc(smem_u32(smem + L::Ones), 256, 128, kSwzNone);
            // every row has read the query sketch (the first key sketch overwrites its columns, and
            // bar_sk must not complete a second time before its slowest waiter has seen the first)
            ok = ok && mbar_spin(&bar_go, 0, status, kErrMma);
            const int tp_last = noncausal ? -1 : tau;
#pragma unroll 1
            for (int tp = 0; tp <= tp_last && ok; ++tp) {
                if (tp > 0) ok = mbar_spin(&bar_pv, (tp - 1) & 1, status, kErrMma);   // K, V, Mk, weights are free
                if (tp > 0 || l == 0) {       // (block l > 0: the first tile was requested above)
                    mbar_expect_tx(&bar_kv, 32768);
                    tma_load_4d(smem + L::K, &mapK, 0, l * b + tp * 128, hi, bi, &bar_kv);
                    tma_load_4d(smem + L::V, &mapV, 0, l * b + tp * 128, hi, bi, &bar_kv);
                }
                ok = ok && mbar_spin(&bar_kv, tp & 1, status, kErrTma);
                FTR(7, tp);
                tc_fence_after();
                if constexpr (LOCAL) {
                    // scores = Q_tile K_tile^T over the head dimension
                    if constexpr (LIN) ok = ok && mbar_spin(&bar_q, 1, status, kErrTma);     // the raw query rows
                    constexpr uint32_t idesc = idesc_bf16(128, 128, false, false);
                    const uint64_t qr = smem_desc(smem_u32(smem + L::Q), 0, 1024, kSwz128);
                    const uint64_t kr = smem_desc(smem_u32(smem + L::K), 0, 1024, kSwz128);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_ss(tm + cS, desc_off(qr, k * 32), desc_off(kr, k * 32), idesc, k > 0);
                    umma_commit(&bar_s);
                } else {
                    issue_sketch<R>(tm + cSk, smem + L::K, smem + L::G);
                    umma_commit(&bar_sk);
                    FTR(8, tp);
                    ok = ok && mbar_spin(&bar_mk, tp & 1, status, kErrMma);
                    FTR(9, tp);
                    tc_fence_after();
                    constexpr uint32_t idesc = idesc_bf16(128, 128, false, false);
#pragma unroll
                    for (int k = 0; k < 3 * R / 16; ++k)
                        umma_ss(tm + cS, desc_off(qd, k * 4096), desc_off(kd, k * 4096), idesc, k > 0);
                    umma_commit(&bar_s);
                }
                FTR(10, tp);
                ok = ok && mbar_spin(&bar_p, tp & 1, status, kErrMma);
                FTR(11, tp);
                tc_fence_after();
                {
                    // numerator += W V; row sums += W 1 (the weights exactly as the value GEMM sees them)
                    constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
                    constexpr uint32_t idesc1 = idesc_bf16(128, 16, false, false);
                    const uint32_t acc0 = (l > 0 || tp > 0) ? 1u : 0u, acc1 = tp > 0 ? 1u : 0u;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        umma_ts(tm + cO, tm + cW + k * 8, desc_off(vd, k * 2048), idesc, k > 0 ? 1u : acc0);
                        umma_ts(tm + cN, tm + cW + k * 8, desc_off(od, k * 512), idesc1, k > 0 ? 1u : acc1);
                    }
                    umma_commit(&bar_pv);
                    FTR(12, tp);
                }
            }
        }
    } else {
        // ================================= rows =================================
        const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
        ok = mbar_wait(&bar_sk, 0, status, kErrMma);
        if (tid == 0) FTR(20, 0);
        tc_fence_after();
        float mq[R];
        read_half_sketch<R>(lane_tm + cSk, mq, 1.f, lin != 0);
        if constexpr (!LOCAL) store_split_rows<R, true>(smem + L::Mq, mq, tid);
        tc_fence_before();
        mbar_arrive(&bar_go);
        if (tid == 0) FTR(21, 0);

        if (has_prefix) {
            if constexpr (F::kCirc) {
                CircGen<R> gen;
                gen.init(mq);
#pragma unroll 1
                for (int C = 0; C < F::NC && ok; ++C) {
                    const int buf = C % kFeatBufs;
                    if (C >= kFeatBufs) {             // the MMAs that read this buffer's previous contents
                        ok = mbar_wait(&bar_a[buf], (C / kFeatBufs - 1) & 1, status, kErrMma);
                        tc_fence_after();
                        if (tid == 0) {               // ... and this stage's: refill it with chunk C's rows
                            mbar_expect_tx(&bar_z[buf], kZStageBytes);
                            tma_load_3d(smem + L::zstage(buf), &mapZ, 0, C * 64, blk, &bar_z[buf]);
                            tma_load_3d(smem + L::zstage(buf) + 8192, &mapZ, 64, C * 64, blk, &bar_z[buf]);
                        }
                    }
                    if (tid == 0) FTR(22, C);
                    uint32_t pk[32];
                    gen.chunk(pk);
                    tmem_st32(lane_tm + cA + buf * 32, pk);
                    tmem_st_wait();
                    tc_fence_before();
                    mbar_arrive(&bar_feat[buf]);
                    if (tid == 0) FTR(23, C);
                }
            } else {
                PackedM<R> pmq;
                pack_half_sketch<R>(mq, pmq);
                static_for<0, F::NC>([&](auto cc) {
                    constexpr int C = decltype(cc)::value;
                    constexpr int buf = C % kFeatBufs;
                    if constexpr (C >= kFeatBufs) {
                        ok = ok && mbar_wait(&bar_a[buf], (C / kFeatBufs - 1) & 1, status, kErrMma);
                        tc_fence_after();
                        if (tid == 0) {
                            mbar_expect_tx(&bar_z[buf], kZStageBytes);
                            tma_load_3d(smem + L::zstage(buf), &mapZ, 0, C * 64, blk, &bar_z[buf]);
                            tma_load_3d(smem + L::zstage(buf) + 8192, &mapZ, 64, C * 64, blk, &bar_z[buf]);
                        }
                    }
                    uint32_t pk[16];
                    gen_features<R, C * 64, 16>(pmq, pk);
                    tmem_st16(lane_tm + cA + buf * 32, pk);
                    gen_features<R, C * 64 + 32, 16>(pmq, pk);
                    tmem_st16(lane_tm + cA + buf * 32 + 16, pk);
                    tmem_st_wait();
                    tc_fence_before();
                    mbar_arrive(&bar_feat[buf]);
                });
            }
        }

        const int tp_last = noncausal ? -1 : tau;
#pragma unroll 1
        for (int tp = 0; tp <= tp_last && ok; ++tp) {
            if constexpr (!LOCAL) {
                ok = mbar_wait(&bar_sk, (tp + 1) & 1, status, kErrMma);
                if (tid == 0) FTR(24, tp);
                tc_fence_after();
                {
                    float mk[R];
                    read_half_sketch<R>(lane_tm + cSk, mk, 1.f, lin != 0);
                    store_split_rows<R, false>(smem + L::Mk, mk, tid);
                }
                fence_proxy_async_smem();
                tc_fence_before();
                mbar_arrive(&bar_mk);
                if (tid == 0) FTR(25, tp);
            }
            ok = ok && mbar_wait(&bar_s, tp & 1, status, kErrMma);
            if (tid == 0) FTR(26, tp);
            tc_fence_after();
            // weights = squared scores (lower triangle on the diagonal tile), packed to bf16 over
            // columns whose fp32 contents have already been read
            // (one loop over the four 32-key groups.  On the diagonal tile a warp's rows
            // 32 w .. 32 w + 31 see group g < w whole, group g > w not at all, and only group
            // g == w through the triangular mask: the mask code runs for one group in four.)
            const int gdiag = (tp == tau) ? warp : 4;
#pragma unroll 1
            for (int gq = 0; gq < 4; ++gq) {
                uint32_t v[32], pk[16];
                tmem_ld32(lane_tm + cS + gq * 32, v);
                tmem_ld_wait();
                if (gq >= gdiag) {
                    const int lim = gq > gdiag ? -1 : (tid & 31);       // keep keys j <= lim of this group
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = j > lim ? 0u : v[j];
                }
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    float w0 = __uint_as_float(v[j]), w1 = __uint_as_float(v[j + 1]);
                    if constexpr (LOCAL) { w0 *= w0; w1 *= w1; }          // (q . k)^2, squared once more below
                    pk[j / 2] = pack_bf16(w0 * w0, w1 * w1);
                }
                tmem_st16(lane_tm + cW + gq * 16, pk);
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&bar_p);
            if (tid == 0) FTR(27, tp);
        }
        if (noncausal)      // the last chunk's MMAs (no same-block tiles follow them)
            ok = ok && mbar_wait(&bar_a[(F::NC - 1) % kFeatBufs], ((F::NC - 1) / kFeatBufs) & 1, status, kErrMma);
        else
            ok = ok && mbar_wait(&bar_pv, tau & 1, status, kErrMma);
        tc_fence_after();
        if (tid == 0) FTR(28, 0);

        // ---- epilogue ----
        float acc[64];
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(lane_tm + cO + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) acc[c0 + j] = __uint_as_float(v[j]);
        }
        float noff = 0.f, rowsum = 0.f;       // normaliser parts: earlier blocks, same block
        {
            uint32_t v[16];
            if (has_prefix) {
                tmem_ld16(lane_tm + cO + 64, v);
                tmem_ld_wait();
                noff = __uint_as_float(v[0]);
            }
            if (!noncausal) {
                tmem_ld16(lane_tm + cN, v);
                tmem_ld_wait();
                rowsum = __uint_as_float(v[0]);
            }
        }
        if constexpr (MODE == 0) {
            const float d = 1.f + rowsum + noff;
            // with centred prefix states (cmean given) the earlier blocks' numerator lacks c * noff
#pragma unroll
            for (int c = 0; c < 64; ++c) acc[c] = fmaf(cm[c], noff, acc[c]);
            const float inv = 1.f / d;
            // rows go out through shared memory and tiled stores: a thread-per-row store pattern
            // would keep the load/store unit busy for thousands of cycles
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint4 v;
                v.x = pack_bf16(acc[8 * c] * inv, acc[8 * c + 1] * inv);
                v.y = pack_bf16(acc[8 * c + 2] * inv, acc[8 * c + 3] * inv);
                v.z = pack_bf16(acc[8 * c + 4] * inv, acc[8 * c + 5] * inv);
                v.w = pack_bf16(acc[8 * c + 6] * inv, acc[8 * c + 7] * inv);
                *reinterpret_cast<uint4*>(smem + L::So + swz128_offset(tid, c)) = v;
            }
            if (keep_oc) {
                // kept for the backward: O - c, rounded to bf16 AFTER the subtraction.  (The rounded
                // O cannot supply it: where the values share a common component |O - c| is far
                // below |O|, and bf16(O) - c would carry O's rounding error, not (O - c)'s.)
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint4 v;
                    v.x = pack_bf16(acc[8 * c] * inv - cm[8 * c], acc[8 * c + 1] * inv - cm[8 * c + 1]);
                    v.y = pack_bf16(acc[8 * c + 2] * inv - cm[8 * c + 2], acc[8 * c + 3] * inv - cm[8 * c + 3]);
                    v.z = pack_bf16(acc[8 * c + 4] * inv - cm[8 * c + 4], acc[8 * c + 5] * inv - cm[8 * c + 5]);
                    v.w = pack_bf16(acc[8 * c + 6] * inv - cm[8 * c + 6], acc[8 * c + 7] * inv - cm[8 * c + 7]);
                    *reinterpret_cast<uint4*>(smem + L::Soc + swz128_offset(tid, c)) = v;
                }
            }
            if (denom != nullptr && ok) denom[(size_t)bh * n + row0 + tid] = d;
            fence_proxy_async_smem();
            consumer_barrier();
            if (tid == 0 && ok) {
                tma_store_4d(&mapO, smem + L::So, 0, row0, hi, bi);
                if (keep_oc) tma_store_4d(&mapOc, smem + L::Soc, 0, bh * n + row0, 0, 0);
                bulk_commit();
                bulk_wait_read();
            }
        } else if (ok) {
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
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float g0 = __uint_as_float(gw[j] << 16), g1 = __uint_as_float(gw[j] & 0xFFFF0000u);
                    const float c0 = cm[c + 2 * j], c1 = cm[c + 2 * j + 1];
                    dot = fmaf(g0, acc[c + 2 * j] - (rowsum + 1.f) * c0, dot);
                    dot = fmaf(g1, acc[c + 2 * j + 1] - (rowsum + 1.f) * c1, dot);
                    ec = fmaf(g0 * inv, c0, ec);
                    ec = fmaf(g1 * inv, c1, ec);
                }
            }
            const float y = -dot * inv;               // -(dO . (O - c))
            y65[row] = y;
            e65h[row] = y * inv - ec;
        }
    }
    if (tid == 0) FTR(29, 0);
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tm, 256);
    if (tid == 0) FTR(30, 0);
}

// Centre of the values of a head: cmean[bh][c] = mean of V[bh][i][c] over at most 1024 rows i
// spread evenly over the sequence (all rows when n <= 1024).  The kernels work with v - cmean
// (and add cmean back times the row's weight sum): an exact identity for ANY constant, which keeps
// the bf16 states free of the common component of the values -- that component otherwise cancels
// only after rounding in the backward.  An estimate of the mean serves that purpose as well as
// the mean itself and costs 128 KB of reads per head instead of the whole tensor.  One CTA per
// head, fixed summation order.
__global__ void __launch_bounds__(1024)
tc_vmean_kernel(const bf16* __restrict__ V, int H, int n, int64_t sb, int64_t sh, int64_t sn,
                float* __restrict__ cmean) {
    __shared__ float part[128][65];
    const int bh = blockIdx.x, tid = threadIdx.x, ch = tid % 8, rg = tid / 8;   // 8 threads x 16 B per row
    const bf16* base = V + (int64_t)(bh / H) * sb + (int64_t)(bh % H) * sh + 8 * ch;
    float s[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j] = 0.f;
    const int stride = n > 1024 ? n / 1024 : 1, count = n > 1024 ? 1024 : n;
    for (int q = rg; q < count; q += 128) {
        const int i = q * stride;
        const uint4 v = *reinterpret_cast<const uint4*>(base + (int64_t)i * sn);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            s[2 * j] += __uint_as_float(w[j] << 16);
            s[2 * j + 1] += __uint_as_float(w[j] & 0xFFFF0000u);
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) part[rg][8 * ch + j] = s[j];
    __syncthreads();
    if (tid < 64) {
        float acc = 0.f;
        for (int r = 0; r < 128; ++r) acc += part[r][tid];
        cmean[(size_t)bh * 64 + tid] = acc / (float)count;
    }
}

// Image of [G1 | G2]^T (set g of the sketch matrices, each [64 x r] row-major) in the layout the
// sketch GEMM reads from shared memory: row nn < 2r = sketch column, 64 head dimensions, swizzled.
// (lin: "G1" = I for r = 64, [I; I] padded with zero rows for r <= 32, "G2" = 0: the sketch GEMM then
// returns the row itself, or the sum of its [hi | lo] halves, see read_half_sketch)
__global__ void __launch_bounds__(128)
tc_gimage_kernel(const bf16* __restrict__ G1, const bf16* __restrict__ G2, int r, int lin, uint8_t* __restrict__ gimg) {
    const int g = blockIdx.x;
    uint8_t* img = gimg + (size_t)g * 2 * r * 128;
    for (int e = threadIdx.x; e < 2 * r * 64; e += 128) {
        const int nn = e / 64, k = e % 64;
        const bf16 v = lin ? __float2bfloat16_rn((nn < r && (k == nn || (r <= 32 && k == r + nn))) ? 1.f : 0.f)
                           : (nn < r ? G1 : G2)[(size_t)g * 64 * r + k * r + (nn % r)];
        *reinterpret_cast<bf16*>(img + swz128_offset(nn, k / 8) + (k % 8) * 2) = v;
    }
}

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------

template <int R>
cudaError_t fwd_impl(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                     void* O, float* denom, char* ws, cudaStream_t s, int* launches) {
    const TcWorkspace w = tc_ws<R>(d, d.keep_states);
    int* status = reinterpret_cast<int*>(ws + w.status);
    bf16* Z = reinterpret_cast<bf16*>(ws + w.Z);
    bf16* Oc = d.keep_states ? reinterpret_cast<bf16*>(ws + w.Oc) : nullptr;
    CUtensorMap mQ, mK, mV, mZ, mO, mOc;
    if (!tc_map_rows(&mQ, Q, d.B, d.H, d.n, d.xsb, d.xsh, d.xsn) || !tc_map_rows(&mK, K, d.B, d.H, d.n, d.xsb, d.xsh, d.xsn) ||
        !tc_map_rows(&mV, V, d.B, d.H, d.n, d.sb, d.sh, d.sn) ||
        !tc_map_states(&mZ, Z, Feat<R>::FP, (int64_t)d.BH() * (d.noncausal ? 1 : d.t)) ||
        !tc_map_rows(&mO, O, d.B, d.H, d.n, d.sb, d.sh, d.sn))
        return cudaErrorInvalidValue;
    if (Oc != nullptr) {
        const int64_t rows = (int64_t)d.BH() * d.n;      // one [rows, 64] bf16 array
        if (!tc_map_rows(&mOc, Oc, 1, 1, (int)rows, rows * 64, rows * 64, 64)) return cudaErrorInvalidValue;
    } else {
        mOc = mO;       // never used
    }
    // keep_states: the backward will read these states, so they are built from centred values
    float* cmean = d.keep_states ? reinterpret_cast<float*>(ws + w.vmean) : nullptr;
    if (cmean != nullptr) PSK_TRY(tc_vmean(d, V, cmean, s, launches));
    uint8_t* gimg = reinterpret_cast<uint8_t*>(ws + w.gimg);
    PSK_TRY(tc_gimage(d, G1, G2, gimg, s, launches));
    PSK_TRY(tc_states(d, mK, mV, gimg, nullptr, nullptr, cmean, cmean ? 1 : 0, Z, false,
                      reinterpret_cast<float*>(ws + w.tot), status, s, launches));
    prof_begin("tc_fwd_out_kernel", s);
    if (d.local && d.sketch_linear) {
        if constexpr (R <= 32) {
            CUtensorMap mQraw, mKraw;
            if (d.rawQ == nullptr || d.rawK == nullptr || !tc_map_rows(&mQraw, d.rawQ, d.B, d.H, d.n, d.sb, d.sh, d.sn) ||
                !tc_map_rows(&mKraw, d.rawK, d.B, d.H, d.n, d.sb, d.sh, d.sn))
                return cudaErrorInvalidValue;
            constexpr size_t smem = OutSmem<R, true>::total + 1024;
            PSK_TRY((set_smem(tc_fwd_out_kernel<R, 0, true, true>, smem)));
            tc_fwd_out_kernel<R, 0, true, true><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
                mQ, mQraw, mKraw, mV, mZ, mO, mOc, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
                denom, nullptr, nullptr, nullptr, Oc != nullptr ? 1 : 0, 0, status);
        } else {
            return cudaErrorInvalidValue;
        }
    } else if (d.local) {
        constexpr size_t smem = OutSmem<R, true>::total + 1024;
        PSK_TRY((set_smem(tc_fwd_out_kernel<R, 0, true, false>, smem)));
        tc_fwd_out_kernel<R, 0, true, false><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
            mQ, mQ, mK, mV, mZ, mO, mOc, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
            denom, nullptr, nullptr, nullptr, Oc != nullptr ? 1 : 0, d.noncausal ? 1 : 0, status);
    } else if (d.sketch_linear) {
        constexpr size_t smem = OutSmem<R, false>::total + 1024;
        PSK_TRY((set_smem(tc_fwd_out_kernel<R, 0, false, true>, smem)));
        tc_fwd_out_kernel<R, 0, false, true><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
            mQ, mQ, mK, mV, mZ, mO, mOc, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
            denom, nullptr, nullptr, nullptr, Oc != nullptr ? 1 : 0, d.noncausal ? 1 : 0, status);
    } else {
        constexpr size_t smem = OutSmem<R, false>::total + 1024;
        PSK_TRY((set_smem(tc_fwd_out_kernel<R, 0, false, false>, smem)));
        tc_fwd_out_kernel<R, 0, false, false><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
            mQ, mQ, mK, mV, mZ, mO, mOc, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
            denom, nullptr, nullptr, nullptr, Oc != nullptr ? 1 : 0, d.noncausal ? 1 : 0, status);
    }
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace

#ifdef PSK_FWD_TRACE
extern "C" int psk_debug_ftrace(long long* host) {
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(host, g_ftr, sizeof(long long) * 64 * 16);
    return 64 * 16;
}
#endif

bool tc_supported(const Dims& d, bool backward) {
    (void)backward;
    // p = 2 (the rows are their own half sketch, r = h) runs the same kernels in "linear" mode;
    // p = 8: CUDA-core kernels (or the tensor cores through the given-half-sketch route of psk_api.cu)
    return d.bf16 && (d.p == 4 || d.p == 2 || d.sketch_linear) && encoder() != nullptr;
}

size_t tc_workspace_bytes(const Dims& d, bool backward) {
    backward = backward || d.keep_states;       // kept states: the forward writes into the backward's layout
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
static cudaError_t recompute_impl(const Dims& d, const CUtensorMap& mQ, const CUtensorMap& mQraw, const CUtensorMap& mK, const CUtensorMap& mV,
                                  const CUtensorMap& mZ, const uint8_t* gimg, const float* cmean,
                                  const float* denom, const bf16* dO, float* y65, float* e65h, int* status,
                                  cudaStream_t s, int* launches) {
    prof_begin("tc_bwd_recompute_kernel", s);
    if (d.local && d.sketch_linear) {
        if constexpr (R <= 32) {
            constexpr size_t smem = OutSmem<R, true>::total + 1024;
            PSK_TRY((set_smem(tc_fwd_out_kernel<R, 1, true, true>, smem)));
            tc_fwd_out_kernel<R, 1, true, true><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
                mQ, mQraw, mK, mV, mZ, mZ, mZ, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
                const_cast<float*>(denom), dO, y65, e65h, 0, 0, status);
        } else {
            return cudaErrorInvalidValue;
        }
    } else if (d.local) {
        constexpr size_t smem = OutSmem<R, true>::total + 1024;
        PSK_TRY((set_smem(tc_fwd_out_kernel<R, 1, true, false>, smem)));
        tc_fwd_out_kernel<R, 1, true, false><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
            mQ, mQ, mK, mV, mZ, mZ, mZ, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
            const_cast<float*>(denom), dO, y65, e65h, 0, d.noncausal ? 1 : 0, status);
    } else if (d.sketch_linear) {
        constexpr size_t smem = OutSmem<R, false>::total + 1024;
        PSK_TRY((set_smem(tc_fwd_out_kernel<R, 1, false, true>, smem)));
        tc_fwd_out_kernel<R, 1, false, true><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
            mQ, mQ, mK, mV, mZ, mZ, mZ, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
            const_cast<float*>(denom), dO, y65, e65h, 0, d.noncausal ? 1 : 0, status);
    } else {
        constexpr size_t smem = OutSmem<R, false>::total + 1024;
        PSK_TRY((set_smem(tc_fwd_out_kernel<R, 1, false, false>, smem)));
        tc_fwd_out_kernel<R, 1, false, false><<<dim3(d.b / 128, d.t, d.BH()), kOutThreads, smem, s>>>(
            mQ, mQ, mK, mV, mZ, mZ, mZ, gimg, d.g_heads, d.H, d.n, d.b, d.t, cmean, d.sb, d.sh, d.sn,
            const_cast<float*>(denom), dO, y65, e65h, 0, d.noncausal ? 1 : 0, status);
    }
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tc_recompute(const Dims& d, const CUtensorMap& mQ, const CUtensorMap& mQraw, const CUtensorMap& mK, const CUtensorMap& mV,
                         const CUtensorMap& mZ, const uint8_t* gimg, const float* cmean, const float* denom,
                         const bf16* dO, float* y65, float* e65h, int* status, cudaStream_t s, int* launches) {
    switch (d.r) {
        case 16: return recompute_impl<16>(d, mQ, mQraw, mK, mV, mZ, gimg, cmean, denom, dO, y65, e65h, status, s, launches);
        case 32: return recompute_impl<32>(d, mQ, mQraw, mK, mV, mZ, gimg, cmean, denom, dO, y65, e65h, status, s, launches);
        case 64: return recompute_impl<64>(d, mQ, mQraw, mK, mV, mZ, gimg, cmean, denom, dO, y65, e65h, status, s, launches);
    }
    return cudaErrorInvalidValue;
}

cudaError_t tc_gimage(const Dims& d, const void* G1, const void* G2, uint8_t* gimg, cudaStream_t s, int* launches) {
    prof_begin("tc_gimage_kernel", s);
    tc_gimage_kernel<<<d.g_heads, 128, 0, s>>>((const bf16*)G1, (const bf16*)G2, d.r, d.sketch_linear ? 1 : 0, gimg);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tc_vmean(const Dims& d, const void* V, float* cmean, cudaStream_t s, int* launches) {
    prof_begin("tc_vmean_kernel", s);
    tc_vmean_kernel<<<d.BH(), 1024, 0, s>>>((const bf16*)V, d.H, d.n, d.sb, d.sh, d.sn, cmean);
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace psk
