// Tensor-core backward of causal Polysketch attention.
//
// With g = dO, E_i = [g_i/d_i | -(g_i.O_i)/d_i], V~_j = [v_j | 1], s_ij = m(q_i).m(k_j):
//   dL/dW_ij = E_i.V~_j (j <= i),  ds_ij = 2 s_ij dW_ij,
//   dm(q_i) = sum_j ds_ij m(k_j),  dm(k_j) = sum_i ds_ij m(q_i),  dV_j = sum_i s_ij^2 E_i[:h].
// Pairs in the same block of b rows go through 128 x 128 tiles; pairs in different blocks go
// through the prefix state Z_l = sum_{blocks<l} phi(K)^T V~ (queries) and the suffix state
// R_l = sum_{blocks>l} phi(Q)^T E (keys, values), in the manner of Section 3.1:
//   d phi_w(q_i) = Z_l E_i,   d phi(k_j) = w * (R_l V~_j),   dV~_j = R_l^T phi_w(k_j),
// and, because every feature is a product m_a m_b, dm = 2 * sum over features of
// (d feature) * (the other factor)  (tc_features.cuh explains the weights w).
// One kernel, two roles: QSIDE rows own (Q, E) and meet keys j <= i; key-side rows own (K, V)
// and meet queries i >= j.  Thread = own row throughout.
#include "tc_common.cuh"

namespace psk {

using namespace tc;

namespace {

// With kept states the forward left Oc = O - c (bf16).  Eight lanes x 8 columns per row (four
// rows per warp):  y65 = -(dO . Oc)  (the last entry of E_i times d_i, paired with centred states),
// e65h = (y65 - dO . c) / d = -(dO . O) / d.  The rows E_i[:h] = dO_i / d_i themselves are never
// formed: the suffix-state kernel reads dO and scales the query features by 1 / d_i instead.
__global__ void __launch_bounds__(256)
tc_bwd_prep_kernel(const bf16* __restrict__ dO, const float* __restrict__ denom, const float* __restrict__ cmean,
                   const bf16* __restrict__ Oc, int H, int n, int total_rows, int64_t sb, int64_t sh, int64_t sn,
                   float* __restrict__ y65, float* __restrict__ e65h) {
    // 128 rows per CTA, four per thread group: all eight 16-byte loads of a thread are in flight
    // before the first is used.  (n and total_rows are multiples of 128: one head per CTA.)
    const int ch = threadIdx.x % 8;
    const int row_base = blockIdx.x * 128 + threadIdx.x / 8;
    const int bh = row_base / n;
    const int64_t head = (int64_t)(bh / H) * sb + (int64_t)(bh % H) * sh + 8 * ch;
    uint4 gv[4], oc[4];
    float dn[4];
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int row = row_base + it * 32;
        gv[it] = *reinterpret_cast<const uint4*>(dO + head + (int64_t)(row % n) * sn);
        oc[it] = *reinterpret_cast<const uint4*>(Oc + (size_t)row * 64 + 8 * ch);
        dn[it] = denom[row];
    }
    const float4 c0 = *reinterpret_cast<const float4*>(cmean + (size_t)bh * 64 + 8 * ch);
    const float4 c1 = *reinterpret_cast<const float4*>(cmean + (size_t)bh * 64 + 8 * ch + 4);
    const float c[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const uint32_t gw[4] = {gv[it].x, gv[it].y, gv[it].z, gv[it].w};
        const uint32_t ow[4] = {oc[it].x, oc[it].y, oc[it].z, oc[it].w};
        float dot = 0.f, gc = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float g0 = __uint_as_float(gw[j] << 16), g1 = __uint_as_float(gw[j] & 0xFFFF0000u);
            dot = fmaf(g0, __uint_as_float(ow[j] << 16), dot);
            dot = fmaf(g1, __uint_as_float(ow[j] & 0xFFFF0000u), dot);
            gc = fmaf(g0, c[2 * j], gc);
            gc = fmaf(g1, c[2 * j + 1], gc);
        }
#pragma unroll
        for (int s = 4; s > 0; s >>= 1) {
            dot += __shfl_xor_sync(0xffffffffu, dot, s);
            gc += __shfl_xor_sync(0xffffffffu, gc, s);
        }
        if (ch == 0) {
            const int row = row_base + it * 32;
            y65[row] = -dot;
            e65h[row] = -(dot + gc) / dn[it];          // -(dO . (O - c) + dO . c) / d
        }
    }
    (void)total_rows;
}

constexpr uint32_t kBoxBytes = 16384;      // two [64 features x 128 B] boxes: state columns 0..63, 64..79

template <int R, bool LOCAL = false, bool QSIDE = false>
struct BwdSmem {
    // every tile: 128 rows x 128 B, 128-byte swizzle
    static constexpr uint32_t kM = HiLoTiles<R>::N * 16384;      // [hi | lo] half-sketch operand
    static constexpr uint32_t Xown = 0, Yown = 16384;
    static constexpr uint32_t G = 32768;
    static constexpr uint32_t ExtA = G + GImage<R>::bytes;       // [128 x 16] un-swizzled
    static constexpr uint32_t Eoth = ExtA + 4096;        // 128 x (1/d, e65h) of the other side's rows
    static constexpr uint32_t U = Eoth + 1024;
    static constexpr uint32_t Box = U;                   // phase B: kSt state boxes
    static constexpr int NC = Feat<R>::NC;
    // stages of the state-chunk ring: four; three on the query side for r = 64 with exact
    // same-block weights, which then fits two CTAs per SM (no split-operand tiles in that variant;
    // the key side, at 255 registers and 225 KB of code, ran slower as two CTAs and keeps four)
    static constexpr int kSt = (R > 32 && LOCAL && QSIDE) ? 3 : 4;
    // Phase C tiles.  r <= 32 (two CTAs per SM): they reuse the boxes' memory, each tile in the
    // stage that the last chunks free first, so the first other-side tile is fetched while the
    // last chunks are still being processed.  r = 64 (one CTA per SM): memory of their own,
    // except with exact same-block weights, where X, Y and the second X buffer are all there is.
    static constexpr bool kAlias = (R <= 32) || LOCAL;
    static constexpr int sX = NC >= kSt ? (NC - kSt) % kSt : 3, sY = NC >= kSt ? (NC - kSt + 1) % kSt : 0;
    static constexpr int sMo = NC >= kSt ? (NC - kSt + 2) % kSt : 1, sMn = NC >= kSt ? (NC - 1) % kSt : 2;
    static constexpr uint32_t C0 = U + kSt * kBoxBytes;
    static constexpr uint32_t Xoth = kAlias ? U + sX * kBoxBytes : C0;
    static constexpr uint32_t Yoth = kAlias ? U + sY * kBoxBytes : C0 + 16384;
    static constexpr uint32_t Moth = kAlias ? U + sMo * kBoxBytes : C0 + 32768;
    static constexpr uint32_t Mown = kAlias ? U + sMn * kBoxBytes : C0 + 32768 + kM;
    static_assert(!kAlias || LOCAL || kM == kBoxBytes, "aliased layout: one tile per stage");
    static_assert(kSt == 4 || NC >= kSt, "three stages: only with many chunks");
    static constexpr uint32_t total = kAlias ? C0 : C0 + 32768 + 2 * kM;
    // output staging (epilogue): dX, dV tiles
    static constexpr uint32_t Sx = U, Sv = U + 16384;
};
constexpr uint32_t kBoxStride = kBoxBytes;

// dm += (d feature) * (the other factor) for the 32 features F0 .. F0+31 held in x
template <int R, int F0>
__device__ __forceinline__ void untensor32(const uint32_t (&x)[32], const float (&m)[R], float (&dm)[R]) {
    static_for<0, 32>([&](auto jc) {
        constexpr int J = decltype(jc)::value;
        constexpr int f = F0 + J;
        if constexpr (f < Feat<R>::F) {
            constexpr int A = Feat<R>::a(f), B = Feat<R>::b(f);
            const float v = __uint_as_float(x[J]);        // weighted by the state row it came through
            dm[A] = fmaf(v, m[B], dm[A]);
            dm[B] = fmaf(v, m[A], dm[B]);
        }
    });
}

// Score GEMM  own rows x 64 other rows over the split half sketches:
//   hi.hi + lo.hi + hi.lo, the [hi | lo] columns of both operands addressed in place.
template <int R>
__device__ __forceinline__ void issue_scores(uint32_t d_tmem, uint32_t own, uint32_t oth) {
    constexpr uint32_t idesc = idesc_bf16(128, 64, false, false);
    constexpr int offA[3] = {0, R, 0}, offB[3] = {0, 0, R};
#pragma unroll
    for (int g = 0; g < 3; ++g) {
#pragma unroll
        for (int kk = 0; kk < R / 16; ++kk) {
            const int ca = offA[g] + kk * 16, cb = offB[g] + kk * 16;
            umma_ss(d_tmem, desc_off(smem_desc(own, 0, 1024, kSwz128), (ca / 64) * 16384 + (ca % 64) * 2),
                    desc_off(smem_desc(oth, 0, 1024, kSwz128), (cb / 64) * 16384 + (cb % 64) * 2), idesc, (g > 0 || kk > 0) ? 1u : 0u);
        }
    }
}

// LOCAL (Section 3.2): same-block pairs carry the exact weights x_ij^4, x_ij = q_i . k_j.  The
// tile scores are then X_own X_other^T over the head dimension (raw bf16 rows: exact products),
// dL/dx_ij = 4 x_ij^3 dW_ij replaces ds_ij, and it multiplies the other side's raw rows straight
// into a dX accumulator that the sketch's backward (phase D) adds to: no half sketch of the other
// tile, no split operands, no dM from the tiles.
// LIN: the rows hold a given half sketch (tc_common.cuh, read_half_sketch); a template parameter, not
// an argument: the key side sits at the register limit, and the flag as an argument cost it 4 %.
template <int R, bool QSIDE, bool LOCAL, bool LIN>
__global__ void __launch_bounds__(128, ((R <= 32 || (LOCAL && QSIDE)) ? 2 : 1))
tc_bwd_rows_kernel(const __grid_constant__ CUtensorMap mapXown, const __grid_constant__ CUtensorMap mapYown,
                   const __grid_constant__ CUtensorMap mapXoth, const __grid_constant__ CUtensorMap mapYoth,
                   const __grid_constant__ CUtensorMap mapS, const __grid_constant__ CUtensorMap mapDX,
                   const __grid_constant__ CUtensorMap mapDV, const __grid_constant__ CUtensorMap mapXownRaw,
                   const __grid_constant__ CUtensorMap mapDXraw, const uint8_t* __restrict__ gimg,
                   int g_heads, int H, int n, int b, int t,
                   const float* __restrict__ y65g, const float* __restrict__ e65h, const float* __restrict__ denom,
                   int noncausal, int* status) {
    constexpr bool lin = LIN;
    using F = Feat<R>;
    using L = BwdSmem<R, LOCAL, QSIDE>;
    constexpr int kStages = L::kSt;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_own, bar_xoth, bar_yoth, bar_mma, bar_phi[2], bar_box[4];
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid / 32, tau = blockIdx.x, l = blockIdx.y, bh = blockIdx.z;
    const int hi = bh % H, bi = bh / H;
    const int g = g_heads == 1 ? 0 : hi;
    const int row0 = l * b + tau * 128;
    // Non-causal: every row tile meets the head's single global state and no same-block tiles.
    const int blk = noncausal ? bh : bh * t + l;
    const int ntiles = b / 128;
    const bool has_state = noncausal || (QSIDE ? (l > 0) : (l < t - 1));

    if (tid == 0) {
        // the own tiles are what everything waits for: their requests go out before anything else
        mbar_init(&bar_own, 1);
        mbar_fence_init();
        mbar_expect_tx(&bar_own, 32768 + GImage<R>::bytes);
        tma_load_4d(smem + L::Xown, &mapXown, 0, row0, hi, bi, &bar_own);
        tma_load_4d(smem + L::Yown, &mapYown, 0, row0, hi, bi, &bar_own);
        bulk_load(smem + L::G, gimg + (size_t)g * GImage<R>::bytes, GImage<R>::bytes, &bar_own);
        mbar_init(&bar_xoth, 1); mbar_init(&bar_yoth, 1); mbar_init(&bar_mma, 1);
        mbar_init(&bar_phi[0], 1); mbar_init(&bar_phi[1], 1);
        for (int s = 0; s < kStages; ++s) mbar_init(&bar_box[s], 1);
        cta_giveup_init();
        mbar_fence_init();
        tma_prefetch_desc(&mapXoth); tma_prefetch_desc(&mapYoth); tma_prefetch_desc(&mapS);
        if (has_state) {
            for (int c = 0; c < kStages && c < F::NC; ++c) {
                mbar_expect_tx(&bar_box[c], kBoxBytes);
                tma_load_3d(smem + L::Box + c * kBoxStride, &mapS, 0, c * 64, blk, &bar_box[c]);
                tma_load_3d(smem + L::Box + c * kBoxStride + 8192, &mapS, 64, c * 64, blk, &bar_box[c]);
            }
        }
        // first other-side tile: at once where its memory is free from the start
        const int orow_first = l * b + (QSIDE ? 0 : tau) * 128;
        if (!noncausal && (!has_state || !L::kAlias || F::NC < kStages)) {
            mbar_expect_tx(&bar_xoth, 16384);
            tma_load_4d(smem + L::Xoth, &mapXoth, 0, orow_first, hi, bi, &bar_xoth);
        }
        if (!noncausal && (!has_state || !L::kAlias)) {
            mbar_expect_tx(&bar_yoth, 16384);
            tma_load_4d(smem + L::Yoth, &mapYoth, 0, orow_first, hi, bi, &bar_yoth);
        }
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    // Query rows work on the raw dO rows g_i (exact bf16 inputs) and apply 1/d_i in fp32 afterwards:
    // dL/dW_ij = (g_i . v_j - g_i . O_i) / d_i cancels heavily when one key dominates a row, and a
    // rounded g_i / d_i would not survive it.  y65 = -(g_i . (O_i - c)) pairs with the centred
    // states, y65h = -(g_i . O_i) with the raw values of the 128 x 128 tiles.  Key rows: 1.
    // (The three row scalars come from HBM.  They are requested here and first used after the half
    // sketch has been read, a few thousand cycles later: the arithmetic on them stays below.)
    const float d_raw = QSIDE ? denom[(size_t)bh * n + row0 + tid] : 1.f;
    const float y65_raw = QSIDE ? y65g[(size_t)bh * n + row0 + tid] : 1.f;
    const float e65h_raw = QSIDE ? e65h[(size_t)bh * n + row0 + tid] : 1.f;
    // key side: the scalars of the first query tile it will meet (thread = that tile's row tid)
    float od_raw = 1.f, oe_raw = 0.f;
    if constexpr (!QSIDE) {
        od_raw = denom[(size_t)bh * n + l * b + tau * 128 + tid];
        oe_raw = e65h[(size_t)bh * n + l * b + tau * 128 + tid];
    }
    *reinterpret_cast<uint4*>(smem + L::ExtA + 2048 + (tid / 8) * 128 + (tid % 8) * 16) = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_slot;
    const uint32_t lane_tm = tm + ((uint32_t)(warp * 32) << 16);
    // tensor-memory columns (256): [0,128) is scratch, reused phase by phase; accumulators follow
    constexpr uint32_t cS = 0, cDW = 64;                  // phase C: scores, dW (64 other rows); then packed dS / W
    constexpr uint32_t cPhi = 0;                          // phase B: d-phi, 2 x 64
    constexpr uint32_t cSk = 0;                           // sketch accumulators (transient, <= 128)
    constexpr uint32_t cdM = 128, cdV = 192;              // accumulators: dM (64), dV (64)
    // r <= 32: the own rows' 64 Y columns also sit in tensor memory (bf16 pairs, 32 columns behind
    // the r <= 32 columns dM needs), as the A operand of every GEMM that multiplies them.  An MMA
    // whose operands both come from shared memory moves 6 KB through the 128 B/clk shared-memory
    // path, which takes as long as its arithmetic and shares that path with everything else.
    constexpr bool kTsA = (R <= 32);
    constexpr uint32_t cYA = cdM + 32;
    constexpr int kNdM = kTsA ? R : 64;                   // columns the dM GEMM writes
    // LOCAL: the tiles' dX accumulator (64 columns).  Query side, r <= 32: the unused dV columns.
    // Otherwise the dM columns -- on the key side with r <= 32 that includes the Y operand's,
    // which phase C then reads from shared memory instead.
    constexpr bool kTsC = kTsA && !(LOCAL && !QSIDE);
    constexpr uint32_t cXl = (kTsA && QSIDE) ? cdV : cdM;
    uint32_t mma_uses = 0;
    bool ok = true;

    // ---- phase A: half sketch of the own rows ----
    ok = mbar_wait(&bar_own, 0, status, kErrTma);
    if (tid == 0) {
        tc_fence_after();
        issue_sketch<R>(tm + cSk, smem + L::Xown, smem + L::G);
        umma_commit(&bar_mma);
    }
    ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
    ++mma_uses;
    tc_fence_after();
    float m[R], dm[R];
    read_half_sketch<R>(lane_tm + cSk, m, 1.f, lin != 0);
    if constexpr (LIN && LOCAL) {
        // The own tile held the given half sketch; the exact same-block scores need the raw rows.
        // The sketch GEMM has completed: fetch them into the same buffer (phase C waits for them).
        if (tid == 0) {
            mbar_expect_tx(&bar_own, 16384);
            tma_load_4d(smem + L::Xown, &mapXownRaw, 0, row0, hi, bi, &bar_own);
        }
    }
#pragma unroll
    for (int c = 0; c < R; ++c) dm[c] = 0.f;
    bool dv_started = false;
    const float d_own = d_raw, inv_own = 1.f / d_own;
    const float y65 = y65_raw, y65h = QSIDE ? e65h_raw * d_own : 1.f;
    // the 65th column of the A operand [Y_own | y65]: first read by phase B's MMAs, after the barrier below
    *reinterpret_cast<uint4*>(smem + L::ExtA + (tid / 8) * 128 + (tid % 8) * 16) = make_uint4(pack_bf16(y65, 0.f), 0, 0, 0);
    fence_proxy_async_smem();
    if constexpr (kTsA) {
        uint32_t ya[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 v = *reinterpret_cast<const uint4*>(smem + L::Yown + swz128_offset(tid, c));
            ya[4 * c] = v.x; ya[4 * c + 1] = v.y; ya[4 * c + 2] = v.z; ya[4 * c + 3] = v.w;
        }
        tmem_st32(lane_tm + cYA, ya);
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // ---- phase B: other blocks through the state ----
    if (has_state) {
        constexpr uint32_t idesc_phi = idesc_bf16(128, 64, false, false);
        // Software pipeline over the 64-feature chunks: while the MMAs of chunk C run, the threads
        // generate chunk C+1's features; while those of chunk C+1 run, they un-tensor chunk C.
        // d-phi is double-buffered in [0,128); during this phase the feature staging buffers sit
        // in the dM accumulator's columns, which only phase C uses.
        constexpr uint32_t cFB = cdM;
        // descriptors are loop invariants: an issue sequence is its MMA instructions and little else
        const uint64_t yd = smem_desc(smem_u32(smem + L::Yown), 0, 1024, kSwz128);
        const uint64_t ed = smem_desc(smem_u32(smem + L::ExtA), 2048, 128, kSwzNone);
        const uint64_t bd0 = smem_desc(smem_u32(smem + L::Box), 0, 1024, kSwz128);
        auto issue_chunk = [&](int C) {           // one thread: the chunk's MMAs, then commit
            const int buf = C & 1, stage = C % kStages;
            const int ksteps = (F::FK - C * 64) >= 64 ? 4 : (F::FK - C * 64) / 16;
            const uint64_t bd = desc_off(bd0, stage * kBoxStride);
            const uint32_t dphi = tm + cPhi + buf * 64;
            // d-phi chunk = [Yown | y65] x box^T: the box's feature rows are a K-major B operand,
            // contraction over the 64 state columns, then the last column (second box)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if constexpr (kTsA) umma_ts(dphi, tm + cYA + k * 8, desc_off(bd, k * 32), idesc_phi, k > 0);
                else umma_ss(dphi, desc_off(yd, k * 32), desc_off(bd, k * 32), idesc_phi, k > 0);
            }
            umma_ss(dphi, ed, desc_off(bd, 8192), idesc_phi, 1);
            if constexpr (!QSIDE) {
                // dV += phi(k) chunk x box (MN-major B: 16 features per K step)
                constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
                const uint32_t fb = tm + cFB + (kTsA ? 0 : buf * 32);   // r <= 32: one staging buffer
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (k < ksteps) umma_ts(tm + cdV, fb + k * 8, desc_off(bd, k * 2048), idesc, (C > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(&bar_phi[buf]);
        };
        auto refill = [&](int C) {                // tid 0: chunk C's box is free
            if (C + kStages < F::NC) {
                const int stage = C % kStages;
                mbar_expect_tx(&bar_box[stage], kBoxBytes);
                tma_load_3d(smem + L::Box + stage * kBoxStride, &mapS, 0, (C + kStages) * 64, blk, &bar_box[stage]);
                tma_load_3d(smem + L::Box + stage * kBoxStride + 8192, &mapS, 64, (C + kStages) * 64, blk, &bar_box[stage]);
            } else if (L::kAlias && !noncausal) {
                // the last chunks free the stages that the first other-side tile goes into
                const int orow_first = l * b + (QSIDE ? 0 : tau) * 128;
                if (F::NC >= kStages && C == F::NC - kStages) {
                    mbar_expect_tx(&bar_xoth, 16384);
                    tma_load_4d(smem + L::Xoth, &mapXoth, 0, orow_first, hi, bi, &bar_xoth);
                }
                if (C == (F::NC >= kStages ? F::NC - kStages + 1 : 0)) {
                    mbar_expect_tx(&bar_yoth, 16384);
                    tma_load_4d(smem + L::Yoth, &mapYoth, 0, orow_first, hi, bi, &bar_yoth);
                }
            }
        };
        if constexpr (F::kCirc) {
            // every chunk is the same code on rotated copies of m: a loop
            CircGen<R> gen;
            CircUntensor<R> ut;
            if constexpr (!QSIDE) gen.init(m);
            ut.init(m);
            auto stage_features = [&](int C) {    // features of the next chunk -> tensor memory
                uint32_t pk[32];
                gen.chunk(pk);
                (void)C;
                tmem_st32(lane_tm + cFB, pk);          // one buffer: its previous reader (chunk C-1's MMAs) is done
                tmem_st_wait();
            };
            if constexpr (!QSIDE) stage_features(0);
            ok = ok && mbar_wait(&bar_box[0], 0, status, kErrTma);
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                issue_chunk(0);
            }
#pragma unroll 1
            for (int C = 0; C < F::NC && ok; ++C) {
                const int buf = C & 1;
                // Key side: chunk C's MMAs read the one staging buffer, so they must have completed
                // before chunk C+1's features go in; query side: chunk C+1 is issued first and runs
                // behind chunk C.
                if constexpr (!QSIDE) {
                    ok = mbar_wait(&bar_phi[buf], (C / 2) & 1, status, kErrMma);
                    tc_fence_after();
                }
                if (C + 1 < F::NC) {
                    if constexpr (!QSIDE) stage_features(C + 1);
                    ok = ok && mbar_wait(&bar_box[(C + 1) % kStages], ((C + 1) / kStages) & 1, status, kErrTma);
                    tc_fence_before();
                    __syncthreads();           // chunk C-1's d-phi has been read by every thread
                    if (tid == 0) {
                        tc_fence_after();
                        issue_chunk(C + 1);
                    }
                }
                if constexpr (QSIDE) {
                    ok = ok && mbar_wait(&bar_phi[buf], (C / 2) & 1, status, kErrMma);
                    tc_fence_after();
                }
                if (tid == 32) refill(C);          // (warp 0 issues the MMAs; the loads go out from warp 1)
                uint32_t x[32];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    tmem_ld32(lane_tm + cPhi + buf * 64 + h * 32, x);
                    tmem_ld_wait();
                    if constexpr (R == 32) {
                        if (h == 0) ut.even(x, m, dm); else { ut.odd(x, m, dm); ut.advance(); }
                    } else {
                        ut.even(x, m, dm);
                        ut.odd(x + 16, m, dm);
                        ut.advance();
                    }
                }
            }
            ut.template finish<F::NC * 64 / (2 * R)>(dm);
        } else {
            PackedM<R> pm;
            if constexpr (!QSIDE) pack_half_sketch<R>(m, pm);
            auto stage_features = [&](auto cc) {
                constexpr int C = decltype(cc)::value;
                uint32_t pk[16];
                gen_features<R, C * 64, 16>(pm, pk);
                tmem_st16(lane_tm + cFB + (C & 1) * 32, pk);
                gen_features<R, C * 64 + 32, 16>(pm, pk);
                tmem_st16(lane_tm + cFB + (C & 1) * 32 + 16, pk);
                tmem_st_wait();
            };
            if constexpr (!QSIDE) stage_features(std::integral_constant<int, 0>{});
            ok = ok && mbar_wait(&bar_box[0], 0, status, kErrTma);
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                issue_chunk(0);
            }
            static_for<0, F::NC>([&](auto cc) {
                constexpr int C = decltype(cc)::value;
                constexpr int buf = C & 1;
                if constexpr (C + 1 < F::NC) {
                    if constexpr (!QSIDE) stage_features(std::integral_constant<int, C + 1>{});
                    ok = ok && mbar_wait(&bar_box[(C + 1) % kStages], ((C + 1) / kStages) & 1, status, kErrTma);
                    tc_fence_before();
                    __syncthreads();           // chunk C-1's d-phi has been read by every thread
                    if (tid == 0) {
                        tc_fence_after();
                        issue_chunk(C + 1);
                    }
                }
                ok = ok && mbar_wait(&bar_phi[buf], (C / 2) & 1, status, kErrMma);
                tc_fence_after();
                if (tid == 32) refill(C);          // (warp 0 issues the MMAs; the loads go out from warp 1)
                {
                    uint32_t x[32];
                    tmem_ld32(lane_tm + cPhi + buf * 64, x);
                    tmem_ld_wait();
                    untensor32<R, C * 64>(x, m, dm);
                    tmem_ld32(lane_tm + cPhi + buf * 64 + 32, x);
                    tmem_ld_wait();
                    untensor32<R, C * 64 + 32>(x, m, dm);
                }
            });
        }
        if constexpr (!QSIDE) dv_started = true;
#pragma unroll
        for (int c = 0; c < R; ++c) dm[c] *= inv_own;
        tc_fence_before();
        __syncthreads();                   // boxes and the scratch columns are dead: phase C reuses them
        tc_fence_after();
    }

    // ---- phase C: same block, other-side tiles, 64 other rows at a time ----
    if constexpr (!LOCAL) store_hilo_tiles<R>(smem + L::Mown, m, tid);
    const int tp_begin = QSIDE ? 0 : tau, tp_end = noncausal ? tp_begin : (QSIDE ? tau + 1 : ntiles);
    bool dm_started = false;
    uint32_t oth_uses = 0;
    float2* oth_col = reinterpret_cast<float2*>(smem + L::Eoth);   // other rows: (1/d, -(g . O)/d)
    const float y65h_inv = y65h * inv_own;
    if constexpr (LIN && LOCAL) ok = ok && mbar_wait(&bar_own, 1, status, kErrTma);      // the raw own rows
#pragma unroll 1
    for (int tp = tp_begin; tp < tp_end && ok; ++tp) {
        const int orow0 = l * b + tp * 128;
        // LOCAL: the other side's raw tiles alternate between two buffers (the second one is the
        // unused split-operand tile), so the next tile's rows can be requested a tile ahead
        const uint32_t xo = (LOCAL && ((tp - tp_begin) & 1)) ? L::Moth : L::Xoth;
        const uint32_t xo_next = (LOCAL && !((tp - tp_begin) & 1)) ? L::Moth : L::Xoth;
        // (this tile's rows were requested ahead: by the prologue, by phase B's last chunks, or
        // by the previous tile as soon as its own copies had been consumed)
        // Every thread is past its wait for the previous tile's last MMAs before the next commit
        // can complete the same barrier again: a waiter that looks after two completions sees
        // the barrier back in the phase it started from.
        __syncthreads();
        if constexpr (!QSIDE) {
            // e65h is already -(g . O) / d.  These two were requested a tile (or a phase) ago; the
            // next tile's are requested now.
            oth_col[tid] = make_float2(1.f / od_raw, oe_raw);
            if (tp + 1 < tp_end) {
                od_raw = denom[(size_t)bh * n + orow0 + 128 + tid];
                oe_raw = e65h[(size_t)bh * n + orow0 + 128 + tid];
            }
        }
        ok = mbar_wait(&bar_xoth, oth_uses & 1, status, kErrTma);
        if constexpr (!LOCAL) {
            if (tid == 0) {
                tc_fence_after();
                issue_sketch<R>(tm + cSk, smem + L::Xoth, smem + L::G);
                umma_commit(&bar_mma);
            }
            ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
            ++mma_uses;
            tc_fence_after();
        }
        ok = ok && mbar_wait(&bar_yoth, oth_uses & 1, status, kErrTma);
        ++oth_uses;
        if constexpr (!LOCAL) {
            float mo[R];
            read_half_sketch<R>(lane_tm + cSk, mo, 1.f, lin != 0);
            store_hilo_tiles<R>(smem + L::Moth, mo, tid);
        }
        const bool diag = (tp == tau);
#pragma unroll 1
        for (int hh = 0; hh < 2; ++hh) {
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                // The X tile has been consumed, and every thread is past its wait for it (a
                // barrier must not complete twice before its slowest waiter has looked): next
                // tile's rows.
                // (LOCAL: the raw rows stay operands to the tile's end; the next ones go to the other buffer)
                if (hh == 0 && tp + 1 < tp_end) {
                    mbar_expect_tx(&bar_xoth, 16384);
                    tma_load_4d(smem + xo_next, &mapXoth, 0, orow0 + 128, hi, bi, &bar_xoth);
                }
                constexpr uint32_t idesc = idesc_bf16(128, 64, false, false);
                if constexpr (LOCAL) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)       // x = own rows . other rows, over the head dimension
                        umma_ss(tm + cS, desc_off(smem_desc(smem_u32(smem + L::Xown), 0, 1024, kSwz128), k * 32),
                                desc_off(smem_desc(smem_u32(smem + xo) + hh * 8192, 0, 1024, kSwz128), k * 32), idesc, k > 0);
                } else {
                    issue_scores<R>(tm + cS, smem_u32(smem + L::Mown), smem_u32(smem + L::Moth) + hh * 8192);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {         // dW without its 65th-column term
                    const uint64_t yod = desc_off(smem_desc(smem_u32(smem + L::Yoth) + hh * 8192, 0, 1024, kSwz128), k * 32);
                    if constexpr (kTsC) umma_ts(tm + cDW, tm + cYA + k * 8, yod, idesc, k > 0);
                    else umma_ss(tm + cDW, desc_off(smem_desc(smem_u32(smem + L::Yown), 0, 1024, kSwz128), k * 32), yod, idesc, k > 0);
                }
                umma_commit(&bar_mma);
            }
            ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
            ++mma_uses;
            tc_fence_after();
            // dW = (own . other + y) / d_i,  ds = 2 s dW,  W / d_i = s^2 / d_i, masked on the diagonal
            // tile; packed to bf16 over columns whose fp32 contents have already been read
            auto tile_math = [&](auto diag_c) {
                constexpr bool DIAG = decltype(diag_c)::value;
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t sv[32], wv[32], pds[16], pw[16];
                    tmem_ld32(lane_tm + cS + c0, sv);
                    tmem_ld32(lane_tm + cDW + c0, wv);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int col = hh * 64 + c0 + j;
                        float s = __uint_as_float(sv[j]);
                        if constexpr (DIAG) s = (QSIDE ? (col <= tid) : (col >= tid)) ? s : 0.f;
                        float inv, yinv;
                        if constexpr (QSIDE) {
                            inv = inv_own; yinv = y65h_inv;
                        } else {
                            const float2 o = oth_col[col];
                            inv = o.x; yinv = o.y;
                        }
                        const float dw = fmaf(__uint_as_float(wv[j]), inv, yinv);
                        if constexpr (LOCAL) {
                            const float s2 = s * s;                     // s is x_ij here
                            sv[j] = __float_as_uint(4.f * s * s2 * dw);
                            wv[j] = __float_as_uint(s2 * (s2 * inv));
                        } else {
                            sv[j] = __float_as_uint((s + s) * dw);
                            wv[j] = __float_as_uint(s * (s * inv));     // weight / d_i: the value side sees g_i / d_i
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        pds[j] = pack_bf16(__uint_as_float(sv[2 * j]), __uint_as_float(sv[2 * j + 1]));
                        pw[j] = pack_bf16(__uint_as_float(wv[2 * j]), __uint_as_float(wv[2 * j + 1]));
                    }
                    tmem_st16(lane_tm + cS + c0 / 2, pds);
                    if constexpr (!QSIDE) tmem_st16(lane_tm + cDW + c0 / 2, pw);
                }
            };
            if (diag) tile_math(std::true_type{}); else tile_math(std::false_type{});
            tmem_st_wait();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
                constexpr uint32_t idesc_dm = idesc_bf16(128, kNdM, false, true);
                if constexpr (LOCAL) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)       // dX_own += dx x X_other
                        umma_ts(tm + cXl, tm + cS + k * 8,
                                desc_off(smem_desc(smem_u32(smem + xo) + hh * 8192, 0, 1024, kSwz128), k * 2048), idesc,
                                (dm_started || k > 0) ? 1u : 0u);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)       // dM_own += dS x M_other (its hi columns)
                        umma_ts(tm + cdM, tm + cS + k * 8,
                                desc_off(smem_desc(smem_u32(smem + L::Moth) + hh * 8192, 0, 1024, kSwz128), k * 2048), idesc_dm,
                                (dm_started || k > 0) ? 1u : 0u);
                }
                if constexpr (!QSIDE) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)       // dV += W x E_other
                        umma_ts(tm + cdV, tm + cDW + k * 8,
                                desc_off(smem_desc(smem_u32(smem + L::Yoth) + hh * 8192, 0, 1024, kSwz128), k * 2048), idesc,
                                (dv_started || k > 0) ? 1u : 0u);
                }
                umma_commit(&bar_mma);
            }
            dm_started = true;
            dv_started = true;
            ok = ok && mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
            ++mma_uses;
            tc_fence_after();
        }
        if (tid == 0 && tp + 1 < tp_end) {        // every MMA that read the Y tile has completed
            mbar_expect_tx(&bar_yoth, 16384);
            tma_load_4d(smem + L::Yoth, &mapYoth, 0, orow0 + 128, hi, bi, &bar_yoth);
        }
    }

    // ---- phase D: through the sketch, dX = ((dM*A2) G1^T + (dM*A1) G2^T) / sqrt(R) ----
    if (ok) {
        // (a given half sketch has no 1/sqrt(R) of its own)
        const float rs = lin ? 1.f : rsqrtf((float)R);
        // dM total = state part (registers) + tile part (tensor memory), scaled by 1/sqrt(R)
        if constexpr (LOCAL) {
#pragma unroll
            for (int c = 0; c < R; ++c) dm[c] *= rs;
        } else {
#pragma unroll
            for (int c0 = 0; c0 < R; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(lane_tm + cdM + c0, v);
                tmem_ld_wait();
                // (no same-block tiles ran: nothing was accumulated there)
#pragma unroll
                for (int j = 0; j < 16; ++j) dm[c0 + j] = (dm[c0 + j] + (dm_started ? __uint_as_float(v[j]) : 0.f)) * rs;
            }
        }
        if constexpr (!LIN) {      // (a given half sketch: dX = dM "G1"^T needs neither A1 nor A2)
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                issue_sketch<R>(tm + cSk, smem + L::Xown, smem + L::G);   // A1, A2 again
                umma_commit(&bar_mma);
            }
            ok = mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
            ++mma_uses;
            tc_fence_after();
        }
    }
    if (ok) {
        // U = [dM*A2 | dM*A1] as a bf16 A operand in tensor memory (2R values -> R columns at cdM).
        // LOCAL: the dM columns may hold the tiles' dX accumulator, so U goes over the sketch
        // columns this thread has just read (dM*A2 from column 0, dM*A1 from column R), and the
        // GEMM adds to that accumulator.
        constexpr uint32_t cU1 = LOCAL ? cSk : cdM, cU2 = LOCAL ? cSk + R : cdM + R / 2;
        constexpr uint32_t cDX = LOCAL ? cXl : cS;
        if constexpr (LIN && LOCAL) {
            // Two gradients leave this kernel: the same-block tiles' one belongs to the raw rows and
            // goes out now; the sketch's belongs to the given half sketch and takes the
            // accumulator over afterwards.  (Every MMA has completed: the staging tile is free.)
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(lane_tm + cXl + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 8)
                    *reinterpret_cast<uint4*>(smem + L::Sx + swz128_offset(tid, (c0 + j) / 8)) =
                        make_uint4(pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1])),
                                   pack_bf16(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])),
                                   pack_bf16(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5])),
                                   pack_bf16(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7])));
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tma_store_4d(&mapDXraw, smem + L::Sx, 0, row0, hi, bi);
                bulk_commit();
                bulk_wait_read();
            }
            __syncthreads();
            tc_fence_after();
        }
#pragma unroll
        for (int c0 = 0; c0 < R; c0 += 16) {
            uint32_t a1[16], a2[16], u1[8], u2[8];
            tmem_ld16(lane_tm + cSk + c0, a1);
            tmem_ld16(lane_tm + cSk + R + c0, a2);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // given half sketch: dX = dM "G1"^T with that identity-like matrix, and nothing through "G2"
                u1[j] = pack_bf16(dm[c0 + 2 * j] * (lin ? 1.f : __uint_as_float(a2[2 * j])),
                                  dm[c0 + 2 * j + 1] * (lin ? 1.f : __uint_as_float(a2[2 * j + 1])));
                u2[j] = pack_bf16(lin ? 0.f : dm[c0 + 2 * j] * __uint_as_float(a1[2 * j]),
                                  lin ? 0.f : dm[c0 + 2 * j + 1] * __uint_as_float(a1[2 * j + 1]));
            }
            tmem_st8(lane_tm + cU1 + c0 / 2, u1);
            tmem_st8(lane_tm + cU2 + c0 / 2, u2);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            constexpr uint32_t idesc = idesc_bf16(128, 64, false, true);
#pragma unroll
            for (int k = 0; k < 2 * R / 16; ++k)    // contraction over the 2R sketch columns
                umma_ts(tm + cDX, tm + (k < R / 16 ? cU1 + k * 8 : cU2 + (k - R / 16) * 8),
                        desc_off(smem_desc(smem_u32(smem + L::G), 0, 1024, kSwz128), k * 2048), idesc, ((LOCAL && !LIN) || k > 0) ? 1u : 0u);
            umma_commit(&bar_mma);
        }
        ok = mbar_wait(&bar_mma, mma_uses & 1, status, kErrMma);
        ++mma_uses;
        tc_fence_after();
    }
    // rows go out through shared memory and tiled stores (every MMA has completed: the other-side
    // tiles' memory is free); a thread-per-row store pattern would keep the load/store unit busy
    // for thousands of cycles
    if (ok) {
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(lane_tm + (LOCAL ? cXl : cS) + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; j += 8)
                *reinterpret_cast<uint4*>(smem + L::Sx + swz128_offset(tid, (c0 + j) / 8)) =
                    make_uint4(pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1])),
                               pack_bf16(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])),
                               pack_bf16(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5])),
                               pack_bf16(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7])));
        }
        if constexpr (!QSIDE) {
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(lane_tm + cdV + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 8)
                    *reinterpret_cast<uint4*>(smem + L::Sv + swz128_offset(tid, (c0 + j) / 8)) =
                        make_uint4(pack_bf16(__uint_as_float(v[j]), __uint_as_float(v[j + 1])),
                                   pack_bf16(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])),
                                   pack_bf16(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5])),
                                   pack_bf16(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7])));
            }
        }
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && ok) {
        tma_store_4d(&mapDX, smem + L::Sx, 0, row0, hi, bi);
        if constexpr (!QSIDE) tma_store_4d(&mapDV, smem + L::Sv, 0, row0, hi, bi);
        bulk_commit();
        bulk_wait_read();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 256);
}

template <int R>
cudaError_t bwd_impl(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                     const void* O, const float* denom, const void* dO, void* dQ, void* dK, void* dV, char* ws,
                     cudaStream_t s, int* launches) {
    const TcWorkspace w = tc_ws<R>(d, true);
    int* status = reinterpret_cast<int*>(ws + w.status);
    bf16* Z = reinterpret_cast<bf16*>(ws + w.Z);
    bf16* Rs = reinterpret_cast<bf16*>(ws + w.Rst);
    float* y65 = reinterpret_cast<float*>(ws + w.y65);
    float* cmean = reinterpret_cast<float*>(ws + w.vmean);
    float* e65h = reinterpret_cast<float*>(ws + w.e65h);
    float* tot = reinterpret_cast<float*>(ws + w.tot);
    if (!d.keep_states) PSK_TRY(tc_vmean(d, V, cmean, s, launches));
    CUtensorMap mQ, mK, mV, mG, mZ, mR, mdQ, mdK, mdV;
    const int64_t nblk = (int64_t)d.BH() * (d.noncausal ? 1 : d.t);
    if (!tc_map_rows(&mQ, Q, d.B, d.H, d.n, d.xsb, d.xsh, d.xsn) || !tc_map_rows(&mK, K, d.B, d.H, d.n, d.xsb, d.xsh, d.xsn) ||
        !tc_map_rows(&mV, V, d.B, d.H, d.n, d.sb, d.sh, d.sn) ||
        !tc_map_rows(&mG, dO, d.B, d.H, d.n, d.sb, d.sh, d.sn) ||
        !tc_map_states(&mZ, Z, Feat<R>::FP, nblk) || !tc_map_states(&mR, Rs, Feat<R>::FP, nblk) ||
        !tc_map_rows(&mdQ, dQ, d.B, d.H, d.n, d.xsb, d.xsh, d.xsn) || !tc_map_rows(&mdK, dK, d.B, d.H, d.n, d.xsb, d.xsh, d.xsn) ||
        !tc_map_rows(&mdV, dV, d.B, d.H, d.n, d.sb, d.sh, d.sn))
        return cudaErrorInvalidValue;
    // given half sketches with exact same-block weights: raw rows in, their gradients out
    CUtensorMap mQraw = mQ, mKraw = mK, mdQraw = mdQ, mdKraw = mdK;
    const bool linloc = d.sketch_linear && d.local;
    if (linloc) {
        const int64_t hs = (int64_t)d.n * 64, bs = (int64_t)d.H * hs;
        if (!d.rawQ || !d.rawK || !d.rawdQ || !d.rawdK || !tc_map_rows(&mQraw, d.rawQ, d.B, d.H, d.n, d.sb, d.sh, d.sn) ||
            !tc_map_rows(&mKraw, d.rawK, d.B, d.H, d.n, d.sb, d.sh, d.sn) || !tc_map_rows(&mdQraw, d.rawdQ, d.B, d.H, d.n, bs, hs, 64) ||
            !tc_map_rows(&mdKraw, d.rawdK, d.B, d.H, d.n, bs, hs, 64))
            return cudaErrorInvalidValue;
    }
    uint8_t* gimg = reinterpret_cast<uint8_t*>(ws + w.gimg);
    PSK_TRY(tc_gimage(d, G1, G2, gimg, s, launches));
    // prefix states of centred values; forward rows again in fp32 -> y65, e65h; suffix states
    if (!d.keep_states) PSK_TRY(tc_states(d, mK, mV, gimg, nullptr, nullptr, cmean, 1, Z, false, tot, status, s, launches));
    if (d.keep_states) {
        const int rows = d.BH() * d.n;
        prof_begin("tc_bwd_prep_kernel", s);
        tc_bwd_prep_kernel<<<rows / 128, 256, 0, s>>>((const bf16*)dO, denom, cmean,
                                                           reinterpret_cast<const bf16*>(ws + w.Oc), d.H, d.n, rows, d.sb,
                                                           d.sh, d.sn, y65, e65h);
        prof_end(s);
        ++*launches;
        PSK_TRY(cudaGetLastError());
    } else {
        PSK_TRY(tc_recompute(d, mQ, mQraw, linloc ? mKraw : mK, mV, mZ, gimg, cmean, denom, (const bf16*)dO, y65, e65h, status, s, launches));
    }
    const dim3 grid(d.b / 128, d.t, d.BH());
    auto rows = [&](auto local_c, auto lin_c) -> cudaError_t {
        constexpr bool LOCAL = decltype(local_c)::value;
        constexpr bool LIN = decltype(lin_c)::value;
        constexpr size_t smem = BwdSmem<R, LOCAL, true>::total + 1024, smem_k = BwdSmem<R, LOCAL, false>::total + 1024;
        PSK_TRY((set_smem(tc_bwd_rows_kernel<R, true, LOCAL, LIN>, smem)));
        PSK_TRY((set_smem(tc_bwd_rows_kernel<R, false, LOCAL, LIN>, smem_k)));
        // query side first: it needs only the prefix states, and the row scalars just written are
        // still in L2; the suffix states (5 GB through L2) come after it
        prof_begin("tc_bwd_q_kernel", s);
        tc_bwd_rows_kernel<R, true, LOCAL, LIN><<<grid, 128, smem, s>>>(mQ, mG, (LOCAL && LIN) ? mKraw : mK, mV, mZ, mdQ, mdQ, mQraw, mdQraw, gimg, d.g_heads, d.H, d.n,
                                                                   d.b, d.t, y65, e65h, denom, d.noncausal ? 1 : 0, status);
        prof_end(s);
        ++*launches;
        PSK_TRY(cudaGetLastError());
        // suffix states: phi(q_i) / d_i against [dO_i | y65_i]
        PSK_TRY(tc_states(d, mQ, mG, gimg, y65, denom, cmean, 2, Rs, true, tot, status, s, launches));
        prof_begin("tc_bwd_k_kernel", s);
        tc_bwd_rows_kernel<R, false, LOCAL, LIN><<<grid, 128, smem_k, s>>>(mK, mV, (LOCAL && LIN) ? mQraw : mQ, mG, mR, mdK, mdV, mKraw, mdKraw, gimg, d.g_heads, d.H, d.n,
                                                                    d.b, d.t, y65, e65h, denom, d.noncausal ? 1 : 0, status);
        prof_end(s);
        ++*launches;
        return cudaGetLastError();
    };
    if (linloc) {
        if constexpr (R <= 32) return rows(std::true_type{}, std::true_type{});
        else return cudaErrorInvalidValue;
    }
    if (d.sketch_linear) return rows(std::false_type{}, std::true_type{});
    return d.local ? rows(std::true_type{}, std::false_type{}) : rows(std::false_type{}, std::false_type{});
}

}  // namespace

cudaError_t tc_bwd(const Dims& d, const void* Q, const void* K, const void* V, const void* G1, const void* G2,
                   const void* O, const float* denom, const void* dO, void* dQ, void* dK, void* dV, char* ws,
                   cudaStream_t s, int* launches) {
    switch (d.r) {
        case 16: return bwd_impl<16>(d, Q, K, V, G1, G2, O, denom, dO, dQ, dK, dV, ws, s, launches);
        case 32: return bwd_impl<32>(d, Q, K, V, G1, G2, O, denom, dO, dQ, dK, dV, ws, s, launches);
        case 64: return bwd_impl<64>(d, Q, K, V, G1, G2, O, denom, dO, dQ, dK, dV, ws, s, launches);
    }
    return cudaErrorInvalidValue;
}

}  // namespace psk
