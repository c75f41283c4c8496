// Prefix states of the block lower-triangular multiply (Section 3.1) on the tensor cores.
//
// State storage (HBM scratch): S[BH][t][FP][80] bf16, one 160-byte row per feature: the 64
// columns of H_l / Z_l, then the normaliser column (the "| 1" of [V | 1], or the last column of E
// in the backward), then zeros.
//
// Sequence runs (the parallel-prefix remark of Section 3.1): with nseg > 1 a head's blocks are cut
// into nseg runs that are processed by different CTAs.  A first launch (kModeTotal) accumulates
// every run but the last from zero and leaves its raw fp32 total in scratch; the second
// (kModePrefix, use_init) starts run s from the sum of the totals of the runs before s and writes
// the prefix states as usual.  Twice the arithmetic, nseg times the parallelism: used when there
// are too few heads to fill the GPU.  The totals pass alone, followed by a small summing kernel,
// gives the single global state of non-causal attention.
#include "tc_common.cuh"

namespace psk {

using namespace tc;

namespace {

constexpr int kModePrefix = 0;         // write the exclusive prefix state at every block boundary
constexpr int kModeTotal = 1;          // write only the raw fp32 total at the end of the run

// ---------------------------------------------------------------------------
// Prefix states of one head, sequentially along the sequence (Section 3.1, Z_l = sum_{j<l} H_j):
//   S[l] = sum over blocks before l (after l when `reverse`) of phi(X_blk)^T [Y_blk | y65]
// for feature tiles [T0, T0+TN).  The running sum never leaves tensor memory (fp32); at every
// block boundary it is rounded to bf16 and written out, then the block's own contribution is
// accumulated on top -- the per-block states H_l and the scan over them are fused away.
//   X: tensor that is sketched (K for the forward state, Q for the backward's reverse state)
//   Y: [V] or [dO];  y65: last column (nullptr = all ones);  fscale: per-token d_i, the
//   features of token i are divided by it (nullptr = not) -- phi(q_i)^T [dO_i | y65_i] / d_i is the
//   suffix state's phi(q_i)^T E_i without E ever being formed
// grid (BH).  Warp roles:
//   NWG generator warpgroups  thread = token: read the half sketches, write their feature tiles
//                             (dealt round-robin) as MN-major A operands into shared memory;
//   1 store warpgroup         thread = feature row: at block boundaries reads the accumulators,
//                             centres, rounds and stores them;
//   1 feeder warp             one thread issues every TMA load, sketch GEMM and state GEMM.
// Stored layout S[blk][FP][80]: one row per feature, 64 state columns, the last column, zeros.
// ---------------------------------------------------------------------------
template <int R, int NWG>
struct StateSmem {
    static constexpr uint32_t X = 0;                     // 2 x 16 KB: rows to sketch
    static constexpr uint32_t Y = 32768;                 // 2 x (16 KB values + 16 KB last-column chunk)
    static constexpr uint32_t kYSlot = 32768;
    static constexpr uint32_t G = Y + 2 * kYSlot;
    static constexpr uint32_t A0 = G + (2 * R * 128 < 1024 ? 1024 : 2 * R * 128);
    static constexpr uint32_t St = A0 + NWG * 32768;     // one state tile on its way out: 128 rows x 160 B
    static constexpr bool kStaged = St + 128 * 160 + 2048 <= 232448;     // where it fits (r <= 32)
    static constexpr uint32_t total = St + (kStaged ? 128 * 160 : 0);
};

// Barrier among the 128 threads of a warpgroup.  The generator and store roles never leave a
// loop early: a wait that gave up returns at once from then on (tc_prims.cuh), so they run the
// remaining iterations through, barriers and arrivals included, and nobody is left waiting at a
// barrier that has lost a participant.
__device__ __forceinline__ void wg_barrier(int wg) {
    asm volatile("bar.sync %0, 128;" ::"r"(wg + 1) : "memory");
}

constexpr int kErrState = 3;

// acc[0..80) of this thread's lane = sum over runs s2 < seg of tot[(row0 + s2 * run_stride) * 80 + ...]
static __device__ __noinline__ void state_init_acc(const float* __restrict__ tot, size_t row0, size_t run_stride, int seg,
                                                   uint32_t acc_tmem) {
#pragma unroll 1
    for (int c0 = 0; c0 < 80; c0 += 16) {
        float a[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) a[q] = 0.f;
        for (int s2 = 0; s2 < seg; ++s2) {
            const float4* src = reinterpret_cast<const float4*>(tot + (row0 + s2 * run_stride) * 80 + c0);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float4 x = src[q];
                a[4 * q] += x.x; a[4 * q + 1] += x.y; a[4 * q + 2] += x.z; a[4 * q + 3] += x.w;
            }
        }
        uint32_t v[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) v[q] = __float_as_uint(a[q]);
        tmem_st16(acc_tmem + c0, v);
    }
}

// SEG = false is the plain walk of a whole head by one CTA (nseg = 1, prefix mode, no start value):
// its run bookkeeping folds away at compile time.
template <int R, int T0, int TN, int NWG, bool SEG>
__global__ void __launch_bounds__(128 * (NWG + 1) + 64)
tc_state_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                const uint8_t* __restrict__ gimg, int g_heads, int H, int n, int b, int t,
                const float* __restrict__ y65, const float* __restrict__ fscale, const float* __restrict__ cmean,
                int center_mode, int reverse, int nseg_arg, int mode_arg, int use_init, float* __restrict__ tot,
                bf16* __restrict__ S, int lin, int* status) {
    using F = Feat<R>;
    using L = StateSmem<R, NWG>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align1024(smem_raw);
    __shared__ uint64_t bar_fullx[2], bar_fully[2], bar_yfree[2], bar_ext[2], bar_sk, bar_mread, bar_drain[2];
    __shared__ uint64_t bar_aready[NWG], bar_afree[NWG], bar_accfull[TN], bar_accread[TN];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(16) float cm[64];
    const int tid = threadIdx.x, wg = tid / 128, wt = tid % 128, warp = tid / 32;
    const int bh = blockIdx.x;
    const int seg = SEG ? (int)blockIdx.y : 0, nseg = SEG ? nseg_arg : 1, mode = SEG ? mode_arg : kModePrefix;
    const int hi = bh % H, bi = bh / H;
    const int g = g_heads == 1 ? 0 : hi;
    const int tpb = b / 128, NJ = n / 128;               // token tiles per block / per head
    const int NJs = NJ / nseg, ts = t / nseg;            // token tiles / blocks of this CTA's run of the sequence
    // a later run of a prefix pass starts from the sum of the earlier runs' totals
    const bool init = SEG && (mode == kModePrefix) && use_init && seg > 0;
    constexpr int kThreads = 128 * (NWG + 1) + 64;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bar_fullx[i], 1); mbar_init(&bar_fully[i], 1); mbar_init(&bar_yfree[i], 1);
            mbar_init(&bar_ext[i], 1);
        }
        mbar_init(&bar_sk, 1); mbar_init(&bar_mread, NWG); mbar_init(&bar_drain[0], 1); mbar_init(&bar_drain[1], 1);
        for (int i = 0; i < NWG; ++i) { mbar_init(&bar_aready[i], 1); mbar_init(&bar_afree[i], 1); }
        for (int i = 0; i < TN; ++i) { mbar_init(&bar_accread[i], 4); mbar_init(&bar_accfull[i], 1); }
        cta_giveup_init();
        mbar_fence_init();
        tma_prefetch_desc(&mapX); tma_prefetch_desc(&mapY);
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    if (tid < 64) cm[tid] = cmean != nullptr ? cmean[(size_t)bh * 64 + tid] : 0.f;
    // last-column chunks of both slots: zero, and column 0 = 1 when the last column is all ones
    for (int e = tid; e < 2 * 1024; e += kThreads) {
        const int s = e / 1024, i = e % 1024;
        reinterpret_cast<uint4*>(smem + L::Y + s * L::kYSlot + 16384)[i] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    if (y65 == nullptr && tid < 128) {
        *reinterpret_cast<bf16*>(smem + L::Y + 16384 + swz128_offset(tid, 0)) = __float2bfloat16_rn(1.f);
        *reinterpret_cast<bf16*>(smem + L::Y + L::kYSlot + 16384 + swz128_offset(tid, 0)) = __float2bfloat16_rn(1.f);
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_slot;
    constexpr uint32_t kAcc = 2 * R;                      // accumulators start after the sketch columns
    // token tile visited at step j of this run (runs and tiles go backwards for suffix sums)
    auto tile_of = [&](int j) { const int gj = seg * NJs + j; return reverse ? (NJ - 1 - gj) : gj; };

    if (wg == NWG + 1) {
        // =============================== feeders ===============================
        // Two issuing threads in two warps.  The first loads the tiles and issues the sketch
        // GEMMs, the second issues the state GEMMs: between two of its MMAs lies as little as
        // possible (each satisfied wait, commit or TMA issue costs a single thread about a
        // hundred cycles, during which the tensor pipe would idle).
        if (tid == 128 * (NWG + 1)) {
            bool ok = true;
            auto load_x = [&](int j) {
                // the first tile's barrier also covers the sketch matrices' image
                mbar_expect_tx(&bar_fullx[j & 1], 16384 + (j == 0 ? GImage<R>::bytes : 0u));
                if (j == 0) bulk_load(smem + L::G, gimg + (size_t)g * GImage<R>::bytes, GImage<R>::bytes, &bar_fullx[0]);
                tma_load_4d(smem + L::X + (j & 1) * 16384, &mapX, 0, tile_of(j) * 128, hi, bi, &bar_fullx[j & 1]);
            };
            auto load_y = [&](int j) {
                mbar_expect_tx(&bar_fully[j & 1], 16384);
                tma_load_4d(smem + L::Y + (j & 1) * L::kYSlot, &mapY, 0, tile_of(j) * 128, hi, bi, &bar_fully[j & 1]);
            };
            load_x(0);
            if (NJs > 1) load_x(1);
            load_y(0);
            ok = mbar_wait(&bar_fullx[0], 0, status, kErrTma);
            tc_fence_after();
            issue_sketch<R>(tm, smem + L::X, smem + L::G);
            umma_commit(&bar_sk);
            for (int j = 0; j + 1 < NJs && ok; ++j) {
                // sketch of the next token tile, as soon as this tile's half sketches are read out
                ok = mbar_wait(&bar_mread, j & 1, status, kErrState);
                ok = ok && mbar_wait(&bar_fullx[(j + 1) & 1], ((j + 1) >> 1) & 1, status, kErrTma);
                tc_fence_after();
                issue_sketch<R>(tm, smem + L::X + ((j + 1) & 1) * 16384, smem + L::G);
                umma_commit(&bar_sk);
                if (j + 2 < NJs) load_x(j + 2);           // its slot: sketch j has completed (it was read)
                // values of the next token tile: their slot held tile j-1
                if (j >= 1) ok = ok && mbar_wait(&bar_yfree[(j + 1) & 1], ((j - 1) >> 1) & 1, status, kErrState);
                load_y(j + 1);
            }
            // drain: every sketch GEMM has completed before tensor memory is released.  (A barrier
            // of its own: completing bar_sk once more, right behind the last sketch, could flip it
            // twice before a generator thread has looked.)
            umma_commit(&bar_drain[0]);
            mbar_wait(&bar_drain[0], 0, status, kErrMma);
        } else if (tid == 128 * (NWG + 1) + 32) {
            constexpr uint32_t idesc_state = idesc_bf16(128, 80, true, true);
            bool ok = true;
            uint32_t a_cnt[NWG];
#pragma unroll
            for (int i = 0; i < NWG; ++i) a_cnt[i] = 0;
            uint64_t ad[NWG];
#pragma unroll
            for (int i = 0; i < NWG; ++i) ad[i] = smem_desc(smem_u32(smem + L::A0 + i * 32768), 16384, 1024, kSwz128);
            const uint64_t yd0 = smem_desc(smem_u32(smem + L::Y), 16384, 1024, kSwz128);
            const int ibase = init ? 0 : 1;               // completions of bar_accread before block 1's
            for (int j = 0; j < NJs && ok; ++j) {
                ok = mbar_spin(&bar_fully[j & 1], (j >> 1) & 1, status, kErrTma);
                if (y65 != nullptr) ok = ok && mbar_spin(&bar_ext[j & 1], (j >> 1) & 1, status, kErrState);
                // block boundary: the store warpgroup has taken (or, for a start from earlier runs,
                // written) the accumulators' values before anything is added to them
                const bool boundary = mode == kModePrefix && (j % tpb == 0) && (j > 0 || init);
                const bool block_end = mode == kModePrefix ? ((j + 1) % tpb == 0) : (j == NJs - 1);
                const uint64_t yd = desc_off(yd0, (j & 1) * L::kYSlot);
                const uint32_t acc0 = (j > 0 || init) ? 1u : 0u;
                static_for<0, TN>([&](auto ic) {
                    constexpr int I = decltype(ic)::value;
                    constexpr int w = I % NWG;
                    // the store warpgroup has taken this accumulator's values for the boundary
                    if (boundary) ok = ok && mbar_spin(&bar_accread[I], ((j / tpb) - ibase) & 1, status, kErrState);
                    ok = ok && mbar_spin(&bar_aready[w], a_cnt[w] & 1, status, kErrState);
                    ++a_cnt[w];
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        umma_ss(tm + kAcc + 80 * I, desc_off(ad[w], k * 2048), desc_off(yd, k * 2048), idesc_state, k > 0 ? 1u : acc0);
                    umma_commit(&bar_afree[w]);
                    // last token tile of a block: this accumulator is complete, and the store
                    // warpgroup may take it while the remaining tiles are still being issued
                    if (block_end) umma_commit(&bar_accfull[I]);
                });
                umma_commit(&bar_yfree[j & 1]);
            }
            // drain: every state GEMM has completed before tensor memory is released
            umma_commit(&bar_drain[1]);
            mbar_wait(&bar_drain[1], 0, status, kErrMma);
        }
    } else if (wg == NWG) {
        // ============================ store warpgroup ============================
        // Tiles leave through shared memory: a warp's 32 rows of 160 B are one contiguous 5 KB
        // piece of the state array, which the warp writes out in ten 512-byte rows of lanes.
        // (Rows stored by their threads directly would be 10 scattered 16-byte stores each: the L1
        // data path, which the MMA operands and the generators' tiles also go through, is this
        // kernel's busiest unit.)
        const uint32_t lane_tm = tm + ((uint32_t)((warp % 4) * 32) << 16);
        uint8_t* stage = smem + L::St;
        if (mode == kModeTotal) {
            // totals: the raw fp32 accumulators at the end of the run
            static_for<0, TN>([&](auto ic) {
                constexpr int I = decltype(ic)::value;
                mbar_wait(&bar_accfull[I], 0, status, kErrMma);
                tc_fence_after();
                float4* out = reinterpret_cast<float4*>(tot + ((((size_t)bh * nseg + seg) * F::NT + (T0 + I)) * 128 + wt) * 80);
                {
#pragma unroll
                    for (int c0 = 0; c0 < 80; c0 += 16) {
                        uint32_t v[16];
                        tmem_ld16(lane_tm + kAcc + 80 * I + c0, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            out[c0 / 4 + q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                          __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                    }
                }
            });
        }
        if (init) {
            // a later run starts from the sum of the earlier runs' totals: into the accumulators
            // first, then block 0 of the run is read back like every other block
            for (int I = 0; I < TN; ++I) state_init_acc(tot, (((size_t)bh * nseg) * F::NT + (T0 + I)) * 128 + wt,
                                                        (size_t)F::NT * 128, seg, lane_tm + kAcc + 80 * I);
            tmem_st_wait();
        }
        for (int p = 0; p < ts && mode == kModePrefix; ++p) {
            const int pg = seg * ts + p;
            const int l = reverse ? (t - 1 - pg) : pg;
            static_for<0, TN>([&](auto ic) {
                constexpr int I = decltype(ic)::value;
                if (p > 0) {
                    mbar_wait(&bar_accfull[I], (p - 1) & 1, status, kErrMma);
                    tc_fence_after();
                }
                const bool live = p > 0 || init;          // the accumulator holds values (else: zeros)
                // 16 accumulator columns (zeros before the first block of a head)
                auto fetch = [&](int c0, uint32_t (&v)[16]) {
                    if (live) {
                        tmem_ld16(lane_tm + kAcc + 80 * I + c0, v);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int q = 0; q < 16; ++q) v[q] = 0u;
                    }
                };
                // centred values, in fp32, without touching the operands (the mode only selects
                // coefficients):  mode 1: sum phi (y - c)^T = H[:, :64] - H[:, 64] c^T
                //                 mode 2: last column H[:, 64] - H[:, :64] c
                float last, corr = 0.f;
                {
                    uint32_t v[16];
                    fetch(64, v);
                    last = __uint_as_float(v[0]);
                }
                const float k1 = center_mode == 1 ? -last : 0.f, k2 = center_mode == 2 ? 1.f : 0.f;
                // the row's pair weight (tc_features.cuh) goes into the stored state; 0 on padding rows
                const float wgt = F::weight((T0 + I) * 128 + wt);
                // this thread's feature row: 80 bf16 = ten 16-byte pieces of the staging tile
                if constexpr (L::kStaged) __syncwarp();       // the previous tile has been read back
                uint4* const grow = reinterpret_cast<uint4*>(S + (((size_t)bh * t + l) * F::FP + (size_t)(T0 + I) * 128 + wt) * 80);
                uint4* dst = L::kStaged ? reinterpret_cast<uint4*>(stage + wt * 160) : grow;
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 16) {
                    uint32_t v[16];
                    fetch(c0, v);
                    if (c0 == 48 && live) {      // last read of this accumulator: hand it (back) to the MMAs
                        tc_fence_before();
                        if (wt % 32 == 0) mbar_arrive(&bar_accread[I]);
                    }
                    uint32_t pk[8];
                    float cv[16];
#pragma unroll
                    for (int q = 0; q < 16; q += 4) {
                        const float4 c4 = *reinterpret_cast<const float4*>(&cm[c0 + q]);
                        cv[q] = c4.x; cv[q + 1] = c4.y; cv[q + 2] = c4.z; cv[q + 3] = c4.w;
                    }
#pragma unroll
                    for (int q = 0; q < 16; q += 2) {
                        const float x0 = fmaf(k1, cv[q], __uint_as_float(v[q]));
                        const float x1 = fmaf(k1, cv[q + 1], __uint_as_float(v[q + 1]));
                        corr = fmaf(k2 * cv[q], x0, corr);
                        corr = fmaf(k2 * cv[q + 1], x1, corr);
                        pk[q / 2] = pack_bf16(x0 * wgt, x1 * wgt);
                    }
                    dst[c0 / 8] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    dst[c0 / 8 + 1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
                dst[8] = make_uint4(pack_bf16((last - corr) * wgt, 0.f), 0, 0, 0);
                dst[9] = make_uint4(0, 0, 0, 0);
                if constexpr (L::kStaged) {
                    __syncwarp();
                    const int w32 = wt & ~31, lane = wt & 31;
                    const uint4* src = reinterpret_cast<const uint4*>(stage + w32 * 160);
                    uint4* out = reinterpret_cast<uint4*>(S + (((size_t)bh * t + l) * F::FP + (size_t)(T0 + I) * 128 + w32) * 80);
#pragma unroll
                    for (int i = 0; i < 10; ++i) out[i * 32 + lane] = src[i * 32 + lane];
                }
            });
        }
    } else {
        // ============================= generators =============================
        const uint32_t lane_tm = tm + ((uint32_t)((warp % 4) * 32) << 16);
        uint8_t* sA = smem + L::A0 + wg * 32768;
        uint32_t a_uses = 0;                              // times this warpgroup's buffer has been filled
        // last-column entry of this thread's token, requested one token tile ahead of its use
        float y_next = (y65 != nullptr && wg == 0) ? y65[(size_t)bh * n + tile_of(0) * 128 + wt] : 0.f;
        float d_next = fscale != nullptr ? fscale[(size_t)bh * n + tile_of(0) * 128 + wt] : 1.f;
        for (int j = 0; j < NJs; ++j) {
            mbar_wait(&bar_sk, j & 1, status, kErrMma);
            tc_fence_after();
            PackedM<R> pm;
            CircGen<R> gen;
            {
                float m[R];
                // features m_a m_b / d: both factors carry 1 / sqrt(d) (d requested a token tile ago)
                const float sc = rsqrtf(d_next);
                if (fscale != nullptr && j + 1 < NJs) d_next = fscale[(size_t)bh * n + tile_of(j + 1) * 128 + wt];
                read_half_sketch<R>(lane_tm, m, sc, lin != 0);
                if constexpr (F::kCirc) gen.init(m); else pack_half_sketch<R>(m, pm);
            }
            tc_fence_before();
            wg_barrier(wg);
            if (wt == 0) mbar_arrive(&bar_mread);
            if (y65 != nullptr && wg == 0) {
                // last-column chunk of this token tile; its slot is free once tile j-2's MMAs are done
                if (j >= 2) mbar_wait(&bar_yfree[j & 1], ((j >> 1) - 1) & 1, status, kErrState);
                const float y = y_next;
                if (j + 1 < NJs) y_next = y65[(size_t)bh * n + tile_of(j + 1) * 128 + wt];
                *reinterpret_cast<bf16*>(smem + L::Y + (j & 1) * L::kYSlot + 16384 + swz128_offset(wt, 0)) =
                    __float2bfloat16_rn(y);
                fence_proxy_async_smem();
                wg_barrier(0);
                if (wt == 0) mbar_arrive(&bar_ext[j & 1]);
            }
            if constexpr (F::kCirc) {
                // this warpgroup's tiles wg, wg + NWG, ...: the same loop body on a rotated copy of m
                static_assert(T0 == 0, "circulant order: one launch covers every tile");
                constexpr int kTileSteps = 128 / (2 * R);
                for (int i = 0; i < wg; ++i) gen.template skip<kTileSteps>();
#pragma unroll 1
                for (int I = wg; I < TN; I += NWG) {
                    if (a_uses > 0) mbar_wait(&bar_afree[wg], (a_uses - 1) & 1, status, kErrMma);
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t pk[32];
                        gen.chunk(pk);
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            *reinterpret_cast<uint4*>(sA + half * 16384 + swz128_offset(wt, c)) =
                                make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                    }
                    fence_proxy_async_smem();
                    wg_barrier(wg);
                    if (wt == 0) mbar_arrive(&bar_aready[wg]);
                    ++a_uses;
                    gen.template skip<(NWG - 1) * kTileSteps>();
                }
            } else {
                static_for<0, TN>([&](auto ic) {
                    constexpr int I = decltype(ic)::value;
                    if (I % NWG == wg) {
                        if (a_uses > 0) mbar_wait(&bar_afree[wg], (a_uses - 1) & 1, status, kErrMma);
                        static_for<0, 16>([&](auto cc) {
                            constexpr int C = decltype(cc)::value;
                            uint32_t pk[4];
                            gen_features<R, (T0 + I) * 128 + C * 8, 4>(pm, pk);
                            *reinterpret_cast<uint4*>(sA + (C / 8) * 16384 + swz128_offset(wt, C % 8)) =
                                make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        });
                        fence_proxy_async_smem();
                        wg_barrier(wg);
                        if (wt == 0) mbar_arrive(&bar_aready[wg]);
                        ++a_uses;
                    }
                });
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}


// Sum of the run totals of a head, centred, weighted and rounded like a stored state: the single
// global state of non-causal attention, written as the head's only block.
template <int R>
__global__ void __launch_bounds__(128)
tc_state_sum_kernel(const float* __restrict__ tot, int nseg, const float* __restrict__ cmean, int center_mode,
                    bf16* __restrict__ S) {
    using F = Feat<R>;
    const int tile = blockIdx.x, bh = blockIdx.y, wt = threadIdx.x;
    const int row = tile * 128 + wt;
    float v[80];
#pragma unroll
    for (int c = 0; c < 80; ++c) v[c] = 0.f;
    for (int s = 0; s < nseg; ++s) {
        const float4* src = reinterpret_cast<const float4*>(tot + ((((size_t)bh * nseg + s) * F::NT + tile) * 128 + wt) * 80);
#pragma unroll
        for (int c = 0; c < 20; ++c) {
            const float4 x = src[c];
            v[4 * c] += x.x; v[4 * c + 1] += x.y; v[4 * c + 2] += x.z; v[4 * c + 3] += x.w;
        }
    }
    const float wgt = F::weight(row);
    const float last = v[64];
    float corr = 0.f;
    uint32_t pk[40];
#pragma unroll
    for (int c = 0; c < 64; c += 2) {
        const float c0 = cmean != nullptr ? cmean[(size_t)bh * 64 + c] : 0.f;
        const float c1 = cmean != nullptr ? cmean[(size_t)bh * 64 + c + 1] : 0.f;
        const float x0 = center_mode == 1 ? v[c] - last * c0 : v[c];
        const float x1 = center_mode == 1 ? v[c + 1] - last * c1 : v[c + 1];
        if (center_mode == 2) corr += c0 * x0 + c1 * x1;
        pk[c / 2] = pack_bf16(x0 * wgt, x1 * wgt);
    }
    pk[32] = pack_bf16((last - corr) * wgt, 0.f);
#pragma unroll
    for (int c = 33; c < 40; ++c) pk[c] = 0u;
    uint4* out = reinterpret_cast<uint4*>(S + ((size_t)bh * F::FP + row) * 80);
#pragma unroll
    for (int c = 0; c < 10; ++c) out[c] = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
}

// ---------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------
struct StateArgs {
    const float *y65, *fscale, *cmean;
    int center_mode;
    bool reverse;
    int nseg, mode, segs_launched;
    bool use_init;
    float* tot;
    bf16* S;
};

template <int R, int T0, int TN, int NWG>
cudaError_t launch_state_group(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const uint8_t* gimg,
                               const StateArgs& a, int* status, cudaStream_t s, int* launches) {
    constexpr size_t smem = StateSmem<R, NWG>::total + 1024;
    prof_begin(a.mode == kModeTotal ? "tc_state_total_kernel" : "tc_state_kernel", s);
    if (a.nseg == 1 && a.mode == kModePrefix) {
        PSK_TRY((set_smem(tc_state_kernel<R, T0, TN, NWG, false>, smem)));
        tc_state_kernel<R, T0, TN, NWG, false><<<dim3(d.BH(), 1), 128 * (NWG + 1) + 64, smem, s>>>(
            mX, mY, gimg, d.g_heads, d.H, d.n, d.b, d.t, a.y65, a.fscale, a.cmean, a.center_mode, a.reverse ? 1 : 0, 1,
            kModePrefix, 0, a.tot, a.S, d.sketch_linear ? 1 : 0, status);
    } else {
        PSK_TRY((set_smem(tc_state_kernel<R, T0, TN, NWG, true>, smem)));
        tc_state_kernel<R, T0, TN, NWG, true><<<dim3(d.BH(), a.segs_launched), 128 * (NWG + 1) + 64, smem, s>>>(
            mX, mY, gimg, d.g_heads, d.H, d.n, d.b, d.t, a.y65, a.fscale, a.cmean, a.center_mode, a.reverse ? 1 : 0, a.nseg,
            a.mode, a.use_init ? 1 : 0, a.tot, a.S, d.sketch_linear ? 1 : 0, status);
    }
    prof_end(s);
    ++*launches;
    return cudaGetLastError();
}

template <int R>
cudaError_t launch_states(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const uint8_t* gimg,
                          const StateArgs& a, int* status, cudaStream_t s, int* launches) {
#define PSK_SG(T0, TN, NWG) PSK_TRY((launch_state_group<R, T0, TN, NWG>(d, mX, mY, gimg, a, status, s, launches)))
    if constexpr (R == 16) {
        PSK_SG(0, 2, 2);
    } else if constexpr (R == 32) {
        PSK_SG(0, 5, 3);
    } else {
        PSK_SG(0, 4, 3); PSK_SG(4, 4, 3); PSK_SG(8, 3, 3); PSK_SG(11, 3, 3); PSK_SG(14, 3, 3);
    }
#undef PSK_SG
    return cudaSuccess;
}

template <int R>
cudaError_t states_impl(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const uint8_t* gimg, const float* y65,
                        const float* fscale, const float* cmean, int center_mode, bf16* S, bool reverse, float* tot,
                        int* status, cudaStream_t s, int* launches) {
    const int nseg = tc_state_segments(d);
    StateArgs a{y65, fscale, cmean, center_mode, reverse, nseg, kModePrefix, nseg, nseg > 1, tot, S};
    if (d.noncausal) {
        // one global state per head: totals of every run, then their sum in the stored format
        a.mode = kModeTotal; a.use_init = false; a.cmean = nullptr; a.center_mode = 0;
        PSK_TRY((launch_states<R>(d, mX, mY, gimg, a, status, s, launches)));
        prof_begin("tc_state_sum_kernel", s);
        tc_state_sum_kernel<R><<<dim3(Feat<R>::NT, d.BH()), 128, 0, s>>>(tot, nseg, cmean, center_mode, S);
        prof_end(s);
        ++*launches;
        return cudaGetLastError();
    }
    if (nseg > 1) {    // totals of every run of blocks but the last (nothing starts after it)
        StateArgs b = a;
        b.mode = kModeTotal; b.segs_launched = nseg - 1; b.use_init = false; b.cmean = nullptr; b.center_mode = 0;
        PSK_TRY((launch_states<R>(d, mX, mY, gimg, b, status, s, launches)));
    }
    return launch_states<R>(d, mX, mY, gimg, a, status, s, launches);
}

}  // namespace

int tc_state_segments(const Dims& d) {
    // units a head's sequence can be cut into: blocks (a run starts at a block boundary), or
    // 128-token tiles when there are no blocks to respect
    const int units = d.noncausal ? d.n / 128 : d.t;
    if (d.seq_segments > 0) return (d.seq_segments <= units && units % d.seq_segments == 0) ? d.seq_segments : 1;
    constexpr long kSMs = 148;
    // Causal: two passes cost twice the arithmetic, so cutting pays from four runs on.
    // Non-causal: the totals pass is all there is, so any cut that fills the GPU pays.
    int s = 1;
    while ((long)d.BH() * s < kSMs && s * 2 <= units && units % (s * 2) == 0 && s < 32) s *= 2;
    if (!d.noncausal && s < 4) s = 1;
    return s;
}

size_t tc_state_total_bytes(const Dims& d) {
    const int nseg = tc_state_segments(d);
    if (nseg <= 1 && !d.noncausal) return 0;
    const size_t nt = d.r == 16 ? Feat<16>::NT : (d.r == 32 ? Feat<32>::NT : Feat<64>::NT);
    return (size_t)d.BH() * nseg * nt * 128 * 80 * sizeof(float);
}

cudaError_t tc_states(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const uint8_t* gimg,
                      const float* y65, const float* fscale, const float* cmean, int center_mode, bf16* S, bool reverse,
                      float* tot, int* status, cudaStream_t s, int* launches) {
    switch (d.r) {
        case 16: return states_impl<16>(d, mX, mY, gimg, y65, fscale, cmean, center_mode, S, reverse, tot, status, s, launches);
        case 32: return states_impl<32>(d, mX, mY, gimg, y65, fscale, cmean, center_mode, S, reverse, tot, status, s, launches);
        case 64: return states_impl<64>(d, mX, mY, gimg, y65, fscale, cmean, center_mode, S, reverse, tot, status, s, launches);
    }
    return cudaErrorInvalidValue;
}

}  // namespace psk
