// Device helpers shared by the tensor-core kernels (forward and backward translation units).
#pragma once

#include "psk_internal.cuh"
#include "tc_features.cuh"

#include <type_traits>

namespace psk {

typedef __nv_bfloat16 bf16;

// host: tensor maps (defined in psk_tc.cu)
// [B,H,n,64] bf16 rows, box 128 rows x 64 columns, 128-byte swizzle
bool tc_map_rows(CUtensorMap* m, const void* base, int B, int H, int n, int64_t sb, int64_t sh, int64_t sn);
// states S[nblk][80][FP] bf16, box 80 rows x 64 features
bool tc_map_states(CUtensorMap* m, const void* base, int FP, int64_t nblk);
// row-major [rows][cols] bf16 matrix, box box_rows x 64 columns
bool tc_map_2d(CUtensorMap* m, const void* base, int cols, int64_t rows, int box_rows);
// contiguous [outer][rows][cols] bf16, box box_rows x box_cols
bool tc_map_3d(CUtensorMap* m, const void* base, int cols, int64_t rows, int64_t outer, int box_cols, int box_rows);
// per-block states of every head + prefix (reverse = false) or suffix (reverse = true) scan
// center_mode 0: states as they are; 1: values centred by the per-head vector cmean
// (columns < 64 become H[:, c] - cmean[c] H[:, 64]); 2: last column becomes H[:, 64] - H[:, :64] cmean.
// `tot`: scratch of tc_state_total_bytes(d) bytes for the segment totals (may be null when that is 0).
// Non-causal (d.noncausal): one state per head, the sum over the whole sequence, stored as block 0.
cudaError_t tc_states(const Dims& d, const CUtensorMap& mX, const CUtensorMap& mY, const uint8_t* gimg,
                      const float* y65, const float* fscale, const float* cmean, int center_mode, bf16* S, bool reverse,
                      float* tot, int* status, cudaStream_t s, int* launches);
// runs a head's blocks are cut into by the state kernel (1 = one CTA group walks the whole head)
int tc_state_segments(const Dims& d);
size_t tc_state_total_bytes(const Dims& d);
// the backward's recomputation of the forward rows: writes y65, e65h (see tc_fwd_out_kernel)
// (mQraw, and mK = the raw key rows: only with a given half sketch and exact same-block weights)
cudaError_t tc_recompute(const Dims& d, const CUtensorMap& mQ, const CUtensorMap& mQraw, const CUtensorMap& mK, const CUtensorMap& mV,
                         const CUtensorMap& mZ, const uint8_t* gimg, const float* cmean, const float* denom,
                         const bf16* dO, float* y65, float* e65h, int* status, cudaStream_t s, int* launches);
// gimg[g] = [G1 | G2]^T of sketch-matrix set g as the shared-memory image of the sketch GEMM's B operand
// (2r rows x 128 B, K-major, 128-byte swizzle): the kernels fetch it with one bulk copy
// (d.sketch_linear: the image of [I | 0] or [I; I | 0] instead, G1 and G2 are not read)
cudaError_t tc_gimage(const Dims& d, const void* G1, const void* G2, uint8_t* gimg, cudaStream_t s, int* launches);
// cmean[bh][c] = mean over the n rows of V[bh][:, c]  (deterministic reduction)
cudaError_t tc_vmean(const Dims& d, const void* V, float* cmean, cudaStream_t s, int* launches);

// Scratch layout of the tensor-core path.
struct TcWorkspace { size_t status, vmean, gimg, tot, Z, Rst, y65, e65h, Oc, total; };

template <int R>
inline TcWorkspace tc_ws(const Dims& d, bool backward) {
    TcWorkspace w{};
    const size_t st = (size_t)d.BH() * (d.noncausal ? 1 : d.t) * tc::Feat<R>::FP * 80 * sizeof(bf16);
    const size_t rows = (size_t)d.BH() * d.n;
    size_t off = 0;
    w.status = off; off += kStatusBytes;
    w.vmean = off; off += align_up((size_t)d.BH() * 64 * sizeof(float));
    w.gimg = off; off += align_up((size_t)d.g_heads * 2 * R * 128);
    w.tot = off; off += align_up(tc_state_total_bytes(d));
    w.Z = off; off += align_up(st);
    if (backward) {
        w.Rst = off; off += align_up(st);
        w.y65 = off; off += align_up(rows * sizeof(float));
        w.e65h = off; off += align_up(rows * sizeof(float));
        if (d.keep_states) { w.Oc = off; off += align_up(rows * 64 * sizeof(bf16)); }   // forward's O - c
    }
    w.total = off;
    return w;
}

#define PSK_TRY(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return e_; } while (0)

template <typename Kern>
inline cudaError_t set_smem(Kern k, size_t bytes) {
    return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

namespace tc {

template <int I, int N, typename Fn>
__device__ __forceinline__ void static_for(Fn&& f) {
    if constexpr (I < N) {
        f(std::integral_constant<int, I>{});
        static_for<I + 1, N>(f);
    }
}

constexpr int kErrTma = 1, kErrMma = 2;

// barrier among the 128 row threads (warps 0-3) of a kernel whose fifth warp issues the MMAs;
// only where every row thread is certain to arrive (never inside a loop a failed wait can leave)
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) {
    return p + ((1024u - (smem_u32(p) & 1023u)) & 1023u);
}

// [G1 | G2]^T as a K-major, 128-byte-swizzled tile: row n (< 2R) holds sketch column n over the 64
// head dimensions.  B operand of the sketch GEMM X [G1 | G2]; built once per call by
// tc_gimage_kernel, then copied into shared memory as it is.
template <int R>
struct GImage { static constexpr uint32_t bytes = 2 * R * 128; };

// Sketch GEMM D[128 tokens x 2R] = X_tile [G1 | G2], 4 K steps of 16 over the head dimension.
template <int R>
__device__ __forceinline__ void issue_sketch(uint32_t d_tmem, const uint8_t* sX, const uint8_t* sG) {
    constexpr uint32_t idesc = idesc_bf16(128, 2 * R, false, false);
#pragma unroll
    for (int k = 0; k < 4; ++k)
        umma_ss(d_tmem, desc_off(smem_desc(smem_u32(sX), 0, 1024, kSwz128), k * 32),
                desc_off(smem_desc(smem_u32(sG), 0, 1024, kSwz128), k * 32), idesc, k > 0);
}

// m[c] = A1[c] A2[c] / sqrt(R) from the sketch accumulator (this thread's lane).
// (`scale`: an extra factor on every entry, folded into the constant)
// `linear`: the half sketch is given, not formed here: the "rows to sketch" are the half sketch
// itself (degree 2: m = x), or its two bf16 terms side by side ([hi | lo]), and the first half of the
// sketch GEMM against an identity-like matrix ([I], [I; I]) just carries it into tensor memory in
// fp32: m[c] = A1[c].
template <int R>
__device__ __forceinline__ void read_half_sketch(uint32_t lane_tmem, float (&m)[R], float scale = 1.f, bool linear = false) {
    const float rs = linear ? scale : rsqrtf((float)R) * scale;
#pragma unroll
    for (int c0 = 0; c0 < R; c0 += 16) {
        uint32_t a1[16], a2[16];
        tmem_ld16(lane_tmem + c0, a1);
        tmem_ld16(lane_tmem + R + c0, a2);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) m[c0 + j] = __uint_as_float(a1[j]) * (linear ? 1.f : __uint_as_float(a2[j])) * rs;
    }
}

// Split of an fp32 half-sketch entry into two bf16 terms, m = hi + lo (+ O(2^-17) |m|).  Scores
// s = m(q).m(k) are formed as hi.hi + hi.lo + lo.hi by one GEMM over 3R columns, the own rows laid
// out as [hi | hi | lo] and the other rows as [hi | lo | hi]; a score is a cancelling sum, so
// rounding m to a single bf16 would cost several percent on rows with few keys.
template <int R, bool OWN>
__device__ __forceinline__ float split_col(const float (&m)[R], int col) {
    const int sec = col / R, c = col % R;
    const float hi = __bfloat162float(__float2bfloat16_rn(m[c]));
    const bool want_lo = OWN ? (sec == 2) : (sec == 1);
    return want_lo ? (m[c] - hi) : hi;
}

// Rows of the 3R-column split operand, K-major and un-swizzled: 8x8 core matrices,
// [k chunk][row/8][row%8][16 B] (K-direction stride 2048 B, 8-row-group stride 128 B).
template <int R, bool OWN>
__device__ __forceinline__ void store_split_rows(uint8_t* dst, const float (&m)[R], int row) {
#pragma unroll
    for (int kc = 0; kc < 3 * R / 8; ++kc) {
        uint4 v;
        v.x = pack_bf16(split_col<R, OWN>(m, kc * 8 + 0), split_col<R, OWN>(m, kc * 8 + 1));
        v.y = pack_bf16(split_col<R, OWN>(m, kc * 8 + 2), split_col<R, OWN>(m, kc * 8 + 3));
        v.z = pack_bf16(split_col<R, OWN>(m, kc * 8 + 4), split_col<R, OWN>(m, kc * 8 + 5));
        v.w = pack_bf16(split_col<R, OWN>(m, kc * 8 + 6), split_col<R, OWN>(m, kc * 8 + 7));
        *reinterpret_cast<uint4*>(dst + kc * 2048 + (row / 8) * 128 + (row % 8) * 16) = v;
    }
}

// The split half sketch as [hi | lo] columns (2R of them) in ceil(2R/64) tiles of
// [128 rows x 128 B], 128-byte-swizzled, zero beyond 2R.  Tile 0 starts with the R `hi` columns,
// so it doubles as the MN-major B operand (N = 64, columns >= R ignored) of the dM GEMMs.
template <int R>
struct HiLoTiles { static constexpr int N = (2 * R + 63) / 64; };

template <int R>
__device__ __forceinline__ void store_hilo_tiles(uint8_t* dst, const float (&m)[R], int row) {
#pragma unroll
    for (int ch = 0; ch < HiLoTiles<R>::N * 8; ++ch) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (ch * 8 < 2 * R) {
            float x[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int col = ch * 8 + j, c = col % R;
                const float hi = __bfloat162float(__float2bfloat16_rn(m[c]));
                x[j] = col < R ? hi : (m[c] - hi);
            }
            v.x = pack_bf16(x[0], x[1]); v.y = pack_bf16(x[2], x[3]);
            v.z = pack_bf16(x[4], x[5]); v.w = pack_bf16(x[6], x[7]);
        }
        *reinterpret_cast<uint4*>(dst + (ch / 8) * 16384 + swz128_offset(row, ch % 8)) = v;
    }
}

}  // namespace tc
}  // namespace psk
