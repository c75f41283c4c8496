// Symmetric feature set of the self-tensored sketch, and its in-register generator.
//
// phi'(x) = m (x) m has r^2 entries but only r(r+1)/2 distinct ones (m_a m_b = m_b m_a), so
// <phi'(q), phi'(k)> = sum_{a<=b} w_ab (q_a q_b)(k_a k_b) with w_ab = 2 for a < b and 1 on the
// diagonal: the same number the r^2-dimensional product of Algorithm 1 gives.  The kernels carry
// only the F = r(r+1)/2 features (a <= b).  States are built from UNWEIGHTED features
// m_a m_b; every consumer that contracts a state with freshly generated features uses the
// WEIGHTED ones w_ab m_a m_b (the factor 2 is exact in bf16).
//
// Feature order (chosen so that runs of consecutive features share `a`):
//   rows p = 0 .. r/2-2, r entries each: first (a = p, b = p+1 .. r-1), then
//                                        (a = r-2-p, b = r-1-p .. r-1);
//   then (a = r/2-1, b = r/2 .. r-1), r/2 entries;  then the diagonal (a, a), r entries.
#pragma once

#include "tc_prims.cuh"

namespace psk {
namespace tc {

template <int R>
struct Feat {
    static constexpr int F = R * (R + 1) / 2;        // distinct features
    static constexpr int FK = (F + 15) / 16 * 16;    // padded to the MMA K step
    static constexpr int NC = (F + 63) / 64;         // 64-feature chunks (A staging / state TMA boxes)
    static constexpr int NT = (F + 127) / 128;       // 128-feature tiles (state accumulators)
    static constexpr int FP = NT * 128;              // padded feature extent of stored states
    static constexpr int kPairRows = (R / 2 - 1) * R;

    __host__ __device__ static constexpr int a(int f) {
        if (f < kPairRows) {
            const int p = f / R, e = f % R;
            return (e < R - 1 - p) ? p : (R - 2 - p);
        }
        const int g = f - kPairRows;
        return (g < R / 2) ? (R / 2 - 1) : (g - R / 2);
    }
    __host__ __device__ static constexpr int b(int f) {
        if (f < kPairRows) {
            const int p = f / R, e = f % R;
            return (e < R - 1 - p) ? (p + 1 + e) : (R - 2 - p + 1 + (e - (R - 1 - p)));
        }
        const int g = f - kPairRows;
        return (g < R / 2) ? (R / 2 + g) : (g - R / 2);
    }
};

// The half sketch of one row as packed bf16 pairs, the generator's working set:
//   e[k] = (m[2k], m[2k+1])   even-aligned pairs,   o[k] = (m[2k+1], m[2k+2])   odd-aligned pairs.
// Consecutive features mostly share `a` and step `b` by one, so a pair of features is one
// packed multiply  (m_a, m_a) * (m_b, m_b+1); the product is rounded to bf16 once more, which
// the tolerance budget covers (relative 2^-9 each, independent across features).
template <int R>
struct PackedM {
    uint32_t e[R / 2], o[R / 2];
};

template <int R>
__device__ __forceinline__ void pack_half_sketch(const float (&m)[R], PackedM<R>& pm) {
#pragma unroll
    for (int k = 0; k < R / 2; ++k) {
        pm.e[k] = pack_bf16(m[2 * k], m[2 * k + 1]);
        pm.o[k] = pack_bf16(m[2 * k + 1], (2 * k + 2 < R) ? m[2 * k + 2] : 0.f);
    }
}

__device__ __forceinline__ uint32_t hmul2_bf16(uint32_t x, uint32_t y) {
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
    return r;
}

// (m_i, m_j) as a packed pair, from the even-aligned registers
template <int R, int I, int J>
__device__ __forceinline__ uint32_t pair_of(const PackedM<R>& pm) {
    constexpr uint32_t sel = (uint32_t)((I % 2) ? 0x32 : 0x10) | ((uint32_t)((J % 2) ? 0x76 : 0x54) << 8);
    return __byte_perm(pm.e[I / 2], pm.e[J / 2], sel);
}

// bf16x2 (feature F0, feature F0 + 1); F0 even.  WEIGHTED doubles the a < b features (exact).
template <int R, int F0, bool WEIGHTED>
__device__ __forceinline__ uint32_t feat_pair(const PackedM<R>& pm) {
    if constexpr (F0 >= Feat<R>::F) {
        return 0u;
    } else {
        static_assert(Feat<R>::F % 2 == 0 && F0 % 2 == 0, "features are generated in pairs");
        constexpr int A1 = Feat<R>::a(F0), B1 = Feat<R>::b(F0), A2 = Feat<R>::a(F0 + 1), B2 = Feat<R>::b(F0 + 1);
        constexpr uint32_t kOne = 0x3F80u, kTwo = 0x4000u;       // bf16 1.0, 2.0
        constexpr uint32_t w = ((WEIGHTED && A1 != B1) ? kTwo : kOne) | (((WEIGHTED && A2 != B2) ? kTwo : kOne) << 16);
        uint32_t x, y;
        if constexpr (A1 == A2 && B2 == B1 + 1) {
            x = pair_of<R, A1, A1>(pm);                           // (m_a, m_a): shared by the whole run
            y = (B1 % 2 == 0) ? pm.e[B1 / 2] : pm.o[B1 / 2];
        } else {
            x = pair_of<R, A1, A2>(pm);
            y = pair_of<R, B1, B2>(pm);
        }
        if constexpr (w != (kOne | (kOne << 16))) x = hmul2_bf16(x, w);   // per run, not per pair
        return hmul2_bf16(x, y);
    }
}

template <int R, int F0, bool WEIGHTED, int J, int N>
struct FeatPack {
    static __device__ __forceinline__ void run(const PackedM<R>& pm, uint32_t (&out)[N]) {
        out[J] = feat_pair<R, F0 + 2 * J, WEIGHTED>(pm);
        FeatPack<R, F0, WEIGHTED, J + 1, N>::run(pm, out);
    }
};
template <int R, int F0, bool WEIGHTED, int N>
struct FeatPack<R, F0, WEIGHTED, N, N> {
    static __device__ __forceinline__ void run(const PackedM<R>&, uint32_t (&)[N]) {}
};

// out[j] = bf16x2(feature F0+2j, feature F0+2j+1), j < N  (2N consecutive features)
template <int R, int F0, bool WEIGHTED, int N>
__device__ __forceinline__ void gen_features(const PackedM<R>& pm, uint32_t (&out)[N]) {
    FeatPack<R, F0, WEIGHTED, 0, N>::run(pm, out);
}

}  // namespace tc
}  // namespace psk
