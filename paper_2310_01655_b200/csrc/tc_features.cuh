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

// One feature from the half sketch held in registers; zero beyond F.
template <int R, int F0, bool WEIGHTED>
__device__ __forceinline__ float feat_value(const float (&m)[R]) {
    if constexpr (F0 >= Feat<R>::F) {
        return 0.f;
    } else {
        constexpr int A = Feat<R>::a(F0), B = Feat<R>::b(F0);
        const float v = m[A] * m[B];
        return (WEIGHTED && A != B) ? 2.f * v : v;
    }
}

template <int R, int F0, bool WEIGHTED, int J, int N>
struct FeatPack {
    static __device__ __forceinline__ void run(const float (&m)[R], uint32_t (&out)[N]) {
        out[J] = pack_bf16(feat_value<R, F0 + 2 * J, WEIGHTED>(m), feat_value<R, F0 + 2 * J + 1, WEIGHTED>(m));
        FeatPack<R, F0, WEIGHTED, J + 1, N>::run(m, out);
    }
};
template <int R, int F0, bool WEIGHTED, int N>
struct FeatPack<R, F0, WEIGHTED, N, N> {
    static __device__ __forceinline__ void run(const float (&)[R], uint32_t (&)[N]) {}
};

// out[j] = bf16x2(feature F0+2j, feature F0+2j+1), j < N  (2N consecutive features)
template <int R, int F0, bool WEIGHTED, int N>
__device__ __forceinline__ void gen_features(const float (&m)[R], uint32_t (&out)[N]) {
    FeatPack<R, F0, WEIGHTED, 0, N>::run(m, out);
}

}  // namespace tc
}  // namespace psk
