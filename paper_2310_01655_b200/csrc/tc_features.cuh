// Symmetric feature set of the self-tensored sketch, and its in-register generators.
//
// phi'(x) = m (x) m has r^2 entries but only r(r+1)/2 distinct ones (m_a m_b = m_b m_a), so
// <phi'(q), phi'(k)> = sum over unordered pairs of w_ab (q_a q_b)(k_a k_b) with w_ab = 2 for
// a != b and 1 on the diagonal: the same number the r^2-dimensional product of Algorithm 1 gives.
// The kernels carry one feature per unordered pair.  Every thread generates UNWEIGHTED products
// m_a m_b; the weights are applied once, to the rows of the stored states (Feat::weight), so
// every contraction of fresh features with a state, and every gradient that flows back through a
// state, already carries them.  With weighted gradients d(feature) the half-sketch gradient is
//   dm[a] += d(feature ab) m[b];   dm[b] += d(feature ab) m[a]        for every stored feature,
// the diagonal included (its two updates coincide, which is the factor 2 of d(m_a^2)).
//
// Two feature orders:
//
//  * circulant (r <= 32): feature (s, a) = m[a] m[(a + s) mod r] for shifts s = 0 .. r/2, stored
//    shift-major in steps of two shifts, f = j * 2r + (s - 2j) * r + a with j = s / 2, for
//    j = 0 .. r/4.  Shift r/2 lists every pair {a, a + r/2} twice, so its weight is 1; shift
//    r/2 + 1 only fills the last step and has weight 0.  Every step is the same code on a
//    rotated copy of m, so generation and its backward are LOOPS over steps: the kernels' code
//    stays small enough for the instruction cache, which is what bounds them otherwise.
//
//  * triangular (r = 64): pairs a <= b enumerated so that runs of consecutive features share
//    `a`; fully unrolled code, one specialised instruction sequence per feature.  (The loop form
//    needs four r-entry register arrays in the backward, which r = 64 does not have.)
//      rows p = 0 .. r/2-2, r entries each: first (a = p, b = p+1 .. r-1), then
//                                           (a = r-2-p, b = r-1-p .. r-1);
//      then (a = r/2-1, b = r/2 .. r-1), r/2 entries;  then the diagonal (a, a), r entries.
#pragma once

#include "tc_prims.cuh"

namespace psk {
namespace tc {

template <int R>
struct Feat {
    static constexpr bool kCirc = (R <= 32);
    static constexpr int kSteps = R / 4 + 1;                         // circulant: steps of two shifts
    static constexpr int F = kCirc ? kSteps * 2 * R : R * (R + 1) / 2;   // stored features
    static constexpr int FK = (F + 15) / 16 * 16;    // padded to the MMA K step
    static constexpr int NC = (F + 63) / 64;         // 64-feature chunks (A staging / state TMA boxes)
    static constexpr int NT = (F + 127) / 128;       // 128-feature tiles (state accumulators)
    static constexpr int FP = NT * 128;              // padded feature extent of stored states
    static constexpr int kPairRows = (R / 2 - 1) * R;

    // triangular order
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
    // weight of stored state row f (0 for padding rows)
    __host__ __device__ static float weight(int f) {
        if (f >= F) return 0.f;
        if (kCirc) {
            const int s = 2 * (f / (2 * R)) + ((f / R) & 1);
            return (s == 0 || s == R / 2) ? 1.f : (s > R / 2 ? 0.f : 2.f);
        }
        return a(f) == b(f) ? 1.f : 2.f;
    }
};

// The half sketch of one row as packed bf16 pairs, the generators' working set:
//   e[k] = (m[2k], m[2k+1])   even-aligned pairs,   o[k] = (m[2k+1], m[2k+2])   odd-aligned pairs
// (o wraps around: its last entry is (m[r-1], m[0]) -- the circulant order needs it, the
// triangular one never reads that half).  A packed multiply of two such pairs yields two
// features; the product is rounded to bf16 once more, which the tolerance budget covers
// (relative 2^-9 each, independent across features).
template <int R>
struct PackedM {
    uint32_t e[R / 2], o[R / 2];
};

template <int R>
__device__ __forceinline__ void pack_half_sketch(const float (&m)[R], PackedM<R>& pm) {
#pragma unroll
    for (int k = 0; k < R / 2; ++k) {
        pm.e[k] = pack_bf16(m[2 * k], m[2 * k + 1]);
        pm.o[k] = pack_bf16(m[2 * k + 1], m[(2 * k + 2) % R]);
    }
}

__device__ __forceinline__ uint32_t hmul2_bf16(uint32_t x, uint32_t y) {
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
    return r;
}

// ---------------------------------------------------------------------------
// circulant order: one step = shifts 2j and 2j+1 = 2r features = r packed words
// ---------------------------------------------------------------------------
// Holds e (fixed) and the copies of e and o rotated by the current step:
//   er[k] = e[(k + j) mod r/2] = (m[2k + 2j], m[2k + 2j + 1]),  orr[k] = o[(k + j) mod r/2].
template <int R>
struct CircGen {
    static constexpr int H = R / 2;
    uint32_t e[H], er[H], orr[H];

    __device__ __forceinline__ void init(const float (&m)[R]) {
#pragma unroll
        for (int k = 0; k < H; ++k) {
            e[k] = pack_bf16(m[2 * k], m[2 * k + 1]);
            er[k] = e[k];
            orr[k] = pack_bf16(m[2 * k + 1], m[(2 * k + 2) % R]);
        }
    }
    // advance by K steps without producing anything
    template <int K>
    __device__ __forceinline__ void skip() {
        uint32_t t[H], u[H];
#pragma unroll
        for (int k = 0; k < H; ++k) { t[k] = er[(k + K) % H]; u[k] = orr[(k + K) % H]; }
#pragma unroll
        for (int k = 0; k < H; ++k) { er[k] = t[k]; orr[k] = u[k]; }
    }
    // out[0 .. H) = features of shift 2j (a = 2k, 2k+1), out[H .. R) = shift 2j+1; then advance
    __device__ __forceinline__ void step(uint32_t* out) {
#pragma unroll
        for (int k = 0; k < H; ++k) {
            out[k] = hmul2_bf16(e[k], er[k]);
            out[H + k] = hmul2_bf16(e[k], orr[k]);
        }
        skip<1>();
    }
    // the next 64 features (32 packed words): 64 / 2r steps
    __device__ __forceinline__ void chunk(uint32_t (&out)[32]) {
        static_assert(R == 16 || R == 32, "circulant order: r = 16 or 32");
#pragma unroll
        for (int s = 0; s < 32 / R; ++s) step(out + s * R);
    }
};

// Backward of the circulant features: with x the (weighted) gradients of the features of one
// step, dm[a] += x m[(a + s) mod r] and dm[(a + s) mod r] += x m[a].  The second term is
// accumulated in the rotated frame (dr[a] collects dm[(a + 2j) mod r]) and folded back at the end.
template <int R>
struct CircUntensor {
    float mr[R], dr[R];

    __device__ __forceinline__ void init(const float (&m)[R]) {
#pragma unroll
        for (int a = 0; a < R; ++a) { mr[a] = m[a]; dr[a] = 0.f; }
    }
    // xe / xo: gradients of the features of shifts 2j / 2j+1 (fp32 bit patterns, a = 0 .. r-1)
    __device__ __forceinline__ void even(const uint32_t* xe, const float (&m)[R], float (&dm)[R]) {
#pragma unroll
        for (int a = 0; a < R; ++a) {
            const float v = __uint_as_float(xe[a]);
            dm[a] = fmaf(v, mr[a], dm[a]);
            dr[a] = fmaf(v, m[a], dr[a]);
        }
    }
    __device__ __forceinline__ void odd(const uint32_t* xo, const float (&m)[R], float (&dm)[R]) {
#pragma unroll
        for (int a = 0; a < R; ++a) {
            const float v = __uint_as_float(xo[a]);
            dm[a] = fmaf(v, mr[(a + 1) % R], dm[a]);
            dr[(a + 1) % R] = fmaf(v, m[a], dr[(a + 1) % R]);
        }
    }
    __device__ __forceinline__ void advance() {
        float t[R], u[R];
#pragma unroll
        for (int a = 0; a < R; ++a) { t[a] = mr[(a + 2) % R]; u[a] = dr[(a + 2) % R]; }
#pragma unroll
        for (int a = 0; a < R; ++a) { mr[a] = t[a]; dr[a] = u[a]; }
    }
    // after TOTAL steps: dr[a] belongs to dm[(a + 2 TOTAL) mod r]
    template <int TOTAL>
    __device__ __forceinline__ void finish(float (&dm)[R]) {
#pragma unroll
        for (int a = 0; a < R; ++a) dm[(a + 2 * TOTAL) % R] += dr[a];
    }
};

// ---------------------------------------------------------------------------
// triangular order: specialised code per feature pair
// ---------------------------------------------------------------------------
// (m_i, m_j) as a packed pair, from the even-aligned registers
template <int R, int I, int J>
__device__ __forceinline__ uint32_t pair_of(const PackedM<R>& pm) {
    constexpr uint32_t sel = (uint32_t)((I % 2) ? 0x32 : 0x10) | ((uint32_t)((J % 2) ? 0x76 : 0x54) << 8);
    return __byte_perm(pm.e[I / 2], pm.e[J / 2], sel);
}

// bf16x2 (feature F0, feature F0 + 1); F0 even
template <int R, int F0>
__device__ __forceinline__ uint32_t feat_pair(const PackedM<R>& pm) {
    if constexpr (F0 >= Feat<R>::F) {
        return 0u;
    } else {
        static_assert(Feat<R>::F % 2 == 0 && F0 % 2 == 0, "features are generated in pairs");
        constexpr int A1 = Feat<R>::a(F0), B1 = Feat<R>::b(F0), A2 = Feat<R>::a(F0 + 1), B2 = Feat<R>::b(F0 + 1);
        uint32_t x, y;
        if constexpr (A1 == A2 && B2 == B1 + 1) {
            x = pair_of<R, A1, A1>(pm);                           // (m_a, m_a): shared by the whole run
            y = (B1 % 2 == 0) ? pm.e[B1 / 2] : pm.o[B1 / 2];
        } else {
            x = pair_of<R, A1, A2>(pm);
            y = pair_of<R, B1, B2>(pm);
        }
        return hmul2_bf16(x, y);
    }
}

template <int R, int F0, int J, int N>
struct FeatPack {
    static __device__ __forceinline__ void run(const PackedM<R>& pm, uint32_t (&out)[N]) {
        out[J] = feat_pair<R, F0 + 2 * J>(pm);
        FeatPack<R, F0, J + 1, N>::run(pm, out);
    }
};
template <int R, int F0, int N>
struct FeatPack<R, F0, N, N> {
    static __device__ __forceinline__ void run(const PackedM<R>&, uint32_t (&)[N]) {}
};

// out[j] = bf16x2(feature F0+2j, feature F0+2j+1), j < N  (2N consecutive features)
template <int R, int F0, int N>
__device__ __forceinline__ void gen_features(const PackedM<R>& pm, uint32_t (&out)[N]) {
    FeatPack<R, F0, 0, N>::run(pm, out);
}

}  // namespace tc
}  // namespace psk
