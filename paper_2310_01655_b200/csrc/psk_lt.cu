// lt(A B^T) C for arbitrary feature matrices by the block algorithm of Section 3.1:
//   H_l = B_l^T C_l,  Z_l = sum_{j<l} H_j,  rows of block l = lt(A_l B_l^T) C_l + A_l Z_l.
// The attention kernels specialise this to A = phi'(Q), B = phi'(K), C = [V | 1] with the
// features generated on the fly; this entry point takes the feature matrices as given (the
// paper applies the same algorithm to other feature maps, Section 4).  fp32 on the CUDA cores.
#include "psk_internal.cuh"

namespace psk {
namespace {

constexpr int kTile = 32;          // rows per tile, features per chunk
constexpr int kColGroups = 8;      // a thread owns the columns c = cx, cx + 8, ...
constexpr int kMaxCols = 16;       // ... at most 16 of them: k <= 128

// H_l[f, c] = sum_{i in block l} B[i, f] C[i, c].  grid (ceil(m/32), t, batch), block (32, 8).
__global__ void __launch_bounds__(256)
lt_state_kernel(const float* __restrict__ B, const float* __restrict__ C, int n, int m, int k, int b, int t,
                float* __restrict__ S) {
    extern __shared__ float smem[];
    float* sB = smem;                       // [32 rows][33]
    float* sC = sB + kTile * 33;            // [32 rows][k]
    const int fx = threadIdx.x, cy = threadIdx.y, tid = cy * 32 + fx;
    const int f0 = blockIdx.x * kTile, l = blockIdx.y, bt = blockIdx.z;
    const size_t row0 = (size_t)bt * n + (size_t)l * b;
    float acc[kMaxCols];
#pragma unroll
    for (int q = 0; q < kMaxCols; ++q) acc[q] = 0.f;
    for (int i0 = 0; i0 < b; i0 += kTile) {
        __syncthreads();
        for (int e = tid; e < kTile * kTile; e += 256) {
            const int r = e / kTile, f = e % kTile;
            sB[r * 33 + f] = (f0 + f < m) ? B[(row0 + i0 + r) * m + f0 + f] : 0.f;
        }
        for (int e = tid; e < kTile * k; e += 256) sC[e] = C[(row0 + i0) * k + e];
        __syncthreads();
        for (int r = 0; r < kTile; ++r) {
            const float bf = sB[r * 33 + fx];
#pragma unroll
            for (int q = 0; q < kMaxCols; ++q) {
                const int c = cy + q * kColGroups;
                if (c < k) acc[q] = fmaf(bf, sC[r * k + c], acc[q]);
            }
        }
    }
    if (f0 + fx < m) {
        float* out = S + (((size_t)bt * t + l) * m + f0 + fx) * k;
#pragma unroll
        for (int q = 0; q < kMaxCols; ++q) {
            const int c = cy + q * kColGroups;
            if (c < k) out[c] = acc[q];
        }
    }
}

// Exclusive prefix over the t states of each batch entry, in place, sequential in l.
__global__ void __launch_bounds__(256)
lt_scan_kernel(float* __restrict__ S, size_t elems, int t) {
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= elems) return;
    float* p = S + (size_t)blockIdx.y * t * elems + e;
    float run = 0.f;
    for (int l = 0; l < t; ++l) { const float v = p[(size_t)l * elems]; p[(size_t)l * elems] = run; run += v; }
}

// Rows i0 .. i0+31 of block l:  A_l Z_l  +  sum over 32-row tiles j0 <= i0 of the block of
// lt-masked (A_tile B_tile^T) C_tile.  grid (b/32, t, batch), block (32 rows, 8 column groups).
__global__ void __launch_bounds__(256)
lt_out_kernel(const float* __restrict__ A, const float* __restrict__ B, const float* __restrict__ C,
              const float* __restrict__ Z, int n, int m, int k, int b, int t, float* __restrict__ Out) {
    extern __shared__ float smem[];
    float* sA = smem;                       // [32 rows][33]   chunk of 32 features
    float* sB = sA + kTile * 33;            // [32 rows][33]
    float* sS = sB + kTile * 33;            // [32][33]        scores of a tile pair
    float* sY = sS + kTile * 33;            // [32][k]         Z chunk or C tile
    const int ry = threadIdx.x, cx = threadIdx.y, tid = cx * 32 + ry;
    const int i0 = blockIdx.x * kTile, l = blockIdx.y, bt = blockIdx.z;
    const size_t blk0 = (size_t)bt * n + (size_t)l * b;
    float acc[kMaxCols];
#pragma unroll
    for (int q = 0; q < kMaxCols; ++q) acc[q] = 0.f;
    // earlier blocks through the prefix state
    if (l > 0) {
        const float* Zl = Z + ((size_t)bt * t + l) * m * k;
        for (int f0 = 0; f0 < m; f0 += kTile) {
            __syncthreads();
            for (int e = tid; e < kTile * kTile; e += 256) {
                const int r = e / kTile, f = e % kTile;
                sA[r * 33 + f] = (f0 + f < m) ? A[(blk0 + i0 + r) * m + f0 + f] : 0.f;
            }
            for (int e = tid; e < kTile * k; e += 256) sY[e] = (f0 + e / k < m) ? Zl[(size_t)f0 * k + e] : 0.f;
            __syncthreads();
            for (int f = 0; f < kTile; ++f) {
                const float a = sA[ry * 33 + f];
#pragma unroll
                for (int q = 0; q < kMaxCols; ++q) {
                    const int c = cx + q * kColGroups;
                    if (c < k) acc[q] = fmaf(a, sY[f * k + c], acc[q]);
                }
            }
        }
    }
    // same block: tiles of 32 other rows up to and including this one
    for (int j0 = 0; j0 <= i0; j0 += kTile) {
        float sc[4] = {0.f, 0.f, 0.f, 0.f};          // scores of row ry against j = cx, cx+8, cx+16, cx+24
        for (int f0 = 0; f0 < m; f0 += kTile) {
            __syncthreads();
            for (int e = tid; e < kTile * kTile; e += 256) {
                const int r = e / kTile, f = e % kTile;
                const bool in = f0 + f < m;
                sA[r * 33 + f] = in ? A[(blk0 + i0 + r) * m + f0 + f] : 0.f;
                sB[r * 33 + f] = in ? B[(blk0 + j0 + r) * m + f0 + f] : 0.f;
            }
            __syncthreads();
            for (int f = 0; f < kTile; ++f) {
                const float a = sA[ry * 33 + f];
#pragma unroll
                for (int q = 0; q < 4; ++q) sc[q] = fmaf(a, sB[(cx + 8 * q) * 33 + f], sc[q]);
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = cx + 8 * q;
            sS[ry * 33 + j] = (j0 + j <= i0 + ry) ? sc[q] : 0.f;      // lt(): keep j <= i
        }
        for (int e = tid; e < kTile * k; e += 256) sY[e] = C[(blk0 + j0) * k + e];
        __syncthreads();
        for (int j = 0; j < kTile; ++j) {
            const float w = sS[ry * 33 + j];
#pragma unroll
            for (int q = 0; q < kMaxCols; ++q) {
                const int c = cx + q * kColGroups;
                if (c < k) acc[q] = fmaf(w, sY[j * k + c], acc[q]);
            }
        }
    }
    float* out = Out + (blk0 + i0 + ry) * k;
#pragma unroll
    for (int q = 0; q < kMaxCols; ++q) {
        const int c = cx + q * kColGroups;
        if (c < k) out[c] = acc[q];
    }
}

bool lt_args_ok(int batch, int n, int m, int k, int b) {
    return batch > 0 && n > 0 && m > 0 && k > 0 && k <= kColGroups * kMaxCols && b > 0 && b % kTile == 0 && n % b == 0 &&
           (int64_t)batch * n < ((int64_t)1 << 31);
}

}  // namespace
}  // namespace psk

using namespace psk;

extern "C" {

size_t psk_lt_multiply_workspace_bytes(int batch, int n, int m, int k, int b) {
    if (!lt_args_ok(batch, n, m, k, b)) return 0;
    return align_up((size_t)batch * (n / b) * m * k * sizeof(float));
}

int psk_lt_multiply(int batch, int n, int m, int k, int b, const float* A, const float* B, const float* C,
                    float* Out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!lt_args_ok(batch, n, m, k, b)) return PSK_ERR_SHAPE;
    if (!A || !B || !C || !Out) return PSK_ERR_INVALID_ARG;
    const size_t need = psk_lt_multiply_workspace_bytes(batch, n, m, k, b);
    if (!workspace || workspace_bytes < need) return PSK_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    float* S = static_cast<float*>(workspace);
    const int t = n / b;
    const dim3 block(32, kColGroups);
    const size_t smem_state = (size_t)(kTile * 33 + kTile * k) * sizeof(float);
    const size_t smem_out = (size_t)(3 * kTile * 33 + kTile * k) * sizeof(float);
    prof_begin("lt_state_kernel", s);
    lt_state_kernel<<<dim3((m + kTile - 1) / kTile, t, batch), block, smem_state, s>>>(B, C, n, m, k, b, t, S);
    prof_end(s);
    const size_t elems = (size_t)m * k;
    prof_begin("lt_scan_kernel", s);
    lt_scan_kernel<<<dim3((unsigned)((elems + 255) / 256), batch), 256, 0, s>>>(S, elems, t);
    prof_end(s);
    prof_begin("lt_out_kernel", s);
    lt_out_kernel<<<dim3(b / kTile, t, batch), block, smem_out, s>>>(A, B, C, S, n, m, k, b, t, Out);
    prof_end(s);
    return cudaGetLastError() == cudaSuccess ? PSK_OK : PSK_ERR_CUDA;
}

}  // extern "C"
