/*
 * psk.h -- C ABI of the causal polynomial-sketch ("Polysketch") attention library
 * for NVIDIA B200 (sm_100a).
 *
 * What the calls compute (PolySketchFormer, arXiv 2310.01655), per (batch, head):
 *   m(x)   = sqrt(1/r) * [(x G1) * (x G2)]              Section 2.2 / Algorithm 1, degree-2 level
 *   phi'(x) = m(x) (x) m(x)   (r^2 features)            Algorithm 1, PolySketchNonNegative, p = 4
 *   O      = D~^{-1} lt(phi'(Q) phi'(K)^T) V            Section 3
 *   D~     = diag(1 + lt(phi'(Q) phi'(K)^T) 1)          Section 3 (the "1 +" is part of it)
 * evaluated in time linear in n by the block lower-triangular multiply of
 * Section 3.1 (diagonal blocks of b rows directly through (L R^T)^2, everything
 * earlier through the prefix sum Z_l of per-block states H_l = phi'(K_l)^T [V_l | 1]).
 * lt() keeps j <= i (diagonal included).  The paper prints no backward pass; the
 * backward call returns the exact derivatives of the formulas above.
 *
 * Conventions
 *   - Every pointer argument marked DEVICE is device memory owned by the caller; the
 *     library allocates nothing and frees nothing.  Scratch space is the caller's
 *     `workspace` (size from psk_workspace_bytes, 256-byte aligned).
 *   - Tensors Q, K, V, O, dO, dQ, dK, dV are [B, H, n, h] with element strides
 *     (stride_b, stride_h, stride_n) and a contiguous last dimension; all eight share
 *     the strides in psk_shape.  G1, G2 are [g_heads, h, r] contiguous, g_heads = 1
 *     (one pair for all heads) or H (one pair per head); the same pair sketches Q and K.
 *   - Q and K are taken as already normalised (the paper applies LayerNorm first,
 *     Section 2.1); dQ and dK are gradients with respect to those inputs.  No
 *     gradient is produced for G1, G2 (random, untrained sketch).
 *   - `dtype` is the storage type of Q, K, V, G1, G2, O and all gradients.  PSK_F32
 *     computes in fp32 on the CUDA cores; PSK_BF16 computes on the tensor cores with
 *     bf16 operands and fp32 accumulation.  `denom` is always fp32.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work and return
 *     without synchronising.  Errors detectable on the host are returned before any
 *     launch and leave the outputs untouched.  A device-side bounded wait that gives
 *     up records a code in the workspace; psk_check() reads it.
 *   - Supported: p = 4, h = 64, r in {16, 32, 64}, b a multiple of 128, n a multiple
 *     of b (Section 3.1 assumes b = n / t).  Anything else: PSK_ERR_UNSUPPORTED or
 *     PSK_ERR_SHAPE.
 *   - Also p = 2 (Algorithm 1 with p/2 = 1): no sketch, m(x) = x, phi'(x) = x (x) x with
 *     h^2 entries, i.e. exact degree-2 polynomial attention with weights (q_i . k_j)^2.
 *     Set r = h; G1 and G2 are not read and may be null.  bf16 storage runs on the tensor
 *     cores (the same kernels, with the rows taken as their own half sketch), fp32 storage on
 *     the CUDA cores.
 *   - Also p = 8 (one more level of Algorithm 1's recursion): two independent degree-2
 *     sketches M1 = sqrt(1/r)[(x Ga1)*(x Ga2)], M2 = sqrt(1/r)[(x Gb1)*(x Gb2)] combined as
 *     m(x) = sqrt(1/r)[(M1 Gc1)*(M2 Gc2)] with Gc1, Gc2 of r x r; phi'(x) = m (x) m as for p = 4,
 *     so the weights approximate (q_i . k_j)^8.  G1 then holds [Ga1; Gb1; Gc1] and G2 holds
 *     [Ga2; Gb2; Gc2], each [g_heads, 2h + r, r] contiguous.  Not with PSK_FLAG_LOCAL_EXACT
 *     (PSK_ERR_UNSUPPORTED).  fp32 storage and r = 64: CUDA-core kernels.  bf16 storage with
 *     r <= 32: the half sketches and the attention on them run on the tensor cores
 *     (PSK_PATH_CUDA_CORES forces the CUDA-core kernels throughout).
 */
#ifndef PSK_H_
#define PSK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PSK_OK = 0,
    PSK_ERR_INVALID_ARG = -1,   /* null pointer, bad enum value                      */
    PSK_ERR_UNSUPPORTED = -2,   /* p not 4, 8 (or 2 with r = h), h != 64, r not in {16,32,64}, bad path */
    PSK_ERR_SHAPE = -3,         /* n % b != 0, b % 128 != 0, non-positive extents    */
    PSK_ERR_ALIGN = -4,         /* pointer or stride not 16-byte aligned             */
    PSK_ERR_WORKSPACE = -5,     /* workspace missing, misaligned or too small        */
    PSK_ERR_CUDA = -6,          /* a CUDA runtime call or launch failed              */
    PSK_ERR_TIMEOUT = -7        /* a bounded device-side wait gave up (psk_check)    */
} psk_status;

typedef enum { PSK_F32 = 0, PSK_BF16 = 1 } psk_dtype;

/* Which implementation runs.  PSK_PATH_AUTO picks by dtype (fp32 -> CUDA cores,
 * bf16 -> tensor cores).  PSK_PATH_CUDA_CORES forces the fp32-arithmetic kernels for
 * either storage type (used to cross-check the tensor-core path). */
typedef enum { PSK_PATH_AUTO = 0, PSK_PATH_CUDA_CORES = 1, PSK_PATH_TENSOR_CORES = 2 } psk_path;

typedef struct {
    int32_t B, H, n, h, r, p, b;
    int32_t dtype;              /* psk_dtype */
    int64_t stride_b, stride_h, stride_n;   /* elements; last dimension contiguous */
    int32_t g_heads;            /* 1 or H */
    int32_t path;               /* psk_path */
    int32_t flags;              /* bit set of psk_flags, 0 for none */
    int32_t seq_segments;       /* tensor-core path: runs of blocks a head's sequence is cut into for the
                                   prefix scan over block states (Section 3.1 notes that the prefix sums
                                   can be computed in parallel); 0 = the library chooses (1 unless there
                                   are too few heads to fill the GPU); must divide n / b */
} psk_shape;

/* PSK_FLAG_KEEP_STATES (tensor-core path; ignored by the CUDA-core path): set on BOTH the
 * forward and the backward call of one training step.  The forward then leaves in its
 * workspace the prefix states Z_l of Section 3.1, the per-head value centres c they are centred
 * by, and O - c (rounded after the subtraction: the caller's rounded O cannot supply it) - for
 * p = 8 and the learnable sketch also the half sketches of Q and K; the
 * backward, given the SAME workspace memory (not written in between) with the same shape and inputs, reads them instead
 * of rebuilding the states from K and V and recomputing the forward rows.  With the flag set
 * psk_workspace_bytes() returns the backward's size for both calls.  Without the flag each
 * call is self-contained.
 *
 * PSK_FLAG_LOCAL_EXACT: "applying exact attention locally" (Section 3.2).  Pairs (i, j) of the
 * same block of b rows get the exact polynomial weight (q_i . k_j)^4 instead of the sketched
 * (m(q_i) . m(k_j))^2, i.e. P_l = lt((Q_l K_l^T)^4) [V_l | 1]; pairs in different blocks are
 * unchanged.  The result now depends on b (more exact pairs with larger blocks; b = n is exact
 * degree-4 polynomial attention).  Set it on the forward and on the backward call alike; the
 * backward sends the same-block part of dQ, dK straight to Q and K instead of through the
 * sketch.  Both paths serve it (bf16 storage: tensor-core kernels, scores from the raw bf16
 * rows with fp32 accumulation; fp32 storage: CUDA-core kernels), and it combines with
 * PSK_FLAG_KEEP_STATES.
 *
 * PSK_FLAG_NONCAUSAL: Polysketch attention without the causal mask (Section 3, first formula):
 *   O = D~^{-1} phi'(Q) phi'(K)^T V,   D~ = diag(1 + phi'(Q) phi'(K)^T 1),
 * evaluated in time linear in n through ONE state phi'(K)^T [V | 1] per head (the sum over the whole
 * sequence) instead of per-block prefix sums; the backward uses that state and the single state
 * phi'(Q)^T E.  b still sets the launch granularity (a multiple of 128 dividing n) but no longer
 * changes the result.  Set it on the forward and on the backward call alike.  Tensor-core path only
 * (bf16 storage, p = 4), not with PSK_FLAG_LOCAL_EXACT: otherwise PSK_ERR_UNSUPPORTED.  Combines
 * with PSK_FLAG_KEEP_STATES. */
typedef enum { PSK_FLAG_KEEP_STATES = 1, PSK_FLAG_LOCAL_EXACT = 2, PSK_FLAG_NONCAUSAL = 4 } psk_flags;

/* Library version (major*100 + minor). */
int psk_version(void);

/* Static, NUL-terminated description of a status code. */
const char* psk_status_string(int status);

/* Bytes of caller-provided scratch the forward (for_backward = 0) or the backward
 * (for_backward = 1) needs for this shape; 0 if the shape is invalid.  Section 3.1:
 * the scratch holds the per-block states H_l / prefix sums Z_l and the half sketches. */
size_t psk_workspace_bytes(const psk_shape* shape, int for_backward);

/* Half sketch and, optionally, the self-tensored features (Algorithm 1).
 *   X        DEVICE [B,H,n,h] storage dtype, strides from `shape`
 *   G1, G2   DEVICE [g_heads,h,r] storage dtype
 *   M_out    DEVICE [B,H,n,r] fp32 contiguous: m(x)
 *   Phi_out  DEVICE [B,H,n,r*r] fp32 contiguous or NULL: phi'(x)[a*r+b] = m_a m_b
 * (row-major Kronecker order of Section 1.2).  Phi_out is meant for tests on small
 * shapes; the attention calls never materialise it in HBM. */
int psk_sketch(const psk_shape* shape, const void* X, const void* G1, const void* G2,
               float* M_out, float* Phi_out, void* stream);

/* Causal Polysketch attention forward (Section 3 through Section 3.1).
 *   Q, K, V  DEVICE inputs; O DEVICE output [B,H,n,h] storage dtype
 *   denom    DEVICE [B,H,n] fp32 or NULL: d_i = 1 + sum_{j<=i} <phi'(q_i), phi'(k_j)>
 *   workspace DEVICE scratch, >= psk_workspace_bytes(shape, 0), 256-byte aligned */
int psk_causal_attn_fwd(const psk_shape* shape, const void* Q, const void* K, const void* V,
                        const void* G1, const void* G2, void* O, float* denom,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Backward of psk_causal_attn_fwd: given dO = dL/dO, writes dQ, dK, dV (storage dtype).
 * O and denom are the forward's outputs (both required).  Derived from Section 3's
 * formula; evaluated with a forward prefix of key states and a reverse prefix of
 * query states in the manner of Section 3.1.
 *   workspace DEVICE scratch, >= psk_workspace_bytes(shape, 1) */
int psk_causal_attn_bwd(const psk_shape* shape, const void* Q, const void* K, const void* V,
                        const void* G1, const void* G2, const void* O, const float* denom,
                        const void* dO, void* dQ, void* dK, void* dV,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Forward pass for callers that must not allocate device memory (no counterpart in the
 * paper: it computes exactly what psk_causal_attn_fwd computes).  Think of a plug-in that
 * runs inside a host application which has already handed the whole GPU to its own
 * memory pool, a real-time loop that may not call the allocator, or code that is not
 * allowed to touch cudaMalloc at all: none of them can size and allocate a workspace.
 * Here the scratch is a fixed array of psk_static_scratch_bytes() bytes (16 MiB) that
 * lives inside the library image; every GPU that loads the library holds it until the
 * process exits.  The caller passes inputs and outputs only.
 *   - Always runs the CUDA-core (fp32 arithmetic) kernels, for either storage type.
 *   - Shapes whose forward scratch (psk_workspace_bytes with path = PSK_PATH_CUDA_CORES)
 *     exceeds the array are refused with PSK_ERR_WORKSPACE before any launch.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.  The address is kept for the life
 *     of the process: do not call cudaDeviceReset on a device between calls.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - All calls on a device share the one array and it keeps the previous call's bytes;
 *     the call zeroes the part that must start at zero.  Two calls that overlap on the
 *     GPU (different streams, or different threads) race on it: serialise them.
 * Arguments and error codes otherwise as psk_causal_attn_fwd. */
size_t psk_static_scratch_bytes(void);
int psk_causal_attn_fwd_static(const psk_shape* shape, const void* Q, const void* K, const void* V,
                               const void* G1, const void* G2, void* O, float* denom, void* stream);

/* Learnable sketches (Algorithm 2 in the appendix, "Replacing Random Projections with Learnable
 * Transformations"; Section 3's paragraph on learnable sketches).  The products x G1 and x G2 of
 * the degree-2 level become f1(x) and f2(x) for two dense networks of equal structure and separate
 * parameters, and the half sketch is
 *     m(x) = sqrt(r) tanh( sqrt(1/r) [ f1(x) * f2(x) ] ),          |m| <= sqrt(r);
 * features m (x) m, the block algorithm and everything else are as for the random sketch.
 * Each network: layer normalisation of the input, dense h -> 8r, gelu, layer normalisation, dense
 * 8r -> r, dense r -> 8r, gelu, dense 8r -> r (output dimension r, hidden layers [8r, r, 8r], gelu after
 * the first and the third, normalisation before the input and before the second hidden layer).
 * Where the paper is silent this library takes: dense layers with biases, normalisations with a
 * learnable gain and bias and eps = 1e-6, gelu(x) = x Phi(x), one pair of networks for all heads.
 *   params   DEVICE fp32 [2][psk_learned_param_count(h, r)]: network 1 then network 2, each packed as
 *            g0[h] c0[h] | W1[h][8r] b1[8r] | g1[8r] c1[8r] | W2[8r][r] b2[r] | W3[r][8r] b3[8r] | W4[8r][r] b4[r]
 *            (gain, bias of a normalisation; row-major weight [in][out], bias of a dense layer)
 *   dparams  DEVICE fp32, same layout: dL/dparams, overwritten by psk_learned_attn_bwd (summed over
 *            the batch, the heads and both uses of the networks, on Q and on K; accumulated with
 *            floating-point atomics, so its last bits are not reproducible from run to run)
 * The other arguments, the workspace rules and the error codes are those of psk_sketch,
 * psk_causal_attn_fwd and psk_causal_attn_bwd; `shape` needs p = 4, g_heads is ignored,
 * PSK_FLAG_LOCAL_EXACT is honoured (the paper's "learned + local" variant), PSK_FLAG_NONCAUSAL is
 * not supported here.  For bf16 storage with r <= 32 (sketched or exact same-block weights) everything
 * runs on the tensor cores: the networks' dense layers (forward with hi + lo pairs of bf16 operands, so
 * the half sketch keeps 2^-17; backward and weight gradients with single bf16 operands) and the
 * attention on their half sketches (`path` = PSK_PATH_CUDA_CORES forces the CUDA-core kernels,
 * PSK_PATH_TENSOR_CORES refuses what the tensor-core route does not serve).  Everything else, and
 * psk_learned_sketch itself, runs on the CUDA cores in fp32.  On the tensor-core route the rows pass
 * through the networks' layers 2^20 at a time (the activations of one such pass are part of the
 * workspace); the environment variable PSK_LEARNED_CHUNK_ROWS (a multiple of 128) overrides that
 * number, provided it does not change between the workspace query and the calls that use it.  Workspace size from
 * psk_learned_workspace_bytes. */
size_t psk_learned_param_count(int h, int r);
size_t psk_learned_workspace_bytes(const psk_shape* shape, int for_backward);
int psk_learned_sketch(const psk_shape* shape, const void* X, const float* params, float* M_out, float* Phi_out,
                       void* stream);
int psk_learned_attn_fwd(const psk_shape* shape, const void* Q, const void* K, const void* V, const float* params,
                         void* O, float* denom, void* workspace, size_t workspace_bytes, void* stream);
int psk_learned_attn_bwd(const psk_shape* shape, const void* Q, const void* K, const void* V, const float* params,
                         const void* O, const float* denom, const void* dO, void* dQ, void* dK, void* dV,
                         float* dparams, void* workspace, size_t workspace_bytes, void* stream);

/* Block lower-triangular multiplication for arbitrary feature matrices (Section 3.1):
 *   Out = lt(A B^T) C,   A, B: [batch, n, m],  C, Out: [batch, n, k],  all fp32, contiguous, DEVICE,
 * computed as  H_l = B_l^T C_l,  Z_l = sum_{j<l} H_j,  rows of block l = lt(A_l B_l^T) C_l + A_l Z_l
 * over blocks of b rows: O(n b (m + k) + n m k) instead of O(n^2 (m + k)).  The attention
 * calls above are this algorithm with A = phi'(Q), B = phi'(K), C = [V | 1] and the features
 * generated on the fly; this call takes any feature matrices (the paper uses it for other
 * feature maps too).  CUDA-core kernels, fp32 arithmetic.  Needs b % 32 == 0, n % b == 0,
 * 1 <= k <= 128 (else PSK_ERR_SHAPE); `workspace` (DEVICE) of at least
 * psk_lt_multiply_workspace_bytes() bytes (0 for a bad shape) holds the t = n / b states
 * of every batch entry.  Enqueues on `stream` and returns. */
size_t psk_lt_multiply_workspace_bytes(int batch, int n, int m, int k, int b);
int psk_lt_multiply(int batch, int n, int m, int k, int b, const float* A, const float* B, const float* C,
                    float* Out, void* workspace, size_t workspace_bytes, void* stream);

/* The same block algorithm (Section 3.1) on the tensor cores for bf16 feature matrices:
 *   Out = lt(A B^T) C,   A, B: [batch, n, m] bf16,  C: [batch, n, 64] bf16,  Out: [batch, n, 64] fp32,
 * all contiguous, DEVICE, 16-byte aligned.  Products of bf16 entries are exact and summed in fp32; the
 * prefix states Z_l and the masked same-block scores are rounded to bf16 once (relative 2^-9)
 * before they are multiplied, as in the attention calls.  Needs m % 64 == 0, k == 64, b = 128 or 256,
 * n % b == 0 (else PSK_ERR_SHAPE).  `workspace` (DEVICE, 256-byte aligned) of at least
 * psk_lt_multiply_bf16_workspace_bytes() bytes (0 for a bad shape): a status word for psk_check,
 * then the t = n / b prefix states of every batch entry.  Enqueues on `stream` and returns. */
size_t psk_lt_multiply_bf16_workspace_bytes(int batch, int n, int m, int k, int b);
int psk_lt_multiply_bf16(int batch, int n, int m, int k, int b, const void* A, const void* B, const void* C,
                         float* Out, void* workspace, size_t workspace_bytes, void* stream);

/* Recurrent form: one new token per (batch, head) per call (inference at O(r^2 h) per token,
 * whatever the context length).  With the running state S (r^2 x 65 per head, fp32)
 *   S <- S + phi'(k_t) [v_t | 1]^T,   N = phi'(q_t)^T S,   d = 1 + N[64],   o_t = N[:64] / d,
 * which is row t of psk_causal_attn_fwd (without PSK_FLAG_LOCAL_EXACT) when the calls are made
 * for t = 0, 1, ... on a state that started as zeros.  q, k, v, o: [B, H, h] contiguous DEVICE
 * arrays of the shape's dtype; G1, G2 as for the other calls; `state`: DEVICE array of
 * psk_decode_state_bytes(shape) bytes, [B*H][r*r][65] fp32, rows in the Kronecker order
 * a*r + b, owned and zero-initialised by the caller, updated in place; `denom` ([B, H] fp32,
 * DEVICE) may be null.  Of the shape only B, H, h, r, p (= 4), dtype, g_heads are read;
 * flags must be 0.  CUDA-core kernel; one pass over the state per call. */
size_t psk_decode_state_bytes(const psk_shape* shape);
int psk_decode_step(const psk_shape* shape, const void* q, const void* k, const void* v, const void* G1,
                    const void* G2, float* state, void* o, float* denom, void* stream);

/* Synchronises `stream`, then reports PSK_ERR_TIMEOUT if a kernel of the last call that
 * used `workspace` abandoned a bounded wait, PSK_ERR_CUDA if the stream is in error,
 * else PSK_OK.  Never traps. */
int psk_check(const void* workspace, void* stream);

/* Self-test of the bounded device-side wait (no counterpart in the paper).  Every wait inside the
 * tensor-core kernels (on a TMA load, an MMA, another warp) is bounded by wall time: a wait that
 * is not satisfied within about one second records a code in the workspace's status word and
 * returns, after which the rest of that thread block runs through without waiting again, so a lost
 * signal costs about a second and can never hang the GPU.  This call exercises exactly that path:
 * it enqueues one small kernel whose 128 threads wait, through the same code with the limit
 * `limit_ns` (1 .. 100 000 000), on a barrier that nobody completes.  Afterwards
 * psk_check(workspace, stream) returns PSK_ERR_TIMEOUT, and four uint64 values at byte offset 64
 * of the workspace (DEVICE) report: nanoseconds the first wait took, nanoseconds a second wait on
 * the same barrier took (it must return at once), and the number of threads whose first / second
 * wait reported failure (128 each).  The next regular call on the workspace clears the status
 * word.  `workspace`: DEVICE, at least 256 bytes, 256-byte aligned. */
int psk_selftest_wait_timeout(void* workspace, size_t workspace_bytes, uint64_t limit_ns, void* stream);

/* Number of kernel launches the last forward / backward call on this thread enqueued
 * (for launch accounting in benchmarks). */
int psk_last_launch_count(void);

/* Measurement aid (no counterpart in the paper).  psk_profile_enable(1) makes every
 * later kernel launch of the library be bracketed by a pair of CUDA events on the launch
 * stream and discards earlier records; psk_profile_enable(0) stops recording and frees
 * them.  psk_profile_count() is the number of launches recorded so far;
 * psk_profile_get(i, name, cap, &ms) waits for launch i to finish and returns its kernel
 * name (HOST buffer, NUL-terminated, truncated to cap) and device duration in ms.
 * Process-wide state; not thread-safe. */
int psk_profile_enable(int enable);
int psk_profile_count(void);
int psk_profile_get(int index, char* name, size_t name_cap, float* ms);

/* Diagnostic, host only (no GPU needed): the feature order of the tensor-core path.
 * Section 2.2's self-tensored sketch phi'(x) = m (x) m has one distinct entry per unordered pair
 * {a, b} of half-sketch coordinates; the tensor-core kernels store one feature per pair (some
 * pairs twice, some padding rows) and weight the rows of their states so that every pair {a, b}
 * carries total weight 2 for a != b and 1 for a == b.  For r in {16, 32, 64} this writes, for
 * stored feature f < count, a[f], b[f] (feature f is m_a m_b) and w[f] (the weight of state row
 * f; 0 for padding) into HOST arrays of capacity `cap` each and returns the number of stored
 * features; PSK_ERR_UNSUPPORTED for another r, PSK_ERR_INVALID_ARG for a null pointer,
 * PSK_ERR_WORKSPACE if cap is too small. */
int psk_feature_table(int r, int* a, int* b, float* w, int cap);

#ifdef __cplusplus
}
#endif
#endif /* PSK_H_ */
