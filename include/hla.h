/*
 * hla.h - C ABI of the B200 (sm_100a) Hadamard Linear Attention operator.
 *
 * The operator is the linear-time form of HLA (paper Section 4.2, Lemma 4.1 and
 * Theorem 4.2, the normaliser paragraph after it, Algorithm 1 steps 4-5 and the
 * 2-/3-factor einsum listings of the appendix):
 *
 *     q_i   = phi_q(Q_i),   k^f_j = phi_{k_f}(K_j),  f = 1..F      (Algorithm 1 step 4)
 *     T_k[j] = k^1_j (x) ... (x) k^F_j,   T_q[i] = q_i (x) ... (x) q_i     in R^P, P = d_phi^F
 *     C = sum_j T_k[j] v_j^T  (P x d),    z = sum_j T_k[j]               (state build)
 *     eta_i = T_q[i] . z,    o_i = (T_q[i]^T C) / (eta_i + eps)          (readout + normaliser)
 *
 * which equals row-normalising A = (.)_f phi_q(Q) phi_{k_f}(K)^T (Eq. "hla") and
 * multiplying by V.  The backward entry point returns the gradients of
 * sum(dO * O) with respect to the inputs.
 *
 * General rules
 *   - All tensor pointers are DEVICE pointers, contiguous, innermost dimension
 *     last, 16-byte aligned.  The caller owns every buffer, including the
 *     workspace and the phi weights; the library allocates no device memory and
 *     borrows pointers only for the work it enqueues.
 *   - hla_ctx is host memory owned by the library (hla_create / hla_destroy).
 *   - hla_forward / hla_backward only enqueue work on `cuda_stream` (a
 *     cudaStream_t passed as void*; NULL = default stream) and return without
 *     synchronising.  They never throw, abort or print: every failure is a
 *     return code, and arguments are validated before anything is launched.
 *   - Device-side waits are bounded; a wait that runs out makes the kernel
 *     record a code in the workspace and return.  hla_last_device_status reads it.
 *     Each wait gives up after two seconds, and the warps of a block that depend
 *     on one another give up one after the other, so a launch that has timed out
 *     can take several times two seconds to return.
 *   - One ctx must not be used from two host threads at once.
 */
#ifndef HLA_H_
#define HLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hla_ctx hla_ctx;

typedef enum {
    HLA_OK = 0,
    HLA_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, non-positive size, bad enum   */
    HLA_ERR_UNSUPPORTED = 2,   /* valid request outside the supported set (see hla_config)  */
    HLA_ERR_WORKSPACE = 3,     /* workspace smaller than hla_workspace_bytes()              */
    HLA_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                        */
    HLA_ERR_DEVICE_TIMEOUT = 5,/* a bounded device-side wait expired (results are invalid)  */
    HLA_ERR_NO_MEMORY = 6      /* host memory for the context could not be obtained          */
} hla_status;

typedef enum { HLA_BF16 = 0, HLA_F32 = 1 } hla_dtype;

typedef enum {
    HLA_PHI_MLP = 0, /* Q, K are raw per-head tensors [B,H,N,d]; the library applies phi_q, phi_k1..F  */
    HLA_PHI_NONE = 1 /* Q is q_phi [B,H,N,d_phi] fp32, K is k_phi [B,H,F,N,d_phi] fp32 (the listings'
                        signature: features are given, must be >= 0 for the normaliser to make sense) */
} hla_phi_mode;

/*
 * Problem statement.  V, O, dO, dV (and Q, K, dQ, dK in HLA_PHI_MLP mode) are
 * [B,H,N,d] in `dtype`.  Features (HLA_PHI_NONE inputs and their gradients) are
 * always fp32.  Supported set: F in {1,2,3,4}, d_phi^F <= 256, d <= 128 and
 * d % 4 == 0.  dtype bf16 with d in {64,128}, (F, d_phi) = (3, 6) or
 * (2, 12) - the paper's two variants - and B*H*N < 2^31 runs on the tensor-core
 * kernels; everything else in the supported set runs on the fp32 SIMT kernels.
 * causal = 1 (Section 4.4 "Causal Attention, Decay Factors and Sequential
 * Updates": token i sees the tokens j <= i, itself included, and the normaliser
 * sums the same entries, o_i = sum_{j<=i} A_ij v_j / (sum_{j<=i} A_ij + eps))
 * is supported for the 3-factor tensor-core set only (bf16, d in {64,128},
 * F = 3, d_phi = 6), forward and backward; any other combination with
 * causal = 1 is HLA_ERR_UNSUPPORTED.  Decay factors (a non-binary mask) are
 * not defined by the paper and not supported.
 */
typedef struct {
    int32_t B, H, N, d;
    int32_t F;        /* number of Hadamard factors; 0 -> 3 (the paper's main model)          */
    int32_t d_phi;    /* feature width; 0 -> 6 if F == 3, 12 if F == 2 (appendix "Defining phi") */
    int32_t phi;      /* hla_phi_mode                                                          */
    int32_t dtype;    /* hla_dtype                                                             */
    float eps;        /* added to the normaliser, o = num / (eta + eps); <= 0 -> 1e-6          */
    int32_t n_splits; /* token splits of the state build per head; 0 -> chosen from the SM count */
    int32_t causal;   /* 0: every token sees every token; 1: token i sees tokens j <= i          */
    int32_t value_mod; /* 1: the workspace also holds the scratch of hla_value_mod_forward / _backward (bf16 with
                          d in {64,128} only; HLA_ERR_UNSUPPORTED otherwise); 0: those calls are refused            */
} hla_config;

/*
 * One feature network (appendix "Defining phi"): feat = ReLU(W2^T GELU(W1^T x + b1) + b2),
 * the erf form of GELU (the tensor-core kernels evaluate its normal CDF with an
 * error below 4e-4 and its derivative with an error below 1.3e-3, both under the bf16
 * rounding of the hidden layer).  Device pointers in the ctx dtype: W1 [d][d] (input index
 * first), b1 [d], W2 [d][d_phi], b2 [d_phi].  One set per map, shared by all
 * batches and heads.
 */
typedef struct {
    const void *W1, *b1, *W2, *b2;
} hla_mlp;

/*
 * One value-modulation network (Section 4.5 "Value Modulation"; appendix "Defining phi"):
 *     phi_v(x) = W2^T GELU(W1^T LN(x) + b1) + b2,   LN(x) = (x - mean) / sqrt(var + 1e-5) * ln_g + ln_b  over the d channels
 * (two Linear layers of width d, no final activation; the paper only says that these maps use a LayerNorm - it is read
 * as acting on the input of the map).  Device pointers in the ctx dtype: ln_g [d], ln_b [d], W1 [d][d] (input index
 * first), b1 [d], W2 [d][d], b2 [d]; W1 and W2 16-byte aligned.
 */
typedef struct {
    const void *ln_g, *ln_b, *W1, *b1, *W2, *b2;
} hla_vmlp;

/*
 * Where hla_backward_weights puts the gradients of one feature network: fp32 device buffers with the shapes of the
 * weights, dW1 [d][d], db1 [d], dW2 [d][d_phi], db2 [d_phi], 16-byte aligned.  The call overwrites them.
 */
typedef struct {
    void *dW1, *db1, *dW2, *db2;
} hla_mlp_grad;

/* Byte offsets of the regions of the workspace that outlive a call (for
 * checking and for callers that want the state).  A region that the
 * configuration does not use has offset (size_t)-1. */
typedef struct {
    size_t status;   /* int32[16]  device status words                                   */
    size_t qf;       /* fp32 [B,H,N,d_phi]     features phi_q(Q)        (HLA_PHI_MLP)   */
    size_t kf;       /* fp32 [B,H,F,N,d_phi]   features phi_kf(K)       (HLA_PHI_MLP)   */
    size_t state;    /* fp32 [B,H,state_rows,state_ld]  columns 0..d-1 = C, column d = z.  state_rows = P = d_phi^F
                        on the SIMT path.  The tensor-core path keeps the state folded over the permutation
                        symmetry of the query tensor q (x) q (x) q: row m = (a <= b <= c) in lexicographic order
                        holds the sum of C over the distinct permutations of (a,b,c); 56 rows for F = 3, d_phi = 6 */
    size_t eta;      /* fp32 [B,H,N]           normaliser before eps                    */
    size_t dstate;   /* fp32 [B,H,state_rows,state_ld]  gradient of the loss w.r.t. that state (after hla_backward) */
    size_t dqf;      /* fp32 [B,H,N,d_phi]     feature gradients        (HLA_PHI_MLP)   */
    size_t dkf;      /* fp32 [B,H,F,N,d_phi]                            (HLA_PHI_MLP)   */
    int32_t state_ld; /* row stride of state / dstate in floats (>= d+1)                */
    int32_t state_rows;
    int32_t n_splits; /* the split count in use                                          */
    int32_t tensor_core; /* 1 if this configuration runs the tcgen05 kernels              */
} hla_ws_layout;

/* Validates the configuration and creates a context.  *out is NULL on failure. */
hla_status hla_create(const hla_config *cfg, hla_ctx **out);

/* HLA_PHI_MLP only: remembers the weight pointers (phi_k points to F entries).
 * The weights must stay valid and unchanged while the ctx is used. */
hla_status hla_set_phi(hla_ctx *ctx, const hla_mlp *phi_q, const hla_mlp *phi_k);

/* Bytes of caller-provided device scratch that forward and backward need. */
size_t hla_workspace_bytes(const hla_ctx *ctx);

hla_status hla_workspace_layout(const hla_ctx *ctx, hla_ws_layout *out);

/*
 * Forward: O = HLA(Q, K, V).  Leaves the features, the state (C, z) and eta in
 * the workspace for a later hla_backward.  With causal = 1 the state left in the
 * workspace is the one after the last token (Eq. "seq.updates": C^N) and eta_i
 * is the masked row sum.  The workspace must be 256-byte
 * aligned and at least hla_workspace_bytes() long.
 */
hla_status hla_forward(hla_ctx *ctx, const void *Q, const void *K, const void *V, void *O,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Sequential updates (Section 4.4, Eq. "seq.updates": C^i = C^{i-1} + T_{k_i} (x) v_i; the context tensor is the state of
 * the sequence).  Contexts created with causal = 1 only.  With carry = 1 every following hla_forward on a workspace
 * starts from the state (C, z) that the previous hla_forward left in that workspace instead of from zero, and leaves
 * the updated state there: a sequence handed over in chunks of N tokens per call gives the outputs of one causal pass
 * over the concatenation (the state is carried in fp32).  The first chunk of a sequence is run with carry = 0 (or on a
 * workspace whose state region the caller has zeroed; hla_workspace_layout gives its offset and size).  hla_backward is
 * HLA_ERR_UNSUPPORTED while carry = 1.  HLA_ERR_INVALID_ARG for a context without the mask or a value other than 0, 1.
 */
hla_status hla_set_carry(hla_ctx *ctx, int carry);

/*
 * Backward of the forward that last wrote `workspace` (same Q, K, V, O; the
 * workspace untouched in between): dQ, dK, dV = d sum(dO * O) / d(Q, K, V).
 * In HLA_PHI_NONE mode dQ, dK are fp32 feature gradients with the shapes of Q, K.
 * In HLA_PHI_MLP mode on the tensor-core kernels dQ and dK must be 32-byte aligned
 * (their rows leave the kernel as 32-byte stores); anything else is refused with
 * HLA_ERR_INVALID_ARG before a launch.
 * Gradients with respect to the phi weights are not computed by this call.
 * With causal = 1, O must be the output of that forward (the call reads it for
 * dO_i . o_i; without the mask it is not read) and V, O, dO, dV must be 16-byte
 * aligned like every tensor.
 */
hla_status hla_backward(hla_ctx *ctx, const void *Q, const void *K, const void *V, const void *O,
                        const void *dO, void *dQ, void *dK, void *dV,
                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The two passes in two halves, for a sequence whose N tokens are split over several devices (one context per device,
 * each created with its own share of N).  Theorem 4.2's state C = sum_j T_k[j] v_j^T and the key-side sum z are sums
 * over the tokens, so the shards' states add: between the two halves of a pass the caller adds the state region of the
 * workspaces of all shards (fp32; hla_workspace_layout gives `state` / `dstate`, state_rows and state_ld; one all-reduce
 * of B*H*state_rows*state_ld floats) and leaves the sum in every workspace.
 *   forward:   hla_forward_keys (feature maps of K, state of the shard)  ->  sum of `state` over the shards  ->
 *              hla_forward_queries (feature map of Q, readout against the summed state, O of the shard's tokens)
 *   backward:  hla_backward_queries (query pass: dQ-side gradients, gradient state of the shard)  ->  sum of `dstate`
 *              over the shards  ->  hla_backward_keys (key pass on the summed gradient state, then the phi backward:
 *              dQ, dK, dV of the shard's tokens)
 * Each half takes the arguments of the whole call and uses those it needs (the key half of the forward K and V, the
 * query half Q and O; both halves of the backward the full list).  With a single shard and no sum in between the two
 * halves give the results of hla_forward / hla_backward bit for bit.  Tensor-core set without the mask only:
 * HLA_ERR_UNSUPPORTED on the fp32 SIMT path and for causal = 1 (a causal pass would need an exclusive scan of the
 * shards' states instead of their sum).  The library itself never communicates between devices.
 */
hla_status hla_forward_keys(hla_ctx *ctx, const void *K, const void *V, void *workspace, size_t workspace_bytes, void *cuda_stream);
hla_status hla_forward_queries(hla_ctx *ctx, const void *Q, void *O, void *workspace, size_t workspace_bytes, void *cuda_stream);
hla_status hla_backward_queries(hla_ctx *ctx, const void *Q, const void *K, const void *V, const void *O,
                                const void *dO, void *dQ, void *dK, void *dV,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);
hla_status hla_backward_keys(hla_ctx *ctx, const void *Q, const void *K, const void *V, const void *O,
                             const void *dO, void *dQ, void *dK, void *dV,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Gradients of sum(dO * O) with respect to the weights of the feature networks (Section 5, "Training Details": the
 * paper trains the phi maps with the rest of the model; Algorithm 1 step 4 defines where they act).  HLA_PHI_MLP
 * contexts on the tensor-core kernels only (HLA_ERR_UNSUPPORTED otherwise).  Call it after hla_backward with the
 * same Q, K and the same workspace: it reads the features the forward kept and the feature gradients the backward
 * left there, recomputes the hidden layer, and sums over all batches, heads and tokens (one weight set per map is
 * shared by all of them).  dphi_q receives the gradients of phi_q, dphi_k points to F entries for phi_k1..F; either
 * may be NULL to skip that side.  The sums are formed in a fixed order: results are bit-reproducible.
 */
hla_status hla_backward_weights(hla_ctx *ctx, const void *Q, const void *K, const hla_mlp_grad *dphi_q, const hla_mlp_grad *dphi_k,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Value modulation of the attention result (Section 4.5):  Out = T + phi_v1(T) (.) phi_v2(V), with T the output of
 * hla_forward and V its value input, both [B,H,N,d]; one weight set per map, shared by all batches and heads.
 * Contexts created with value_mod = 1 only.  hla_set_phi_v remembers the weight pointers (they must stay valid).
 * The forward keeps nothing for the backward; the backward recomputes both maps and returns
 *     dT = dOut + J1^T (dOut (.) phi_v2(V)),     dV = J2^T (dOut (.) phi_v1(T))      (J: Jacobian of a map w.r.t. its input)
 * the gradients of sum(dOut * Out) with respect to T and V (weights fixed).  With accumulate_dV != 0 the V-side
 * gradient is added to what dV already holds (the dV that hla_backward wrote for the same step), else dV is overwritten.
 * Out, dT, dV must be 32-byte aligned.  Out may not alias T or V.  hla_value_mod_forward clears the device status words
 * like hla_forward does (read hla_last_device_status before it if the record of hla_forward matters); the backward
 * keeps them.  A whole step is then
 *     hla_forward -> hla_value_mod_forward;   hla_value_mod_backward -> hla_backward(dO = dT) with accumulate_dV = 0 and
 *     the two dV added by the caller, or hla_backward first and hla_value_mod_backward with accumulate_dV = 1.
 */
hla_status hla_set_phi_v(hla_ctx *ctx, const hla_vmlp *v1, const hla_vmlp *v2);
hla_status hla_value_mod_forward(hla_ctx *ctx, const void *T, const void *V, void *Out, void *workspace, size_t workspace_bytes,
                                 void *cuda_stream);
hla_status hla_value_mod_backward(hla_ctx *ctx, const void *T, const void *V, const void *dOut, void *dT, void *dV,
                                  int32_t accumulate_dV, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Forward without a caller-provided workspace (no counterpart in the paper: a
 * deployment aid).  Some callers of this library cannot obtain device memory
 * at the time they need the operator: a plug-in running inside a host
 * application that owns the allocator, a real-time loop that forbids
 * allocation after start-up, code that only receives the tensors it is
 * handed.  For them the library carries its own scratch: one array of
 * HLA_STATIC_WS_BYTES bytes that is part of the loaded module, so every GPU
 * that loads the library holds that much memory until the process exits.
 * This call computes exactly what hla_forward computes, with that array as the
 * workspace, and calls no memory-allocating routine.
 *
 *   - Contexts whose hla_workspace_bytes() exceeds HLA_STATIC_WS_BYTES are
 *     refused with HLA_ERR_WORKSPACE before anything is enqueued.
 *   - The first call on a device looks up the array's device address (with
 *     that device current) and remembers it; make that first call outside any
 *     stream capture.  Later calls on the same device only enqueue work.
 *   - All contexts and all calls share the one array, and it keeps what the
 *     previous call left in it.  Everything a call reads from it is written
 *     earlier in the same call (the status words are cleared at the start),
 *     so back-to-back calls on one stream are independent; two calls that can
 *     overlap on the GPU (different streams without an ordering between them)
 *     race on it and must not be made.
 *   - If `scratch_out` is not NULL it receives the array's device address:
 *     pass it as `workspace` to hla_last_device_status, to hla_backward (the
 *     state of the forward lives there), or add hla_workspace_layout offsets
 *     to read eta or the state.
 */
#define HLA_STATIC_WS_BYTES (16u * 1024u * 1024u)
hla_status hla_forward_static(hla_ctx *ctx, const void *Q, const void *K, const void *V, void *O,
                              void *cuda_stream, void **scratch_out);

/* Synchronises `cuda_stream`, reads the device status words of `workspace`
 * and returns HLA_OK, HLA_ERR_DEVICE_TIMEOUT or HLA_ERR_CUDA. */
hla_status hla_last_device_status(hla_ctx *ctx, const void *workspace, void *cuda_stream);

/*
 * Self-test of the failure path (no counterpart in the paper).  Every wait inside the kernels is bounded; this
 * call enqueues a one-block kernel that waits, with a 1 ms limit, on a barrier that nothing arrives at.  The wait
 * must run out, the kernel must return normally, and a following hla_last_device_status(ctx, workspace, stream)
 * must report HLA_ERR_DEVICE_TIMEOUT.  The status words are cleared by the next hla_forward.
 */
hla_status hla_selftest_bounded_wait(hla_ctx *ctx, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Number of kernels the last hla_forward / hla_backward on this ctx launched. */
int32_t hla_last_launch_count(const hla_ctx *ctx);

/*
 * Optional per-kernel timing (no counterpart in the paper: a measurement aid).
 * While enabled, every kernel launch of hla_forward / hla_backward is bracketed
 * by CUDA events on the launching stream.  After the caller has synchronised
 * the stream, hla_timing_collect folds the recorded launches into per-kernel
 * totals (replacing earlier totals) and returns how many distinct kernels
 * there are; hla_timing_get returns entry i: a static name, the summed device
 * time in milliseconds and the number of launches.
 */
hla_status hla_timing_enable(hla_ctx *ctx, int32_t on);
int32_t hla_timing_collect(hla_ctx *ctx);
hla_status hla_timing_get(const hla_ctx *ctx, int32_t i, const char **name, double *total_ms, int64_t *launches);

hla_status hla_destroy(hla_ctx *ctx);

const char *hla_status_string(hla_status s);

#ifdef __cplusplus
}
#endif
#endif /* HLA_H_ */
