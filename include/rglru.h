/*
 * rglru.h -- C ABI of the B200 (sm_100a) RG-LRU temporal-core library.
 *
 * The library computes the temporal core of the Griffin/Hawk recurrent block:
 * a causal depthwise Conv1D of temporal width 4 (Section 2.3, "Recurrent block"),
 * followed by the RG-LRU layer (Section 2.4, Eq. 1-4) with the decay evaluated in
 * log space (Appendix A) and block-diagonal gate matrices (Section 4.1, "Model parallelism", paragraph "Recurrent Block"):
 *
 *     u_t = b_c + sum_{j=0..3} w[j] * x_{t-j}                 (Conv1D, tap j hits x_{t-j})
 *     r_t = sigmoid(W_a u_t + b_a)                            (Eq. 1)
 *     i_t = sigmoid(W_x u_t + b_x)                            (Eq. 2)
 *     a_t = sigmoid(Lambda)^(c r_t) = exp(-c softplus(-Lambda) r_t)   (Eq. 3, Appendix A)
 *     h_t = a_t * h_{t-1} + sqrt(1 - a_t^2) * (i_t * u_t),  y_t = h_t (Eq. 4)
 *
 * Conventions that hold for every entry point unless stated otherwise:
 *  - Data pointers are DEVICE pointers owned by the caller.  The library never allocates,
 *    frees or keeps them.  All tensors are dense, row-major, innermost dimension D.
 *  - "io" tensors (x, y, dy, dx, conv_w, W_a, W_x, conv_state) have the dtype named in
 *    rglru_shape_t.io; per-channel vectors (conv_b, b_a, b_x, lambda), the recurrent state
 *    (h0, h_T, h) and all parameter gradients are fp32.  The state is carried in fp32.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *    stream) and return without synchronising.  Argument errors are detected on the host
 *    before anything is launched and are reported by the return code; nothing is printed,
 *    thrown or aborted.  Conditions found on the device (a bounded wait that ran out) are
 *    recorded in the workspace and read back by rglru_query_status.
 *  - `workspace` is caller-owned device scratch of at least rglru_workspace_bytes(...)
 *    bytes, 256-byte aligned.  Its contents need not be preserved between calls; calls
 *    that share a workspace must be ordered on one stream.
 *  - Shapes without a kernel return RGLRU_ERR_UNSUPPORTED.  There is no CPU fallback.
 *  - Kernels.  bf16 io with a head width D_h that is a multiple of 32 up to 256 runs on tensor-core kernels (prefill, decode
 *    step, backward; the backward needs T % 8 == 0).  Section 4.1 fixes 16 blocks, so D_h is 256 only at D_RNN = 4096; it is 96
 *    at D_RNN = 1536, 128 at 2048 and 160 at 2560.  Narrower heads share, or occupy alone, groups of 256 channel slots whose
 *    weight tile is block-diagonal; the slots a width leaves unused are idle work.  Every other shape with D_h <= 1024, fp32
 *    or bf16, runs on shape-generic CUDA-core kernels.
 */
#ifndef RGLRU_H_
#define RGLRU_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RGLRU_OK = 0,
    RGLRU_ERR_NULL = 1,        /* a required pointer is NULL */
    RGLRU_ERR_SHAPE = 2,       /* B, T, D, H <= 0, D % H != 0, or c <= 0 */
    RGLRU_ERR_UNSUPPORTED = 3, /* no kernel for this dtype / head width */
    RGLRU_ERR_ALIGN = 4,       /* a pointer is not 16-byte aligned (workspace: 256) */
    RGLRU_ERR_WORKSPACE = 5,   /* workspace_bytes too small */
    RGLRU_ERR_CUDA = 6,        /* a CUDA runtime call failed (launch, copy) */
    RGLRU_ERR_TIMEOUT = 7,     /* device side: a bounded wait on another block's carry ran out */
    RGLRU_ERR_ALIAS = 8        /* y aliases x, or dx aliases an input */
} rglru_status_t;

typedef enum { RGLRU_F32 = 0, RGLRU_BF16 = 1 } rglru_dtype_t;

typedef enum { RGLRU_OP_PREFILL = 0, RGLRU_OP_DECODE = 1, RGLRU_OP_BACKWARD = 2 } rglru_op_t;

/* flags */
#define RGLRU_FLAG_NONE 0u
#define RGLRU_FLAG_FORCE_GENERIC 1u /* use the shape-generic CUDA-core kernels even where a tensor-core kernel exists */
/* Test hook of the failure path, honoured by the tensor-core rglru_prefill only: tiles that wait for another tile's carry
 * record look for a tag that is never published, so the bounded wait (rglru_set_wait_limit_ns) runs out, the kernel drains
 * and returns, and rglru_query_status reports RGLRU_ERR_TIMEOUT.  Outputs are undefined after such a call. */
#define RGLRU_FLAG_TEST_CARRY_NEVER_ARRIVES 0x40000000u

typedef struct {
    int32_t B;     /* sequences */
    int32_t T;     /* tokens per sequence (ignored by rglru_decode_step) */
    int32_t D;     /* D_RNN, channels */
    int32_t H;     /* heads = diagonal blocks of W_a and W_x; head width D_h = D / H */
    int32_t io;    /* rglru_dtype_t of the io tensors */
    float c;       /* exponent scale of Eq. 3; the paper fixes 8 */
    uint32_t flags;
} rglru_shape_t;

typedef struct {
    const void *conv_w;  /* [4, D] io; row j multiplies x_{t-j} */
    const float *conv_b; /* [D] or NULL (zero) */
    const void *W_a;     /* [H, D_h, D_h] io; W[h][out][in], Eq. 1 */
    const float *b_a;    /* [D] */
    const void *W_x;     /* [H, D_h, D_h] io, Eq. 2 */
    const float *b_x;    /* [D] */
    const float *lambda; /* [D]; a = sigmoid(lambda), Section 2.4 */
} rglru_params_t;

/* Version of this ABI (major * 100 + minor). */
int32_t rglru_abi_version(void);

/* Text for a status code; never NULL; static storage. */
const char *rglru_status_string(int32_t status);

/*
 * Device scratch needed by one call of `op` (rglru_op_t) on `shape`.  Host-only; returns 0
 * for an invalid or unsupported shape.  The value is at least 256 so that the status word
 * always has a home.
 */
size_t rglru_workspace_bytes(const rglru_shape_t *shape, int32_t op);

/*
 * Forward over T tokens (Conv1D + Eq. 1-4), also the inference prefill: returns the state
 * that a later rglru_prefill or rglru_decode_step continues from (Appendix F.4, "Cache sizes": the
 * recurrent state has size D_RNN, the convolution state (4-1) D_RNN per sequence).
 *   x              [B,T,D] io, in
 *   h0             [B,D] fp32, in, or NULL for a zero state
 *   conv_state_in  [B,3,D] io, in, the raw inputs x_{-3}, x_{-2}, x_{-1} (oldest first), or NULL for zeros
 *   y              [B,T,D] io, out (rounded to nearest even for bf16); must not overlap x
 *   h_T            [B,D] fp32, out: the unrounded state after the last token; may alias h0
 *   conv_state_out [B,3,D] io, out: last three rows of concat(conv_state_in, x), bit-exact copies; may alias conv_state_in
 */
int32_t rglru_prefill(const rglru_shape_t *shape, const rglru_params_t *params, const void *x, const float *h0,
                      const void *conv_state_in, void *y, float *h_T, void *conv_state_out, void *workspace,
                      size_t workspace_bytes, void *cuda_stream);

/*
 * rglru_prefill with optional extras (NULL, or a struct whose members may each be NULL; with all of them NULL the call is
 * rglru_prefill):
 *   gate_branch [B,T,D] io, in: the second branch of the recurrent block (Section 2.3: a GeLU on that branch, then the two
 *               branches are merged by element-wise multiplication).  The call then writes
 *               y_t = h_t * GeLU(gate_branch_t), GeLU(v) = v Phi(v), the merge as the epilogue of the scan, so that h is
 *               not written and read again by a separate kernel; h_T stays the raw state.  Must not overlap y.
 *   a_prod      [B,D] fp32, out: prod_t a_t over the T tokens of the call (Eq. 3).  Eq. 4 is affine in the incoming state,
 *               h_T = a_prod * h0 + (h_T from a zero state), so with h0 = NULL the pair (a_prod, h_T) describes the whole call
 *               as one step of the recurrence: what ranks that split a sequence in time exchange (Section 4.1 shards the
 *               recurrent block over heads without communication; along time one exchange of this pair per rank suffices).
 * Other arguments, ownership, asynchrony and errors as for rglru_prefill; RGLRU_ERR_ALIGN also for an extra that is not
 * 16-byte aligned, RGLRU_ERR_ALIAS also when gate_branch overlaps y.
 */
typedef struct {
    const void *gate_branch;
    float *a_prod;
} rglru_prefill_extras_t;

int32_t rglru_prefill_ex(const rglru_shape_t *shape, const rglru_params_t *params, const void *x, const float *h0,
                         const void *conv_state_in, void *y, float *h_T, void *conv_state_out,
                         const rglru_prefill_extras_t *extras, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * One decode step for B sequences (Section 5.1, "A simple model of the decode step", and Appendix F.4): the T = 1 case of the
 * forward with the state updated in place.
 *   x          [B,D] io, in
 *   h          [B,D] fp32, in/out
 *   conv_state [B,3,D] io, in/out: rows shift by one (bit-exact) and x becomes row 2
 *   y          [B,D] io, out
 * The tensor-core kernel is launched so that it may start while the preceding kernel on the stream is still finishing
 * (programmatic dependent launch): it reads the parameters (conv_w, conv_b, W_a, b_a, W_x, b_x, lambda) before it waits
 * for that kernel, and x, h and conv_state after.  A kernel that writes the parameters (a cast, an optimiser step) must
 * therefore not be the one directly before this call on the stream; put any other work, or an event, in between.
 * After RGLRU_ERR_TIMEOUT (rglru_query_status) h and conv_state are undefined: conv_state may already hold the shifted rows
 * while h has not been advanced.
 */
int32_t rglru_decode_step(const rglru_shape_t *shape, const rglru_params_t *params, const void *x, float *h,
                          void *conv_state, void *y, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Backward of rglru_prefill for an upstream gradient dy on y (the paper states no backward;
 * this is reverse-mode differentiation of Eq. 1-4 and the Conv1D: a reverse-time scan
 * g_t = dy_t + a_{t+1} g_{t+1} followed by the gate and convolution adjoints).  With
 * `state` given, the call also differentiates through the carried state, so that a sequence cut
 * into segments (truncated back-propagation through time, Section 7) is differentiated segment by
 * segment, last segment first: what a segment returns in dh0 and dconv_state_in is what the segment
 * before it takes as dh_T and dconv_state_out.
 *   x, h0, conv_state_in : as given to the forward
 *   y              [B,T,D] io, the forward output, or NULL (the state is then recomputed)
 *   dy             [B,T,D] io, in
 *   dx             [B,T,D] io, out; must not overlap x, y or dy
 *   dconv_w [4,D], dconv_b [D] (may be NULL), dW_a, dW_x [H,D_h,D_h], db_a, db_x, dlambda [D]:
 *                  fp32, out, overwritten (not accumulated), summed over batch and time.
 *   state          NULL (no gradient through the state), or a struct of four device pointers, each of which may be NULL:
 *       dh_T            [B,D] fp32, in: gradient arriving on h_T
 *       dconv_state_out [B,3,D] io, in: gradient arriving on conv_state_out (a copy of the last three rows of
 *                       concat(conv_state_in, x), so it is added to the gradient of the rows it copies)
 *       dh0             [B,D] fp32, out: gradient of h0 (= a_0 g_0)
 *       dconv_state_in  [B,3,D] io, out: gradient of the three carried inputs x_{-3..-1}
 */
typedef struct rglru_state_grads {
    const float *dh_T;
    const void *dconv_state_out;
    float *dh0;
    void *dconv_state_in;
} rglru_state_grads_t;

int32_t rglru_backward(const rglru_shape_t *shape, const rglru_params_t *params, const void *x, const float *h0,
                       const void *conv_state_in, const void *y, const void *dy, void *dx, float *dconv_w,
                       float *dconv_b, float *dW_a, float *db_a, float *dW_x, float *db_x, float *dlambda,
                       const rglru_state_grads_t *state, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * rglru_prefill for callers whose activations live in HOST memory (pinned memory makes the
 * copies asynchronous).  x_host is copied to `staging`, the forward runs there, and y, h_T and
 * conv_state_out are copied back to the host pointers; the call returns without synchronising and work
 * enqueued on `cuda_stream` afterwards sees the results.  The batch is cut into chunks of sequences whose
 * host-to-device copy, forward and device-to-host copy overlap on two internal streams (created on first use
 * per device); calls on one device must not be made from several host threads at once.  These two streams and the
 * events that tie them to `cuda_stream` are the one thing the library creates and keeps (per device, until the process
 * exits): the rule above that nothing is allocated or retained holds for device memory, not for them.
 * params, h0, conv_state_in, staging and workspace are device pointers.
 *   staging : device scratch of at least rglru_host_staging_bytes(shape) bytes, 256-byte aligned.
 */
size_t rglru_host_staging_bytes(const rglru_shape_t *shape);
int32_t rglru_prefill_host(const rglru_shape_t *shape, const rglru_params_t *params, const void *x_host,
                           const float *h0, const void *conv_state_in, void *y_host, float *h_T_host,
                           void *conv_state_out_host, void *staging, size_t staging_bytes, void *workspace,
                           size_t workspace_bytes, void *cuda_stream);

/*
 * rglru_prefill for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment convenience).  A serving loop that runs on a memory pool sized and frozen at
 * start-up, code under a framework allocator that forbids side allocations, or a process whose
 * device memory is fully handed to other components has no way to provide the workspace that
 * rglru_prefill asks for.  Here the scratch of the tensor-core prefill kernel lives in one array of
 * RGLRU_STATIC_SCRATCH_BYTES that is part of the library image; the call allocates and frees nothing.
 *   - Arguments x ... conv_state_out are those of rglru_prefill (device pointers, same aliasing rules).
 *   - status_word: optional device pointer to a 4-byte-aligned uint32 owned by the caller, zero before the
 *     first use.  A device-side wait that runs out is recorded there, and the pointer may be given to
 *     rglru_query_status in place of a workspace.  NULL: such a condition is not reported.
 *   - Only shapes served by the tensor-core prefill (bf16 io, head width a multiple of 32 up to 256) are accepted; others return
 *     RGLRU_ERR_UNSUPPORTED.  A shape whose scratch (256 bytes + rglru_workspace_bytes(shape, PREFILL))
 *     exceeds RGLRU_STATIC_SCRATCH_BYTES returns RGLRU_ERR_WORKSPACE; nothing is launched.
 *   - Every GPU on which the library is loaded holds the array until the process exits.
 *   - All calls on a device share the array: calls that overlap on the GPU (different streams without
 *     ordering) race.  Order them on one stream or with events.  The array keeps the previous call's
 *     contents; the call clears what has to start at zero on `cuda_stream` before its launch.
 *   - The first call on each device looks up the array's device address (with that device current) and
 *     caches it; make that first call outside any stream capture.
 */
#define RGLRU_STATIC_SCRATCH_BYTES ((size_t)8 << 20)
int32_t rglru_prefill_static_scratch(const rglru_shape_t *shape, const rglru_params_t *params, const void *x,
                                     const float *h0, const void *conv_state_in, void *y, float *h_T,
                                     void *conv_state_out, void *status_word, void *cuda_stream);

/*
 * Time limit of every device-side wait (a CTA waiting for another CTA's carry record, for a copy or for the tensor
 * core).  A wait that runs out makes the kernel record RGLRU_ERR_TIMEOUT in the workspace header, let work in flight
 * land, release its resources and return; nothing hangs and the context stays usable.  The default is 2 s, far above
 * any legitimate wait; ns = 0 restores it.  Process-wide; takes effect for calls issued afterwards.  Returns the
 * previous value.
 */
uint64_t rglru_set_wait_limit_ns(uint64_t ns);

/*
 * Synchronises `cuda_stream` and returns the device-side status recorded in `workspace` by the
 * calls issued so far (RGLRU_OK, RGLRU_ERR_TIMEOUT, or RGLRU_ERR_CUDA if the stream itself
 * reports an error), then clears it.
 */
int32_t rglru_query_status(void *workspace, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RGLRU_H_ */
