// extern "C" entry points of the RG-LRU library: host-side validation, workspace planning,
// kernel selection.  Every error is a return code; nothing here allocates device memory.
#include <cuda_runtime.h>

#include <mutex>

#include "rglru_internal.h"

using namespace rglru;

namespace {

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t io_bytes(int io) { return io == RGLRU_BF16 ? 2 : 4; }

int32_t check_shape(const rglru_shape_t *s, bool need_T) {
    if (s == nullptr) return RGLRU_ERR_NULL;
    if (s->B <= 0 || s->D <= 0 || s->H <= 0 || (need_T && s->T <= 0)) return RGLRU_ERR_SHAPE;
    if (s->D % s->H != 0) return RGLRU_ERR_SHAPE;
    if (!(s->c > 0.0f)) return RGLRU_ERR_SHAPE;
    if (s->io != RGLRU_F32 && s->io != RGLRU_BF16) return RGLRU_ERR_UNSUPPORTED;
    if (s->D / s->H > GENERIC_MAX_DH) return RGLRU_ERR_UNSUPPORTED;
    return RGLRU_OK;
}

int32_t check_params(const rglru_params_t *p) {
    if (p == nullptr) return RGLRU_ERR_NULL;
    if (!p->conv_w || !p->W_a || !p->b_a || !p->W_x || !p->b_x || !p->lambda) return RGLRU_ERR_NULL;
    if (!aligned(p->conv_w, 16) || !aligned(p->W_a, 16) || !aligned(p->W_x, 16) || !aligned(p->b_a, 16) ||
        !aligned(p->b_x, 16) || !aligned(p->lambda, 16) || !aligned(p->conv_b, 16))
        return RGLRU_ERR_ALIGN;
    return RGLRU_OK;
}

inline bool overlap(const void *a, size_t na, const void *b, size_t nb) {
    if (!a || !b) return false;
    uintptr_t pa = (uintptr_t)a, pb = (uintptr_t)b;
    return pa < pb + nb && pb < pa + na;
}

bool use_sm100_prefill(const rglru_shape_t *s) {
    return !(s->flags & RGLRU_FLAG_FORCE_GENERIC) && sm100_prefill_supported(s->B, s->T, s->D, s->H, s->io);
}

// Two helper streams and the events that tie them to the caller's stream for rglru_prefill_host, one set per device,
// created on first use (streams and events are not device memory).  Calls on one device are serialised by the mutex.
struct HostPipe {
    static constexpr int MAX_CHUNKS = 16;
    std::mutex mutex;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, done = nullptr, copied[MAX_CHUNKS] = {}, computed[MAX_CHUNKS] = {};
    bool ready = false;
};

HostPipe *host_pipe() {
    static HostPipe pipes[64];
    static std::mutex setup;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(setup);
    HostPipe &hp = pipes[dev];
    if (!hp.ready) {
        bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.done, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < HostPipe::MAX_CHUNKS; ++i)
            ok = cudaEventCreateWithFlags(&hp.copied[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.computed[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        hp.ready = true;
    }
    return &hp;
}

bool use_sm100_backward(const rglru_shape_t *s) {
    return !(s->flags & RGLRU_FLAG_FORCE_GENERIC) && sm100_backward_supported(s->B, s->T, s->D, s->H, s->io);
}

FwdArgs make_fwd(const rglru_shape_t *s, const rglru_params_t *p) {
    FwdArgs a{};
    a.B = s->B; a.T = s->T; a.D = s->D; a.H = s->H; a.c = s->c;
    a.conv_w = p->conv_w; a.conv_b = p->conv_b; a.W_a = p->W_a; a.W_x = p->W_x;
    a.b_a = p->b_a; a.b_x = p->b_x; a.lambda = p->lambda;
    a.flags = s->flags;
    return a;
}

}  // namespace

extern "C" {

int32_t rglru_abi_version(void) { return 102; }

const char *rglru_status_string(int32_t status) {
    switch (status) {
        case RGLRU_OK: return "ok";
        case RGLRU_ERR_NULL: return "a required pointer is NULL";
        case RGLRU_ERR_SHAPE: return "invalid shape (B, T, D, H must be positive, D divisible by H, c > 0)";
        case RGLRU_ERR_UNSUPPORTED: return "no kernel for this dtype or head width";
        case RGLRU_ERR_ALIGN: return "pointer not sufficiently aligned (16 bytes; workspace and staging 256)";
        case RGLRU_ERR_WORKSPACE: return "workspace or staging buffer too small";
        case RGLRU_ERR_CUDA: return "a CUDA runtime call failed";
        case RGLRU_ERR_TIMEOUT: return "device-side bounded wait for a carry ran out";
        case RGLRU_ERR_ALIAS: return "output buffer overlaps an input buffer";
        default: return "unknown status";
    }
}

size_t rglru_workspace_bytes(const rglru_shape_t *s, int32_t op) {
    if (check_shape(s, op != RGLRU_OP_DECODE) != RGLRU_OK) return 0;
    size_t body = 0;
    switch (op) {
        case RGLRU_OP_PREFILL:
            if (use_sm100_prefill(s)) body = sm100_prefill_workspace_bytes(s->B, s->T, s->D, s->H);
            break;
        case RGLRU_OP_DECODE: break;
        case RGLRU_OP_BACKWARD:
            body = use_sm100_backward(s) ? sm100_backward_workspace_bytes(s->B, s->T, s->D, s->H)
                                         : generic_backward_workspace_bytes(s->B, s->T, s->D, s->H);
            break;
        default: return 0;
    }
    return WS_HEADER_BYTES + body;
}

int32_t rglru_prefill(const rglru_shape_t *s, const rglru_params_t *p, const void *x, const float *h0,
                      const void *conv_state_in, void *y, float *h_T, void *conv_state_out, void *workspace,
                      size_t workspace_bytes, void *cuda_stream) {
    return rglru_prefill_ex(s, p, x, h0, conv_state_in, y, h_T, conv_state_out, nullptr, workspace, workspace_bytes, cuda_stream);
}

int32_t rglru_prefill_ex(const rglru_shape_t *s, const rglru_params_t *p, const void *x, const float *h0,
                         const void *conv_state_in, void *y, float *h_T, void *conv_state_out, const rglru_prefill_extras_t *extras,
                         void *workspace, size_t workspace_bytes, void *cuda_stream) {
    int32_t rc = check_shape(s, true);
    if (rc != RGLRU_OK) return rc;
    if ((rc = check_params(p)) != RGLRU_OK) return rc;
    if (!x || !y || !h_T || !conv_state_out || !workspace) return RGLRU_ERR_NULL;
    const void *gate_branch = extras ? extras->gate_branch : nullptr;
    float *a_prod = extras ? extras->a_prod : nullptr;
    if (!aligned(x, 16) || !aligned(y, 16) || !aligned(h_T, 16) || !aligned(conv_state_out, 16) || !aligned(h0, 16) ||
        !aligned(conv_state_in, 16) || !aligned(workspace, 256) || !aligned(gate_branch, 16) || !aligned(a_prod, 16))
        return RGLRU_ERR_ALIGN;
    const size_t need = rglru_workspace_bytes(s, RGLRU_OP_PREFILL);
    if (workspace_bytes < need) return RGLRU_ERR_WORKSPACE;
    const size_t nbytes = (size_t)s->B * s->T * s->D * io_bytes(s->io);
    if (overlap(x, nbytes, y, nbytes) || (gate_branch && overlap(gate_branch, nbytes, y, nbytes))) return RGLRU_ERR_ALIAS;

    FwdArgs a = make_fwd(s, p);
    a.x = x; a.h0 = h0; a.cs_in = conv_state_in; a.y = y; a.h_T = h_T; a.cs_out = conv_state_out;
    a.gate_branch = gate_branch; a.a_prod = a_prod;
    a.status = (uint32_t *)workspace;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (use_sm100_prefill(s))
        e = sm100_prefill(a, (char *)workspace + WS_HEADER_BYTES, workspace_bytes - WS_HEADER_BYTES, st);
    else
        e = generic_prefill(a, s->io, st);
    return e == cudaSuccess ? RGLRU_OK : RGLRU_ERR_CUDA;
}

int32_t rglru_decode_step(const rglru_shape_t *s, const rglru_params_t *p, const void *x, float *h, void *conv_state,
                          void *y, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    int32_t rc = check_shape(s, false);
    if (rc != RGLRU_OK) return rc;
    if ((rc = check_params(p)) != RGLRU_OK) return rc;
    if (!x || !h || !conv_state || !y || !workspace) return RGLRU_ERR_NULL;
    if (!aligned(x, 16) || !aligned(h, 16) || !aligned(conv_state, 16) || !aligned(y, 16) || !aligned(workspace, 256))
        return RGLRU_ERR_ALIGN;
    if (workspace_bytes < rglru_workspace_bytes(s, RGLRU_OP_DECODE)) return RGLRU_ERR_WORKSPACE;
    const size_t nbytes = (size_t)s->B * s->D * io_bytes(s->io);
    if (overlap(x, nbytes, y, nbytes)) return RGLRU_ERR_ALIAS;

    FwdArgs a = make_fwd(s, p);
    a.T = 1;
    a.x = x; a.y = y; a.h_T = h; a.cs_out = conv_state;
    a.status = (uint32_t *)workspace;
    cudaError_t e;
    if (!(s->flags & RGLRU_FLAG_FORCE_GENERIC) && sm100_decode_supported(s->B, s->D, s->H, s->io))
        e = sm100_decode(a, (cudaStream_t)cuda_stream);
    else
        e = generic_decode(a, s->io, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? RGLRU_OK : RGLRU_ERR_CUDA;
}

int32_t rglru_backward(const rglru_shape_t *s, const rglru_params_t *p, const void *x, const float *h0,
                       const void *conv_state_in, const void *y, const void *dy, void *dx, float *dconv_w,
                       float *dconv_b, float *dW_a, float *db_a, float *dW_x, float *db_x, float *dlambda,
                       const rglru_state_grads_t *state, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    int32_t rc = check_shape(s, true);
    if (rc != RGLRU_OK) return rc;
    if ((rc = check_params(p)) != RGLRU_OK) return rc;
    if (!x || !dy || !dx || !dconv_w || !dW_a || !db_a || !dW_x || !db_x || !dlambda || !workspace) return RGLRU_ERR_NULL;
    if (!aligned(x, 16) || !aligned(dy, 16) || !aligned(dx, 16) || !aligned(y, 16) || !aligned(h0, 16) ||
        !aligned(conv_state_in, 16) || !aligned(dconv_w, 16) || !aligned(dconv_b, 16) || !aligned(dW_a, 16) ||
        !aligned(db_a, 16) || !aligned(dW_x, 16) || !aligned(db_x, 16) || !aligned(dlambda, 16) || !aligned(workspace, 256))
        return RGLRU_ERR_ALIGN;
    if (state && (!aligned(state->dh_T, 16) || !aligned(state->dconv_state_out, 16) || !aligned(state->dh0, 16) ||
                  !aligned(state->dconv_state_in, 16)))
        return RGLRU_ERR_ALIGN;
    if (workspace_bytes < rglru_workspace_bytes(s, RGLRU_OP_BACKWARD)) return RGLRU_ERR_WORKSPACE;
    const size_t nbytes = (size_t)s->B * s->T * s->D * io_bytes(s->io);
    if (overlap(dx, nbytes, x, nbytes) || overlap(dx, nbytes, dy, nbytes) || overlap(dx, nbytes, y, nbytes)) return RGLRU_ERR_ALIAS;

    FwdArgs f = make_fwd(s, p);
    f.x = x; f.h0 = h0; f.cs_in = conv_state_in;
    f.status = (uint32_t *)workspace;
    BwdArgs q{};
    q.B = s->B; q.T = s->T; q.D = s->D; q.H = s->H; q.c = s->c;
    q.x = x; q.conv_w = p->conv_w; q.W_a = p->W_a; q.W_x = p->W_x; q.cs_in = conv_state_in; q.dy = dy;
    q.lambda = p->lambda; q.dx = dx;
    q.dconv_w = dconv_w; q.dconv_b = dconv_b; q.dW_a = dW_a; q.db_a = db_a; q.dW_x = dW_x; q.db_x = db_x; q.dlambda = dlambda;
    if (state) { q.dh_T = state->dh_T; q.dcs_out = state->dconv_state_out; q.dh0 = state->dh0; q.dcs_in = state->dconv_state_in; }
    cudaError_t e;
    if (use_sm100_backward(s))
        e = sm100_backward(f, q, y, (char *)workspace + WS_HEADER_BYTES, workspace_bytes - WS_HEADER_BYTES, (uint32_t *)workspace,
                           (cudaStream_t)cuda_stream);
    else
        e = generic_backward(f, q, s->io, (char *)workspace + WS_HEADER_BYTES, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? RGLRU_OK : RGLRU_ERR_CUDA;
}

size_t rglru_host_staging_bytes(const rglru_shape_t *s) {
    if (check_shape(s, true) != RGLRU_OK) return 0;
    const size_t xb = ((size_t)s->B * s->T * s->D * io_bytes(s->io) + 255) & ~(size_t)255;
    const size_t hb = ((size_t)s->B * s->D * sizeof(float) + 255) & ~(size_t)255;
    const size_t cb = ((size_t)s->B * 3 * s->D * io_bytes(s->io) + 255) & ~(size_t)255;
    return 2 * xb + hb + cb;
}

int32_t rglru_prefill_host(const rglru_shape_t *s, const rglru_params_t *p, const void *x_host, const float *h0,
                           const void *conv_state_in, void *y_host, float *h_T_host, void *conv_state_out_host,
                           void *staging, size_t staging_bytes, void *workspace, size_t workspace_bytes,
                           void *cuda_stream) {
    int32_t rc = check_shape(s, true);
    if (rc != RGLRU_OK) return rc;
    if (!x_host || !y_host || !h_T_host || !conv_state_out_host || !staging) return RGLRU_ERR_NULL;
    if (!aligned(staging, 256)) return RGLRU_ERR_ALIGN;
    if (staging_bytes < rglru_host_staging_bytes(s)) return RGLRU_ERR_WORKSPACE;
    const size_t io = io_bytes(s->io);
    const size_t seq_x = (size_t)s->T * s->D * io, seq_h = (size_t)s->D * sizeof(float), seq_c = (size_t)3 * s->D * io;
    const size_t xbytes = (size_t)s->B * seq_x, hbytes = (size_t)s->B * seq_h, cbytes = (size_t)s->B * seq_c;
    const size_t xb = (xbytes + 255) & ~(size_t)255, hb = (hbytes + 255) & ~(size_t)255;
    char *sx = (char *)staging, *sy = sx + xb, *sh = sy + xb, *sc = sh + hb;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    // Sequences are independent, so the batch is cut into chunks that move through three stages at once: host-to-device
    // copy of chunk c+1, forward of chunk c, device-to-host copy of chunk c-1 (PCIe carries both directions at the same
    // time).  Chunk boundaries must keep every pointer 16-byte aligned; otherwise the whole batch is one chunk.
    HostPipe *hp = host_pipe();
    const bool splittable = hp != nullptr && s->B > 1 && seq_x % 16 == 0 && seq_h % 16 == 0 && seq_c % 16 == 0;
    const int nchunks = splittable ? (s->B < HostPipe::MAX_CHUNKS ? s->B : HostPipe::MAX_CHUNKS) : 1;
    if (nchunks == 1) {
        if (cudaMemcpyAsync(sx, x_host, xbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return RGLRU_ERR_CUDA;
        rc = rglru_prefill(s, p, sx, h0, conv_state_in, sy, (float *)sh, sc, workspace, workspace_bytes, cuda_stream);
        if (rc != RGLRU_OK) return rc;
        if (cudaMemcpyAsync(y_host, sy, xbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return RGLRU_ERR_CUDA;
        if (cudaMemcpyAsync(h_T_host, sh, hbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return RGLRU_ERR_CUDA;
        if (cudaMemcpyAsync(conv_state_out_host, sc, cbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return RGLRU_ERR_CUDA;
        return RGLRU_OK;
    }
    std::lock_guard<std::mutex> lock(hp->mutex);
#define CK(call) do { if ((call) != cudaSuccess) return RGLRU_ERR_CUDA; } while (0)
    CK(cudaEventRecord(hp->start, st));                      // everything below follows the work already on the stream
    CK(cudaStreamWaitEvent(hp->in, hp->start, 0));
    CK(cudaStreamWaitEvent(hp->out, hp->start, 0));
    for (int c = 0; c < nchunks; ++c) {
        const int b0 = (int)((long long)s->B * c / nchunks), b1 = (int)((long long)s->B * (c + 1) / nchunks);
        rglru_shape_t sc_shape = *s;
        sc_shape.B = b1 - b0;
        const size_t xo = (size_t)b0 * seq_x, ho = (size_t)b0 * seq_h, co = (size_t)b0 * seq_c, xn = (size_t)(b1 - b0) * seq_x;
        CK(cudaMemcpyAsync(sx + xo, (const char *)x_host + xo, xn, cudaMemcpyHostToDevice, hp->in));
        CK(cudaEventRecord(hp->copied[c], hp->in));
        CK(cudaStreamWaitEvent(st, hp->copied[c], 0));
        rc = rglru_prefill(&sc_shape, p, sx + xo, h0 ? (const float *)((const char *)h0 + ho) : nullptr,
                           conv_state_in ? (const char *)conv_state_in + co : nullptr, sy + xo, (float *)(sh + ho), sc + co, workspace,
                           workspace_bytes, cuda_stream);
        if (rc != RGLRU_OK) return rc;
        CK(cudaEventRecord(hp->computed[c], st));
        CK(cudaStreamWaitEvent(hp->out, hp->computed[c], 0));
        CK(cudaMemcpyAsync((char *)y_host + xo, sy + xo, xn, cudaMemcpyDeviceToHost, hp->out));
    }
    CK(cudaMemcpyAsync(h_T_host, sh, hbytes, cudaMemcpyDeviceToHost, hp->out));
    CK(cudaMemcpyAsync(conv_state_out_host, sc, cbytes, cudaMemcpyDeviceToHost, hp->out));
    CK(cudaEventRecord(hp->done, hp->out));
    CK(cudaStreamWaitEvent(st, hp->done, 0));                // later work on the caller's stream sees the results
#undef CK
    return RGLRU_OK;
}

uint64_t rglru_set_wait_limit_ns(uint64_t ns) {
    const uint64_t prev = g_spin_limit_ns;
    g_spin_limit_ns = ns == 0 ? 2000000000ull : ns;
    return prev;
}

int32_t rglru_query_status(void *workspace, void *cuda_stream) {
    if (!workspace) return RGLRU_ERR_NULL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return RGLRU_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return RGLRU_ERR_CUDA;
    if ((word & 0xFFFFFF00u) != STATUS_MAGIC) return RGLRU_OK;  // nothing recorded
    if (cudaMemsetAsync(workspace, 0, sizeof(word), st) != cudaSuccess) return RGLRU_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return RGLRU_ERR_CUDA;
    return (int32_t)(word & 0xFFu);
}

}  // extern "C"
