// rglru_prefill_static_scratch: the tensor-core prefill for callers that cannot allocate device memory.
//
// Some callers of this library run where cudaMalloc is not an option: inside a serving loop whose
// memory pool was sized and frozen at start-up, under a framework allocator that forbids side
// allocations, or in a process whose device memory is fully handed out to other components.  The
// regular entry point asks them for a workspace they have no way to provide.  This variant keeps the
// scratch of the prefill kernel (the per-tile carry records of the time split, the private copies of
// an aliased incoming state, and the status word) in one file-scope device array that is part of the
// library image, so the caller passes inputs and outputs only.
//
// Consequences of the shared array, all of them documented in include/rglru.h as well:
//  - every GPU that loads the library holds STATIC_SCRATCH_BYTES of device memory until the process exits;
//  - shapes whose scratch exceeds that size are rejected with RGLRU_ERR_WORKSPACE;
//  - all calls on one device use the same array, so two calls that overlap on the GPU (different
//    streams, no ordering) race; calls must be ordered on one stream or by events;
//  - the array keeps what the last call wrote: carry records are told apart by a per-call tag, and
//    the status word is cleared on the stream before every launch.
//
// Host code cannot use the array's name as a pointer: in host code that name is only a handle for
// cudaGetSymbolAddress.  The device address is looked up once per device (with that device current)
// on the first call there and cached; that first call should be made outside any stream capture.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "rglru_internal.h"

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = (size_t)8 << 20;  // 8 MiB; see RGLRU_STATIC_SCRATCH_BYTES in rglru.h
static_assert(STATIC_SCRATCH_BYTES == RGLRU_STATIC_SCRATCH_BYTES, "header and implementation disagree on the scratch size");

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[MAX_DEVICES] = {};

// Device address of the scratch array on the current device; nullptr (and *err set) on failure.
void *scratch_for_current_device(cudaError_t *err) {
    int dev = -1;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= MAX_DEVICES) { *err = cudaErrorInvalidDevice; return nullptr; }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void *ptr = nullptr;
        *err = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (*err != cudaSuccess) return nullptr;
        g_scratch_addr[dev] = ptr;
    }
    return g_scratch_addr[dev];
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int32_t rglru_prefill_static_scratch(const rglru_shape_t *s, const rglru_params_t *p, const void *x,
                                                const float *h0, const void *conv_state_in, void *y, float *h_T,
                                                void *conv_state_out, void *status_word, void *cuda_stream) {
    using namespace rglru;
    if (s == nullptr || p == nullptr) return RGLRU_ERR_NULL;
    if (s->B <= 0 || s->T <= 0 || s->D <= 0 || s->H <= 0 || s->D % s->H != 0 || !(s->c > 0.0f)) return RGLRU_ERR_SHAPE;
    if (!sm100_prefill_supported(s->B, s->T, s->D, s->H, s->io)) return RGLRU_ERR_UNSUPPORTED;
    if (!p->conv_w || !p->W_a || !p->b_a || !p->W_x || !p->b_x || !p->lambda) return RGLRU_ERR_NULL;
    if (!x || !y || !h_T || !conv_state_out) return RGLRU_ERR_NULL;
    if (!aligned16(p->conv_w) || !aligned16(p->conv_b) || !aligned16(p->W_a) || !aligned16(p->W_x) || !aligned16(p->b_a) ||
        !aligned16(p->b_x) || !aligned16(p->lambda) || !aligned16(x) || !aligned16(y) || !aligned16(h_T) ||
        !aligned16(conv_state_out) || !aligned16(h0) || !aligned16(conv_state_in) ||
        (reinterpret_cast<uintptr_t>(status_word) & 3u) != 0)
        return RGLRU_ERR_ALIGN;
    const size_t body = sm100_prefill_workspace_bytes(s->B, s->T, s->D, s->H);
    if (WS_HEADER_BYTES + body > STATIC_SCRATCH_BYTES) return RGLRU_ERR_WORKSPACE;  // shape too large for the built-in scratch
    const size_t nbytes = (size_t)s->B * s->T * s->D * sizeof(__nv_bfloat16);
    {
        const uintptr_t px = (uintptr_t)x, py = (uintptr_t)y;
        if (px < py + nbytes && py < px + nbytes) return RGLRU_ERR_ALIAS;
    }

    cudaError_t e;
    unsigned char *scratch = (unsigned char *)scratch_for_current_device(&e);
    if (scratch == nullptr) return RGLRU_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // the status word must start at zero; everything else in the array is tagged per call
    if (cudaMemsetAsync(scratch, 0, WS_HEADER_BYTES, st) != cudaSuccess) return RGLRU_ERR_CUDA;

    FwdArgs a{};
    a.B = s->B; a.T = s->T; a.D = s->D; a.H = s->H; a.c = s->c;
    a.conv_w = p->conv_w; a.conv_b = p->conv_b; a.W_a = p->W_a; a.W_x = p->W_x;
    a.b_a = p->b_a; a.b_x = p->b_x; a.lambda = p->lambda;
    a.x = x; a.h0 = h0; a.cs_in = conv_state_in; a.y = y; a.h_T = h_T; a.cs_out = conv_state_out;
    // a wait that runs out on the device is recorded in the caller's word when there is one (readable with
    // rglru_query_status), else in the array's header, where nothing reads it back
    a.status = status_word ? (uint32_t *)status_word : (uint32_t *)scratch;
    e = sm100_prefill(a, scratch + WS_HEADER_BYTES, STATIC_SCRATCH_BYTES - WS_HEADER_BYTES, st);
    return e == cudaSuccess ? RGLRU_OK : RGLRU_ERR_CUDA;
}
