// Internal declarations shared by the translation units of the RG-LRU CUDA library.
// Not part of the public ABI (that is include/rglru.h).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <mutex>

#include "rglru.h"

namespace rglru {

// Function attributes belong to a device's context, so the opt-in to more than 48 KB of dynamic shared memory has to be made
// once per device (with that device current), not once per process.  Thread-safe; `T` is a kernel function pointer type.
struct PerDeviceOptIn {
    std::mutex mutex;
    bool done[64] = {};
    template <typename T> cudaError_t ensure(T kernel, int smem_bytes) {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mutex);
        if (!done[dev]) {
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
            if (e != cudaSuccess) return e;
            done[dev] = true;
        }
        return cudaSuccess;
    }
};

// The first 256 bytes of every workspace hold the device-side status: word 0 carries
// STATUS_MAGIC | code once a kernel has recorded a condition.  A word without the magic
// (fresh, uninitialised scratch) reads as "nothing recorded".
constexpr uint32_t STATUS_MAGIC = 0x52474C00u;  // 'R','G','L', code in the low byte
constexpr size_t WS_HEADER_BYTES = 256;

struct FwdArgs {
    int B, T, D, H;
    float c;
    const void *x;            // [B,T,D] io  (decode: [B,D])
    const void *conv_w;       // [4,D] io
    const float *conv_b;      // [D] or null
    const void *W_a, *W_x;    // [H,Dh,Dh] io
    const float *b_a, *b_x, *lambda;
    const float *h0;          // [B,D] or null
    const void *cs_in;        // [B,3,D] io or null
    void *y;                  // [B,T,D] io
    float *h_T;               // [B,D]
    void *cs_out;             // [B,3,D] io
    // optional fp32 saves for the backward, each [B,T,D] (null when not saving)
    float *save_u, *save_r, *save_i, *save_hprev;
    uint32_t *status;         // workspace header
    uint32_t flags;           // RGLRU_FLAG_* of the call
    const void *gate_branch;  // [B,T,D] io or null: y_t = h_t * GeLU(gate_branch_t) (prefill only)
    float *a_prod;            // [B,D] or null: prod_t a_t over the call (prefill only)
};

struct BwdArgs {
    int B, T, D, H;
    float c;
    const void *x, *conv_w, *W_a, *W_x, *cs_in, *dy;
    const float *lambda;
    void *dx;
    float *dconv_w, *dconv_b, *dW_a, *db_a, *dW_x, *db_x, *dlambda;
    // gradient through the carried state (each may be null): in dh_T [B,D], dcs_out [B,3,D] io; out dh0 [B,D], dcs_in [B,3,D] io
    const float *dh_T;
    const void *dcs_out;
    float *dh0;
    void *dcs_in;
    // workspace arrays, each [B,T,D] fp32: u, r -> dz_a, i -> dz_x, hprev -> du
    float *u, *r, *gi, *hp;
    float *part_vec;   // [B][3][D]        partial sums of dlambda, db_a, db_x
    float *part_conv;  // [B*nchunk][5][D] partial sums of dconv_w (4 rows) and dconv_b
    float *part_dw;    // [S][2][H*Dh*Dh]  partial sums of dW_a, dW_x
    int nchunk, S;
};

// ---- shape-generic CUDA-core kernels (any D_h <= GENERIC_MAX_DH, fp32 or bf16 io) ----
constexpr int GENERIC_MAX_DH = 1024;
constexpr int GENERIC_BWD_CHUNK = 64;  // tokens per thread in the conv backward
size_t generic_backward_workspace_bytes(int B, int T, int D, int H);
cudaError_t generic_prefill(const FwdArgs &a, int io, cudaStream_t st);
cudaError_t generic_decode(const FwdArgs &a, int io, cudaStream_t st);
cudaError_t generic_backward(const FwdArgs &fwd, BwdArgs &b, int io, void *ws_body, cudaStream_t st);

// ---- sm_100a tensor-core kernels (bf16 io, D_h = 256) ----
bool sm100_prefill_supported(int B, int T, int D, int H, int io);
size_t sm100_prefill_workspace_bytes(int B, int T, int D, int H);
cudaError_t sm100_prefill(const FwdArgs &a, void *ws_body, size_t ws_body_bytes, cudaStream_t st);
bool sm100_decode_supported(int B, int D, int H, int io);
cudaError_t sm100_decode(const FwdArgs &a, cudaStream_t st);
extern unsigned long long g_spin_limit_ns;  // every device-side wait gives up after this many nanoseconds
// Tiled-TMA descriptor of a dense bf16 tensor [d2][d1][d0] (d0 innermost) with a box of box1 x box0 elements;
// swizzle128 selects the 128-byte shared-memory swizzle that tcgen05.mma operands use.  False if the driver
// entry point is unavailable or rejects the shape.
bool encode_bf16_map_3d(CUtensorMap *tm, const void *ptr, uint64_t d0, uint64_t d1, uint64_t d2, uint32_t box0, uint32_t box1,
                        bool swizzle128);
// The general form for any 16-bit element type: dims (innermost first), byte strides of dims 1 and 2, box extents.
bool encode_map16_3d(CUtensorMap *tm, const void *ptr, const uint64_t dims[3], const uint64_t strides_bytes[2], const uint32_t box[3],
                     bool swizzle128);
// ---- sm_100a backward (bf16 io, D_h = 256, T a multiple of 8): tensor-core GEMMs around element-wise scan kernels
bool sm100_backward_supported(int B, int T, int D, int H, int io);
size_t sm100_backward_workspace_bytes(int B, int T, int D, int H);
cudaError_t sm100_backward(const FwdArgs &fwd, BwdArgs &b, const void *y_saved, void *ws_body, size_t ws_body_bytes, uint32_t *status,
                           cudaStream_t st);
// Gradient of the three carried conv inputs, dcs_in[r] = sum_j w[j] du_{r-3+j} (0 <= r-3+j < T), and the gradient that arrives
// on conv_state_out added to the rows it copies (dx_{T-3+k} is recomputed from du with the term added, so it is rounded once;
// rows of conv_state_in when T < 3).  du is [B,T,D] of DUT (float or __half); io tensors are IOT.  No-op without dcs_in / dcs_out.
cudaError_t state_conv_grads(const BwdArgs &q, int io, const void *du, bool du_is_half, cudaStream_t st);
// out[i] = sum over p of in[p * stride + i] in ascending p (fixed order: run-to-run identical results)
cudaError_t reduce_partials(const float *in, int nparts, size_t stride, float *out, size_t n, cudaStream_t st);
// A row of n0 + n1 + n2 values summed over the parts and split over up to three output arrays (any of them may be null or
// empty); four interleaved running sums over ascending p, added at the end: also a fixed order.
cudaError_t reduce_partials3(const float *in, int nparts, size_t stride, float *out0, size_t n0, float *out1, size_t n1, float *out2,
                             size_t n2, cudaStream_t st);

}  // namespace rglru
