// del_head_argmax_static: the exit head's arg-max for callers that must not allocate device memory.
//
// Who needs it: code that runs where cudaMalloc is off limits — inside a serving loop whose memory pool
// was sized and frozen at start-up, in a plug-in that is handed tensors but no allocator, or in a
// process that already filled the device on purpose.  The regular path keeps the LM-head kernel's
// per-CTA (max, index) partials in the caller's workspace; this variant keeps them in a fixed array
// that is part of the library image, so the call needs nothing beyond its inputs and its output.
//
// Consequences of the fixed array (also stated in include/del.h):
//   * every GPU that loads the library holds DEL_STATIC_SCRATCH_BYTES until the process exits;
//   * sizes are capped (rows <= 64, grid <= 1024 CTAs) and larger requests are rejected;
//   * all calls on a device share the array: two calls that overlap on the GPU (different streams)
//     race; calls on one stream are ordered and safe.  The array keeps the previous call's contents;
//     everything a call reads from it is rewritten by that call first;
//   * the first call on a device looks up the array's device address; make that call before starting
//     a stream capture.
#include "../../include/del.h"
#include "kernels.h"

#include <cstring>

namespace {

constexpr int MAX_CTAS = 1024;
constexpr size_t PART_BYTES = (size_t)MAX_CTAS * DEL_ROWS_MAX * 4;
constexpr size_t SCRATCH_BYTES = 2 * PART_BYTES;
static_assert(SCRATCH_BYTES <= DEL_STATIC_SCRATCH_BYTES, "static scratch larger than documented");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress, never an address.
static __device__ __align__(256) unsigned char g_static_scratch[DEL_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
unsigned char *g_scratch_ptr[MAX_DEVICES] = {nullptr};   // device address of the array, per device

// one block per row: reduce the per-CTA partials, ties to the lowest token id
__global__ void __launch_bounds__(256) static_argmax_kernel(const float *pv, const int32_t *pi, int n_part, int32_t *tokens) {
    __shared__ float sv[8];
    __shared__ int si[8];
    const int c = blockIdx.x;
    float v = -INFINITY;
    int idx = 0x7fffffff;
    for (int p = threadIdx.x; p < n_part; p += 256) {
        const float v2 = pv[(size_t)p * DEL_ROWS_MAX + c];
        const int i2 = pi[(size_t)p * DEL_ROWS_MAX + c];
        if (v2 > v || (v2 == v && i2 < idx)) { v = v2; idx = i2; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xffffffffu, v, o);
        const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
        if (v2 > v || (v2 == v && i2 < idx)) { v = v2; idx = i2; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = v; si[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (sv[w] > v || (sv[w] == v && si[w] < idx)) { v = sv[w]; idx = si[w]; }
        tokens[c] = idx;
    }
}

}  // namespace

extern "C" int del_head_argmax_static(const void *x, const void *lm_head, int rows, int vocab, int d_model, int32_t *tokens,
                                      void *cuda_stream) {
    if (!x || !lm_head || !tokens) return DEL_EINVAL;
    if (rows < 1 || rows > DEL_ROWS_MAX) return DEL_EINVAL;              // beyond the static scratch
    if (vocab < 16 || vocab % 16 || d_model < 256 || d_model % 8) return DEL_EINVAL;
    int dev = 0, n_sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return DEL_ECUDA;
    if (cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return DEL_ECUDA;
    if (!g_scratch_ptr[dev]) {
        // once per device, with that device current: the array's address on THIS device
        unsigned char *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_static_scratch) != cudaSuccess || !p) return DEL_ECUDA;
        g_scratch_ptr[dev] = p;
    }
    unsigned char *scratch = g_scratch_ptr[dev];
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int n_items = vocab / 16;
    const int n_part = rowgemm_lmhead_grid(n_items, rows, n_sms, 2);
    if (n_part > MAX_CTAS) return DEL_EINVAL;                            // beyond the static scratch

    GemmArgs a;
    memset(&a, 0, sizeof(a));
    a.D.d = d_model; a.D.V = vocab; a.D.S = 1; a.D.B = 1; a.D.n_sst = d_model / 16;
    a.plan.m = rows;
    a.K = d_model;
    a.n_items = n_items;
    a.X = reinterpret_cast<const bf16 *>(x);
    a.W0 = reinterpret_cast<const bf16 *>(lm_head);
    a.x_by_row = 1;
    a.ctas_per_sm = 2;
    a.B.LPV = reinterpret_cast<float *>(scratch);
    a.B.LPI = reinterpret_cast<int32_t *>(scratch + PART_BYTES);

    if (launch_rowgemm(EPI_LMHEAD, a, rows, n_sms, st, false) != cudaSuccess) return DEL_ECUDA;
    static_argmax_kernel<<<rows, 256, 0, st>>>(a.B.LPV, a.B.LPI, n_part, tokens);
    if (cudaGetLastError() != cudaSuccess) return DEL_ECUDA;
    return DEL_OK;
}
