// river_argmax_noalloc: greedy next-token selection over caller-provided logits that allocates nothing.
//
// The decode step's own argmax keeps its per-CTA partial maxima in the caller's workspace.  Some callers have no
// workspace to give and may not allocate one at that point: a sampler hook that runs inside a serving loop whose
// device memory was handed to the KV cache in full at start-up, or a latency-critical loop in which a cudaMalloc
// would serialise the whole device.  For them this variant keeps its scratch (partial maxima and the per-row
// arrival counters) in a fixed array that lives in the library's device image: every GPU that loads the library
// holds those 66 KB until the process exits.  The tie rule is the decode step's: the lowest token id wins.
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "../../include/river.h"

namespace {

constexpr int kMaxRows = RIVER_NOALLOC_MAX_ROWS;
constexpr int kParts = 128;  // CTAs that share one row's vocabulary
constexpr int kMaxDevices = 64;

struct Partial {
    float val;
    int32_t idx;
};
struct Scratch {
    Partial part[kMaxRows][kParts];
    unsigned arrived[kMaxRows];  // CTAs of a row that have published their partial; must be zero at launch
};

// Scratch in the device image.  In host code this name is only a stand-in for the symbol: the device address is
// obtained once per device with cudaGetSymbolAddress and handed to the kernel as an ordinary pointer.
static __device__ __align__(256) unsigned char g_scratch[sizeof(Scratch)];

Scratch *g_scratch_addr[kMaxDevices];  // per device, filled by the first call made with that device current

__device__ __forceinline__ bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

// grid (kParts, rows): CTA (p, r) scans its share of row r, publishes (max, lowest id of the max); the last CTA of
// a row to arrive (atomic counter, no spinning) merges the row's partials and writes the token.
__global__ void __launch_bounds__(256) argmax_noalloc_kernel(const float *logits, int V, int32_t *next_tok,
                                                             Scratch *s) {
    const int part = blockIdx.x, row = blockIdx.y;
    const float *x = logits + (size_t)row * V;
    const int per = (V + kParts - 1) / kParts;
    const int v0 = part * per, v1 = min(V, v0 + per);
    float bv = -CUDART_INF_F;
    int bi = 0x7fffffff;
    for (int v = v0 + threadIdx.x; v < v1; v += blockDim.x) {
        const float f = x[v];
        if (better(f, v, bv, bi)) { bv = f; bi = v; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    __shared__ float sv[8];
    __shared__ int si[8];
    __shared__ bool last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (better(sv[w], si[w], bv, bi)) { bv = sv[w]; bi = si[w]; }
        s->part[row][part] = Partial{bv, bi};
        __threadfence();
        last = atomicAdd(&s->arrived[row], 1u) == kParts - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    bv = -CUDART_INF_F;
    bi = 0x7fffffff;
    if (threadIdx.x < kParts) {
        const volatile Partial *p = &s->part[row][threadIdx.x];
        bv = p->val;
        bi = p->idx;
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    __syncthreads();
    if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w)
            if (better(sv[w], si[w], bv, bi)) { bv = sv[w]; bi = si[w]; }
        next_tok[row] = bi == 0x7fffffff ? 0 : bi;  // a row without any comparable value (all NaN) yields token 0
        s->arrived[row] = 0;
    }
}

}  // namespace

extern "C" int river_argmax_noalloc(const float *logits, int n_rows, int V, int32_t *next_tok, void *cuda_stream) {
    if (!logits || !next_tok || n_rows <= 0 || V <= 0 || V > 0x7fffffff - kParts) return RIVER_E_BADARG;
    if (n_rows > kMaxRows) return RIVER_E_NOMEM;  // beyond the fixed scratch: split the batch
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RIVER_E_DEVICE;
    if (!g_scratch_addr[dev]) {
        // one-time set-up for this device (it is current): the device address of the scratch symbol
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) return RIVER_E_DEVICE;
        g_scratch_addr[dev] = static_cast<Scratch *>(p);
    }
    Scratch *s = g_scratch_addr[dev];
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the last call left and the counters have to start at zero: this memset is what the
    // call relies on (the kernel also returns them to zero, so an aborted earlier launch cannot poison a later one)
    if (cudaMemsetAsync(s->arrived, 0, sizeof(unsigned) * n_rows, st) != cudaSuccess) return RIVER_E_DEVICE;
    argmax_noalloc_kernel<<<dim3(kParts, n_rows), 256, 0, st>>>(logits, V, next_tok, s);
    return cudaGetLastError() == cudaSuccess ? RIVER_OK : RIVER_E_DEVICE;
}
