// Shared device-side definitions of the early-exit decode step (sm_100a): small helpers, the per-step metadata
// block, row lists, weight handles and the KV-pool addressing used by every kernel file.
//
// One decode step = embed -> per layer { QKV projection + RoPE + paged KV write, paged GQA decode attention,
// O projection + residual, gate/up + SwiGLU, down + residual, exit score (Eq. 1), row compaction } ->
// final norm + LM head + argmax.  Rows still in the backbone read the bf16 weights, rows that left it read the
// 4-bit exit-layer copy of the same block and write K/V to the very same cache slots (paper Section 4.1).
// Which rows are where is decided on the device; every kernel reads the row lists and counts from device memory.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace river {

constexpr int kPage = 16;         // tokens per KV page
constexpr int kMaxBatch = 1024;   // rows per step (one CTA scans the exit flags)

enum DevErr : int { DEV_OK = 0, DEV_BAD_FORCED = 1, DEV_BAD_TOKEN = 2, DEV_BAD_PAGE = 3, DEV_WAIT_TIMEOUT = 4, DEV_INTERNAL = 5 };

// ---------------------------------------------------------------- small helpers
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ float bf16f(uint16_t v) { return __uint_as_float(((uint32_t)v) << 16); }

__device__ __forceinline__ uint4 ldg_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ uint16_t ldg_u16(const void *p) {
    uint16_t v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Activation rows sit in shared memory in a lane-interleaved order so that a lane that owns the E consecutive
// inputs of "chunk" c reads them with conflict-free 128-bit loads: index of input k (c = k / E, j = k % E).
template <int E>
__device__ __forceinline__ int xs_index(int k) {
    if constexpr (E == 0) return k;  // plain order
    const int c = k / (E ? E : 1), j = k % (E ? E : 1);
    return (c >> 5) * (32 * E) + (j >> 2) * 128 + (c & 31) * 4 + (j & 3);
}
// KV splits per (row, KV head) of the small-step attention kernel: about one CTA per SM.
__host__ __device__ inline int small_attn_splits(int num_sms, int n_rows, int Hkv) {
    const int s = num_sms / (n_rows * Hkv);
    return s < 1 ? 1 : (s > 64 ? 64 : s);
}
__host__ __device__ inline int xs_stride(int K, int E) { return ((K + 32 * E - 1) / (32 * E)) * (32 * E); }

// ---------------------------------------------------------------- per-step parameters shared by the kernels
struct StepMeta {  // device-resident, rewritten by the host before every step
    int32_t n_rows;
    int32_t n_updates;
    int32_t n_head_rows;
    int32_t attn_chunk;   // positions per KV split of the attention kernel (multiple of 64)
    int32_t attn_splits;  // split slots per (row, head) in the partial buffers
    int32_t hint_act;     // rows still in the backbone as of the latest compaction (reset to n_rows by the host)
    int32_t pad[2];       // small-step attention: positions per split, splits per (row, KV head)
    int32_t pad2[2];      // [0]: query tiles of a prefill chunk (attn_prefill_kernel)
    // the caller's device buffers of this step (read through here so that a captured launch sequence never changes)
    const int32_t *tok;
    const float *tau;
    const int32_t *forced;  // may be null
    float *logits;          // may be null
    int32_t *next_tok;
    int32_t *exit_layer;
    float *scores;          // may be null
};
constexpr int kMetaHdr = sizeof(StepMeta) / sizeof(int32_t);

struct Lists {  // rows entering each block, per layer index 0..L
    int32_t *act_idx;  // [(L+1)][max_batch]
    int32_t *riv_idx;
    int32_t *n_act;    // [(L+1)]
    int32_t *n_riv;
    int32_t max_batch;
};

struct W4 {
    const uint8_t *codes;
    const uint16_t *scale;
    const uint16_t *zero;
};

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Stable partition of the rows by the sticky exit flag, run by ONE CTA (any number of threads >= 32, multiple of
// 32): ascending row ids of the rows still in the backbone and of the rows in the exit layers, and their counts.
__device__ __forceinline__ void build_lists(int n, const uint8_t *exited, int l, const Lists &lists,
                                            int32_t *hint_act, int *s_cnt /* shared, 2 * 32 + 2 ints */) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    int32_t *A = lists.act_idx + (size_t)l * lists.max_batch;
    int32_t *R = lists.riv_idx + (size_t)l * lists.max_batch;
    if (tid == 0) { s_cnt[64] = 0; s_cnt[65] = 0; }
    __syncthreads();
    for (int b0 = 0; b0 < n; b0 += blockDim.x) {
        const int b = b0 + tid;
        const bool valid = b < n;
        const bool gone = valid && exited[b] != 0;
        const unsigned ma = __ballot_sync(0xffffffffu, valid && !gone);
        const unsigned mr = __ballot_sync(0xffffffffu, valid && gone);
        if (lane == 0) { s_cnt[warp] = __popc(ma); s_cnt[32 + warp] = __popc(mr); }
        __syncthreads();
        int base_a = s_cnt[64], base_r = s_cnt[65], tot_a = 0, tot_r = 0;
        for (int w = 0; w < nwarps; ++w) {
            if (w < warp) { base_a += s_cnt[w]; base_r += s_cnt[32 + w]; }
            tot_a += s_cnt[w];
            tot_r += s_cnt[32 + w];
        }
        const unsigned lt = (1u << lane) - 1u;
        if (valid) {
            if (!gone) A[base_a + __popc(ma & lt)] = b;
            else R[base_r + __popc(mr & lt)] = b;
        }
        __syncthreads();
        if (tid == 0) { s_cnt[64] += tot_a; s_cnt[65] += tot_r; }
        __syncthreads();
    }
    if (tid == 0) {
        lists.n_act[l] = s_cnt[64];
        lists.n_riv[l] = s_cnt[65];
        *hint_act = s_cnt[64];
    }
}

// ---------------------------------------------------------------- shared by the projection kernels
// What feeds a projection: either rows of an fp32 buffer as they are, or their RMSNorm (x = h * rsqrt(mean h^2 +
// eps) * gain), computed by every CTA for itself.
struct ProjIn {
    const float *src;      // [rows][K]
    const uint16_t *gain;  // bf16 [K] or nullptr = no normalisation
    float eps;
};

struct KvAddr {
    __nv_bfloat16 *pool;  // [L][n_pages][2][Hkv][16][dh]
    const int32_t *page_tbl;
    const int32_t *row_slot, *row_pos;
    const int32_t *row_page;  // page that holds each row's new position (host-computed: no table walk on the write path)
    int n_pages, max_pages_per_seq, Hkv, dh;
    int layer0;
    __device__ __forceinline__ size_t base(int page, int kv, int kvh, int inpage) const {
        return ((((size_t)layer0 * n_pages + page) * 2 + kv) * Hkv + kvh) * (size_t)(kPage * dh) + (size_t)inpage * dh;
    }
};

}  // namespace river
