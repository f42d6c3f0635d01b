// Device code of the early-exit decode step (sm_100a).
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
    const int c = k / E, j = k % E;
    return (c >> 5) * (32 * E) + (j >> 2) * 128 + (c & 31) * 4 + (j & 3);
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
    int32_t pad[2];
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

// ---------------------------------------------------------------- step prologue
// Applies the page-table updates of this step, embeds the tokens (a0), resets the per-row exit state and the
// score diagnostics, and tabulates cos/sin of the rotary angles of every row's position.
__global__ void step_begin_kernel(const StepMeta *meta, const int32_t *upd, /* [3][max_batch]: slot, idx, page */
                                  int32_t *page_tbl, int max_pages_per_seq, int max_batch,
                                  const uint16_t *embed, int d, int V, float *h0, const int32_t *row_pos,
                                  const double *inv_freq, int half_dh, float2 *rope_cs,
                                  int L, int entry_layer, uint8_t *exited,
                                  int *dev_err, Lists lists, int32_t *hint_act, unsigned *ticket) {
    __shared__ int s_cnt[66];
    __shared__ bool s_last;
    pdl_launch();
    pdl_wait();
    const int b = blockIdx.x;
    const int n_rows = meta->n_rows;
    const int32_t *tok = meta->tok, *forced = meta->forced;
    int32_t *exit_layer = meta->exit_layer;
    float *scores = meta->scores;
    if (b == 0) {
        for (int i = threadIdx.x; i < meta->n_updates; i += blockDim.x)
            page_tbl[(size_t)upd[i] * max_pages_per_seq + upd[max_batch + i]] = upd[2 * max_batch + i];
    }
    if (b < n_rows) {
        int t = tok[b];
        if (t < 0 || t >= V) {
            if (threadIdx.x == 0) atomicExch(dev_err, DEV_BAD_TOKEN);
            t = 0;
        }
        const uint16_t *e = embed + (size_t)t * d;
        for (int i = threadIdx.x; i < d; i += blockDim.x) h0[(size_t)b * d + i] = bf16f(e[i]);
        const int pos = row_pos[b];
        for (int i = threadIdx.x; i < half_dh; i += blockDim.x) {
            double s, c;
            sincos((double)pos * inv_freq[i], &s, &c);
            rope_cs[(size_t)b * half_dh + i] = make_float2((float)c, (float)s);
        }
        if (scores)
            for (int i = threadIdx.x; i < L; i += blockDim.x) scores[(size_t)b * L + i] = CUDART_NAN_F;
        if (threadIdx.x == 0) {
            int f = forced ? forced[b] : -1;
            if (f >= 0 && (f > L || f < entry_layer)) {
                atomicExch(dev_err, DEV_BAD_FORCED);
                f = L;
            }
            const bool gone = (f == 0);
            exited[b] = gone ? 1 : 0;
            exit_layer[b] = gone ? 0 : L;
        }
    }
    // the last CTA to finish builds the row lists entering block 1 (a7)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (s_last) {
        __threadfence();
        build_lists(n_rows, exited, 0, lists, hint_act, s_cnt);
        if (threadIdx.x == 0) *ticket = 0;
    }
}

// ---------------------------------------------------------------- a6 + a7: exit score, decision, compaction
// One CTA per row of the step.  A row still in the backbone gets s = <h_in, h_out> / (|h_in| |h_out|) (Eq. 1) in
// fp32 with a fixed reduction order and the flag s > tau (strict; NaN fails; a zero norm gives s = 0).  The last
// CTA to finish (atomic ticket, no spinning) applies the eligibility window entry_layer <= l < L, the forced-exit
// hook and the batch mode to the flags, updates the sticky exit state and emits the two ascending row lists
// (a stable partition, bit-exact) and their counts for block l+1.
__global__ void __launch_bounds__(256) score_compact_kernel(const StepMeta *meta, int l, int L, int entry_layer,
                                                            int exit_mode, const float *h_in, const float *h_out,
                                                            int d, uint8_t *pass, uint8_t *exited, Lists lists,
                                                            int32_t *hint_act, unsigned *ticket) {
    __shared__ float red[3][8];
    __shared__ int s_cnt[66];
    __shared__ bool s_last;
    __shared__ int s_allpass;
    pdl_launch();
    // per-step constants (uploaded before the step's first kernel): fetched while the predecessor still runs, so the
    // decision below waits for nothing but the scores
    const int n = meta->n_rows;
    const float *tau = meta->tau;
    const int32_t *forced = meta->forced;
    int32_t *exit_layer = meta->exit_layer;
    float *scores = meta->scores;
    const int row = blockIdx.x;
    const float tau_row = row < n ? tau[row] : 0.f;
    int forced_mine = -1;  // thread b of the deciding CTA keeps row b's forced exit layer (rows beyond blockDim: read later)
    if (forced && (int)threadIdx.x < n) forced_mine = forced[threadIdx.x];
    pdl_wait();
    const bool eligible = (l >= 1) && (l >= entry_layer) && (l < L);
    if (n == 1 && gridDim.x == 1) {
        // A step of one row: its exit flag and both state vectors are requested together (one round trip), and one
        // thread takes the decision and writes the two one-element lists - no ballots, no second pass over flags.
        const int gone_before = exited[0];
        float ab = 0.f, aa = 0.f, bb = 0.f;
        if (eligible || scores) {
            const float4 *a = reinterpret_cast<const float4 *>(h_in);
            const float4 *b = reinterpret_cast<const float4 *>(h_out);
            for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
                const float4 x = __ldcg(a + i), y = __ldcg(b + i);
                ab += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
                aa += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
                bb += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
            }
            ab = warp_sum(ab); aa = warp_sum(aa); bb = warp_sum(bb);
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            if (lane == 0) { red[0][warp] = ab; red[1][warp] = aa; red[2][warp] = bb; }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            bool pass1 = false;
            if (gone_before == 0 && (eligible || scores)) {
                ab = aa = bb = 0.f;
                for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { ab += red[0][w]; aa += red[1][w]; bb += red[2][w]; }
                float sc = 0.f;
                if (aa > 0.f && bb > 0.f) sc = ab / (sqrtf(aa) * sqrtf(bb));
                pass1 = sc > tau_row;
                if (scores) scores[l - 1] = sc;
            }
            bool gone = gone_before != 0;
            if (!gone) {
                bool leave = eligible && pass1;  // with one row the batch minimum is the row itself
                if (forced_mine >= 0) leave = (forced_mine == l) && (l < L);
                if (leave) {
                    exited[0] = 1;
                    exit_layer[0] = l;
                    gone = true;
                }
            }
            (gone ? lists.riv_idx : lists.act_idx)[(size_t)l * lists.max_batch] = 0;
            lists.n_act[l] = gone ? 0 : 1;
            lists.n_riv[l] = gone ? 1 : 0;
            *hint_act = gone ? 0 : 1;
        }
        return;
    }
    if (row < n && exited[row] == 0 && (eligible || scores)) {
        const float4 *a = reinterpret_cast<const float4 *>(h_in + (size_t)row * d);
        const float4 *b = reinterpret_cast<const float4 *>(h_out + (size_t)row * d);
        float ab = 0.f, aa = 0.f, bb = 0.f;
        const int nv = d / 4;
        for (int i0 = 0; i0 < nv; i0 += 4 * 256) {  // four loads of each vector in flight per thread
            float4 x[4], y[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * 256 + threadIdx.x;
                x[u] = i < nv ? __ldcg(a + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                y[u] = i < nv ? __ldcg(b + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                ab += x[u].x * y[u].x + x[u].y * y[u].y + x[u].z * y[u].z + x[u].w * y[u].w;
                aa += x[u].x * x[u].x + x[u].y * x[u].y + x[u].z * x[u].z + x[u].w * x[u].w;
                bb += y[u].x * y[u].x + y[u].y * y[u].y + y[u].z * y[u].z + y[u].w * y[u].w;
            }
        }
        ab = warp_sum(ab); aa = warp_sum(aa); bb = warp_sum(bb);
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        if (lane == 0) { red[0][warp] = ab; red[1][warp] = aa; red[2][warp] = bb; }
        __syncthreads();
        if (threadIdx.x == 0) {
            ab = aa = bb = 0.f;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { ab += red[0][w]; aa += red[1][w]; bb += red[2][w]; }
            float s = 0.f;
            if (aa > 0.f && bb > 0.f) s = ab / (sqrtf(aa) * sqrtf(bb));
            pass[row] = (s > tau_row) ? 1 : 0;
            if (scores) scores[(size_t)row * L + (l - 1)] = s;
        }
    }
    if (gridDim.x > 1) {  // a single CTA is its own last arriver
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    } else {
        __syncthreads();
    }
    // ---- decision for every row still in the backbone
    if (threadIdx.x == 0) s_allpass = 1;
    __syncthreads();
    if (exit_mode == 1) {
        for (int b = threadIdx.x; b < n; b += blockDim.x)
            if (exited[b] == 0 && !(eligible && pass[b])) atomicAnd(&s_allpass, 0);
        __syncthreads();
    }
    for (int b = threadIdx.x; b < n; b += blockDim.x) {
        if (exited[b] != 0) continue;
        bool leave = eligible && (exit_mode == 1 ? (s_allpass != 0) : (pass[b] != 0));
        const int f = forced ? (b == (int)threadIdx.x ? forced_mine : forced[b]) : -1;
        if (f >= 0) leave = (f == l) && (l < L);
        if (leave) {
            exited[b] = 1;
            exit_layer[b] = l;
        }
    }
    __syncthreads();
    build_lists(n, exited, l, lists, hint_act, s_cnt);
    if (threadIdx.x == 0 && gridDim.x > 1) *ticket = 0;
}

// ---------------------------------------------------------------- a6 + a7 as the tail of the kernel that ends a block
// An alternative to the score kernel above for small steps (RIVER_F_FUSED_SCORE): the kernel that writes the block
// output (the down projection) finishes it: the last CTA to arrive (atomic ticket, no spinning)
// computes Eq. 1 for every row still in the backbone, takes the decisions and emits the row lists, exactly as
// score_compact_kernel does.
struct ScoreTail {
    const StepMeta *meta;   // null: the kernel has no tail
    int l, L, entry_layer, exit_mode, d;
    const float *h_in, *h_out;
    uint8_t *pass, *exited;
    Lists lists;
    int32_t *hint_act;
    unsigned *ticket;
};

__device__ __forceinline__ void score_tail(const ScoreTail &t) {
    __shared__ float red[3][32];
    __shared__ int s_cnt[66];
    __shared__ bool s_last;
    __shared__ int s_allpass;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(t.ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const int n = t.meta->n_rows, l = t.l, L = t.L, d = t.d;
    const float *tau = t.meta->tau;
    const int32_t *forced = t.meta->forced;
    int32_t *exit_layer = t.meta->exit_layer;
    float *scores = t.meta->scores;
    const bool eligible = (l >= 1) && (l >= t.entry_layer) && (l < L);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int row = 0; row < n; ++row) {
        if (t.exited[row] != 0 || !(eligible || scores)) continue;  // uniform
        const float4 *a = reinterpret_cast<const float4 *>(t.h_in + (size_t)row * d);
        const float4 *b = reinterpret_cast<const float4 *>(t.h_out + (size_t)row * d);
        float ab = 0.f, aa = 0.f, bb = 0.f;
        for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
            const float4 x = __ldcg(a + i), y = __ldcg(b + i);
            ab += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
            aa += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
            bb += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
        }
        ab = warp_sum(ab); aa = warp_sum(aa); bb = warp_sum(bb);
        __syncthreads();
        if (lane == 0) { red[0][warp] = ab; red[1][warp] = aa; red[2][warp] = bb; }
        __syncthreads();
        if (threadIdx.x == 0) {
            ab = aa = bb = 0.f;
            for (int w = 0; w < nwarps; ++w) { ab += red[0][w]; aa += red[1][w]; bb += red[2][w]; }
            float s = 0.f;
            if (aa > 0.f && bb > 0.f) s = ab / (sqrtf(aa) * sqrtf(bb));
            t.pass[row] = (s > tau[row]) ? 1 : 0;
            if (scores) scores[(size_t)row * L + (l - 1)] = s;
        }
    }
    if (threadIdx.x == 0) s_allpass = 1;
    __syncthreads();
    if (t.exit_mode == 1) {
        for (int b = threadIdx.x; b < n; b += blockDim.x)
            if (t.exited[b] == 0 && !(eligible && t.pass[b])) atomicAnd(&s_allpass, 0);
        __syncthreads();
    }
    for (int b = threadIdx.x; b < n; b += blockDim.x) {
        if (t.exited[b] != 0) continue;
        bool leave = eligible && (t.exit_mode == 1 ? (s_allpass != 0) : (t.pass[b] != 0));
        const int f = forced ? forced[b] : -1;
        if (f >= 0) leave = (f == l) && (l < L);
        if (leave) {
            t.exited[b] = 1;
            exit_layer[b] = l;
        }
    }
    __syncthreads();
    build_lists(n, t.exited, l, t.lists, t.hint_act, s_cnt);
    if (threadIdx.x == 0) *t.ticket = 0;
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

// ---------------------------------------------------------------- a3: paged GQA decode attention, plain version
// (a debugging aid selected by RIVER_F_SIMPLE_ATTN; the production kernel is in attn_decode.cuh)
// One CTA per (row, kv head): its GQ query heads share every K/V load.  A warp walks positions warp, warp+W, ...;
// a lane owns DH/32 head dims; softmax is online in fp32; the warps' partial states merge through shared memory.
template <int DH, int GQ>
__global__ void __launch_bounds__(128) attn_decode_kernel(const StepMeta *meta, const float *q, KvAddr kv,
                                                          float scale, int Hq, float *out) {
    constexpr int VE = DH / 32;
    constexpr int NW = 4;
    const int row = blockIdx.y, kvh = blockIdx.x;
    if (row >= meta->n_rows) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pos = kv.row_pos[row], slot = kv.row_slot[row];
    float qr[GQ][VE], acc[GQ][VE], m[GQ], l[GQ];
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
        m[g] = -CUDART_INF_F;
        l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < VE; ++e) {
            qr[g][e] = q[(size_t)row * Hq * DH + (size_t)(kvh * GQ + g) * DH + lane * VE + e] * scale;
            acc[g][e] = 0.f;
        }
    }
    for (int p = warp; p <= pos; p += NW) {
        const int page = kv.page_tbl[(size_t)slot * kv.max_pages_per_seq + p / kPage];
        const __nv_bfloat16 *kp = kv.pool + kv.base(page, 0, kvh, p % kPage) + lane * VE;
        const __nv_bfloat16 *vp = kv.pool + kv.base(page, 1, kvh, p % kPage) + lane * VE;
        float kf[VE], vf[VE];
#pragma unroll
        for (int e = 0; e < VE; ++e) { kf[e] = __bfloat162float(kp[e]); vf[e] = __bfloat162float(vp[e]); }
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < VE; ++e) s = fmaf(qr[g][e], kf[e], s);
            s = warp_sum(s);
            const float mn = fmaxf(m[g], s);
            const float corr = __expf(m[g] - mn), pr = __expf(s - mn);
            l[g] = l[g] * corr + pr;
#pragma unroll
            for (int e = 0; e < VE; ++e) acc[g][e] = fmaf(pr, vf[e], acc[g][e] * corr);
            m[g] = mn;
        }
    }
    __shared__ float s_m[NW][GQ], s_l[NW][GQ], s_acc[NW][GQ][DH];
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
        if (lane == 0) { s_m[warp][g] = m[g]; s_l[warp][g] = l[g]; }
#pragma unroll
        for (int e = 0; e < VE; ++e) s_acc[warp][g][lane * VE + e] = acc[g][e];
    }
    __syncthreads();
    for (int t = threadIdx.x; t < GQ * DH; t += blockDim.x) {
        const int g = t / DH, e = t % DH;
        float M = -CUDART_INF_F;
        for (int w = 0; w < NW; ++w) M = fmaxf(M, s_m[w][g]);
        float num = 0.f, den = 0.f;
        for (int w = 0; w < NW; ++w) {
            const float c = (s_m[w][g] == -CUDART_INF_F) ? 0.f : __expf(s_m[w][g] - M);
            num = fmaf(c, s_acc[w][g][e], num);
            den = fmaf(c, s_l[w][g], den);
        }
        out[(size_t)row * Hq * DH + (size_t)(kvh * GQ + g) * DH + e] = num / den;
    }
}

// ---------------------------------------------------------------- cache copy in / out (bf16 [n][Hkv][dh])
__global__ void kv_copy_kernel(KvAddr kv, int slot, int pos0, int n, __nv_bfloat16 *k_io, __nv_bfloat16 *v_io,
                               int to_cache) {
    const int i = blockIdx.x;  // position index
    if (i >= n) return;
    const int pos = pos0 + i;
    const int page = kv.page_tbl[(size_t)slot * kv.max_pages_per_seq + pos / kPage];
    const int w = kv.Hkv * kv.dh;
    for (int t = threadIdx.x; t < w; t += blockDim.x) {
        const int kvh = t / kv.dh, e = t % kv.dh;
        const size_t ok = kv.base(page, 0, kvh, pos % kPage) + e, ov = kv.base(page, 1, kvh, pos % kPage) + e;
        if (to_cache) {
            kv.pool[ok] = k_io[(size_t)i * w + t];
            kv.pool[ov] = v_io[(size_t)i * w + t];
        } else {
            k_io[(size_t)i * w + t] = kv.pool[ok];
            v_io[(size_t)i * w + t] = kv.pool[ov];
        }
    }
}

}  // namespace river
