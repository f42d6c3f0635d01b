// Weight-streaming projections on CUDA cores for small row counts (sm_100a).
//
// Every weight byte of a decode-step projection is used once per activation row, so the kernel is a stream: a warp
// owns R output features at a time, its lanes pull 16-byte pieces of those weight rows straight from HBM into
// registers (eight independent 128-bit loads in flight per lane), multiply them with up to N activation rows held
// in shared memory in fp32 and reduce with shuffles; latency is hidden by tens of such warps per SM.  The launch
// geometry is chosen per projection so that every warp gets the same number of tasks.  Weights never depend on the
// previous kernel, so with programmatic dependent launch each warp issues the first loads of its first task BEFORE
// the grid dependency resolves and the HBM stream keeps running across kernel boundaries.  The same launch serves
// the rows still in the backbone (bf16 weights) and the rows in the exit layers (4-bit codes + bf16 scale / zero
// per group, dequantised on the fly as (q - z) * s); which set is non-empty is read on the device.
#pragma once
#include "river_common.cuh"

namespace river {

// ---------------------------------------------------------------- problems
// A problem tells where the R rows of task t live (NRUN runs of R/NRUN consecutive rows) and what to do with the
// R x N results of a task.
struct RowLists {
    const int32_t *act_idx, *n_act, *riv_idx, *n_riv;
    const int32_t *hint_act;  // backbone row count as of the latest compaction; never under-counts (a prefetch hint)
    const int32_t *n_rows;    // rows of the step (per-step metadata, stable while the step runs)
    const uint8_t *state;     // sticky exit flags of the rows entering this block (steps of up to four rows build
                              // their lists from these: one load instead of count -> index)
};

struct QkvProblem {
    static constexpr int NRUN = 2;
    const uint16_t *wq, *wk, *wv;
    W4 rq, rk, rv;
    int K, Hq, Hkv, dh, group;
    const float2 *rope_cs;
    float *q_out;
    KvAddr kv;
    int *dev_err;
    template <int R>
    __device__ int n_tasks() const { return (Hq + 2 * Hkv) * (dh / 2) / (R / 2); }
    // task -> (matrix, head, first pair index)
    template <int R>
    __device__ void locate(int t, int &which, int &hl, int &i0) const {
        const int per_head = (dh / 2) / (R / 2);
        const int hh = t / per_head;
        i0 = (t % per_head) * (R / 2);
        if (hh < Hq) { which = 0; hl = hh; }
        else if (hh < Hq + Hkv) { which = 1; hl = hh - Hq; }
        else { which = 2; hl = hh - Hq - Hkv; }
    }
    template <int R>
    __device__ size_t run_row(int t, int run) const {  // first row of the run inside its matrix
        int which, hl, i0;
        locate<R>(t, which, hl, i0);
        return (size_t)hl * dh + i0 + run * (dh / 2);
    }
    template <int R>
    __device__ const uint16_t *bf16_base(int t, int) const {
        int which, hl, i0;
        locate<R>(t, which, hl, i0);
        return which == 0 ? wq : (which == 1 ? wk : wv);
    }
    template <int R>
    __device__ W4 w4_base(int t, int) const {
        int which, hl, i0;
        locate<R>(t, which, hl, i0);
        return which == 0 ? rq : (which == 1 ? rk : rv);
    }
    // results: res[r] for stage rows r = run * (R/2) + j  <->  features i0 + j (+ dh/2 for run 1)
    template <int R>
    __device__ void epilogue(int t, int row, const float (&res)[R]) const {
        int which, hl, i0;
        locate<R>(t, which, hl, i0);
        const int half = dh / 2;
        const int pos = kv.row_pos[row];
        int page = 0;
        if (which != 0) {
            page = kv.row_page[row];
            if (page < 0 || page >= kv.n_pages) { atomicExch(dev_err, DEV_BAD_PAGE); return; }
        }
#pragma unroll
        for (int j = 0; j < R / 2; ++j) {
            float lo = res[j], hi = res[R / 2 + j];
            const int i = i0 + j;
            if (which != 2) {
                const float2 cs = rope_cs[(size_t)row * half + i];
                const float rl = lo * cs.x - hi * cs.y, rh = hi * cs.x + lo * cs.y;
                lo = rl; hi = rh;
            }
            if (which == 0) {
                float *q = q_out + (size_t)row * (Hq * dh) + (size_t)hl * dh;
                q[i] = lo;
                q[i + half] = hi;
            } else {
                const size_t o = kv.base(page, which - 1, hl, pos % kPage);
                kv.pool[o + i] = __float2bfloat16_rn(lo);
                kv.pool[o + i + half] = __float2bfloat16_rn(hi);
            }
        }
    }
    // What the epilogue of a two-row task reads besides the dot products, requested BEFORE the dot products are
    // computed so that the loads travel meanwhile: rotary cos / sin, position and write page of the row.
    __device__ void epi_pre(int t, int row, float (&e)[4]) const {
        int which, hl, i0;
        locate<2>(t, which, hl, i0);
        if (which != 2) {
            const float2 cs = rope_cs[(size_t)row * (dh / 2) + i0];
            e[0] = cs.x;
            e[1] = cs.y;
        }
        if (which != 0) {
            e[2] = __int_as_float(kv.row_pos[row]);
            e[3] = __int_as_float(kv.row_page[row]);
        }
    }
    __device__ void epilogue_pre(int t, int row, const float (&res)[2], const float (&e)[4]) const {
        int which, hl, i0;
        locate<2>(t, which, hl, i0);
        const int half = dh / 2;
        float lo = res[0], hi = res[1];
        if (which != 2) {
            const float rl = lo * e[0] - hi * e[1], rh = hi * e[0] + lo * e[1];
            lo = rl; hi = rh;
        }
        if (which == 0) {
            float *q = q_out + (size_t)row * (Hq * dh) + (size_t)hl * dh;
            q[i0] = lo;
            q[i0 + half] = hi;
        } else {
            const int pos = __float_as_int(e[2]), page = __float_as_int(e[3]);
            if (page < 0 || page >= kv.n_pages) { atomicExch(dev_err, DEV_BAD_PAGE); return; }
            const size_t o = kv.base(page, which - 1, hl, pos % kPage);
            kv.pool[o + i0] = __float2bfloat16_rn(lo);
            kv.pool[o + i0 + half] = __float2bfloat16_rn(hi);
        }
    }
};

struct ResidProblem {  // out[row][o] = resid[row][o] + W[o] . x[row]
    static constexpr int NRUN = 1;
    const uint16_t *w;
    W4 rw;
    int K, out_dim, group;
    const float *resid;
    float *out;
    template <int R> __device__ int n_tasks() const { return out_dim / R; }
    template <int R> __device__ size_t run_row(int t, int) const { return (size_t)t * R; }
    template <int R> __device__ const uint16_t *bf16_base(int, int) const { return w; }
    template <int R> __device__ W4 w4_base(int, int) const { return rw; }
    template <int R>
    __device__ void epilogue(int t, int row, const float (&res)[R]) const {
        const size_t o = (size_t)row * out_dim + (size_t)t * R;
#pragma unroll
        for (int r = 0; r < R; ++r) out[o + r] = __ldcg(resid + o + r) + res[r];  // L2: written by other SMs
    }
    __device__ void epi_pre(int t, int row, float (&e)[4]) const {
        const float2 v = __ldcg(reinterpret_cast<const float2 *>(resid + (size_t)row * out_dim + (size_t)t * 2));
        e[0] = v.x;
        e[1] = v.y;
    }
    __device__ void epilogue_pre(int t, int row, const float (&res)[2], const float (&e)[4]) const {
        *reinterpret_cast<float2 *>(out + (size_t)row * out_dim + (size_t)t * 2) = make_float2(e[0] + res[0], e[1] + res[1]);
    }
};

struct GateUpProblem {  // act[row][f] = silu(Wg[f] . y) * (Wu[f] . y)
    static constexpr int NRUN = 2;
    const uint16_t *wg, *wu;
    W4 rg, ru;
    int K, F, group;
    float *act;
    template <int R> __device__ int n_tasks() const { return F / (R / 2); }
    template <int R> __device__ size_t run_row(int t, int) const { return (size_t)t * (R / 2); }
    template <int R> __device__ const uint16_t *bf16_base(int, int run) const { return run == 0 ? wg : wu; }
    template <int R> __device__ W4 w4_base(int, int run) const { return run == 0 ? rg : ru; }
    template <int R>
    __device__ void epilogue(int t, int row, const float (&res)[R]) const {
#pragma unroll
        for (int j = 0; j < R / 2; ++j) {
            const float g = res[j], u = res[R / 2 + j];
            act[(size_t)row * F + (size_t)t * (R / 2) + j] = g / (1.f + __expf(-g)) * u;
        }
    }
    __device__ void epi_pre(int, int, float (&)[4]) const {}
    __device__ void epilogue_pre(int t, int row, const float (&res)[2], const float (&)[4]) const { epilogue<2>(t, row, res); }
};


// The exit decision of the block that has just finished, taken by the kernel that consumes its output (steps of up
// to four rows): Eq. 1 on the block's input and output, strict s > tau in fp32, the eligibility window
// entry_layer <= l < L, the forced-exit hook and the batch mode.  Every CTA of the launch computes it from the same
// data with the same reduction order (all CTAs of a launch have the same shape), so all CTAs agree on which weight
// set every row takes and no kernel boundary is spent on the decision; CTA 0 publishes exit flags, exit layers,
// scores, the two row lists and the prefetch hint for the kernels and host queries that follow.
struct DecideArgs {
    const StepMeta *meta;      // null: this launch takes no decision
    int l;                     // the block being scored (1-based); its output is this launch's input rows
    int L, entry_layer, exit_mode;
    const float *h_prev;       // input of block l, fp32 [rows][K]
    const uint8_t *state_in;   // exit flags entering block l
    uint8_t *state_out;        // exit flags entering block l + 1
    Lists lists;
    int32_t *hint_act;
    int32_t *fail;             // optional [slots][L + 1]: set to 1 where a row's score does NOT pass its threshold (the
    const int32_t *row_slot;   // prefill pass that looks for the unified depth); row_slot maps rows to sequence slots
};

// Activation rows of the exit layers as 16-bit block floating point (the A16 of the paper's W4A16, Section 4.1): every
// 32-input chunk of a row shares one fp32 scale (max |x| / 16383), an input is a signed 15-bit integer v = 128 hi + lo
// split into two byte digits, so that a 4-bit code times an input is an exact integer product and four of them are ONE
// dp4a.  Per chunk c the digits sit in four 16-byte pieces [hi of code words 0-1 | hi of words 2-3 | lo of words 0-1 |
// lo of words 2-3], a piece holding (even inputs of word a, odd inputs of word a, even of word b, odd of word b) - the
// byte order of the isolated even / odd nibbles of a code word; piece p of the 32 chunks of a group is contiguous, so
// a lane that owns a chunk reads its pieces with conflict-free 128-bit loads.  xsc[c] is the scale, xsum[c] = scale *
// sum of v over the chunk (what the zero-point multiplies).  Rows are read in plain fp32 order from xs.
__host__ __device__ inline int xq_stride16(int K) { return (((K >> 5) + 31) >> 5) * 128; }  // uint4 per row

template <int N>
__device__ __forceinline__ void stream_quantise_rows(const float *xs, int K, int xstride, uint4 *xq, float *xsc,
                                                     float *xsum) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int nw = K >> 3, nch = K >> 5;  // 8-input words (four per chunk: four adjacent lanes share a chunk)
    const int total = N * nw;
    uint32_t *xq32 = reinterpret_cast<uint32_t *>(xq);
    for (int u0 = 0; u0 < total; u0 += nthr) {
        const int unit = u0 + tid;
        const bool valid = unit < total;
        const int n = valid ? unit / nw : 0, w = valid ? unit % nw : 0;
        const int c = w >> 2, wd = w & 3;
        float x[8];
        if (valid) {
            const float4 a = *reinterpret_cast<const float4 *>(xs + n * xstride + 8 * w);
            const float4 b = *reinterpret_cast<const float4 *>(xs + n * xstride + 8 * w + 4);
            x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = 0.f;
        }
        float m = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(x[i]));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
        const float inv = m > 0.f ? 16383.f / m : 0.f;
        int v[8], sv = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { v[i] = __float2int_rn(x[i] * inv); sv += v[i]; }
        sv += __shfl_xor_sync(0xffffffffu, sv, 1);
        sv += __shfl_xor_sync(0xffffffffu, sv, 2);
        if (valid) {
            auto pack = [](int b0, int b1, int b2, int b3) {
                return (uint32_t)(b0 & 255) | ((uint32_t)(b1 & 255) << 8) | ((uint32_t)(b2 & 255) << 16) | ((uint32_t)(b3 & 255) << 24);
            };
            const uint32_t hi_e = pack(v[0] >> 7, v[2] >> 7, v[4] >> 7, v[6] >> 7), hi_o = pack(v[1] >> 7, v[3] >> 7, v[5] >> 7, v[7] >> 7);
            const uint32_t lo_e = pack(v[0] & 127, v[2] & 127, v[4] & 127, v[6] & 127), lo_o = pack(v[1] & 127, v[3] & 127, v[5] & 127, v[7] & 127);
            uint32_t *row = xq32 + (size_t)n * xq_stride16(K) * 4;
            const int g = c >> 5, cl = c & 31;
            uint32_t *ph = row + ((g * 4 + (wd >> 1)) * 32 + cl) * 4 + (wd & 1) * 2;
            uint32_t *pl = row + ((g * 4 + 2 + (wd >> 1)) * 32 + cl) * 4 + (wd & 1) * 2;
            *reinterpret_cast<uint2 *>(ph) = make_uint2(hi_e, hi_o);
            *reinterpret_cast<uint2 *>(pl) = make_uint2(lo_e, lo_o);
            if (wd == 0) {
                const float sc = m * (1.f / 16383.f);
                xsc[n * nch + c] = sc;
                xsum[n * nch + c] = sc * (float)sv;
            }
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------- activation rows -> shared memory
// All threads of the CTA load up to N rows idx[i0..], optionally RMS-normalise them, and store them fp32 in the
// lane-interleaved order for E inputs per chunk (8: bf16 weights) or in plain order (E = 0: the exit-layer rows, which
// the caller then turns into block-floating-point digits).
template <int N, int E>
__device__ __forceinline__ void stream_load_rows(const ProjIn &in, const int32_t *idx, int i0, int cnt, int K,
                                                 int xstride, float *xs, float *red) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    for (int n = 0; n < N; ++n) {
        float *dst = xs + n * xstride;
        if (i0 + n >= cnt) {
            for (int k = tid; k < xstride; k += nthr) dst[k] = 0.f;
            continue;
        }
        const float4 *src = reinterpret_cast<const float4 *>(in.src + (size_t)idx[i0 + n] * K);
        const int nv = K >> 2;
        float ss = 0.f;
        for (int v0 = 0; v0 < nv; v0 += nthr * 4) {
            float4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = v0 + u * nthr + tid;
                x[u] = v < nv ? __ldcg(src + v) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = v0 + u * nthr + tid;
                if (v < nv) {
                    ss += x[u].x * x[u].x + x[u].y * x[u].y + x[u].z * x[u].z + x[u].w * x[u].w;
                    *reinterpret_cast<float4 *>(dst + xs_index<E>(4 * v)) = x[u];
                }
            }
        }
        if (in.gain) {
            ss = warp_sum(ss);
            if ((tid & 31) == 0) red[tid >> 5] = ss;
            __syncthreads();
            ss = 0.f;
            for (int w = 0; w < (nthr >> 5); ++w) ss += red[w];
            const float scale = rsqrtf(ss / (float)K + in.eps);
            __syncthreads();
            for (int v = tid; v < nv; v += nthr) {
                float4 *p = reinterpret_cast<float4 *>(dst + xs_index<E>(4 * v));
                const uint2 gw = *reinterpret_cast<const uint2 *>(in.gain + 4 * v);
                float4 x = *p;
                x.x *= scale * bf16lo(gw.x); x.y *= scale * bf16hi(gw.x);
                x.z *= scale * bf16lo(gw.y); x.w *= scale * bf16hi(gw.y);
                *p = x;
            }
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------- one task = R weight rows against N activation rows
constexpr int kStreamPF = 4;  // 16-byte loads per weight row issued together (R * kStreamPF in flight per lane)

template <int R>
__device__ __forceinline__ void stream_issue_bf16(const uint16_t *const (&wrow)[R], int nch, int it0, int lane,
                                                  uint4 (&w)[R][kStreamPF]) {
#pragma unroll
    for (int u = 0; u < kStreamPF; ++u) {
        const int c = (it0 + u) * 32 + lane;
#pragma unroll
        for (int r = 0; r < R; ++r)
            w[r][u] = c < nch ? ldg_stream16(wrow[r] + (size_t)c * 8) : make_uint4(0u, 0u, 0u, 0u);
    }
}

// bf16 weights: lane owns the 8-input chunks lane, lane + 32, ...; `pre` holds the first kStreamPF chunks per row if
// they were loaded before the grid dependency resolved.
template <int N, int R>
__device__ __forceinline__ void stream_dots_bf16(const uint16_t *const (&wrow)[R], const float *xs, int K, int xstride,
                                                 bool have_pre, uint4 (&pre)[R][kStreamPF], float (&acc)[R][N]) {
    const int lane = threadIdx.x & 31;
    const int nch = K >> 3, nit = (nch + 31) >> 5;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
    for (int it0 = 0; it0 < nit; it0 += kStreamPF) {
        uint4 w[R][kStreamPF];
        if (it0 == 0 && have_pre) {
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int u = 0; u < kStreamPF; ++u) w[r][u] = pre[r][u];
        } else {
            stream_issue_bf16<R>(wrow, nch, it0, lane, w);
        }
#pragma unroll
        for (int u = 0; u < kStreamPF; ++u) {
            const int c = (it0 + u) * 32 + lane;
            if (c < nch) {
                const float *xb = xs + (c >> 5) * 256 + lane * 4;
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    const float4 x0 = *reinterpret_cast<const float4 *>(xb + n * xstride);
                    const float4 x1 = *reinterpret_cast<const float4 *>(xb + n * xstride + 128);
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const uint4 v = w[r][u];
                        float a0 = bf16lo(v.x) * x0.x, a1 = bf16hi(v.x) * x0.y;
                        a0 = fmaf(bf16lo(v.y), x0.z, a0); a1 = fmaf(bf16hi(v.y), x0.w, a1);
                        a0 = fmaf(bf16lo(v.z), x1.x, a0); a1 = fmaf(bf16hi(v.z), x1.y, a1);
                        a0 = fmaf(bf16lo(v.w), x1.z, a0); a1 = fmaf(bf16hi(v.w), x1.w, a1);
                        acc[r][n] += a0 + a1;
                    }
                }
            }
        }
    }
}

// 4-bit weights: lane owns the 32-input chunks lane, lane + 32, ... (16 bytes of codes each) and multiplies them with
// the block-floating-point digits of the activations: the even and the odd nibbles of a code word, isolated with one
// mask each, are four byte operands of dp4a, so eight weights cost three logic operations and four integer dot
// products (two digits), and the chunk's scale and zero-point enter once per 32 weights.
template <int R>
struct W4Batch {
    static constexpr int PF = R <= 2 ? kStreamPF : kStreamPF / 2;  // chunks per row in flight: 8 code loads per lane
    uint4 q[R][kStreamPF];      // (sized for the bf16 prefetch that shares these registers)
    uint32_t sz[R][PF];         // scale (low half) and zero (high half) of the chunk's group, bf16 bits
};

template <int R>
__device__ __forceinline__ void stream_issue_w4(const W4 (&wrow)[R], int nch, int gshift, int it0, int lane,
                                                W4Batch<R> &b) {
#pragma unroll
    for (int u = 0; u < W4Batch<R>::PF; ++u) {
        const int c = (it0 + u) * 32 + lane;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (c < nch) {
                b.q[r][u] = ldg_stream16(wrow[r].codes + (size_t)c * 16);
                b.sz[r][u] = (uint32_t)ldg_u16(wrow[r].scale + (c >> gshift)) |
                             ((uint32_t)ldg_u16(wrow[r].zero + (c >> gshift)) << 16);
            } else {
                b.q[r][u] = make_uint4(0u, 0u, 0u, 0u);
                b.sz[r][u] = 0u;
            }
        }
    }
}

// One batch of chunks (already in registers) against the staged rows: the inner step of the pipelined passes below.
template <int N, int R>
__device__ __forceinline__ void stream_fma_bf16(const uint4 (&w)[R][kStreamPF], const float *xs, int xstride, int it0,
                                                int nch, int lane, float (&acc)[R][N]) {
#pragma unroll
    for (int u = 0; u < kStreamPF; ++u) {
        const int c = (it0 + u) * 32 + lane;
        if (c < nch) {
            const float *xb = xs + (c >> 5) * 256 + lane * 4;
#pragma unroll
            for (int n = 0; n < N; ++n) {
                const float4 x0 = *reinterpret_cast<const float4 *>(xb + n * xstride);
                const float4 x1 = *reinterpret_cast<const float4 *>(xb + n * xstride + 128);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const uint4 v = w[r][u];
                    float a0 = bf16lo(v.x) * x0.x, a1 = bf16hi(v.x) * x0.y;
                    a0 = fmaf(bf16lo(v.y), x0.z, a0); a1 = fmaf(bf16hi(v.y), x0.w, a1);
                    a0 = fmaf(bf16lo(v.z), x1.x, a0); a1 = fmaf(bf16hi(v.z), x1.y, a1);
                    a0 = fmaf(bf16lo(v.w), x1.z, a0); a1 = fmaf(bf16hi(v.w), x1.w, a1);
                    acc[r][n] += a0 + a1;
                }
            }
        }
    }
}

template <int N, int R>
__device__ __forceinline__ void stream_fma_w4(const W4Batch<R> &b, const uint4 *xq, const float *xsc, const float *xsum,
                                              int xqs, int it0, int nch, int lane, float (&acc)[R][N]) {
#pragma unroll
    for (int u = 0; u < W4Batch<R>::PF; ++u) {
        const int c = (it0 + u) * 32 + lane;
        if (c < nch) {
#pragma unroll
            for (int n = 0; n < N; ++n) {
                const uint4 *xb = xq + n * xqs + (c >> 5) * 128 + lane;
                const uint4 h01 = xb[0], h23 = xb[32], l01 = xb[64], l23 = xb[96];
                const float sc = xsc[n * nch + c], sx = xsum[n * nch + c];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const uint4 q = b.q[r][u];
                    int dh = 0, dl = 0;
                    uint32_t e, o;
                    e = q.x & 0x0f0f0f0fu; o = (q.x >> 4) & 0x0f0f0f0fu;  // bytes: even / odd inputs of the code word
                    dh = __dp4a((int)e, (int)h01.x, dh); dh = __dp4a((int)o, (int)h01.y, dh);
                    dl = __dp4a((int)e, (int)l01.x, dl); dl = __dp4a((int)o, (int)l01.y, dl);
                    e = q.y & 0x0f0f0f0fu; o = (q.y >> 4) & 0x0f0f0f0fu;
                    dh = __dp4a((int)e, (int)h01.z, dh); dh = __dp4a((int)o, (int)h01.w, dh);
                    dl = __dp4a((int)e, (int)l01.z, dl); dl = __dp4a((int)o, (int)l01.w, dl);
                    e = q.z & 0x0f0f0f0fu; o = (q.z >> 4) & 0x0f0f0f0fu;
                    dh = __dp4a((int)e, (int)h23.x, dh); dh = __dp4a((int)o, (int)h23.y, dh);
                    dl = __dp4a((int)e, (int)l23.x, dl); dl = __dp4a((int)o, (int)l23.y, dl);
                    e = q.w & 0x0f0f0f0fu; o = (q.w >> 4) & 0x0f0f0f0fu;
                    dh = __dp4a((int)e, (int)h23.z, dh); dh = __dp4a((int)o, (int)h23.w, dh);
                    dl = __dp4a((int)e, (int)l23.z, dl); dl = __dp4a((int)o, (int)l23.w, dl);
                    // sum_k (q_k - z) s x_k = s (scale * sum_k q_k v_k - z * scale * sum_k v_k), the integer sum exact
                    const float s = bf16lo(b.sz[r][u]), z = bf16hi(b.sz[r][u]);
                    acc[r][n] = fmaf(s, fmaf(sc, (float)(dh * 128 + dl), -z * sx), acc[r][n]);
                }
            }
        }
    }
}

// ---------------------------------------------------------------- the kernel
template <class P, int R>
__device__ __forceinline__ void stream_rows_bf16(const P &p, int t, const uint16_t *(&rows)[R]) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int run = r / (R / P::NRUN), j = r % (R / P::NRUN);
        rows[r] = p.template bf16_base<R>(t, run) + (p.template run_row<R>(t, run) + j) * (size_t)p.K;
    }
}
template <class P, int R>
__device__ __forceinline__ void stream_rows_w4(const P &p, int t, W4 (&rows)[R]) {
    const int ng = p.K / p.group;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int run = r / (R / P::NRUN), j = r % (R / P::NRUN);
        const W4 b = p.template w4_base<R>(t, run);
        const size_t row = p.template run_row<R>(t, run) + j;
        rows[r] = W4{b.codes + row * (size_t)(p.K >> 1), b.scale + row * ng, b.zero + row * ng};
    }
}

// Eq. 1 score from the three sums, as the score kernel computes it: a zero norm gives 0, no epsilon.
__device__ __forceinline__ float transition_score(float ab, float aa, float bb) {
    return (aa > 0.f && bb > 0.f) ? ab / (sqrtf(aa) * sqrtf(bb)) : 0.f;
}

// The decision for up to four rows from their scores (every thread computes the same): flags entering block l + 1.
// CTA 0 / thread 0 publishes.  gone_in / sc are indexed by row; returns the new flags as bits.
template <int N>
__device__ __forceinline__ uint32_t stream_decide(const DecideArgs &dec, int n, uint32_t gone_in, const float (&sc)[N],
                                                  const float (&tau)[N], const int (&forced)[N]) {
    const int l = dec.l;
    const bool eligible = (l >= 1) && (l >= dec.entry_layer) && (l < dec.L);
    bool allpass = true;
#pragma unroll
    for (int b = 0; b < N; ++b)
        if (b < n && !((gone_in >> b) & 1u) && !(eligible && sc[b] > tau[b])) allpass = false;
    uint32_t gone = gone_in;
#pragma unroll
    for (int b = 0; b < N; ++b) {
        if (b >= n || ((gone_in >> b) & 1u)) continue;
        bool leave = eligible && (dec.exit_mode == 1 ? allpass : (sc[b] > tau[b]));
        if (forced[b] >= 0) leave = (forced[b] == l) && (l < dec.L);
        if (leave) gone |= 1u << b;
    }
    return gone;
}

template <int N>
__device__ __forceinline__ void stream_publish(const DecideArgs &dec, int n, uint32_t gone_in, uint32_t gone,
                                               const float (&sc)[N], const float (&tau)[N]) {
    const int l = dec.l;
    int32_t *exit_layer = dec.meta->exit_layer;
    float *scores = dec.meta->scores;
    int32_t *A = dec.lists.act_idx + (size_t)l * dec.lists.max_batch;
    int32_t *Rv = dec.lists.riv_idx + (size_t)l * dec.lists.max_batch;
    int na = 0, nr = 0;
#pragma unroll
    for (int b = 0; b < N; ++b) {
        if (b >= n) continue;
        const bool was = (gone_in >> b) & 1u, is = (gone >> b) & 1u;
        dec.state_out[b] = is ? 1 : 0;
        if (!was) {
            if (scores) scores[(size_t)b * dec.L + (l - 1)] = sc[b];
            if (is) exit_layer[b] = l;
            if (dec.fail && !(sc[b] > tau[b])) dec.fail[(size_t)dec.row_slot[b] * (dec.L + 1) + l] = 1;
        }
        if (is) Rv[nr++] = b;
        else A[na++] = b;
    }
    dec.lists.n_act[l] = na;
    dec.lists.n_riv[l] = nr;
    *dec.hint_act = na;
}

// A step of ONE row (the latency-critical case): exit flag, the row and (when this launch decides) the previous
// block's input are requested together - one memory round trip after the grid dependency - then Eq. 1, the decision
// (published by CTA 0), the RMS norm, and the row in shared memory in the layout of the weight set it takes: fp32 in
// the lane-interleaved order for the bf16 weights, block-floating-point digits for the 4-bit ones.  Returns whether
// the row is on the exit layers.  gr: the norm gain of this thread's pieces, fetched before the wait.
template <int XF>
__device__ __forceinline__ bool stream_stage_one(const ProjIn &in, const DecideArgs &dec, const uint8_t *state, int K,
                                                 int xstride, float *red, float *xs, uint4 *xq, float *xsc, float *xsum,
                                                 const uint2 (&gr)[XF], float tau0, int forced0) {
    const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31, nwarps = nthr >> 5;
    const int nv = K >> 2;
    const uint8_t flag_in = __ldcg(state);
    float4 xr[XF];
    float bb = 0.f, ab = 0.f, aa = 0.f;
    const float4 *src = reinterpret_cast<const float4 *>(in.src);
#pragma unroll
    for (int k = 0; k < XF; ++k) {
        const int v = tid + k * nthr;
        xr[k] = v < nv ? __ldcg(src + v) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (dec.meta) {
        const float4 *prv = reinterpret_cast<const float4 *>(dec.h_prev);
        float4 xp[XF];
#pragma unroll
        for (int k = 0; k < XF; ++k) {
            const int v = tid + k * nthr;
            xp[k] = v < nv ? __ldcg(prv + v) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < XF; ++k) {
            ab += xp[k].x * xr[k].x + xp[k].y * xr[k].y + xp[k].z * xr[k].z + xp[k].w * xr[k].w;
            aa += xp[k].x * xp[k].x + xp[k].y * xp[k].y + xp[k].z * xp[k].z + xp[k].w * xp[k].w;
        }
    }
#pragma unroll
    for (int k = 0; k < XF; ++k) bb += xr[k].x * xr[k].x + xr[k].y * xr[k].y + xr[k].z * xr[k].z + xr[k].w * xr[k].w;
    bool riv = flag_in != 0;
    if (in.gain || dec.meta) {
        bb = warp_sum(bb);
        if (dec.meta) { ab = warp_sum(ab); aa = warp_sum(aa); }
        if (lane == 0) { red[warp] = bb; red[16 + warp] = ab; red[32 + warp] = aa; }
        __syncthreads();
        bb = ab = aa = 0.f;
        for (int w = 0; w < nwarps; ++w) { bb += red[w]; ab += red[16 + w]; aa += red[32 + w]; }
    }
    if (dec.meta) {
        const float sc[1] = {transition_score(ab, aa, bb)}, tau[1] = {tau0};
        const int forced[1] = {forced0};
        const uint32_t gone_in = flag_in ? 1u : 0u;
        const uint32_t gone = stream_decide<1>(dec, 1, gone_in, sc, tau, forced);
        if (blockIdx.x == 0 && tid == 0) stream_publish<1>(dec, 1, gone_in, gone, sc, tau);
        riv = gone != 0;
    }
    const float scale = in.gain ? rsqrtf(bb / (float)K + in.eps) : 1.f;
#pragma unroll
    for (int k = 0; k < XF; ++k) {
        const int v = tid + k * nthr;
        if (v < nv) {
            float4 y = xr[k];
            if (in.gain) {
                y.x *= scale * bf16lo(gr[k].x); y.y *= scale * bf16hi(gr[k].x);
                y.z *= scale * bf16lo(gr[k].y); y.w *= scale * bf16hi(gr[k].y);
            }
            if (riv) *reinterpret_cast<float4 *>(xs + 4 * v) = y;
            else *reinterpret_cast<float4 *>(xs + xs_index<8>(4 * v)) = y;
        }
    }
    __syncthreads();
    if (riv) stream_quantise_rows<1>(xs, K, xstride, xq, xsc, xsum);
    return riv;
}

// ---------------------------------------------------------------- the two passes over a CTA's tasks
// A warp walks its tasks batch by batch (kStreamPF chunks of each of the R rows) with the NEXT batch's loads - the
// same task's next chunks or the next task's first ones - issued before the current batch is multiplied, so its
// loads are in flight during the arithmetic, the warp reduction and the epilogue of a task as well as across task
// boundaries.  The very first batch may have been loaded before the grid dependency resolved.
template <class P, int N, int R>
__device__ __forceinline__ void stream_pass_bf16(const P &p, const ProjIn &in, const int32_t *act_idx, int na, int xstride,
                                                 float *xs, float *red, int t0, int t1, bool prestaged,
                                                 bool fast, bool have_pre, uint4 (&pre)[R][kStreamPF]) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int K = p.K, nch = K >> 3, nit = (nch + 31) >> 5;
    constexpr bool PIPE = N * R <= 2;  // more rows: the second register set would spill
    for (int i0 = 0; i0 < na; i0 += N) {
        if (!prestaged) {
            __syncthreads();
            stream_load_rows<N, 8>(in, act_idx, i0, na, K, xstride, xs, red);
        }
        int t = t0 + warp;
        if (t >= t1) continue;
        const uint16_t *rows[R];
        stream_rows_bf16<P, R>(p, t, rows);
        bool loaded = have_pre && i0 == 0;  // `pre` already holds the batch that comes next
        if constexpr (PIPE) {
            if (!loaded) stream_issue_bf16<R>(rows, nch, 0, lane, pre);
        }
        for (; t < t1; t += nwarps) {
            float acc[R][N];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
            float ep[4] = {0.f, 0.f, 0.f, 0.f};
            if constexpr (N == 1 && R == 2) {
                if (fast && lane == 0) p.epi_pre(t, 0, ep);  // travels while the dot products are computed
            }
            for (int it0 = 0; it0 < nit; it0 += kStreamPF) {
                if constexpr (PIPE) {
                    uint4 w[R][kStreamPF];
#pragma unroll
                    for (int r = 0; r < R; ++r)
#pragma unroll
                        for (int u = 0; u < kStreamPF; ++u) w[r][u] = pre[r][u];
                    if (it0 + kStreamPF < nit) {
                        stream_issue_bf16<R>(rows, nch, it0 + kStreamPF, lane, pre);
                    } else if (t + nwarps < t1) {
                        const uint16_t *nrows[R];
                        stream_rows_bf16<P, R>(p, t + nwarps, nrows);
                        stream_issue_bf16<R>(nrows, nch, 0, lane, pre);
                    }
                    stream_fma_bf16<N, R>(w, xs, xstride, it0, nch, lane, acc);
                } else {
                    if (!loaded) stream_issue_bf16<R>(rows, nch, it0, lane, pre);
                    loaded = false;
                    stream_fma_bf16<N, R>(pre, xs, xstride, it0, nch, lane, acc);
                }
            }
#pragma unroll
            for (int n2 = 0; n2 < N; ++n2) {
                float res[R];
#pragma unroll
                for (int r = 0; r < R; ++r) res[r] = warp_sum(acc[r][n2]);
                if (lane == n2 && i0 + n2 < na) {
                    if constexpr (N == 1 && R == 2) {
                        if (fast) p.epilogue_pre(t, 0, res, ep);
                        else p.template epilogue<R>(t, act_idx[i0 + n2], res);
                    } else {
                        p.template epilogue<R>(t, act_idx[i0 + n2], res);
                    }
                }
            }
            if (t + nwarps < t1) stream_rows_bf16<P, R>(p, t + nwarps, rows);
        }
    }
}

template <class P, int N, int R, bool PRE>
__device__ __forceinline__ void stream_pass_w4(const P &p, const ProjIn &in, const int32_t *riv_idx, int nr, int xstride,
                                               float *xs, uint4 *xq, float *xsc, float *xsum, float *red, int t0, int t1,
                                               bool prestaged,
                                               bool fast, W4Batch<R> &pre) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int K = p.K, nch = K >> 5, nit = (nch + 31) >> 5;
    const int gshift = (p.group == 64) ? 1 : (p.group == 32 ? 0 : 2);
    constexpr int PF = W4Batch<R>::PF;
    const int xqs = xq_stride16(K);
    constexpr bool PIPE = false;  // measured: issuing the next batch early makes the 4-bit pass slower, not faster
    for (int i0 = 0; i0 < nr; i0 += N) {
        if (!prestaged) {
            __syncthreads();
            stream_load_rows<N, 0>(in, riv_idx, i0, nr, K, xstride, xs, red);
            stream_quantise_rows<N>(xs, K, xstride, xq, xsc, xsum);
        }
        int t = t0 + warp;
        if (t >= t1) continue;
        W4 rows[R];
        stream_rows_w4<P, R>(p, t, rows);
        bool loaded = PRE && i0 == 0;
        if constexpr (PIPE) {
            if (!loaded) stream_issue_w4<R>(rows, nch, gshift, 0, lane, pre);
        }
        for (; t < t1; t += nwarps) {
            float acc[R][N];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
            float ep[4] = {0.f, 0.f, 0.f, 0.f};
            if constexpr (N == 1 && R == 2) {
                if (fast && lane == 0) p.epi_pre(t, 0, ep);
            }
            for (int it0 = 0; it0 < nit; it0 += PF) {
                if constexpr (PIPE) {
                    const W4Batch<R> b = pre;
                    if (it0 + PF < nit) {
                        stream_issue_w4<R>(rows, nch, gshift, it0 + PF, lane, pre);
                    } else if (t + nwarps < t1) {
                        W4 nrows[R];
                        stream_rows_w4<P, R>(p, t + nwarps, nrows);
                        stream_issue_w4<R>(nrows, nch, gshift, 0, lane, pre);
                    }
                    stream_fma_w4<N, R>(b, xq, xsc, xsum, xqs, it0, nch, lane, acc);
                } else {
                    if (!loaded) stream_issue_w4<R>(rows, nch, gshift, it0, lane, pre);
                    loaded = false;
                    stream_fma_w4<N, R>(pre, xq, xsc, xsum, xqs, it0, nch, lane, acc);
                }
            }
#pragma unroll
            for (int n2 = 0; n2 < N; ++n2) {
                float res[R];
#pragma unroll
                for (int r = 0; r < R; ++r) res[r] = warp_sum(acc[r][n2]);
                if (lane == n2 && i0 + n2 < nr) {
                    if constexpr (N == 1 && R == 2) {
                        if (fast) p.epilogue_pre(t, 0, res, ep);
                        else p.template epilogue<R>(t, riv_idx[i0 + n2], res);
                    } else {
                        p.template epilogue<R>(t, riv_idx[i0 + n2], res);
                    }
                }
            }
            if (t + nwarps < t1) stream_rows_w4<P, R>(p, t + nwarps, rows);
        }
    }
}

template <class P, int N, int R>
__global__ void __launch_bounds__(512) stream_proj_kernel(const P p, const ProjIn in, const RowLists rl, int has_river,
                                                          int xstride, int skip_backbone, const DecideArgs dec) {
    extern __shared__ __align__(16) float stream_smem[];
    const int K = p.K;
    float *red = stream_smem;            // 64: block reductions (up to three sums x 16 warps)
    const int nchp = ((K >> 5) + 3) & ~3;  // keeps what follows 16-byte aligned
    float *xsum = stream_smem + 64;      // N * K/32
    float *xsc = xsum + N * nchp;        // N * K/32
    float *xs = xsc + N * nchp;          // N * xstride
    uint4 *xq = reinterpret_cast<uint4 *>(xs + N * xstride);  // N * xq_stride16(K): digits of the exit-layer rows
    __shared__ int32_t s_act[4], s_riv[4];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    pdl_launch();

    const int tasks = p.template n_tasks<R>();
    const int t0 = (int)(((long long)tasks * blockIdx.x) / gridDim.x);
    const int t1 = (int)(((long long)tasks * (blockIdx.x + 1)) / gridDim.x);

    // ---- before the grid dependency: the first loads of this warp's first task (weights depend on nothing).  The hint never under-counts the backbone rows: positive, the
    // bf16 set is (almost certainly) needed; zero, every row has left the backbone and the 4-bit set is.
    W4Batch<R> pre4;   // its q registers also carry the bf16 weights when that set is prefetched
    int pre_kind = 0;  // 1: pre4.q holds bf16 weights, 2: pre4 holds codes with their scales / zeros
    const int gshift = (p.group == 64) ? 1 : (p.group == 32 ? 0 : 2);
    if (t0 + warp < t1) {
        const int hint = *reinterpret_cast<const volatile int32_t *>(rl.hint_act);
        if (hint > 0 && !skip_backbone) {
            const uint16_t *rows[R];
            stream_rows_bf16<P, R>(p, t0 + warp, rows);
            stream_issue_bf16<R>(rows, K >> 3, 0, lane, pre4.q);
            pre_kind = 1;
        } else if (hint == 0 && has_river == 1) {
            W4 rows[R];
            stream_rows_w4<P, R>(p, t0 + warp, rows);
            stream_issue_w4<R>(rows, K >> 5, gshift, 0, lane, pre4);
            pre_kind = 2;
        }
    }
    // Per-step constants of the decision and the norm gain, fetched before the wait.
    constexpr int XF = R == 2 ? 4 : 2;  // 128-bit pieces of a row a thread keeps in registers (one-row steps)
    const int nv = K >> 2, tid = threadIdx.x, nthr = blockDim.x;
    const int n = *rl.n_rows;
    const bool small = n <= N;       // the whole step in one pass: lists come from the exit flags
    const bool fast = N == 1 && n == 1 && nv <= XF * nthr && has_river != 2;
    float tau[N];
    int forced[N];
#pragma unroll
    for (int b = 0; b < N; ++b) { tau[b] = 0.f; forced[b] = -1; }
    if (dec.meta && small) {
        const float *tp = dec.meta->tau;
        const int32_t *fp = dec.meta->forced;
#pragma unroll
        for (int b = 0; b < N; ++b)
            if (b < n) {
                tau[b] = tp[b];
                if (fp) forced[b] = fp[b];
            }
    }
    uint2 gr[XF];
    if (fast && in.gain) {
#pragma unroll
        for (int k = 0; k < XF; ++k) {
            const int v = tid + k * nthr;
            gr[k] = v < nv ? *reinterpret_cast<const uint2 *>(in.gain + 4 * v) : make_uint2(0u, 0u);
        }
    }
    pdl_wait();
    int na, nr;
    bool prestaged = false;
    const int32_t *act_idx = rl.act_idx, *riv_idx = rl.riv_idx;
    if (fast) {
        const bool riv = stream_stage_one<XF>(in, dec, dec.meta ? dec.state_in : rl.state, K, xstride, red, xs, xq, xsc, xsum,
                                              gr, tau[0], forced[0]);
        if (tid == 0) { s_act[0] = 0; s_riv[0] = 0; }
        __syncthreads();
        na = (riv || skip_backbone) ? 0 : 1;
        nr = (riv && has_river) ? 1 : 0;
        act_idx = s_act;
        riv_idx = s_riv;
        prestaged = true;
    } else if (small) {
        // ---- up to four rows: flags (and, when this launch decides, Eq. 1 for every row: the warps split over the
        // rows, the per-row sums meet in shared memory in a fixed order), then the lists in shared memory
        uint32_t gone = 0u;
        const uint8_t *st = dec.meta ? dec.state_in : rl.state;
#pragma unroll
        for (int b = 0; b < N; ++b)
            if (b < n && __ldcg(st + b)) gone |= 1u << b;
        if (dec.meta) {
            const int wpr = nwarps / n;  // warps per row (n <= 4 <= nwarps)
            const int row = warp % n, member = warp / n;
            float ab = 0.f, aa = 0.f, bb = 0.f;
            if (member < wpr) {
                const float4 *a4 = reinterpret_cast<const float4 *>(dec.h_prev + (size_t)row * K);
                const float4 *b4 = reinterpret_cast<const float4 *>(in.src + (size_t)row * K);
                const int stride = wpr * 32;
                for (int v0 = member * 32 + lane; v0 < nv; v0 += 4 * stride) {
                    float4 x[4], y[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int v = v0 + u * stride;
                        x[u] = v < nv ? __ldcg(a4 + v) : make_float4(0.f, 0.f, 0.f, 0.f);
                        y[u] = v < nv ? __ldcg(b4 + v) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        ab += x[u].x * y[u].x + x[u].y * y[u].y + x[u].z * y[u].z + x[u].w * y[u].w;
                        aa += x[u].x * x[u].x + x[u].y * x[u].y + x[u].z * x[u].z + x[u].w * x[u].w;
                        bb += y[u].x * y[u].x + y[u].y * y[u].y + y[u].z * y[u].z + y[u].w * y[u].w;
                    }
                }
            }
            ab = warp_sum(ab); aa = warp_sum(aa); bb = warp_sum(bb);
            if (lane == 0) { red[warp] = ab; red[16 + warp] = aa; red[32 + warp] = bb; }
            __syncthreads();
            float sc[N];
#pragma unroll
            for (int b = 0; b < N; ++b) {
                sc[b] = 0.f;
                if (b >= n) continue;
                float sab = 0.f, saa = 0.f, sbb = 0.f;
                for (int m = 0; m < wpr; ++m) { sab += red[m * n + b]; saa += red[16 + m * n + b]; sbb += red[32 + m * n + b]; }
                sc[b] = transition_score(sab, saa, sbb);
            }
            const uint32_t gone_in = gone;
            gone = stream_decide<N>(dec, n, gone_in, sc, tau, forced);
            if (blockIdx.x == 0 && tid == 0) stream_publish<N>(dec, n, gone_in, gone, sc, tau);
        }
        na = 0; nr = 0;
        if (tid == 0) {
            int a = 0, r = 0;
#pragma unroll
            for (int b = 0; b < N; ++b)
                if (b < n) {
                    if ((gone >> b) & 1u) s_riv[r++] = b;
                    else s_act[a++] = b;
                }
        }
        na = n - __popc(gone);
        nr = has_river ? __popc(gone) : 0;
        if (skip_backbone) na = 0;
        act_idx = s_act;
        riv_idx = s_riv;
        __syncthreads();
    } else {
        // skip_backbone: the backbone rows of this step are served by the tensor-core kernel
        na = skip_backbone ? 0 : *rl.n_act;
        nr = has_river ? *rl.n_riv : 0;
    }

    // has_river == 2 (State Propagation, Section 3): this launch serves the rows that have LEFT the backbone, on the bf16
    // weights - the two lists trade places and nothing runs on 4-bit codes
    if (has_river == 2) {
        const int32_t *t = act_idx; act_idx = riv_idx; riv_idx = t;
        na = nr;
        nr = 0;
    }
    // hint == 0 promised that no row is left in the backbone: then only the 4-bit pass runs, with the prefetched
    // registers; otherwise the bf16 pass (which may hold prefetched registers) and the 4-bit pass without them, so
    // that neither pass keeps the other's prefetch registers alive
    if (pre_kind == 2) {
        if (na == 0)
            stream_pass_w4<P, N, R, true>(p, in, riv_idx, nr, xstride, xs, xq, xsc, xsum, red, t0, t1, prestaged, fast, pre4);
    } else {
        stream_pass_bf16<P, N, R>(p, in, act_idx, na, xstride, xs, red, t0, t1, prestaged, fast, pre_kind == 1, pre4.q);
        stream_pass_w4<P, N, R, false>(p, in, riv_idx, nr, xstride, xs, xq, xsc, xsum, red, t0, t1, prestaged, fast, pre4);
    }
}

// ---------------------------------------------------------------- a8: final norm + LM head + argmax partials
// logits = W_lm . RMSNorm(h) for the rows that need them (all rows of a decode step; the last prompt position in
// prefill), written as fp32 if the caller gave a buffer, and the greedy next token: every CTA keeps the best
// (value, id) of its share of the vocabulary (ties -> lowest id), a second small kernel merges the CTAs.
struct HeadArgs {
    const uint16_t *w;  // [V][d]
    ProjIn in;
    int d, V;
    const int32_t *rows;  // rows that need logits
    const StepMeta *meta; // n_head_rows, logits [n_head_rows][V] or nullptr (indexed by position in `rows`)
    float *part_val;      // [max_batch][gridDim.x]
    int32_t *part_idx;
};

template <int N, int R>
__global__ void __launch_bounds__(256) lm_head_kernel(const HeadArgs a, int xstride) {
    extern __shared__ __align__(16) float stream_smem[];
    float *red = stream_smem;
    float *xs = stream_smem + 32;
    __shared__ float s_val[8][N];
    __shared__ int s_idx[8][N];
    const int K = a.d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    pdl_launch();
    const int tasks = a.V / R;
    const int t0 = (int)(((long long)tasks * blockIdx.x) / gridDim.x);
    const int t1 = (int)(((long long)tasks * (blockIdx.x + 1)) / gridDim.x);
    uint4 pre[R][kStreamPF];
    bool have_pre = false;
    if (t0 + warp < t1) {  // the LM head always runs: start its first weight loads before the dependency resolves
        const uint16_t *rows[R];
#pragma unroll
        for (int r = 0; r < R; ++r) rows[r] = a.w + ((size_t)(t0 + warp) * R + r) * K;
        stream_issue_bf16<R>(rows, K >> 3, 0, lane, pre);
        have_pre = true;
    }
    pdl_wait();
    const int cnt = a.meta->n_head_rows;
    float *logits = a.meta->logits;
    for (int i0 = 0; i0 < cnt; i0 += N) {
        __syncthreads();
        stream_load_rows<N, 8>(a.in, a.rows, i0, cnt, K, xstride, xs, red);
        float best[N];
        int besti[N];
#pragma unroll
        for (int n = 0; n < N; ++n) { best[n] = -CUDART_INF_F; besti[n] = 0x7fffffff; }
        for (int t = t0 + warp; t < t1; t += nwarps) {
            const size_t o0 = (size_t)t * R;
            const uint16_t *rows[R];
#pragma unroll
            for (int r = 0; r < R; ++r) rows[r] = a.w + (o0 + r) * K;
            float acc[R][N];
            stream_dots_bf16<N, R>(rows, xs, K, xstride, have_pre && i0 == 0 && t == t0 + warp, pre, acc);
#pragma unroll
            for (int n = 0; n < N; ++n)
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float v = warp_sum(acc[r][n]);
                    if (v > best[n]) { best[n] = v; besti[n] = (int)(o0 + r); }  // ascending ids: first max wins
                    if (logits && lane == n * R + r && i0 + n < cnt) logits[(size_t)(i0 + n) * a.V + o0 + r] = v;
                }
        }
        if (lane == 0)
#pragma unroll
            for (int n = 0; n < N; ++n) { s_val[warp][n] = best[n]; s_idx[warp][n] = besti[n]; }
        __syncthreads();
        if (threadIdx.x < N && i0 + (int)threadIdx.x < cnt) {
            const int n = threadIdx.x;
            float bv = -CUDART_INF_F;
            int bi = 0x7fffffff;
            for (int w = 0; w < nwarps; ++w) {
                const float v = s_val[w][n];
                const int id = s_idx[w][n];
                if (v > bv || (v == bv && id < bi)) { bv = v; bi = id; }
            }
            a.part_val[(size_t)(i0 + n) * gridDim.x + blockIdx.x] = bv;
            a.part_idx[(size_t)(i0 + n) * gridDim.x + blockIdx.x] = bi;
        }
    }
}

// exit_hist (decode steps only, else null): [L + 1] counters of the exit layers taken so far - the head rows of a decode
// step are its rows, and their exit layers are final by now.
static __global__ void argmax_final_kernel(const StepMeta *meta, const float *part_val, const int32_t *part_idx, int nparts,
                                           unsigned long long *exit_hist) {
    pdl_launch();
    pdl_wait();
    const int i = blockIdx.x;
    if (i >= meta->n_head_rows) return;
    if (exit_hist && threadIdx.x == 0) atomicAdd(exit_hist + meta->exit_layer[i], 1ull);
    int32_t *next_tok = meta->next_tok;  // indexed by position in the head-row list
    float bv = -CUDART_INF_F;
    int bi = 0x7fffffff;
    for (int p = threadIdx.x; p < nparts; p += blockDim.x) {
        const float v = part_val[(size_t)i * nparts + p];
        const int id = part_idx[(size_t)i * nparts + p];
        if (v > bv || (v == bv && id < bi)) { bv = v; bi = id; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    __shared__ float sv[32];
    __shared__ int si[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
            if (sv[w] > bv || (sv[w] == bv && si[w] < bi)) { bv = sv[w]; bi = si[w]; }
        next_tok[i] = bi == 0x7fffffff ? 0 : bi;  // a row without any comparable logit (all NaN) yields token 0
    }
}

inline size_t stream_smem_bytes(int N, int K) {
    return sizeof(float) * (64 + 2 * (size_t)N * (((K >> 5) + 3) & ~3) + (size_t)N * xs_stride(K, 32)) +
           16 * (size_t)N * xq_stride16(K);
}

}  // namespace river
