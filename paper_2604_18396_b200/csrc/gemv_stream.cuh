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
#include "river_kernels.cuh"

namespace river {

// ---------------------------------------------------------------- problems
// A problem tells where the R rows of task t live (NRUN runs of R/NRUN consecutive rows) and what to do with the
// R x N results of a task.
struct RowLists {
    const int32_t *act_idx, *n_act, *riv_idx, *n_riv;
    const int32_t *hint_act;  // backbone row count as of the latest compaction; never under-counts (a prefetch hint)
    const int32_t *n_rows;    // rows of the step (per-step metadata, stable while the step runs)
    const uint8_t *exited;    // the sticky exit flags the lists were built from
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


// Sums of every 32-input chunk of the rows staged in the E = 32 order (all threads of the CTA; ends with a barrier).
template <int N>
__device__ __forceinline__ void stream_chunk_sums(const float *xs, float *xsum, int K, int xstride) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int nch = K >> 5;
    for (int t = tid; t < N * nch; t += nthr) {
        const int n = t / nch, c = t % nch;
        const float *xb = xs + n * xstride + (c >> 5) * 1024 + (c & 31) * 4;
        float sx = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float4 v = *reinterpret_cast<const float4 *>(xb + j * 128);
            sx += (v.x + v.y) + (v.z + v.w);
        }
        xsum[n * nch + c] = sx;
    }
    __syncthreads();
}

// ---------------------------------------------------------------- activation rows -> shared memory
// All threads of the CTA load up to N rows idx[i0..], optionally RMS-normalise them, and store them fp32 in the
// lane-interleaved order for E inputs per chunk (8: bf16 weights, 32: 4-bit codes, plus the sums of every chunk).
template <int N, int E>
__device__ __forceinline__ void stream_load_rows(const ProjIn &in, const int32_t *idx, int i0, int cnt, int K,
                                                 int xstride, float *xs, float *xsum, float *red) {
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
    if (E == 32) stream_chunk_sums<N>(xs, xsum, K, xstride);
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

// 4-bit weights: lane owns the 32-input chunks lane, lane + 32, ... (16 bytes of codes each).
// sum_k (q_k - z) s x_k over a chunk = s * (sum_k (128 + q_k) x_k - (z + 128) * sum_k x_k), with 128 + q read off
// the bf16 bit pattern 0x4300 | q; the chunk sums of x are precomputed.
template <int N, int R>
__device__ __forceinline__ void stream_dots_w4(const W4 (&wrow)[R], const float *xs, const float *xsum, int K,
                                               int xstride, int group, float (&acc)[R][N]) {
    const int lane = threadIdx.x & 31;
    const int nch = K >> 5;
    const int gshift = (group == 64) ? 1 : (group == 32 ? 0 : 2);
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
#pragma unroll 4
    for (int c = lane; c < nch; c += 32) {
        uint4 q[R];
        float s[R], zz[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            q[r] = ldg_stream16(wrow[r].codes + (size_t)c * 16);
            s[r] = bf16f(ldg_u16(wrow[r].scale + (c >> gshift)));
            zz[r] = bf16f(ldg_u16(wrow[r].zero + (c >> gshift))) + 128.f;
        }
#pragma unroll
        for (int n = 0; n < N; ++n) {
            const float *xb = xs + n * xstride + (c >> 5) * 1024 + lane * 4;
            float p0[R], p1[R];
#pragma unroll
            for (int r = 0; r < R; ++r) { p0[r] = 0.f; p1[r] = 0.f; }
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {  // code word wd holds inputs 8*wd .. 8*wd+7 of the chunk
                const float4 x0 = *reinterpret_cast<const float4 *>(xb + (2 * wd) * 128);
                const float4 x1 = *reinterpret_cast<const float4 *>(xb + (2 * wd + 1) * 128);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const uint32_t v = wd == 0 ? q[r].x : (wd == 1 ? q[r].y : (wd == 2 ? q[r].z : q[r].w));
                    const uint32_t b0 = (v & 0x000f000fu) | 0x43004300u;          // inputs 0, 4
                    const uint32_t b1 = ((v >> 4) & 0x000f000fu) | 0x43004300u;   // inputs 1, 5
                    const uint32_t b2 = ((v >> 8) & 0x000f000fu) | 0x43004300u;   // inputs 2, 6
                    const uint32_t b3 = ((v >> 12) & 0x000f000fu) | 0x43004300u;  // inputs 3, 7
                    p0[r] = fmaf(bf16lo(b0), x0.x, p0[r]); p1[r] = fmaf(bf16lo(b1), x0.y, p1[r]);
                    p0[r] = fmaf(bf16lo(b2), x0.z, p0[r]); p1[r] = fmaf(bf16lo(b3), x0.w, p1[r]);
                    p0[r] = fmaf(bf16hi(b0), x1.x, p0[r]); p1[r] = fmaf(bf16hi(b1), x1.y, p1[r]);
                    p0[r] = fmaf(bf16hi(b2), x1.z, p0[r]); p1[r] = fmaf(bf16hi(b3), x1.w, p1[r]);
                }
            }
            const float sx = xsum[n * nch + c];
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r][n] = fmaf(s[r], (p0[r] + p1[r]) - zz[r] * sx, acc[r][n]);
        }
    }
}

// ---------------------------------------------------------------- the kernel
template <class P, int N, int R>
__device__ __forceinline__ void stream_rows_bf16(const P &p, int t, const uint16_t *(&rows)[R]) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int run = r / (R / P::NRUN), j = r % (R / P::NRUN);
        rows[r] = p.template bf16_base<R>(t, run) + (p.template run_row<R>(t, run) + j) * (size_t)p.K;
    }
}

template <class P, int N, int R>
__global__ void __launch_bounds__(512) stream_proj_kernel(const P p, const ProjIn in, const RowLists rl, int has_river,
                                                          int xstride, int skip_backbone, const ScoreTail tail) {
    extern __shared__ __align__(16) float stream_smem[];
    const int K = p.K;
    float *red = stream_smem;            // 32
    float *xsum = stream_smem + 32;      // N * K/32
    float *xs = xsum + N * (K >> 5);     // N * xstride
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    pdl_launch();

    const int tasks = p.template n_tasks<R>();
    const int t0 = (int)(((long long)tasks * blockIdx.x) / gridDim.x);
    const int t1 = (int)(((long long)tasks * (blockIdx.x + 1)) / gridDim.x);

    // ---- before the grid dependency: the first loads of this warp's first backbone task (weights depend on
    // nothing).  The hint never under-counts the backbone rows, so zero means they are certainly not needed.
    uint4 pre[R][kStreamPF];
    bool have_pre = false;
    if (!skip_backbone && t0 + warp < t1 && *reinterpret_cast<const volatile int32_t *>(rl.hint_act) > 0) {
        const uint16_t *rows[R];
        stream_rows_bf16<P, N, R>(p, t0 + warp, rows);
        stream_issue_bf16<R>(rows, K >> 3, 0, lane, pre);
        have_pre = true;
    }
    // A step of ONE row (the latency-critical case): which weight set the row takes follows from its exit flag, its
    // index is 0, and its data can be requested at once - one memory round trip after the grid dependency instead of
    // three (count -> index -> data).  The norm gain, a constant, is fetched before the wait.
    constexpr int XF = 4;  // 128-bit pieces of the row a thread keeps in registers
    const int nv = K >> 2, tid = threadIdx.x, nthr = blockDim.x;
    const bool single = N == 1 && *rl.n_rows == 1;
    const bool fast = single && nv <= XF * nthr;
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
    __shared__ int32_t s_row0;
    const int32_t *act_idx = rl.act_idx, *riv_idx = rl.riv_idx;
    if (single) {
        if (tid == 0) s_row0 = 0;
        const bool riv = rl.exited[0] != 0;
        na = (riv || skip_backbone) ? 0 : 1;
        nr = (riv && has_river) ? 1 : 0;
        act_idx = riv_idx = &s_row0;
        if (fast && na + nr == 1) {
            float4 xr[XF];
            float ss = 0.f;
            const float4 *src = reinterpret_cast<const float4 *>(in.src);
#pragma unroll
            for (int k = 0; k < XF; ++k) {
                const int v = tid + k * nthr;
                xr[k] = v < nv ? __ldcg(src + v) : make_float4(0.f, 0.f, 0.f, 0.f);
                ss += xr[k].x * xr[k].x + xr[k].y * xr[k].y + xr[k].z * xr[k].z + xr[k].w * xr[k].w;
            }
            float scale = 1.f;
            if (in.gain) {
                ss = warp_sum(ss);
                if (lane == 0) red[warp] = ss;
                __syncthreads();
                ss = 0.f;
                for (int w = 0; w < nwarps; ++w) ss += red[w];
                scale = rsqrtf(ss / (float)K + in.eps);
            }
#pragma unroll
            for (int k = 0; k < XF; ++k) {
                const int v = tid + k * nthr;
                if (v < nv) {
                    float4 y = xr[k];
                    if (in.gain) {
                        y.x *= scale * bf16lo(gr[k].x); y.y *= scale * bf16hi(gr[k].x);
                        y.z *= scale * bf16lo(gr[k].y); y.w *= scale * bf16hi(gr[k].y);
                    }
                    if (riv) *reinterpret_cast<float4 *>(xs + xs_index<32>(4 * v)) = y;
                    else *reinterpret_cast<float4 *>(xs + xs_index<8>(4 * v)) = y;
                }
            }
            __syncthreads();
            if (riv) stream_chunk_sums<1>(xs, xsum, K, xstride);
            prestaged = true;
        } else {
            __syncthreads();  // s_row0
        }
    } else {
        // skip_backbone: the backbone rows of this step are served by the tensor-core kernel
        na = skip_backbone ? 0 : *rl.n_act;
        nr = has_river ? *rl.n_riv : 0;
    }

    for (int i0 = 0; i0 < na; i0 += N) {
        if (!prestaged) {
            __syncthreads();
            stream_load_rows<N, 8>(in, act_idx, i0, na, K, xstride, xs, xsum, red);
        }
        for (int t = t0 + warp; t < t1; t += nwarps) {
            const uint16_t *rows[R];
            stream_rows_bf16<P, N, R>(p, t, rows);
            float acc[R][N];
            float ep[4] = {0.f, 0.f, 0.f, 0.f};
            if constexpr (N == 1 && R == 2) {
                if (single && lane == 0) p.epi_pre(t, 0, ep);  // travels while the dot products are computed
            }
            stream_dots_bf16<N, R>(rows, xs, K, xstride, have_pre && i0 == 0 && t == t0 + warp, pre, acc);
#pragma unroll
            for (int n = 0; n < N; ++n) {
                float res[R];
#pragma unroll
                for (int r = 0; r < R; ++r) res[r] = warp_sum(acc[r][n]);
                if (lane == n && i0 + n < na) {
                    if constexpr (N == 1 && R == 2) {
                        if (single) p.epilogue_pre(t, 0, res, ep);
                        else p.template epilogue<R>(t, act_idx[i0 + n], res);
                    } else {
                        p.template epilogue<R>(t, single ? 0 : act_idx[i0 + n], res);
                    }
                }
            }
        }
    }
    for (int i0 = 0; i0 < nr; i0 += N) {
        if (!prestaged) {
            __syncthreads();
            stream_load_rows<N, 32>(in, riv_idx, i0, nr, K, xstride, xs, xsum, red);
        }
        const int ng = K / p.group;
        for (int t = t0 + warp; t < t1; t += nwarps) {
            W4 rows[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int run = r / (R / P::NRUN), j = r % (R / P::NRUN);
                const W4 b = p.template w4_base<R>(t, run);
                const size_t row = p.template run_row<R>(t, run) + j;
                rows[r] = W4{b.codes + row * (K >> 1), b.scale + row * ng, b.zero + row * ng};
            }
            float acc[R][N];
            float ep[4] = {0.f, 0.f, 0.f, 0.f};
            if constexpr (N == 1 && R == 2) {
                if (single && lane == 0) p.epi_pre(t, 0, ep);
            }
            stream_dots_w4<N, R>(rows, xs, xsum, K, xstride, p.group, acc);
#pragma unroll
            for (int n = 0; n < N; ++n) {
                float res[R];
#pragma unroll
                for (int r = 0; r < R; ++r) res[r] = warp_sum(acc[r][n]);
                if (lane == n && i0 + n < nr) {
                    if constexpr (N == 1 && R == 2) {
                        if (single) p.epilogue_pre(t, 0, res, ep);
                        else p.template epilogue<R>(t, riv_idx[i0 + n], res);
                    } else {
                        p.template epilogue<R>(t, single ? 0 : riv_idx[i0 + n], res);
                    }
                }
            }
        }
    }
    if (tail.meta) score_tail(tail);  // the kernel that ends a block also scores it (small steps)
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
        stream_load_rows<N, 8>(a.in, a.rows, i0, cnt, K, xstride, xs, nullptr, red);
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

__global__ void argmax_final_kernel(const StepMeta *meta, const float *part_val, const int32_t *part_idx, int nparts) {
    pdl_launch();
    pdl_wait();
    const int i = blockIdx.x;
    if (i >= meta->n_head_rows) return;
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
        next_tok[i] = bi;
    }
}

inline size_t stream_smem_bytes(int N, int K) {
    return sizeof(float) * (32 + (size_t)N * (K >> 5) + (size_t)N * xs_stride(K, 32));
}

}  // namespace river
