// Weight-streaming projections for small row counts (sm_100a).
//
// One CTA per SM owns a contiguous range of output-feature tasks.  A producer warp streams the weight rows of those
// tasks through a shared-memory ring with bulk TMA copies (cp.async.bulk + mbarrier complete_tx); it starts before
// the kernel's grid dependency resolves, because weights never depend on the previous kernel, so the HBM stream does
// not stop at kernel boundaries (programmatic dependent launch).  A stage holds R weight rows (one K-slice of them).
// All eight consumer warps work on every stage together, each thread on its own columns, against up to N activation
// rows held in shared memory in fp32, so that only the stage being read is out of flight.  Partial sums are reduced
// with shuffles inside a warp and through shared memory across warps: the warps take turns (task number mod 8) to
// wait, bounded, for all eight partials of a task, add them in a fixed order and run the projection's epilogue, so
// that the epilogue's memory latency never holds a ring slot and is spread over all warps.
// The same launch serves the rows still in the backbone (bf16 weights) and the rows in the exit layers (4-bit codes +
// bf16 scale / zero per group, dequantised on the fly as (q - z) * s); which set is non-empty is read on the device.
#pragma once
#include "attn_decode.cuh"
#include "river_kernels.cuh"

namespace river {

constexpr int kRingConsumers = 8;
constexpr int kRingCThreads = 32 * kRingConsumers;
constexpr int kRingThreads = kRingCThreads + 32;
constexpr int kRingStageBytes = 18432;  // 16 KB of weights or codes + up to 2 KB of scales and zeros
constexpr int kRingMaxSlots = 8;
constexpr int kRingTaskDepth = 16;  // partial-sum buffers in flight: more than the ring depth, so none is overwritten early

__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kRingCThreads) : "memory"); }

// ---------------------------------------------------------------- problems
// A problem tells where the R rows of task t live (NRUN runs of R/NRUN consecutive rows) and what to do with the
// R x N results of a task.
struct RowLists {
    const int32_t *act_idx, *n_act, *riv_idx, *n_riv;
    const int32_t *hint_act;  // latest backbone row count any compaction has published (may lag: a hint only)
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
        const int pos = kv.row_pos[row], slot = kv.row_slot[row];
        int page = 0;
        if (which != 0) {
            page = kv.page_tbl[(size_t)slot * kv.max_pages_per_seq + pos / kPage];
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
        for (int r = 0; r < R; ++r) out[o + r] = resid[o + r] + res[r];
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
};

// ---------------------------------------------------------------- activation rows -> shared memory
// The consumer warps load up to N rows idx[i0..], optionally RMS-normalise them, and store them fp32 in the
// lane-interleaved order for E inputs per chunk (8: bf16 weights, 32: 4-bit codes, plus the sums of every chunk).
// Only the consumer threads call this; it synchronises them with their named barrier.
template <int N, int E>
__device__ __forceinline__ void ring_load_rows(const ProjIn &in, const int32_t *idx, int i0, int cnt, int K,
                                               int xstride, float *xs, float *xsum, float *red, int tid) {
    constexpr int nthr = kRingCThreads;
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
            consumer_sync();
            ss = 0.f;
#pragma unroll
            for (int w = 0; w < kRingConsumers; ++w) ss += red[w];
            const float scale = rsqrtf(ss / (float)K + in.eps);
            consumer_sync();
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
    consumer_sync();
    if (E == 32) {
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
        consumer_sync();
    }
}

// ---------------------------------------------------------------- consumer math on one stage
// bf16: the stage holds R rows x ks columns (row-major); thread tid owns the 8-column chunks tid, tid + 256, ...
template <int N, int R>
__device__ __forceinline__ void stage_dots_bf16(const uint8_t *stage, int k0, int ks, const float *xs, int xstride,
                                                float (&acc)[R][N], int tid) {
    const int nch = ks >> 3;
#pragma unroll 2
    for (int c = tid; c < nch; c += kRingCThreads) {
        uint4 w[R];
#pragma unroll
        for (int r = 0; r < R; ++r) w[r] = *reinterpret_cast<const uint4 *>(stage + (size_t)r * ks * 2 + c * 16);
        const int cc = (k0 >> 3) + c;
        const float *xb = xs + (cc >> 5) * 256 + (cc & 31) * 4;
#pragma unroll
        for (int n = 0; n < N; ++n) {
            const float4 x0 = *reinterpret_cast<const float4 *>(xb + n * xstride);
            const float4 x1 = *reinterpret_cast<const float4 *>(xb + n * xstride + 128);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float a0 = bf16lo(w[r].x) * x0.x, a1 = bf16hi(w[r].x) * x0.y;
                a0 = fmaf(bf16lo(w[r].y), x0.z, a0); a1 = fmaf(bf16hi(w[r].y), x0.w, a1);
                a0 = fmaf(bf16lo(w[r].z), x1.x, a0); a1 = fmaf(bf16hi(w[r].z), x1.y, a1);
                a0 = fmaf(bf16lo(w[r].w), x1.z, a0); a1 = fmaf(bf16hi(w[r].w), x1.w, a1);
                acc[r][n] += a0 + a1;
            }
        }
    }
}

// 4-bit: the stage holds codes [R][K/2], then scales [R][K/G] and zeros [R][K/G] (bf16).  A 32-input chunk of one
// row is one item; thread tid owns items tid, tid + 256, ... of the R * K/32 items (row = item / (K/32)).
// sum_k (q_k - z) s x_k over a chunk = s * (sum_k (128 + q_k) x_k - (z + 128) * sum_k x_k), with 128 + q read off
// the bf16 bit pattern 0x4300 | q.  K/32 is a multiple of 32, so a warp's 32 items of one pass share their row.
template <int N, int R, int UMAX>
__device__ __forceinline__ void stage_dots_w4(const uint8_t *stage, int K, int group, const float *xs, int xstride,
                                              const float *xsum, float (&acc)[UMAX][N], int tid) {
    const int nch = K >> 5, ng = K / group, items = R * nch;
    const int gshift = (group == 64) ? 1 : (group == 32 ? 0 : 2);
    const uint16_t *sc = reinterpret_cast<const uint16_t *>(stage + (size_t)R * (K >> 1));
    const uint16_t *zr = sc + (size_t)R * ng;
#pragma unroll
    for (int u = 0; u < UMAX; ++u) {
        const int item = tid + u * kRingCThreads;
        if (item < items) {
            const int r = item / nch, c = item - r * nch;
            const uint4 q = *reinterpret_cast<const uint4 *>(stage + (size_t)r * (K >> 1) + c * 16);
            const float s = bf16f(sc[r * ng + (c >> gshift)]);
            const float zz = bf16f(zr[r * ng + (c >> gshift)]) + 128.f;
#pragma unroll
            for (int n = 0; n < N; ++n) {
                const float *xb = xs + n * xstride + (c >> 5) * 1024 + (c & 31) * 4;
                float p0 = 0.f, p1 = 0.f;
#pragma unroll
                for (int wd = 0; wd < 4; ++wd) {  // code word wd holds inputs 8*wd .. 8*wd+7 of the chunk
                    const float4 x0 = *reinterpret_cast<const float4 *>(xb + (2 * wd) * 128);
                    const float4 x1 = *reinterpret_cast<const float4 *>(xb + (2 * wd + 1) * 128);
                    const uint32_t v = wd == 0 ? q.x : (wd == 1 ? q.y : (wd == 2 ? q.z : q.w));
                    const uint32_t b0 = (v & 0x000f000fu) | 0x43004300u;          // inputs 0, 4
                    const uint32_t b1 = ((v >> 4) & 0x000f000fu) | 0x43004300u;   // inputs 1, 5
                    const uint32_t b2 = ((v >> 8) & 0x000f000fu) | 0x43004300u;   // inputs 2, 6
                    const uint32_t b3 = ((v >> 12) & 0x000f000fu) | 0x43004300u;  // inputs 3, 7
                    p0 = fmaf(bf16lo(b0), x0.x, p0); p1 = fmaf(bf16lo(b1), x0.y, p1);
                    p0 = fmaf(bf16lo(b2), x0.z, p0); p1 = fmaf(bf16lo(b3), x0.w, p1);
                    p0 = fmaf(bf16hi(b0), x1.x, p0); p1 = fmaf(bf16hi(b1), x1.y, p1);
                    p0 = fmaf(bf16hi(b2), x1.z, p0); p1 = fmaf(bf16hi(b3), x1.w, p1);
                }
                acc[u][n] = s * ((p0 + p1) - zz * xsum[n * nch + c]);
            }
        }
    }
}

// ---------------------------------------------------------------- the kernel
struct RingGeom {
    int n_slots;     // ring depth (<= kRingMaxSlots)
    int ks;          // bf16 K-slice (columns) per stage: R * ks * 2 bytes <= 16 KB
    int xstride;     // floats per activation row in shared memory
};

template <class P, int N, int RB, int RW>
__global__ void __launch_bounds__(kRingThreads) ring_proj_kernel(const P p, const ProjIn in, const RowLists rl,
                                                                 const RingGeom geom, int has_river, int *dev_err) {
    extern __shared__ __align__(128) uint8_t ring_smem[];
    constexpr int RMAX = RB > RW ? RB : RW;
    const int K = p.K, xstride = geom.xstride, S = geom.n_slots, KSB = geom.ks;
    uint8_t *ring = ring_smem;
    float *xs = reinterpret_cast<float *>(ring + (size_t)S * kRingStageBytes);
    float *xsum = xs + N * xstride;
    float *red = xsum + N * (K >> 5);                       // rms scratch [8]
    float *part = red + 8;                                  // [16 tasks][8 warps][RMAX * N] per-warp partial sums
    int *cnt = reinterpret_cast<int *>(part + kRingTaskDepth * kRingConsumers * RMAX * N);  // [16] arrivals per task
    uint64_t *bars = reinterpret_cast<uint64_t *>(cnt + kRingTaskDepth);  // full[S], empty[S]
    __shared__ int s_abort, s_na, s_nr, s_pref, s_pref_w;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    grid_dep_launch();
    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[S + s]), kRingConsumers);
        }
        for (int s = 0; s < kRingTaskDepth; ++s) cnt[s] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    volatile int *abortp = &s_abort;

    // this CTA's tasks
    const int tasks_b_all = p.template n_tasks<RB>(), tasks_w_all = p.template n_tasks<RW>();
    const int tb0 = (int)(((long long)tasks_b_all * blockIdx.x) / gridDim.x);
    const int tb1 = (int)(((long long)tasks_b_all * (blockIdx.x + 1)) / gridDim.x);
    const int tw0 = (int)(((long long)tasks_w_all * blockIdx.x) / gridDim.x);
    const int tw1 = (int)(((long long)tasks_w_all * (blockIdx.x + 1)) / gridDim.x);
    const int ntb = tb1 - tb0, ntw = tw1 - tw0;
    const int nsl_b = (K + KSB - 1) / KSB;

    // ---- producer side: stage seq of the bf16 set = (chunk, task, slice) in that order
    auto issue_bf16 = [&](int seq, int t, int slice) {
        const int slot = seq % S;
        if (seq >= S && !mbar_wait(smem_u32(&bars[S + slot]), ((seq / S) - 1) & 1, abortp, dev_err)) return false;
        const int k0 = slice * KSB, ks = min(KSB, K - k0);
        const uint32_t full = smem_u32(&bars[slot]);
        mbar_expect_tx(full, (uint32_t)(RB * ks * 2));
        const uint32_t dst = smem_u32(ring + (size_t)slot * kRingStageBytes);
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const int run = r / (RB / P::NRUN), j = r % (RB / P::NRUN);
            const uint16_t *base = p.template bf16_base<RB>(t, run);
            const size_t row = p.template run_row<RB>(t, run) + j;
            bulk_load(dst + r * ks * 2, base + row * K + k0, (uint32_t)(ks * 2), full);
        }
        return true;
    };
    auto produce_bf16 = [&](int from, int to) {  // stages [from, to)
        const int per_chunk = ntb * nsl_b;
        if (per_chunk == 0) return true;
        int seq = (from / per_chunk) * per_chunk;
        while (seq < to) {
            for (int t = 0; t < ntb; ++t)
                for (int sl = 0; sl < nsl_b; ++sl, ++seq) {
                    if (seq < from) continue;
                    if (seq >= to) return true;
                    if (!issue_bf16(seq, tb0 + t, sl)) return false;
                }
        }
        return true;
    };
    auto issue_w4 = [&](int seq, int t) {
        const int slot = seq % S;
        if (seq >= S && !mbar_wait(smem_u32(&bars[S + slot]), ((seq / S) - 1) & 1, abortp, dev_err)) return false;
        const int ng = K / p.group;
        constexpr int RR = RW / P::NRUN;
        const uint32_t full = smem_u32(&bars[slot]);
        mbar_expect_tx(full, (uint32_t)(RW * ((K >> 1) + 4 * ng)));
        const uint32_t dst = smem_u32(ring + (size_t)slot * kRingStageBytes);
        const uint32_t dsc = dst + RW * (K >> 1), dzr = dsc + RW * ng * 2;
#pragma unroll
        for (int run = 0; run < P::NRUN; ++run) {
            const W4 b = p.template w4_base<RW>(t, run);
            const size_t row = p.template run_row<RW>(t, run);
            bulk_load(dst + run * RR * (K >> 1), b.codes + row * (K >> 1), (uint32_t)(RR * (K >> 1)), full);
            bulk_load(dsc + run * RR * ng * 2, b.scale + row * ng, (uint32_t)(RR * ng * 2), full);
            bulk_load(dzr + run * RR * ng * 2, b.zero + row * ng, (uint32_t)(RR * ng * 2), full);
        }
        return true;
    };

    // ---- before the grid dependency: the producer fills the ring with the weights of the set that the hint
    // predicts.  The hint never under-counts the backbone rows (exits are sticky and the host resets it with the
    // step's metadata), so zero means that every row is in the exit layers; a wrong "backbone" guess is drained.
    if (tid == kRingCThreads) {
        int prefetched = 0, prefetched_w = 0;
        const int hint = *reinterpret_cast<const volatile int32_t *>(rl.hint_act);
        if (hint > 0) {
            prefetched = min(S, ntb * nsl_b);
            produce_bf16(0, prefetched);
        } else if (has_river) {
            prefetched_w = min(S, ntw);
            for (int t = 0; t < prefetched_w; ++t) issue_w4(t, tw0 + t);
        }
        s_pref = prefetched;
        s_pref_w = prefetched_w;
    }
    grid_dep_wait();
    if (tid == 0) {
        s_na = *rl.n_act;
        s_nr = has_river ? *rl.n_riv : 0;
    }
    __syncthreads();
    const int na = s_na, nr = s_nr, prefetched = s_pref, prefetched_w = s_pref_w;
    const int chunks_b = (na + N - 1) / N, chunks_w = (nr + N - 1) / N;
    const int stages_b = na > 0 ? chunks_b * ntb * nsl_b : prefetched;  // a wrong prefetch is drained without compute
    // both sets use one stage numbering: the 4-bit stages follow the bf16 stages in the same ring

    if (warp == kRingConsumers) {
        // ================= producer
        if (lane == 0) {
            bool ok = produce_bf16(prefetched, stages_b);
            int seq = stages_b;
            for (int ch = 0; ch < chunks_w && ok; ++ch)
                for (int t = 0; t < ntw && ok; ++t, ++seq)
                    if (seq - stages_b >= prefetched_w) ok = issue_w4(seq, tw0 + t);
        }
    } else {
        // ================= consumers: every warp walks every stage in order
        int seq = 0;
        auto wait_full = [&](int i) { return mbar_wait(smem_u32(&bars[i % S]), (i / S) & 1, abortp, dev_err); };
        auto release = [&](int i) {
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[S + i % S]));
        };
        // Publish this warp's partial sums of task number tq and, if it is this warp's turn, wait for the other
        // seven, add all eight in warp order and hand the R results of activation row `lane` to the epilogue.
        int tq = 0;
        auto publish = [&](const float *vals, int nvals) {  // lane 0 holds vals[0..nvals)
            float *mine = part + ((size_t)(tq & (kRingTaskDepth - 1)) * kRingConsumers + warp) * (RMAX * N);
            if (lane == 0) {
                for (int i = 0; i < nvals; ++i) mine[i] = vals[i];
                __threadfence_block();
                atomicAdd(&cnt[tq & (kRingTaskDepth - 1)], 1);
            }
            __syncwarp();
        };
        auto my_turn = [&]() {
            if ((tq & (kRingConsumers - 1)) != warp) return false;
            volatile int *c = &cnt[tq & (kRingTaskDepth - 1)];
            uint32_t it = 0;
            while (*c < kRingConsumers) {
                if (++it > kWaitLimit || *abortp) { *abortp = 1; return false; }
            }
            __threadfence_block();
            return true;
        };
        bool ok = true;
        if (na == 0) {  // drain a wrong prefetch
            for (; seq < stages_b && ok; ++seq) {
                ok = wait_full(seq);
                if (ok) release(seq);
            }
        }
        for (int ch = 0; ch < (na > 0 ? chunks_b : 0) && ok; ++ch) {
            consumer_sync();
            ring_load_rows<N, 8>(in, rl.act_idx, ch * N, na, K, xstride, xs, xsum, red, tid);
            for (int t = 0; t < ntb && ok; ++t) {
                float acc[RB][N];
#pragma unroll
                for (int r = 0; r < RB; ++r)
#pragma unroll
                    for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
                for (int sl = 0; sl < nsl_b; ++sl, ++seq) {
                    ok = wait_full(seq);
                    if (!ok) break;
                    const int k0 = sl * KSB, ks = min(KSB, K - k0);
                    stage_dots_bf16<N, RB>(ring + (size_t)(seq % S) * kRingStageBytes, k0, ks, xs, xstride, acc, tid);
                    release(seq);
                }
                if (!ok) break;
                // cross-warp reduction
                float vals[RB * N];
#pragma unroll
                for (int r = 0; r < RB; ++r)
#pragma unroll
                    for (int n = 0; n < N; ++n) vals[r * N + n] = warp_sum(acc[r][n]);
                publish(vals, RB * N);
                if (my_turn()) {
                    const float *all = part + (size_t)(tq & (kRingTaskDepth - 1)) * kRingConsumers * (RMAX * N);
                    if (lane < N && ch * N + lane < na) {
                        float res[RB];
#pragma unroll
                        for (int r = 0; r < RB; ++r) {
                            float v = 0.f;
#pragma unroll
                            for (int w = 0; w < kRingConsumers; ++w) v += all[w * (RMAX * N) + r * N + lane];
                            res[r] = v;
                        }
                        p.template epilogue<RB>(tb0 + t, rl.act_idx[ch * N + lane], res);
                    }
                    __syncwarp();
                    if (lane == 0) cnt[tq & (kRingTaskDepth - 1)] = 0;
                }
                ++tq;
            }
        }
        // -- exit-layer set: one stage per task
        constexpr int UMAX = 4;  // RW * K/32 items over 256 threads: <= 4 passes for every supported shape
        const int nch = K >> 5;
        for (int ch = 0; ch < chunks_w && ok; ++ch) {
            consumer_sync();
            ring_load_rows<N, 32>(in, rl.riv_idx, ch * N, nr, K, xstride, xs, xsum, red, tid);
            for (int t = 0; t < ntw && ok; ++t, ++seq) {
                ok = wait_full(seq);
                if (!ok) break;
                const int slot = seq % S;
                float acc[UMAX][N];
#pragma unroll
                for (int u = 0; u < UMAX; ++u)
#pragma unroll
                    for (int n = 0; n < N; ++n) acc[u][n] = 0.f;
                stage_dots_w4<N, RW, UMAX>(ring + (size_t)slot * kRingStageBytes, K, p.group, xs, xstride, xsum, acc, tid);
                release(seq);
                // per-warp partials by row: a warp's pass u covers one row (K/32 is a multiple of 32)
                float vals[RW * N];
#pragma unroll
                for (int i = 0; i < RW * N; ++i) vals[i] = 0.f;
#pragma unroll
                for (int u = 0; u < UMAX; ++u) {
                    const int item = (warp << 5) + u * kRingCThreads;
                    if (item < RW * nch) {
                        const int r = item / nch;
#pragma unroll
                        for (int n = 0; n < N; ++n) {
                            const float v = warp_sum(acc[u][n]);
#pragma unroll
                            for (int rr = 0; rr < RW; ++rr)
                                if (rr == r) vals[rr * N + n] += v;
                        }
                    }
                }
                publish(vals, RW * N);
                if (my_turn()) {
                    const float *all = part + (size_t)(tq & (kRingTaskDepth - 1)) * kRingConsumers * (RMAX * N);
                    if (lane < N && ch * N + lane < nr) {
                        float res[RW];
#pragma unroll
                        for (int r = 0; r < RW; ++r) {
                            float v = 0.f;
#pragma unroll
                            for (int w = 0; w < kRingConsumers; ++w) v += all[w * (RMAX * N) + r * N + lane];
                            res[r] = v;
                        }
                        p.template epilogue<RW>(tw0 + t, rl.riv_idx[ch * N + lane], res);
                    }
                    __syncwarp();
                    if (lane == 0) cnt[tq & (kRingTaskDepth - 1)] = 0;
                }
                ++tq;
            }
        }
    }
    if (s_abort) {
        for (int i = 0; i < 2000; ++i) __nanosleep(100);
    }
}

inline size_t ring_smem_bytes(int n_slots, int N, int K, int rmax) {
    const int xstride = xs_stride(K, 32);
    return (size_t)n_slots * kRingStageBytes +
           sizeof(float) * ((size_t)N * xstride + (size_t)N * (K >> 5) + 8 +
                            (size_t)kRingTaskDepth * kRingConsumers * rmax * N) +
           sizeof(int) * kRingTaskDepth + 2 * kRingMaxSlots * sizeof(uint64_t) + 128;
}

}  // namespace river
