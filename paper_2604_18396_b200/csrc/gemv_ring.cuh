// Weight-streaming projections for small row counts (sm_100a).
//
// One CTA per SM slot owns a contiguous range of output-feature tasks.  A producer warp streams the weight rows of
// those tasks through a shared-memory ring with bulk TMA copies (cp.async.bulk + mbarrier complete_tx); it starts
// before the kernel's grid dependency resolves, because weights never depend on the previous kernel, so the HBM
// stream does not stop at kernel boundaries (programmatic dependent launch).  Four consumer warps each take whole
// stages: a stage is R weight rows (one K-slice of them), the warp multiplies them with up to N activation rows
// held in shared memory in fp32, reduces with shuffles and runs the projection's epilogue.  The same launch serves
// the rows still in the backbone (bf16 weights) and the rows in the exit layers (4-bit codes + bf16 scale / zero
// per group, dequantised on the fly as (q - z) * s); which of the two sets is non-empty is read on the device.
#pragma once
#include "attn_decode.cuh"
#include "river_kernels.cuh"

namespace river {

constexpr int kRingConsumers = 4;
constexpr int kRingThreads = 32 * (kRingConsumers + 1);
constexpr int kRingStageBytes = 18432;  // 16 KB of weights or codes + up to 2 KB of scales and zeros
constexpr int kRingSlice = 4096;        // bf16 K-slice per stage row

__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kRingConsumers) : "memory"); }

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
    constexpr int nthr = 32 * kRingConsumers;
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
// bf16: stage holds R rows x ks columns (row-major); lane owns 8-column chunks lane, lane+32, ...
template <int N, int R>
__device__ __forceinline__ void stage_dots_bf16(const uint8_t *stage, int k0, int ks, const float *xs, int xstride,
                                                float (&acc)[R][N], int lane) {
    const int nch = ks >> 3;
#pragma unroll 2
    for (int c = lane; c < nch; c += 32) {
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
                float a = acc[r][n];
                a = fmaf(bf16lo(w[r].x), x0.x, a); a = fmaf(bf16hi(w[r].x), x0.y, a);
                a = fmaf(bf16lo(w[r].y), x0.z, a); a = fmaf(bf16hi(w[r].y), x0.w, a);
                a = fmaf(bf16lo(w[r].z), x1.x, a); a = fmaf(bf16hi(w[r].z), x1.y, a);
                a = fmaf(bf16lo(w[r].w), x1.z, a); a = fmaf(bf16hi(w[r].w), x1.w, a);
                acc[r][n] = a;
            }
        }
    }
}

// 4-bit: stage holds codes [R][K/2], then scales [R][K/G] and zeros [R][K/G] (bf16); lane owns 32-input chunks.
// sum_k (q_k - z) s x_k over a chunk = s * (sum_k (128 + q_k) x_k - (z + 128) * sum_k x_k), with 128 + q read off
// the bf16 bit pattern 0x4300 | q.
template <int N, int R>
__device__ __forceinline__ void stage_dots_w4(const uint8_t *stage, int K, int group, const float *xs, int xstride,
                                              const float *xsum, float (&acc)[R][N], int lane) {
    const int nch = K >> 5, ng = K / group;
    const int gshift = (group == 64) ? 1 : (group == 32 ? 0 : 2);
    const uint16_t *sc = reinterpret_cast<const uint16_t *>(stage + (size_t)R * (K >> 1));
    const uint16_t *zr = sc + (size_t)R * ng;
    for (int c = lane; c < nch; c += 32) {
        uint4 q[R];
        float s[R], zz[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            q[r] = *reinterpret_cast<const uint4 *>(stage + (size_t)r * (K >> 1) + c * 16);
            s[r] = bf16f(sc[r * ng + (c >> gshift)]);
            zz[r] = bf16f(zr[r * ng + (c >> gshift)]) + 128.f;
        }
#pragma unroll
        for (int n = 0; n < N; ++n) {
            float part[R];
#pragma unroll
            for (int r = 0; r < R; ++r) part[r] = 0.f;
            const float *xb = xs + n * xstride + (c >> 5) * 1024 + (c & 31) * 4;
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {  // code word wd holds inputs 8*wd .. 8*wd+7 of the chunk
                const float4 x0 = *reinterpret_cast<const float4 *>(xb + (2 * wd) * 128);
                const float4 x1 = *reinterpret_cast<const float4 *>(xb + (2 * wd + 1) * 128);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const uint32_t v = wd == 0 ? q[r].x : (wd == 1 ? q[r].y : (wd == 2 ? q[r].z : q[r].w));
                    const uint32_t p0 = (v & 0x000f000fu) | 0x43004300u;          // inputs 0, 4
                    const uint32_t p1 = ((v >> 4) & 0x000f000fu) | 0x43004300u;   // inputs 1, 5
                    const uint32_t p2 = ((v >> 8) & 0x000f000fu) | 0x43004300u;   // inputs 2, 6
                    const uint32_t p3 = ((v >> 12) & 0x000f000fu) | 0x43004300u;  // inputs 3, 7
                    float a = part[r];
                    a = fmaf(bf16lo(p0), x0.x, a); a = fmaf(bf16lo(p1), x0.y, a);
                    a = fmaf(bf16lo(p2), x0.z, a); a = fmaf(bf16lo(p3), x0.w, a);
                    a = fmaf(bf16hi(p0), x1.x, a); a = fmaf(bf16hi(p1), x1.y, a);
                    a = fmaf(bf16hi(p2), x1.z, a); a = fmaf(bf16hi(p3), x1.w, a);
                    part[r] = a;
                }
            }
            const float sx = xsum[n * nch + c];
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r][n] = fmaf(s[r], part[r] - zz[r] * sx, acc[r][n]);
        }
    }
}

// ---------------------------------------------------------------- the kernel
struct RingGeom {
    int n_stages;   // ring depth
    int xstride;    // floats per activation row in shared memory
};

// Stage sequence of one weight set: for every chunk of N rows, for every group of kRingConsumers tasks, for every
// K-slice, one stage per task of the group; consumer warp w takes the stages of the group's w-th task.
struct SetPlan {
    int tasks;       // tasks of this CTA
    int n_slices;    // K-slices per task
    int n_chunks;    // row chunks
    __device__ int stages_per_chunk() const { return tasks * n_slices; }
    __device__ int total() const { return n_chunks * tasks * n_slices; }
};

template <class P, int N, int RB, int RW>
__global__ void __launch_bounds__(kRingThreads) ring_proj_kernel(const P p, const ProjIn in, const RowLists rl,
                                                                 const RingGeom geom, int has_river, int *dev_err) {
    extern __shared__ __align__(128) uint8_t ring_smem[];
    uint8_t *smem = ring_smem;
    const int S = geom.n_stages, K = p.K, xstride = geom.xstride;
    uint8_t *ring = smem;
    float *xs = reinterpret_cast<float *>(ring + (size_t)S * kRingStageBytes);
    float *xsum = xs + N * xstride;
    float *red = xsum + N * (K >> 5);
    uint64_t *bars = reinterpret_cast<uint64_t *>(red + 8);  // full[S], empty[S]
    __shared__ int s_abort, s_na, s_nr, s_pref;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    grid_dep_launch();
    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[S + s]), 1);
        }
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
    const int nsl_b = (K + kRingSlice - 1) / kRingSlice;

    auto issue_bf16 = [&](int seq, int local_task, int slice) {
        const int slot = seq % S;
        if (seq >= S && !mbar_wait(smem_u32(&bars[S + slot]), ((seq / S) - 1) & 1, abortp, dev_err)) return false;
        const int t = tb0 + local_task;
        const int k0 = slice * kRingSlice, ks = min(kRingSlice, K - k0);
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
    auto issue_w4 = [&](int seq, int local_task) {
        const int slot = seq % S;
        if (seq >= S && !mbar_wait(smem_u32(&bars[S + slot]), ((seq / S) - 1) & 1, abortp, dev_err)) return false;
        const int t = tw0 + local_task;
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
    // A consumer warp only sees its own stages, so the slot's barrier may still be one use behind when the warp
    // gets there, and a parity wait would then succeed at once on the wrong phase.  Waiting first for the release
    // of the slot's previous occupant (a phase every later one is ordered after) rules that out.
    auto wait_stage = [&](int i) {
        const int slot = i % S;
        if (i >= S && !mbar_wait(smem_u32(&bars[S + slot]), ((i / S) - 1) & 1, abortp, dev_err)) return false;
        return mbar_wait(smem_u32(&bars[slot]), (i / S) & 1, abortp, dev_err);
    };
    // stage order inside one row chunk: group-major, then slice, then task of the group
    auto decode = [&](int i, int tasks, int nsl, int &local_task, int &slice) {
        const int per_group = kRingConsumers * nsl;
        const int g = i / per_group, rem = i % per_group;
        const int gtasks = min(kRingConsumers, tasks - g * kRingConsumers);
        slice = rem / gtasks;
        local_task = g * kRingConsumers + rem % gtasks;
    };

    // ---- before the grid dependency: the producer fills the ring with backbone weights if the hint says that
    // rows are still in the backbone (a wrong hint only costs the prefetch)
    int prefetched = 0;
    if (tid == kRingConsumers * 32) {
        const int hint = *reinterpret_cast<const volatile int32_t *>(rl.hint_act);
        if (hint > 0) {
            const int first = min(S, (tb1 - tb0) * nsl_b);
            for (int i = 0; i < first; ++i) {
                int lt, sl;
                decode(i, tb1 - tb0, nsl_b, lt, sl);
                issue_bf16(i, lt, sl);
            }
            prefetched = first;
        }
        s_pref = prefetched;
    }
    grid_dep_wait();
    if (tid == 0) {
        s_na = *rl.n_act;
        s_nr = has_river ? *rl.n_riv : 0;
    }
    __syncthreads();
    const int na = s_na, nr = s_nr;
    prefetched = s_pref;

    // ---- plans
    SetPlan pb{tb1 - tb0, nsl_b, (na + N - 1) / N};
    SetPlan pw{tw1 - tw0, 1, (nr + N - 1) / N};
    const int stages_b = na > 0 ? pb.total() : prefetched;  // a wrong prefetch is drained without compute
    const int stages_w = nr > 0 ? pw.total() : 0;

    if (warp == kRingConsumers) {
        // ================= producer
        if (lane == 0) {
            bool ok = true;
            for (int i = prefetched; i < stages_b && ok; ++i) {
                int lt, sl;
                decode(i % pb.stages_per_chunk(), pb.tasks, nsl_b, lt, sl);
                ok = issue_bf16(i, lt, sl);
            }
            for (int i = 0; i < stages_w && ok; ++i) {
                int lt, sl;
                decode(i % pw.stages_per_chunk(), pw.tasks, 1, lt, sl);
                ok = issue_w4(stages_b + i, lt);
            }
        }
    } else {
        // ================= consumers
        // -- backbone set (or the drain of a wrong prefetch)
        if (na == 0) {
            for (int i = warp; i < stages_b; i += kRingConsumers) {  // any fixed split of the drain works
                if (!wait_stage(i)) break;
                if (lane == 0) mbar_arrive(smem_u32(&bars[S + i % S]));
            }
        }
        for (int ch = 0; ch < (na > 0 ? pb.n_chunks : 0); ++ch) {
            consumer_sync();
            ring_load_rows<N, 8>(in, rl.act_idx, ch * N, na, K, xstride, xs, xsum, red, tid);
            const int base = ch * pb.stages_per_chunk();
            for (int g0 = 0; g0 < pb.tasks; g0 += kRingConsumers) {
                const int gtasks = min(kRingConsumers, pb.tasks - g0);
                if (warp >= gtasks) continue;
                float acc[RB][N];
#pragma unroll
                for (int r = 0; r < RB; ++r)
#pragma unroll
                    for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
                bool ok = true;
                for (int sl = 0; sl < nsl_b && ok; ++sl) {
                    const int i = base + g0 * nsl_b + sl * gtasks + warp;
                    ok = wait_stage(i);
                    if (!ok) break;
                    const int k0 = sl * kRingSlice, ks = min(kRingSlice, K - k0);
                    stage_dots_bf16<N, RB>(ring + (size_t)(i % S) * kRingStageBytes, k0, ks, xs, xstride, acc, lane);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars[S + i % S]));
                }
                if (!ok) break;
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    float res[RB];
#pragma unroll
                    for (int r = 0; r < RB; ++r) res[r] = warp_sum(acc[r][n]);
                    if (lane == n && ch * N + n < na) p.template epilogue<RB>(tb0 + g0 + warp, rl.act_idx[ch * N + n], res);
                }
            }
        }
        // -- exit-layer set
        for (int ch = 0; ch < (nr > 0 ? pw.n_chunks : 0); ++ch) {
            consumer_sync();
            ring_load_rows<N, 32>(in, rl.riv_idx, ch * N, nr, K, xstride, xs, xsum, red, tid);
            const int base = stages_b + ch * pw.stages_per_chunk();
            for (int g0 = 0; g0 < pw.tasks; g0 += kRingConsumers) {
                const int gtasks = min(kRingConsumers, pw.tasks - g0);
                if (warp >= gtasks) continue;
                float acc[RW][N];
#pragma unroll
                for (int r = 0; r < RW; ++r)
#pragma unroll
                    for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
                const int i = base + g0 + warp;
                if (!wait_stage(i)) break;
                stage_dots_w4<N, RW>(ring + (size_t)(i % S) * kRingStageBytes, K, p.group, xs, xstride, xsum, acc, lane);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars[S + i % S]));
#pragma unroll
                for (int n = 0; n < N; ++n) {
                    float res[RW];
#pragma unroll
                    for (int r = 0; r < RW; ++r) res[r] = warp_sum(acc[r][n]);
                    if (lane == n && ch * N + n < nr) p.template epilogue<RW>(tw0 + g0 + warp, rl.riv_idx[ch * N + n], res);
                }
            }
        }
    }
    if (s_abort) {
        for (int i = 0; i < 2000; ++i) __nanosleep(100);
    }
}

inline size_t ring_smem_bytes(int S, int N, int K) {
    const int xstride = xs_stride(K, 32);
    return (size_t)S * kRingStageBytes + sizeof(float) * ((size_t)N * xstride + (size_t)N * (K >> 5) + 8) +
           2 * (size_t)S * sizeof(uint64_t) + 128;
}

}  // namespace river
