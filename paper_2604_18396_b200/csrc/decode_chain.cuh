// One persistent kernel for the layer chain of a small-batch decode step (rows <= 4, sm_100a).
//
// At one to four rows every projection is a weight stream and what a step costs beyond the weight bytes is the chain
// of dependent launches: QKV -> attention -> O -> gate/up -> down -> exit score, 32 times.  This kernel runs the whole
// chain, and the LM head, as phases of ONE cooperative launch with one CTA per SM:
//   * phases are separated by a grid barrier (arrive counter in global memory, bounded spin);
//   * a phase splits its weight rows evenly over the CTAs and, inside a CTA, splits (row pair, K slice) units evenly
//     over the warps, so every warp streams the same number of bytes whatever the projection's shape; the partial
//     dot products of a row pair meet in shared memory in a fixed order (deterministic);
//   * a warp that has finished its share of a phase asks the L2 for the first weights it will need in the NEXT phase
//     (cp.async.bulk.prefetch.L2), so HBM keeps streaming through phase tails, barriers, the attention phase and the
//     activation staging of the next phase;
//   * attention (split over KV positions, merged by the last-arriving CTA of a head), the Eq. 1 score, the exit
//     decision and the row lists are computed in-kernel; the decision is taken redundantly and identically by every
//     CTA, so no extra barrier is needed for it.
// Rows still in the backbone use the bf16 weights, rows that left it the 4-bit exit-layer copy (Section 4.1); both
// write K/V to the same cache slots.
#pragma once
#include "gemv_stream.cuh"

namespace river {

struct LayerDev {  // device-resident copy of one block's weight pointers
    const uint16_t *attn_norm, *ffn_norm, *wq, *wk, *wv, *wo, *wg, *wu, *wd;
    W4 rq, rk, rv, ro, rg, ru, rd;
    int32_t has_river, pad;
};

struct ChainArgs {
    const StepMeta *meta;
    const LayerDev *layers;
    int L, d, Hq, Hkv, dh, F, V, group, entry_layer, exit_mode;
    float eps, qscale;  // qscale = log2(e) / sqrt(dh)
    float *h[3], *qbuf, *obuf, *act;
    const float2 *rope_cs;
    KvAddr kv;  // layer0 is set per layer
    float *part_o;      // [row][Hq][splits][dh]
    float2 *part_ml;    // [row][Hq][splits]
    unsigned *attn_tickets;  // [row][Hkv], zero between steps
    uint8_t *exited;    // [max_batch] in: state after the step prologue; out: final state
    Lists lists;
    const uint16_t *lm_head, *final_norm;
    const int32_t *head_rows;
    float *part_val;    // [row][gridDim.x]
    int32_t *part_idx;
    unsigned *bar;      // arrive counter, zero at launch
    int *dev_err;
    unsigned long long *stamps;  // optional [2 + 6 L]: globaltimer at the phase boundaries seen by CTA 0
    unsigned long long *sub;     // optional [5][8]: time CTA 0 spent staging / streaming / finishing / waiting, per phase kind
    int part_cap;       // unit slots for partial dot products
    int pf_bytes;       // bytes of the next phase each warp asks the L2 for
    int xs_floats;      // capacity of the activation staging area
    int part_floats;    // capacity of the partial-sum area
};

constexpr int kChainThreads = 512;
constexpr int kChainWarps = kChainThreads / 32;
constexpr int kChainR = 2;           // weight rows per task
constexpr unsigned kChainSpinLimit = 1u << 20;

__device__ __forceinline__ unsigned long long chain_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Ask the L2 to fetch [p, p + bytes) (never a byte outside the range; 16-byte granules).
__device__ __forceinline__ void l2_prefetch(const void *p, size_t bytes) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    uintptr_t a0 = (a + 15) & ~(uintptr_t)15;
    if (a0 - a >= bytes) return;
    size_t n = (bytes - (a0 - a)) & ~(size_t)15;
    while (n) {
        const uint32_t c = n > 32768 ? 32768u : (uint32_t)n;
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a0), "r"(c) : "memory");
        a0 += c;
        n -= c;
    }
}

// Optional timing probe of CTA 0 / thread 0: time since the previous mark is added to acc[k] (profiling runs only).
struct ChainProbe {
    unsigned long long *acc;
    unsigned long long last;
    __device__ __forceinline__ void mark(int k) {
        if (acc) {
            const unsigned long long t = chain_now();
            acc[k] += t - last;
            last = t;
        }
    }
};

// ---------------------------------------------------------------- grid barrier
// Every CTA arrives once per barrier on a counter that only grows during the launch.  The wait is bounded: a CTA
// that gives up flags DEV_WAIT_TIMEOUT, and every other CTA leaves as soon as it sees the flag.
__device__ __forceinline__ bool chain_grid_sync(unsigned *bar, unsigned &target, int *dev_err, int *s_dead) {
    target += gridDim.x;
    __syncthreads();
    if (threadIdx.x == 0) {
        // release: the CTA's writes (ordered before this thread by the barrier above) become visible before the count
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
        unsigned it = 0;
        for (;;) {
            unsigned v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(bar) : "memory");
            if ((int)(v - target) >= 0) break;
            ++it;
            if (it > kChainSpinLimit) {
                atomicExch(dev_err, DEV_WAIT_TIMEOUT);
                *s_dead = 1;
                break;
            }
            if ((it & 63u) == 0 && *reinterpret_cast<volatile int *>(dev_err) == DEV_WAIT_TIMEOUT) {
                *s_dead = 1;
                break;
            }
        }
    }
    __syncthreads();
    return *s_dead == 0;
}

// ---------------------------------------------------------------- the share of a phase a CTA / warp owns
struct ChainShare {
    int t0, T;        // first task and task count of this CTA
    int nsl;          // K slices per task
    int units;        // T * nsl
};
__device__ __forceinline__ ChainShare chain_share(int tasks, int nit, int its_per_slice) {
    ChainShare s;
    s.t0 = (int)(((long long)tasks * blockIdx.x) / gridDim.x);
    s.T = (int)(((long long)tasks * (blockIdx.x + 1)) / gridDim.x) - s.t0;
    s.nsl = max(1, (nit + its_per_slice - 1) / its_per_slice);
    s.units = s.T * s.nsl;
    return s;
}

// ---------------------------------------------------------------- units: bf16 weights
constexpr int kBfIts = 4;  // 32-lane x 16-byte iterations per slice (1024 inputs)

template <int N, int R>
__device__ __forceinline__ void chain_fma_bf16(const uint4 (&w)[R][kBfIts], const float *xs, int xstride, int it0, int nch,
                                               int lane, float (&acc)[R][N]) {
#pragma unroll
    for (int u = 0; u < kBfIts; ++u) {
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

// ---------------------------------------------------------------- units: 4-bit weights
constexpr int kW4Its = 2;  // 32-lane x 16-byte iterations per slice (2048 inputs)

struct W4Regs {
    uint4 q;
    float s, zz;
};

template <int R>
__device__ __forceinline__ void chain_issue_w4(const W4 (&wrow)[R], int nch, int gshift, int it0, int lane,
                                               W4Regs (&w)[R][kW4Its]) {
#pragma unroll
    for (int u = 0; u < kW4Its; ++u) {
        const int c = (it0 + u) * 32 + lane;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (c < nch) {
                w[r][u].q = ldg_stream16(wrow[r].codes + (size_t)c * 16);
                w[r][u].s = bf16f(ldg_u16(wrow[r].scale + (c >> gshift)));
                w[r][u].zz = bf16f(ldg_u16(wrow[r].zero + (c >> gshift))) + 128.f;
            } else {
                w[r][u].q = make_uint4(0u, 0u, 0u, 0u);
                w[r][u].s = 0.f;
                w[r][u].zz = 0.f;
            }
        }
    }
}

// sum_k (q_k - z) s x_k over a 32-input chunk = s * (sum_k (128 + q_k) x_k - (z + 128) * sum_k x_k); 128 + q is the
// bf16 bit pattern 0x4300 | q, the chunk sums of x are precomputed while staging.
template <int N, int R>
__device__ __forceinline__ void chain_fma_w4(const W4Regs (&w)[R][kW4Its], const float *xs, const float *xsum, int xstride,
                                             int it0, int nch, int lane, float (&acc)[R][N]) {
#pragma unroll
    for (int u = 0; u < kW4Its; ++u) {
        const int c = (it0 + u) * 32 + lane;
        if (c < nch) {
#pragma unroll
            for (int n = 0; n < N; ++n) {
                const float *xb = xs + n * xstride + (c >> 5) * 1024 + lane * 4;
                float p0[R], p1[R];
#pragma unroll
                for (int r = 0; r < R; ++r) { p0[r] = 0.f; p1[r] = 0.f; }
#pragma unroll
                for (int wd = 0; wd < 4; ++wd) {
                    const float4 x0 = *reinterpret_cast<const float4 *>(xb + (2 * wd) * 128);
                    const float4 x1 = *reinterpret_cast<const float4 *>(xb + (2 * wd + 1) * 128);
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const uint4 q = w[r][u].q;
                        const uint32_t v = wd == 0 ? q.x : (wd == 1 ? q.y : (wd == 2 ? q.z : q.w));
                        const uint32_t b0 = (v & 0x000f000fu) | 0x43004300u;
                        const uint32_t b1 = ((v >> 4) & 0x000f000fu) | 0x43004300u;
                        const uint32_t b2 = ((v >> 8) & 0x000f000fu) | 0x43004300u;
                        const uint32_t b3 = ((v >> 12) & 0x000f000fu) | 0x43004300u;
                        p0[r] = fmaf(bf16lo(b0), x0.x, p0[r]); p1[r] = fmaf(bf16lo(b1), x0.y, p1[r]);
                        p0[r] = fmaf(bf16lo(b2), x0.z, p0[r]); p1[r] = fmaf(bf16lo(b3), x0.w, p1[r]);
                        p0[r] = fmaf(bf16hi(b0), x1.x, p0[r]); p1[r] = fmaf(bf16hi(b1), x1.y, p1[r]);
                        p0[r] = fmaf(bf16hi(b2), x1.z, p0[r]); p1[r] = fmaf(bf16hi(b3), x1.w, p1[r]);
                    }
                }
                const float sx = xsum[n * nch + c];
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r][n] = fmaf(w[r][u].s, (p0[r] + p1[r]) - w[r][u].zz * sx, acc[r][n]);
            }
        }
    }
}

template <class P, int R>
__device__ __forceinline__ void chain_rows_w4(const P &p, int t, W4 (&rows)[R]) {
    const int K = p.K, ng = K / p.group;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int run = r / (R / P::NRUN), j = r % (R / P::NRUN);
        const W4 b = p.template w4_base<R>(t, run);
        const size_t row = p.template run_row<R>(t, run) + j;
        rows[r] = W4{b.codes + row * (size_t)(K >> 1), b.scale + row * (size_t)ng, b.zero + row * (size_t)ng};
    }
}

// ---------------------------------------------------------------- L2 prefetch of the first units of a phase
// Units are consumed in index order, so the CTA asks for its first kChainWarps * (pf_bytes / unit bytes) units;
// thread i of the CTA takes (unit i / R, row i % R).
template <class P, int R>
__device__ __forceinline__ void chain_prefetch(const P &p, bool want_bf16, bool want_w4, int pf_bytes) {
    const int K = p.K;
    const int tasks = p.template n_tasks<R>();
    const int i = threadIdx.x;
    if (want_bf16) {
        const int nch = K >> 3;
        const ChainShare sh = chain_share(tasks, (nch + 31) >> 5, kBfIts);
        const int per = kBfIts * 32 * 8;  // inputs per slice
        const int count = min(sh.units, kChainWarps * max(1, pf_bytes / (R * per * 2)));
        const int u = i / R, r = i % R;
        if (u < count) {
            const int t = sh.t0 + u / sh.nsl, sl = u % sh.nsl;
            const int run = r / (R / P::NRUN), j = r % (R / P::NRUN);
            const uint16_t *row = p.template bf16_base<R>(t, run) + (p.template run_row<R>(t, run) + j) * (size_t)K;
            const int k0 = sl * per;
            if (k0 < K) l2_prefetch(row + k0, (size_t)min(per, K - k0) * 2);
        }
    }
    if (want_w4) {
        const int nch = K >> 5;
        const ChainShare sh = chain_share(tasks, (nch + 31) >> 5, kW4Its);
        const int per = kW4Its * 32 * 32;
        const int count = min(sh.units, kChainWarps * max(1, pf_bytes / (R * (per / 2 + 4 * per / p.group))));
        const int u = i / R, r = i % R;
        if (u < count) {
            const int t = sh.t0 + u / sh.nsl, sl = u % sh.nsl;
            W4 rows[R];
            chain_rows_w4<P, R>(p, t, rows);
            const int k0 = sl * per;
            if (k0 < K) {
                const int len = min(per, K - k0);
                l2_prefetch(rows[r].codes + (k0 >> 1), (size_t)len >> 1);
                l2_prefetch(rows[r].scale + k0 / p.group, (size_t)(len / p.group) * 2);
                l2_prefetch(rows[r].zero + k0 / p.group, (size_t)(len / p.group) * 2);
            }
        }
    }
}

// ---------------------------------------------------------------- one pass of a phase over staged activation rows
// The CTA's share of the phase is T tasks x nsl K-slices = units of equal size.  Warps take units from a shared
// counter (a warp that met slow memory simply takes fewer), keep the next unit's loads in flight while they
// multiply the current one, and leave each unit's R x N partial dot products in its own slot; then the CTA's
// threads add a task's slices in slice order (deterministic, whoever computed them) and finish the task:
// epi(task, n, res[R]) gets the R dot products of activation row n of the pass.
template <class P, int N, int R, bool W4M, class PF, class EP>
__device__ __forceinline__ void chain_stream(const P &p, const float *xs, const float *xsum, int xstride, float *part,
                                             int part_cap, int *dev_err, bool do_pf, PF &&prefetch_next, EP &&epi,
                                             int *s_next, ChainProbe &probe, int pk) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int K = p.K;
    const int nch = W4M ? (K >> 5) : (K >> 3);
    constexpr int ITS = W4M ? kW4Its : kBfIts;
    const ChainShare sh = chain_share(p.template n_tasks<R>(), (nch + 31) >> 5, ITS);
    const int nsl = sh.nsl;
    int units = sh.units;
    if (units > part_cap) {  // cannot happen with the host's sizing; flagged rather than trusted
        if (threadIdx.x == 0) atomicExch(dev_err, DEV_INTERNAL);
        units = 0;
    }
    if (threadIdx.x == 0) *s_next = kChainWarps;
    __syncthreads();
    float acc[R][N];
    auto store_unit = [&](int u) {
        float *dst = part + (size_t)u * (R * N);
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int n = 0; n < N; ++n) {
                const float v = warp_sum(acc[r][n]);
                if (lane == 0) dst[r * N + n] = v;
            }
    };
    auto next_unit = [&]() {
        int un = 0;
        if (lane == 0) un = atomicAdd(s_next, 1);
        return __shfl_sync(0xffffffffu, un, 0);
    };
    int u = warp;
    if constexpr (!W4M) {
        uint4 wn[R][kBfIts];
        if (u < units) {
            const int t = u / nsl;
            const uint16_t *rows[R];
            stream_rows_bf16<P, N, R>(p, sh.t0 + t, rows);
            stream_issue_bf16<R>(rows, nch, (u - t * nsl) * ITS, lane, wn);
        }
        while (u < units) {
            uint4 wc[R][kBfIts];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < kBfIts; ++i) wc[r][i] = wn[r][i];
            const int un = next_unit();
            if (un < units) {
                const int tn = un / nsl;
                const uint16_t *rows[R];
                stream_rows_bf16<P, N, R>(p, sh.t0 + tn, rows);
                stream_issue_bf16<R>(rows, nch, (un - tn * nsl) * ITS, lane, wn);
            }
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
            chain_fma_bf16<N, R>(wc, xs, xstride, (u % nsl) * ITS, nch, lane, acc);
            store_unit(u);
            u = un;
        }
    } else {
        const int gshift = (p.group == 64) ? 1 : (p.group == 32 ? 0 : 2);
        W4Regs wn[R][kW4Its];
        if (u < units) {
            const int t = u / nsl;
            W4 rows[R];
            chain_rows_w4<P, R>(p, sh.t0 + t, rows);
            chain_issue_w4<R>(rows, nch, gshift, (u - t * nsl) * ITS, lane, wn);
        }
        while (u < units) {
            W4Regs wc[R][kW4Its];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < kW4Its; ++i) wc[r][i] = wn[r][i];
            const int un = next_unit();
            if (un < units) {
                const int tn = un / nsl;
                W4 rows[R];
                chain_rows_w4<P, R>(p, sh.t0 + tn, rows);
                chain_issue_w4<R>(rows, nch, gshift, (un - tn * nsl) * ITS, lane, wn);
            }
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int n = 0; n < N; ++n) acc[r][n] = 0.f;
            chain_fma_w4<N, R>(wc, xs, xsum, xstride, (u % nsl) * ITS, nch, lane, acc);
            store_unit(u);
            u = un;
        }
    }
    probe.mark(pk + 1);
    if (do_pf) prefetch_next();
    __syncthreads();
    if (!W4M) probe.mark((pk & ~7) + 7);
    if (units > 0)
        for (int e = threadIdx.x; e < sh.T * N; e += blockDim.x) {
            const int tl = e / N, n = e - tl * N;
            float res[R];
#pragma unroll
            for (int r = 0; r < R; ++r) res[r] = 0.f;
            const float *src = part + (size_t)tl * nsl * (R * N) + n;
            for (int sl = 0; sl < nsl; ++sl)
#pragma unroll
                for (int r = 0; r < R; ++r) res[r] += src[(sl * R + r) * N];
            epi(sh.t0 + tl, n, res);
        }
    __syncthreads();
    probe.mark(pk + 2);
}

struct ChainSmem {
    float *red, *xsum, *part, *xs;
};

// A projection phase: the rows still in the backbone against the bf16 weights, then the rows in the exit layers
// against the 4-bit copy, N rows per pass.
template <class P, int N, class PF>
__device__ __forceinline__ void chain_project(const ChainArgs &a, const P &p, const ProjIn &in, const int *s_act, int na,
                                              const int *s_riv, int nr, const ChainSmem &sm, PF &&prefetch_next,
                                              int *s_next, ChainProbe &probe, int pk, bool prestaged = false) {
    constexpr int R = kChainR;
    const int K = p.K;
    const int xstride = xs_stride(K, 32);
    const int passes_a = (na + N - 1) / N, passes_r = (nr + N - 1) / N;
    for (int ps = 0; ps < passes_a; ++ps) {
        const int i0 = ps * N;
        if (!(prestaged && ps == 0)) stream_load_rows<N, 8>(in, s_act, i0, na, K, xstride, sm.xs, sm.xsum, sm.red);
        probe.mark(pk);
        chain_stream<P, N, R, false>(p, sm.xs, sm.xsum, xstride, sm.part, a.part_cap, a.dev_err,
                                     ps + 1 == passes_a && passes_r == 0, prefetch_next,
                                     [&](int t, int n, const float(&res)[R]) {
                                         if (i0 + n < na) p.template epilogue<R>(t, s_act[i0 + n], res);
                                     }, s_next, probe, pk);
    }
    for (int ps = 0; ps < passes_r; ++ps) {
        const int i0 = ps * N;
        if (!(prestaged && ps == 0 && passes_a == 0)) stream_load_rows<N, 32>(in, s_riv, i0, nr, K, xstride, sm.xs, sm.xsum, sm.red);
        probe.mark(pk + 4);
        chain_stream<P, N, R, true>(p, sm.xs, sm.xsum, xstride, sm.part, a.part_cap, a.dev_err, ps + 1 == passes_r,
                                    prefetch_next, [&](int t, int n, const float(&res)[R]) {
                                        if (i0 + n < nr) p.template epilogue<R>(t, s_riv[i0 + n], res);
                                    }, s_next, probe, pk + 4);
    }
    if (passes_a + passes_r == 0) prefetch_next();
}

// ---------------------------------------------------------------- a3 inside the chain: split-KV decode attention
// Work item = (row, kv head, split of the positions).  A warp takes four consecutive positions of one page at a
// time (a lane owns DH/32 head dims of K and V), keeps a base-2 online softmax per query head of the group, the
// warps of the CTA merge through shared memory and the CTA writes one partial per item; the last CTA of a (row, kv
// head) to arrive merges the splits in split order (deterministic) and writes the attention output.
struct ChainFlags {
    int exited[4], act[4], riv[4], pass[4];
    int na, nr, dead, flag, next;
    // per-step constants of the decision, read once (the per-layer decision then touches no global memory to decide)
    float tau[4];
    int forced[4];
    float *scores;
    int32_t *exit_layer;
};

__device__ __forceinline__ float chain_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Raw K and V bits of one cached position for this lane's DH / 32 head dims.
template <int VE>
__device__ __forceinline__ void attn_load_raw(const KvAddr &kv, int page, int kvh, int p, int lane, uint2 &k, uint2 &v) {
    const __nv_bfloat16 *kp = kv.pool + kv.base(page, 0, kvh, p % kPage) + lane * VE;
    const __nv_bfloat16 *vp = kv.pool + kv.base(page, 1, kvh, p % kPage) + lane * VE;
    if constexpr (VE == 4) {
        k = __ldcg(reinterpret_cast<const uint2 *>(kp));
        v = __ldcg(reinterpret_cast<const uint2 *>(vp));
    } else {
        k = make_uint2(__ldcg(reinterpret_cast<const uint32_t *>(kp)), 0u);
        v = make_uint2(__ldcg(reinterpret_cast<const uint32_t *>(vp)), 0u);
    }
}

// The cached positions of this warp's first batch of the CTA's first work item, requested BEFORE the grid barrier
// that ends the QKV phase: everything but the position written in this very step is already in the cache.
struct AttnPre {
    uint2 k[4], v[4];
    unsigned mask;  // bit u: position u of the batch is in k[u], v[u]
};
template <int DH>
__device__ __forceinline__ void chain_attention_preload(const ChainArgs &a, const KvAddr &kv, int n_rows, int S, int chunk,
                                                        AttnPre &pre) {
    constexpr int VE = DH / 32, U = 4;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pre.mask = 0u;
    const int item = blockIdx.x;
    if (item >= n_rows * a.Hkv * S) return;
    const int sp = item % S, kvh = (item / S) % a.Hkv, row = item / (S * a.Hkv);
    const int pos = kv.row_pos[row], slot = kv.row_slot[row];
    const int p0 = sp * chunk, p1 = min(pos + 1, p0 + chunk);
    const int pb = p0 + warp * U;
    if (pb >= p1) return;
    const int page = kv.page_tbl[(size_t)slot * kv.max_pages_per_seq + pb / kPage];
    if (page < 0 || page >= kv.n_pages) return;  // the attention phase itself reports it
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int p = pb + u;
        if (p < p1 && p != pos) {
            attn_load_raw<VE>(kv, page, kvh, p, lane, pre.k[u], pre.v[u]);
            pre.mask |= 1u << u;
        }
    }
}

template <int DH, int GQ>
__device__ __forceinline__ void chain_attention(const ChainArgs &a, const KvAddr &kv, int n_rows, int S, int chunk,
                                                float *sm, ChainFlags *fl, const AttnPre &pre) {
    constexpr int VE = DH / 32, U = 4, NW = kChainWarps;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float *s_m = sm, *s_l = sm + NW * GQ, *s_acc = sm + 2 * NW * GQ;  // [NW][GQ], [NW][GQ], [NW][GQ][DH]
    const int items = n_rows * a.Hkv * S;
    const int Hq = a.Hq;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int sp = item % S, kvh = (item / S) % a.Hkv, row = item / (S * a.Hkv);
        const int pos = kv.row_pos[row], slot = kv.row_slot[row];
        const int p0 = sp * chunk, p1 = min(pos + 1, p0 + chunk);
        float qr[GQ][VE], acc[GQ][VE], m[GQ], l[GQ];
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            m[g] = -CUDART_INF_F;
            l[g] = 0.f;
            const float *qp = a.qbuf + (size_t)row * Hq * DH + (size_t)(kvh * GQ + g) * DH + lane * VE;
            if constexpr (VE == 4) {
                const float4 q4 = __ldcg(reinterpret_cast<const float4 *>(qp));
                qr[g][0] = q4.x * a.qscale; qr[g][1] = q4.y * a.qscale; qr[g][2] = q4.z * a.qscale; qr[g][3] = q4.w * a.qscale;
            } else {
                const float2 q2 = __ldcg(reinterpret_cast<const float2 *>(qp));
                qr[g][0] = q2.x * a.qscale; qr[g][1] = q2.y * a.qscale;
            }
#pragma unroll
            for (int e = 0; e < VE; ++e) acc[g][e] = 0.f;
        }
        const int32_t *pt = kv.page_tbl + (size_t)slot * kv.max_pages_per_seq;
        for (int pb = p0 + warp * U; pb < p1; pb += NW * U) {  // pb is a multiple of 4: one page per batch
            int page = pt[pb / kPage];
            if (page < 0 || page >= kv.n_pages) {
                if (lane == 0) atomicExch(a.dev_err, DEV_BAD_PAGE);
                page = 0;
            }
            float kf[U][VE], vf[U][VE];
            const bool first = item == (int)blockIdx.x && pb == p0 + warp * U;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int p = pb + u;
                if (p < p1) {
                    uint2 kr, vr;
                    if (first && ((pre.mask >> u) & 1u)) { kr = pre.k[u]; vr = pre.v[u]; }
                    else attn_load_raw<VE>(kv, page, kvh, p, lane, kr, vr);
                    kf[u][0] = bf16lo(kr.x); kf[u][1] = bf16hi(kr.x);
                    vf[u][0] = bf16lo(vr.x); vf[u][1] = bf16hi(vr.x);
                    if constexpr (VE == 4) {
                        kf[u][2] = bf16lo(kr.y); kf[u][3] = bf16hi(kr.y);
                        vf[u][2] = bf16lo(vr.y); vf[u][3] = bf16hi(vr.y);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < VE; ++e) { kf[u][e] = 0.f; vf[u][e] = 0.f; }
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (pb + u < p1) {  // warp-uniform
#pragma unroll
                    for (int g = 0; g < GQ; ++g) {
                        float s = 0.f;
#pragma unroll
                        for (int e = 0; e < VE; ++e) s = fmaf(qr[g][e], kf[u][e], s);
                        s = warp_sum(s);
                        const float mn = fmaxf(m[g], s);
                        const float corr = chain_ex2(m[g] - mn), pr = chain_ex2(s - mn);
                        l[g] = l[g] * corr + pr;
#pragma unroll
                        for (int e = 0; e < VE; ++e) acc[g][e] = fmaf(pr, vf[u][e], acc[g][e] * corr);
                        m[g] = mn;
                    }
                }
            }
        }
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            if (lane == 0) { s_m[warp * GQ + g] = m[g]; s_l[warp * GQ + g] = l[g]; }
#pragma unroll
            for (int e = 0; e < VE; ++e) s_acc[(warp * GQ + g) * DH + lane * VE + e] = acc[g][e];
        }
        __syncthreads();
        for (int t = threadIdx.x; t < GQ * DH; t += blockDim.x) {
            const int g = t / DH, e = t % DH;
            float M = -CUDART_INF_F;
            for (int w = 0; w < NW; ++w) M = fmaxf(M, s_m[w * GQ + g]);
            float num = 0.f, den = 0.f;
            for (int w = 0; w < NW; ++w) {
                const float mw = s_m[w * GQ + g];
                const float c = (mw == -CUDART_INF_F) ? 0.f : chain_ex2(mw - M);
                num = fmaf(c, s_acc[(w * GQ + g) * DH + e], num);
                den = fmaf(c, s_l[w * GQ + g], den);
            }
            const int head = kvh * GQ + g;
            if (S == 1) {
                a.obuf[(size_t)row * Hq * DH + (size_t)head * DH + e] = num / den;
            } else {
                const size_t pi = ((size_t)row * Hq + head) * S + sp;
                a.part_o[pi * DH + e] = num;
                if (e == 0) a.part_ml[pi] = make_float2(M, den);
            }
        }
        if (S > 1) {
            __syncthreads();  // the CTA's partial is written ...
            if (threadIdx.x == 0) {
                __threadfence();  // ... and made visible before the ticket (one fence, cumulative over the barrier)
                const unsigned tk = atomicAdd(a.attn_tickets + row * a.Hkv + kvh, 1u);
                fl->flag = (tk == (unsigned)(S - 1));
                __threadfence();
            }
            __syncthreads();
            if (fl->flag) {
                // (max, sum) of every (head, split) into shared memory, then every thread owns one (head, dim) and
                // pulls the splits' partial outputs in batches of independent loads
                float *s_mx = s_acc, *s_sm = s_acc + GQ * 64;
                for (int t = threadIdx.x; t < GQ * S; t += blockDim.x) {
                    const int g = t / S, s2 = t % S;
                    const float2 ml = __ldcg(&a.part_ml[((size_t)row * Hq + kvh * GQ + g) * S + s2]);
                    s_mx[g * 64 + s2] = ml.x;
                    s_sm[g * 64 + s2] = ml.y;
                }
                __syncthreads();
                for (int t = threadIdx.x; t < GQ * DH; t += blockDim.x) {
                    const int g = t / DH, e = t % DH;
                    const float *po = a.part_o + ((size_t)row * Hq + kvh * GQ + g) * S * DH + e;
                    float M = -CUDART_INF_F;
                    for (int s2 = 0; s2 < S; ++s2) M = fmaxf(M, s_mx[g * 64 + s2]);
                    float num = 0.f, den = 0.f;
                    for (int s0 = 0; s0 < S; s0 += 8) {
                        float v[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) v[k] = (s0 + k < S) ? __ldcg(po + (size_t)(s0 + k) * DH) : 0.f;
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            if (s0 + k < S) {
                                const float mx = s_mx[g * 64 + s0 + k];
                                const float c = (mx == -CUDART_INF_F) ? 0.f : chain_ex2(mx - M);
                                num = fmaf(c, v[k], num);
                                den = fmaf(c, s_sm[g * 64 + s0 + k], den);
                            }
                    }
                    a.obuf[(size_t)row * Hq * DH + (size_t)(kvh * GQ + g) * DH + e] = num / den;
                }
                if (threadIdx.x == 0) a.attn_tickets[row * a.Hkv + kvh] = 0u;
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------- the same attention as a kernel of its own
// For steps of 1-4 rows in the one-kernel-per-stage plan: one CTA per (row, KV head, split).  The cached positions do
// of a decode step do not depend on the preceding QKV kernel (it writes only each row's newest position), so they
// are requested before griddepcontrol.wait; after it only q and the newest position remain.  (Larger steps use the
// TMA-fed kernel.)
template <int DH, int GQ>
__global__ void __launch_bounds__(kChainThreads) attn_small_kernel(const ChainArgs a, int layer0, int early) {
    extern __shared__ __align__(16) float attn_small_smem[];
    __shared__ ChainFlags fl;
    pdl_launch();
    KvAddr kv = a.kv;
    kv.layer0 = layer0;
    const int n = a.meta->n_rows, S = a.meta->pad[1], chunk = a.meta->pad[0];
    AttnPre pre;
    pre.mask = 0u;
    // early: every row of the step belongs to a different sequence (a decode step), so the QKV kernel in flight
    // writes nothing but each row's newest position.  Prefill chunks hold consecutive positions of one sequence and
    // must wait.
    if (early) chain_attention_preload<DH>(a, kv, n, S, chunk, pre);
    pdl_wait();
    chain_attention<DH, GQ>(a, kv, n, S, chunk, attn_small_smem, &fl, pre);
}

// ---------------------------------------------------------------- a6 + a7 inside the chain
// Eq. 1 for every row still in the backbone, the exit decision and the row lists entering block l + 1.  Every CTA
// runs this on the same inputs with the same reduction order, so all CTAs hold identical lists; CTA 0 publishes
// them (and the scores / exit layers) to global memory for the host-side queries.
__device__ __forceinline__ void chain_decide(const ChainArgs &a, int l, const float *h_in, const float *h_out, int n,
                                             float *red, ChainFlags *fl) {
    const int L = a.L, d = a.d;
    const bool eligible = (l >= 1) && (l >= a.entry_layer) && (l < L);
    float *scores = fl->scores;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int row = 0; row < n; ++row) {
        if (fl->exited[row] != 0 || !(eligible || scores)) continue;  // uniform across the CTA
        const float4 *x = reinterpret_cast<const float4 *>(h_in + (size_t)row * d);
        const float4 *y = reinterpret_cast<const float4 *>(h_out + (size_t)row * d);
        float ab = 0.f, aa = 0.f, bb = 0.f;
        for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
            const float4 u = __ldcg(x + i), v = __ldcg(y + i);
            ab += u.x * v.x + u.y * v.y + u.z * v.z + u.w * v.w;
            aa += u.x * u.x + u.y * u.y + u.z * u.z + u.w * u.w;
            bb += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ab = warp_sum(ab); aa = warp_sum(aa); bb = warp_sum(bb);
        __syncthreads();
        if (lane == 0) { red[warp] = ab; red[32 + warp] = aa; red[64 + warp] = bb; }
        __syncthreads();
        if (threadIdx.x == 0) {
            ab = aa = bb = 0.f;
            for (int w = 0; w < kChainWarps; ++w) { ab += red[w]; aa += red[32 + w]; bb += red[64 + w]; }
            float s = 0.f;
            if (aa > 0.f && bb > 0.f) s = ab / (sqrtf(aa) * sqrtf(bb));
            fl->pass[row] = (s > fl->tau[row]) ? 1 : 0;
            if (scores && blockIdx.x == 0) scores[(size_t)row * L + (l - 1)] = s;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int allpass = 1;
        if (a.exit_mode == 1)
            for (int b = 0; b < n; ++b)
                if (fl->exited[b] == 0 && !(eligible && fl->pass[b])) allpass = 0;
        int na = 0, nr = 0;
        for (int b = 0; b < n; ++b) {
            if (fl->exited[b] == 0) {
                bool leave = eligible && (a.exit_mode == 1 ? (allpass != 0) : (fl->pass[b] != 0));
                const int f = fl->forced[b];
                if (f >= 0) leave = (f == l) && (l < L);
                if (leave) {
                    fl->exited[b] = 1;
                    if (blockIdx.x == 0) { fl->exit_layer[b] = l; a.exited[b] = 1; }
                }
            }
            if (fl->exited[b] == 0) fl->act[na++] = b;
            else fl->riv[nr++] = b;
        }
        fl->na = na;
        fl->nr = nr;
        if (blockIdx.x == 0) {
            int32_t *A = a.lists.act_idx + (size_t)l * a.lists.max_batch, *R = a.lists.riv_idx + (size_t)l * a.lists.max_batch;
            for (int i = 0; i < na; ++i) A[i] = fl->act[i];
            for (int i = 0; i < nr; ++i) R[i] = fl->riv[i];
            a.lists.n_act[l] = na;
            a.lists.n_riv[l] = nr;
        }
    }
    __syncthreads();
}

// ---------------------------------------------------------------- a6 + a7 fused with the next block's first staging
// The block output that Eq. 1 scores is also the input of the next block's attention norm: one pass loads it
// (and the block input of the rows that still need a score), yields dot product, both squared norms (the second
// is the RMS statistic), takes the decision, and writes the normalised rows of the next QKV phase's first pass
// straight from registers.  Returns false (and falls back to chain_decide) when a row does not fit in two 128-bit
// values per thread.
template <int N>
__device__ __forceinline__ bool chain_decide_stage(const ChainArgs &a, int l, const float *h_in, const float *h_out, int n,
                                                   const uint16_t *gain_next, const ChainSmem &sm, ChainFlags *fl) {
    const int L = a.L, d = a.d, nv = d >> 2;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
    if (nv > 2 * nthr) {
        chain_decide(a, l, h_in, h_out, n, sm.red, fl);
        return false;
    }
    const bool eligible = (l >= 1) && (l >= a.entry_layer) && (l < L);
    float *scores = fl->scores;
    float4 v[N][2];  // the step has at most N rows
    float ab[N], aa[N], bb[N];
#pragma unroll
    for (int b = 0; b < N; ++b) {
        ab[b] = aa[b] = bb[b] = 0.f;
#pragma unroll
        for (int k = 0; k < 2; ++k) v[b][k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (b < n) {
            const bool need = fl->exited[b] == 0 && (eligible || scores);  // uniform across the CTA
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int i = tid + k * nthr;
                if (i < nv) {
                    const float4 y = __ldcg(reinterpret_cast<const float4 *>(h_out + (size_t)b * d) + i);
                    v[b][k] = y;
                    bb[b] += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
                    if (need) {
                        const float4 x = __ldcg(reinterpret_cast<const float4 *>(h_in + (size_t)b * d) + i);
                        ab[b] += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
                        aa[b] += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
                    }
                }
            }
        }
    }
    float *red = sm.red;  // [3][4][kChainWarps]
#pragma unroll
    for (int b = 0; b < N; ++b) {
        if (b < n) {
            const float sab = warp_sum(ab[b]), saa = warp_sum(aa[b]), sbb = warp_sum(bb[b]);
            if (lane == 0) {
                red[(0 * 4 + b) * kChainWarps + warp] = sab;
                red[(1 * 4 + b) * kChainWarps + warp] = saa;
                red[(2 * 4 + b) * kChainWarps + warp] = sbb;
            }
        }
    }
    __syncthreads();
    float bbt[N];
#pragma unroll
    for (int b = 0; b < N; ++b) {
        bbt[b] = 0.f;
        if (b < n)
            for (int w = 0; w < kChainWarps; ++w) bbt[b] += red[(2 * 4 + b) * kChainWarps + w];
    }
    if (tid == 0) {
        for (int b = 0; b < n; ++b) {
            fl->pass[b] = 0;
            if (fl->exited[b] == 0 && (eligible || scores)) {
                float tab = 0.f, taa = 0.f;
                for (int w = 0; w < kChainWarps; ++w) { tab += red[(0 * 4 + b) * kChainWarps + w]; taa += red[(1 * 4 + b) * kChainWarps + w]; }
                float sc = 0.f;
                if (taa > 0.f && bbt[b] > 0.f) sc = tab / (sqrtf(taa) * sqrtf(bbt[b]));
                fl->pass[b] = (sc > fl->tau[b]) ? 1 : 0;
                if (scores && blockIdx.x == 0) scores[(size_t)b * L + (l - 1)] = sc;
            }
        }
        int allpass = 1;
        if (a.exit_mode == 1)
            for (int b = 0; b < n; ++b)
                if (fl->exited[b] == 0 && !(eligible && fl->pass[b])) allpass = 0;
        int na = 0, nr = 0;
        for (int b = 0; b < n; ++b) {
            if (fl->exited[b] == 0) {
                bool leave = eligible && (a.exit_mode == 1 ? (allpass != 0) : (fl->pass[b] != 0));
                const int f = fl->forced[b];
                if (f >= 0) leave = (f == l) && (l < L);
                if (leave) {
                    fl->exited[b] = 1;
                    if (blockIdx.x == 0) { fl->exit_layer[b] = l; a.exited[b] = 1; }
                }
            }
            if (fl->exited[b] == 0) fl->act[na++] = b;
            else fl->riv[nr++] = b;
        }
        fl->na = na;
        fl->nr = nr;
        if (blockIdx.x == 0) {
            int32_t *A = a.lists.act_idx + (size_t)l * a.lists.max_batch, *R = a.lists.riv_idx + (size_t)l * a.lists.max_batch;
            for (int i = 0; i < na; ++i) A[i] = fl->act[i];
            for (int i = 0; i < nr; ++i) R[i] = fl->riv[i];
            a.lists.n_act[l] = na;
            a.lists.n_riv[l] = nr;
        }
    }
    __syncthreads();
    if (l >= L) return false;  // the LM head stages its own rows
    // ---- first pass of the next QKV phase: the backbone rows if any are left, else the exit-layer rows
    const bool bf = fl->na > 0;
    const int *list = bf ? fl->act : fl->riv;
    const int len = bf ? fl->na : fl->nr;
    const int xstride = xs_stride(d, 32);
#pragma unroll
    for (int j = 0; j < N; ++j) {
        float *dst = sm.xs + j * xstride;
        if (j >= len) {
            for (int k = tid; k < xstride; k += nthr) dst[k] = 0.f;
            continue;
        }
        const int rowid = list[j];
        float4 x[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
        float ssq = 0.f;
#pragma unroll
        for (int b = 0; b < N; ++b)
            if (b == rowid) { x[0] = v[b][0]; x[1] = v[b][1]; ssq = bbt[b]; }
        const float scale = rsqrtf(ssq / (float)d + a.eps);
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int i = tid + k * nthr;
            if (i < nv) {
                const uint2 gw = *reinterpret_cast<const uint2 *>(gain_next + 4 * i);
                float4 y = x[k];
                y.x *= scale * bf16lo(gw.x); y.y *= scale * bf16hi(gw.x);
                y.z *= scale * bf16lo(gw.y); y.w *= scale * bf16hi(gw.y);
                if (bf) *reinterpret_cast<float4 *>(dst + xs_index<8>(4 * i)) = y;
                else *reinterpret_cast<float4 *>(dst + xs_index<32>(4 * i)) = y;
            }
        }
    }
    __syncthreads();
    if (!bf) stream_chunk_sums<N>(sm.xs, sm.xsum, d, xstride);
    return true;
}

// ---------------------------------------------------------------- a8 inside the chain: LM head as a stream problem
struct HeadProblem {
    static constexpr int NRUN = 1;
    const uint16_t *w;
    int K, V, group;
    template <int R> __device__ int n_tasks() const { return V / R; }
    template <int R> __device__ size_t run_row(int t, int) const { return (size_t)t * R; }
    template <int R> __device__ const uint16_t *bf16_base(int, int) const { return w; }
    template <int R> __device__ W4 w4_base(int, int) const { return W4{nullptr, nullptr, nullptr}; }
};

struct NoProblem {  // "nothing follows"
    static constexpr int NRUN = 1;
    int K, group;
    template <int R> __device__ int n_tasks() const { return 0; }
    template <int R> __device__ size_t run_row(int, int) const { return 0; }
    template <int R> __device__ const uint16_t *bf16_base(int, int) const { return nullptr; }
    template <int R> __device__ W4 w4_base(int, int) const { return W4{nullptr, nullptr, nullptr}; }
};

// ---------------------------------------------------------------- the kernel
// N = activation rows per pass (1, 2 or 4; the host picks the smallest that holds the step's rows, or fewer if the
// widest input does not fit in shared memory N times).  Launched cooperatively: gridDim.x CTAs are co-resident.
template <int N, int DH, int GQ>
__global__ void __launch_bounds__(kChainThreads, 1) decode_chain_kernel(const ChainArgs a) {
    extern __shared__ __align__(16) float chain_smem[];
    __shared__ ChainFlags fl;
    __shared__ LayerDev s_layer[2];  // this block's and the next block's weight pointers (fetched one block ahead)
    __shared__ float s_best[kChainWarps];
    __shared__ int s_besti[kChainWarps];
    constexpr int R = kChainR;
    const int Kmax = max(max(a.d, a.F), a.Hq * a.dh);
    ChainSmem sm;
    sm.red = chain_smem;                                  // 256
    sm.xsum = chain_smem + 256;                            // N * Kmax / 32
    sm.part = sm.xsum + ((N * (Kmax >> 5) + 3) & ~3);     // kChainWarps * part_cap * R * N
    sm.xs = sm.part + a.part_floats;
    const int n = a.meta->n_rows;
    const int L = a.L;
    unsigned target = 0;
    if (threadIdx.x == 0) {
        fl.dead = 0;
        fl.flag = 0;
        int na = 0, nr = 0;
        fl.scores = a.meta->scores;
        fl.exit_layer = a.meta->exit_layer;
        for (int b = 0; b < n && b < 4; ++b) {
            fl.tau[b] = a.meta->tau[b];
            fl.forced[b] = a.meta->forced ? a.meta->forced[b] : -1;
            fl.exited[b] = a.exited[b];
            fl.pass[b] = 0;
            if (fl.exited[b] == 0) fl.act[na++] = b;
            else fl.riv[nr++] = b;
        }
        fl.na = na;
        fl.nr = nr;
    }
    {
        constexpr int kWords = (int)(sizeof(LayerDev) / sizeof(unsigned long long));
        static_assert(sizeof(LayerDev) % sizeof(unsigned long long) == 0, "LayerDev is copied in 8-byte words");
        const int t = threadIdx.x - 32;  // warp 1 copies; warp 0's thread 0 is busy above
        if (t >= 0 && t < kWords) reinterpret_cast<unsigned long long *>(&s_layer[0])[t] = reinterpret_cast<const unsigned long long *>(&a.layers[0])[t];
        if (t >= 0 && t < kWords && a.L > 1) reinterpret_cast<unsigned long long *>(&s_layer[1])[t] = reinterpret_cast<const unsigned long long *>(&a.layers[1])[t];
    }
    __syncthreads();
    const bool stamp = a.stamps != nullptr && blockIdx.x == 0 && threadIdx.x == 0;
    int si = 0;
    if (stamp) a.stamps[si++] = chain_now();
    ChainProbe probe{stamp ? a.sub : nullptr, chain_now()};
    const int S = a.meta->pad[1], chunk = a.meta->pad[0];
    int hi = 0;
    bool prestaged = false;  // the QKV phase's first rows were staged by the previous block's decision pass
    for (int l = 1; l <= L; ++l) {
        const LayerDev &w = s_layer[(l - 1) & 1];
        float *h_in = a.h[hi], *h_mid = a.h[(hi + 1) % 3], *h_out = a.h[(hi + 2) % 3];
        const int na = fl.na, nr = w.has_river ? fl.nr : 0;
        const bool riv = nr > 0, act = na > 0;

        QkvProblem pq{};
        pq.wq = w.wq; pq.wk = w.wk; pq.wv = w.wv; pq.rq = w.rq; pq.rk = w.rk; pq.rv = w.rv;
        pq.K = a.d; pq.Hq = a.Hq; pq.Hkv = a.Hkv; pq.dh = a.dh; pq.group = a.group;
        pq.rope_cs = a.rope_cs; pq.q_out = a.qbuf; pq.kv = a.kv; pq.kv.layer0 = l - 1; pq.dev_err = a.dev_err;
        ResidProblem po{};
        po.w = w.wo; po.rw = w.ro; po.K = a.Hq * a.dh; po.out_dim = a.d; po.group = a.group; po.resid = h_in; po.out = h_mid;
        GateUpProblem pg{};
        pg.wg = w.wg; pg.wu = w.wu; pg.rg = w.rg; pg.ru = w.ru; pg.K = a.d; pg.F = a.F; pg.group = a.group; pg.act = a.act;
        ResidProblem pd{};
        pd.w = w.wd; pd.rw = w.rd; pd.K = a.F; pd.out_dim = a.d; pd.group = a.group; pd.resid = h_mid; pd.out = h_out;

        // ---- a2
        chain_project<QkvProblem, N>(a, pq, ProjIn{h_in, w.attn_norm, a.eps}, fl.act, na, fl.riv, nr, sm,
                                     [&]() { chain_prefetch<ResidProblem, R>(po, act, riv, a.pf_bytes); }, &fl.next, probe, 0, prestaged);
        AttnPre apre;
        chain_attention_preload<DH>(a, pq.kv, n, S, chunk, apre);  // cached positions travel across the barrier
        if (!chain_grid_sync(a.bar, target, a.dev_err, &fl.dead)) return;
        probe.mark(3);
        if (stamp) a.stamps[si++] = chain_now();
        // ---- a3
        chain_attention<DH, GQ>(a, pq.kv, n, S, chunk, sm.xs, &fl, apre);
        probe.mark(32);
        if (!chain_grid_sync(a.bar, target, a.dev_err, &fl.dead)) return;
        probe.mark(35);
        if (stamp) a.stamps[si++] = chain_now();
        // ---- a4
        chain_project<ResidProblem, N>(a, po, ProjIn{a.obuf, nullptr, 0.f}, fl.act, na, fl.riv, nr, sm,
                                       [&]() { chain_prefetch<GateUpProblem, R>(pg, act, riv, a.pf_bytes); }, &fl.next, probe, 8);
        if (!chain_grid_sync(a.bar, target, a.dev_err, &fl.dead)) return;
        probe.mark(11);
        if (stamp) a.stamps[si++] = chain_now();
        // ---- a5: gate / up + SwiGLU
        chain_project<GateUpProblem, N>(a, pg, ProjIn{h_mid, w.ffn_norm, a.eps}, fl.act, na, fl.riv, nr, sm,
                                        [&]() { chain_prefetch<ResidProblem, R>(pd, act, riv, a.pf_bytes); }, &fl.next, probe, 16);
        if (!chain_grid_sync(a.bar, target, a.dev_err, &fl.dead)) return;
        probe.mark(19);
        if (stamp) a.stamps[si++] = chain_now();
        // ---- a5: down + residual; what follows is block l + 1 with the lists as they stand (an exit at this layer
        // makes the bf16 part of that request useless, once per token), or the LM head
        chain_project<ResidProblem, N>(a, pd, ProjIn{a.act, nullptr, 0.f}, fl.act, na, fl.riv, nr, sm, [&]() {
            if (l < L) {
                const LayerDev &wn = s_layer[l & 1];
                QkvProblem pn = pq;
                pn.wq = wn.wq; pn.wk = wn.wk; pn.wv = wn.wv; pn.rq = wn.rq; pn.rk = wn.rk; pn.rv = wn.rv;
                chain_prefetch<QkvProblem, R>(pn, act, wn.has_river && fl.nr > 0, a.pf_bytes);
            } else {
                HeadProblem ph{a.lm_head, a.d, a.V, a.group};
                chain_prefetch<HeadProblem, R>(ph, true, false, a.pf_bytes);
            }
        }, &fl.next, probe, 24);
        if (!chain_grid_sync(a.bar, target, a.dev_err, &fl.dead)) return;
        probe.mark(27);
        if (stamp) a.stamps[si++] = chain_now();
        // ---- a6 + a7
        prestaged = chain_decide_stage<N>(a, l, h_in, h_out, n, l < L ? s_layer[l & 1].attn_norm : nullptr, sm, &fl);
        probe.mark(36);
        if (stamp) a.stamps[si++] = chain_now();
        if (l + 1 < L) {  // block l + 2's pointers into the slot block l used (its last reader is behind the barrier above)
            constexpr int kWords = (int)(sizeof(LayerDev) / sizeof(unsigned long long));
            const int t = threadIdx.x;
            if (t < kWords) reinterpret_cast<unsigned long long *>(&s_layer[(l + 1) & 1])[t] = reinterpret_cast<const unsigned long long *>(&a.layers[l + 1])[t];
        }
        hi = (hi + 2) % 3;
    }

    // ---- a8: final norm + LM head + per-CTA argmax partials (merged by argmax_final_kernel)
    const int n_head = a.meta->n_head_rows;
    if (n_head > 0) {
        HeadProblem ph{a.lm_head, a.d, a.V, a.group};
        float *logits = a.meta->logits;
        const ProjIn in{a.h[hi], a.final_norm, a.eps};
        const int xstride = xs_stride(a.d, 32);
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int i0 = 0; i0 < n_head; i0 += N) {
            stream_load_rows<N, 8>(in, a.head_rows, i0, n_head, a.d, xstride, sm.xs, sm.xsum, sm.red);
            float best[N];
            int besti[N];
#pragma unroll
            for (int k = 0; k < N; ++k) { best[k] = -CUDART_INF_F; besti[k] = 0x7fffffff; }
            NoProblem none{a.d, a.group};
            chain_stream<HeadProblem, N, R, false>(ph, sm.xs, sm.xsum, xstride, sm.part, a.part_cap, a.dev_err, false,
                                                   [&]() { (void)none; }, [&](int t, int k, const float(&res)[R]) {
                                                       if (i0 + k >= n_head) return;
#pragma unroll
                                                       for (int r = 0; r < R; ++r) {
                                                           const int id = t * R + r;
                                                           if (logits) logits[(size_t)(i0 + k) * a.V + id] = res[r];
#pragma unroll
                                                           for (int kk = 0; kk < N; ++kk)
                                                               if (kk == k && (res[r] > best[kk] || (res[r] == best[kk] && id < besti[kk]))) {
                                                                   best[kk] = res[r];
                                                                   besti[kk] = id;
                                                               }
                                                       }
                                                   }, &fl.next, probe, 40);
#pragma unroll
            for (int k = 0; k < N; ++k) {
                float bv = best[k];
                int bi = besti[k];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                }
                if (lane == 0) { s_best[warp] = bv; s_besti[warp] = bi; }
                __syncthreads();
                if (threadIdx.x == 0 && i0 + k < n_head) {
                    for (int w2 = 1; w2 < kChainWarps; ++w2)
                        if (s_best[w2] > bv || (s_best[w2] == bv && s_besti[w2] < bi)) { bv = s_best[w2]; bi = s_besti[w2]; }
                    a.part_val[(size_t)(i0 + k) * gridDim.x + blockIdx.x] = bv;
                    a.part_idx[(size_t)(i0 + k) * gridDim.x + blockIdx.x] = bi;
                }
                __syncthreads();
            }
        }
    }
    if (stamp) a.stamps[si++] = chain_now();
}

// Shared memory the kernel needs for N rows per pass.
struct ChainLayout {
    int xs_floats, part_floats;
    size_t bytes;
};
// Shared memory of the kernel for N rows per pass: reduction scratch, chunk sums, unit slots, staging area (fp32
// rows, or the attention scratch).
inline ChainLayout chain_layout(int N, int Kmax, int part_cap, int dh, int gq) {
    ChainLayout l;
    const size_t xs = std::max<size_t>((size_t)N * xs_stride(Kmax, 32), (size_t)kChainWarps * gq * (dh + 2));
    l.xs_floats = (int)((xs + 3) & ~(size_t)3);
    l.part_floats = (int)(((size_t)part_cap * kChainR * N + 3) & ~(size_t)3);
    l.bytes = sizeof(float) * (256 + (((size_t)N * (Kmax >> 5) + 3) & ~(size_t)3) + l.part_floats + l.xs_floats);
    return l;
}

}  // namespace river
