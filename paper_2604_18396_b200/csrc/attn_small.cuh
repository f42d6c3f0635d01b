// Paged GQA decode attention for steps of one to four rows (sm_100a).
//
// At these sizes the step is a chain of short dependent kernels and the cache of a row (a few MB) is far below what
// it takes to keep HBM busy, so what matters is the length of the dependency chain, not the copy engine: one
// 512-thread CTA per (row, KV head, split of the positions), a warp takes four consecutive positions of one page at a
// time (a lane owns DH / 32 head dims), base-2 online softmax per query head in fp32, the warps merge through shared
// memory and the splits through a ticket (the last CTA of a (row, KV head) to arrive merges them in split order).
// In a decode step every row belongs to a different sequence, so the QKV kernel still in flight writes nothing but
// each row's newest position: all other cached positions of the warp's first batch are requested BEFORE
// griddepcontrol.wait, and after it only q and the newest position remain to be fetched.
#pragma once
#include "river_common.cuh"

namespace river {

constexpr int kSmallAttnThreads = 512;
constexpr int kSmallAttnWarps = kSmallAttnThreads / 32;

struct SmallAttnArgs {
    const StepMeta *meta;  // n_rows; pad[0] = positions per split (whole pages), pad[1] = splits per (row, KV head)
    int Hq, Hkv;
    float qscale;          // log2(e) / sqrt(dh)
    const float *qbuf;     // [row][Hq][dh]
    float *obuf;           // [row][Hq][dh]
    KvAddr kv;
    float *part_o;            // [row][Hq][splits][dh]
    float2 *part_ml;          // [row][Hq][splits]
    unsigned *attn_tickets;   // [row][Hkv], zero between launches
    int *dev_err;
    const uint8_t *skip;      // rows whose flag is set do not attend (they have left and run nothing here), or null
    const uint8_t *pos_depth; // KV Mask: [slot][depth_stride] backbone blocks the token at each position ran, or null
    int depth_stride, layer1; // ... a position is visible in block layer1 if that number is >= layer1 (or it is the row's own)
};

__device__ __forceinline__ float small_ex2(float x) {
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

// The cached positions of this warp's first batch of the CTA's first work item, requested BEFORE the grid dependency
// on the QKV kernel resolves: everything but the position written in this very step is already in the cache.
struct AttnPre {
    uint2 k[4], v[4];
    unsigned mask;  // bit u: position u of the batch is in k[u], v[u]
};
template <int DH>
__device__ __forceinline__ void small_attn_preload(const SmallAttnArgs &a, const KvAddr &kv, int n_rows, int S, int chunk,
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
    if (page < 0 || page >= kv.n_pages) return;  // the attention proper reports it
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
__device__ __forceinline__ void small_attn_body(const SmallAttnArgs &a, const KvAddr &kv, int n_rows, int S, int chunk,
                                                float *sm, int *s_flag, const AttnPre &pre) {
    constexpr int VE = DH / 32, U = 4, NW = kSmallAttnWarps;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float *s_m = sm, *s_l = sm + NW * GQ, *s_acc = sm + 2 * NW * GQ;  // [NW][GQ], [NW][GQ], [NW][GQ][DH]
    const int items = n_rows * a.Hkv * S;
    const int Hq = a.Hq;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int sp = item % S, kvh = (item / S) % a.Hkv, row = item / (S * a.Hkv);
        if (a.skip && a.skip[row]) continue;
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
            uint32_t dw = 0xffffffffu;  // depth bytes of positions pb .. pb + 3 (pb is a multiple of 4)
            if (a.pos_depth) dw = *reinterpret_cast<const uint32_t *>(a.pos_depth + (size_t)slot * a.depth_stride + pb);
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
                // warp-uniform; KV Mask: a position whose token skipped this block has no entry here (its slot may hold
                // anything) and is not seen - the row's own position always is
                if (pb + u < p1 && (pb + u == pos || (int)((dw >> (8 * u)) & 0xffu) >= a.layer1)) {
#pragma unroll
                    for (int g = 0; g < GQ; ++g) {
                        float s = 0.f;
#pragma unroll
                        for (int e = 0; e < VE; ++e) s = fmaf(qr[g][e], kf[u][e], s);
                        s = warp_sum(s);
                        const float mn = fmaxf(m[g], s);
                        const float corr = small_ex2(m[g] - mn), pr = small_ex2(s - mn);
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
                const float c = (mw == -CUDART_INF_F) ? 0.f : small_ex2(mw - M);
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
                *s_flag = (tk == (unsigned)(S - 1));
                __threadfence();
            }
            __syncthreads();
            if (*s_flag) {
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
                                const float c = (mx == -CUDART_INF_F) ? 0.f : small_ex2(mx - M);
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
// ---------------------------------------------------------------- the kernel: one CTA per (row, KV head, split)
template <int DH, int GQ>
__global__ void __launch_bounds__(kSmallAttnThreads) attn_small_kernel(const SmallAttnArgs a, int layer0, int early) {
    extern __shared__ __align__(16) float attn_small_smem[];
    __shared__ int s_flag;
    pdl_launch();
    KvAddr kv = a.kv;
    kv.layer0 = layer0;
    const int n = a.meta->n_rows, S = a.meta->pad[1], chunk = a.meta->pad[0];
    AttnPre pre;
    pre.mask = 0u;
    // early: every row of the step belongs to a different sequence (a decode step), so the QKV kernel in flight
    // writes nothing but each row's newest position.  Prefill chunks hold consecutive positions of one sequence and
    // must wait.
    if (early) small_attn_preload<DH>(a, kv, n, S, chunk, pre);
    pdl_wait();
    small_attn_body<DH, GQ>(a, kv, n, S, chunk, attn_small_smem, &s_flag, pre);
}

}  // namespace river
