// a3: ragged GQA decode attention over the paged bf16 KV cache (sm_100a).
//
// Work item = (row, kv head, KV split).  A producer warp stages K/V pages of the split in shared memory with TMA
// (2-D tiled copies, 128-byte swizzle, one mbarrier pair per pipeline stage); eight consumer warps each own one half
// page (8 positions) of every 64-position tile and run an independent online softmax over their share: a lane owns one
// position and a quarter of the head dim for q.K (the GQ query heads of the group share every K/V read, and no K or V
// element is unpacked twice), the tile maximum and the probabilities move with warp shuffles, and for P.V a lane owns
// DH/32 head dims.  The eight warp states merge through shared memory (the pipeline stages, free by then) into one
// partial (max, sum, unnormalised output) per (row, head, split); the last split of a (row, kv head) to finish merges
// the splits.  All arithmetic is fp32, exponentials are base 2 (q is pre-scaled by log2 e).
//
// Groups of up to four query heads run the two contractions on the warp-level tensor cores instead (MMA = true; the
// CUDA-core consumers above retire ~1500 warp instructions per 8 KB page and are bound by instruction issue at half the
// HBM rate).  Four consumer warps, one page of every tile each:
//   * S = Q K^T as mma.sync m16n8k16 with the pre-scaled queries as the A operand, held in registers for the whole
//     kernel: row g carries the bf16 head of q_g, row 4 + g its bf16 remainder (q = hi + lo keeps 16 mantissa bits);
//     the K page is the B operand, read from the swizzled stage with ldmatrix exactly as TMA laid it down;
//   * the two partial scores of a head meet with one shuffle; the online softmax runs in the accumulator layout (a lane
//     holds one head row and four positions of the page);
//   * O^T = V^T P^T: the V page is the A operand (ldmatrix.trans of the same swizzled rows), the probabilities are the
//     B operand - again split p = hi + lo into columns g and 4 + g - and the accumulator layout of S is already the
//     fragment layout of that operand, so nothing is exchanged between lanes; O^T keeps DH x 8 fp32 values per warp.
//   Cache rows past the row's position are never multiplied: their scores are replaced, their V fragments zeroed.
#pragma once
#include "mbar_tma.cuh"
#include "mma_sync.cuh"

namespace river {

constexpr int kAttnTile = 64;      // positions per pipeline stage (4 pages)
constexpr int kAttnStages = 2;     // two stages of 32 KB (head dim 128): three CTAs per SM, 24 consumer warps
constexpr int kAttnConsumers = 4;  // pages per tile
constexpr int kAttnWarps = 2 * kAttnConsumers;         // CUDA-core consumer warps: two per page, 8 positions each
__host__ __device__ constexpr int attn_threads(bool mma) { return 32 * ((mma ? kAttnConsumers : kAttnWarps) + 1); }  // consumers + producer
struct AttnArgs {
    const StepMeta *meta;
    const float *q;        // [rows][Hq*DH]
    const int32_t *page_tbl, *row_slot, *row_pos;
    const int32_t *order;  // grid z -> row (longest context first), a permutation of the step's rows
    int n_pages, max_pages_per_seq, Hkv, Hq, layer0;
    float qscale;          // log2(e) / sqrt(DH)
    float *part_o;         // [(row*Hq + head)*splits + split][DH]  unnormalised
    float2 *part_ml;       // same index: (max, sum) in the base-2 domain
    unsigned *tickets;     // [rows][Hkv], zero between launches: the last split of a (row, kv head) merges them all
    float *out;            // [rows][Hq*DH]
    int *dev_err;
    const uint8_t *skip;   // rows whose flag is set do not attend (they have left and run nothing here), or null
    const uint8_t *pos_depth;  // KV Mask: [slot][depth_stride] backbone blocks the token at each position ran, or null
    int depth_stride, layer1;  // ... a position is visible in block layer1 if that number is >= layer1 (or it is the row's own)
    int early;             // 1: every row is a different sequence (a decode step): the kernel still in flight writes nothing
                           // but each row's newest position, so tiles that end before it are requested BEFORE the wait
};

template <int DH, int GQ, bool MMA>
__global__ void __launch_bounds__(attn_threads(MMA)) attn_split_kernel(const __grid_constant__ CUtensorMap tmap,
                                                                       const AttnArgs a) {
    static_assert(!MMA || GQ <= 4, "the tensor-core consumers carry hi and lo parts of four heads in eight columns");
    constexpr int NW = MMA ? kAttnConsumers : kAttnWarps;  // consumer warps
    constexpr int kAttnThreads = attn_threads(MMA);
    constexpr int HP = kPage / 2;                // positions per warp and tile
    constexpr int NB = DH / 64;                  // 128-byte boxes per cache row
    constexpr int PAGE_BYTES = kPage * DH * 2;   // one page of K (or V) of one kv head
    constexpr int STAGE_BYTES = 2 * kAttnConsumers * PAGE_BYTES;
    constexpr int NCH = DH / 32;                 // 16-byte chunks per lane quarter in q.K
    constexpr int VE = DH / 32;                  // head dims per lane in P.V

    const int split = blockIdx.x, kvh = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch();

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *stages = smem;                                            // kAttnStages * STAGE_BYTES, 1024-aligned
    float *sq = reinterpret_cast<float *>(stages + kAttnStages * STAGE_BYTES);  // [GQ][DH]
    float *sp = sq + GQ * DH;                                          // [NW warps][8 positions][GQ]
    float *sm = reinterpret_cast<float *>(stages);                     // merge: [NW][GQ][DH + 2], in the drained stages
    uint64_t *bars = reinterpret_cast<uint64_t *>(sp + NW * HP * GQ);  // full[S], empty[S]
    __shared__ int s_abort;
    __shared__ bool s_last;
    const bool is_producer = tid == NW * 32;
    if (is_producer) {  // nothing here depends on the previous kernel
        s_abort = 0;
        for (int s = 0; s < kAttnStages; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);
            mbar_init(smem_u32(&bars[kAttnStages + s]), NW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (!a.early) pdl_wait();
    // (the step metadata and the page table are the host's: complete before the step's first kernel)
    // independent loads first, decisions after (every index below is valid for any row of the grid)
    const int n_rows = a.meta->n_rows, chunk = a.meta->attn_chunk, n_splits = a.meta->attn_splits;
    const int row = a.order[blockIdx.z];  // (entries past the step's rows hold 0 or an earlier step's row id)
    const int pos = a.row_pos[row], slot = a.row_slot[row];
    if ((int)blockIdx.z >= n_rows || (a.skip && a.skip[row])) return;
    const int p0 = split * chunk;
    if (p0 > pos) return;
    const int p1 = min(p0 + chunk, pos + 1);     // positions [p0, p1)
    const int n_tiles = (p1 - p0 + kAttnTile - 1) / kAttnTile;
    volatile int *abortp = &s_abort;

    // The producer WARP issues the TMA copies of a tile, at most kAttnStages tiles ahead - one copy per lane (a tile is
    // 2 NB copies per page: a single lane, retiring an instruction every few tens of cycles, would take about as long
    // to issue them as the tile takes to arrive); the first tiles go out before anything else.  Called by all lanes.
    static_assert(kAttnConsumers * 2 * NB <= 32, "one copy per producer lane");
    auto issue_tile = [&](int t) {
        const int s = t % kAttnStages;
        if (t >= kAttnStages) {
            int ok = 1;
            if (lane == 0)
                ok = mbar_wait(smem_u32(&bars[kAttnStages + s]), ((t / kAttnStages) - 1) & 1, abortp, a.dev_err) ? 1 : 0;
            if (!__shfl_sync(0xffffffffu, ok, 0)) return false;
        }
        const int first_page = (p0 + t * kAttnTile) / kPage;
        const int n_valid = min(kAttnConsumers, (p1 - 1) / kPage - first_page + 1);
        const uint32_t full = smem_u32(&bars[s]);
        if (lane == 0) mbar_expect_tx(full, (uint32_t)(n_valid * 2 * PAGE_BYTES));
        __syncwarp();
        if (lane < n_valid * 2 * NB) {
            const int j = lane / (2 * NB), kv = (lane / NB) & 1, b = lane % NB;  // page of the tile, K or V, 128-byte box
            int page = a.page_tbl[(size_t)slot * a.max_pages_per_seq + first_page + j];
            if (page < 0 || page >= a.n_pages) { atomicExch(a.dev_err, DEV_BAD_PAGE); page = 0; }
            // cache rows of (layer, page, K|V, kv head): 16 consecutive rows of the [rows][DH] view
            const int y = ((((a.layer0 * a.n_pages + page) * 2 + kv) * a.Hkv) + kvh) * kPage;
            const uint32_t dst = smem_u32(stages + s * STAGE_BYTES + (kv * kAttnConsumers + j) * PAGE_BYTES) + b * (kPage * 128);
            tma_load_2d(dst, &tmap, b * 64, y, full);
        }
        return true;
    };
    if (warp == NW) {
        __syncwarp();  // the barriers lane 0 initialised
        for (int t = 0; t < min(n_tiles, kAttnStages); ++t)
            if (!a.early || p0 + (t + 1) * kAttnTile <= pos) issue_tile(t);  // (early: only tiles the row's new position is not in)
    }
    if (a.early) {
        pdl_wait();
        if (warp == NW)
            for (int t = 0; t < min(n_tiles, kAttnStages); ++t)
                if (p0 + (t + 1) * kAttnTile > pos) issue_tile(t);
    }
    if constexpr (!MMA) {
        for (int i = tid; i < GQ * DH; i += kAttnThreads)
            sq[i] = a.q[(size_t)row * a.Hq * DH + (size_t)kvh * GQ * DH + i] * a.qscale;
    }
    __syncthreads();

    if constexpr (MMA) {
        // ---------------- tensor-core consumers: warp w owns page w of every tile
        constexpr int KS = DH / 16;  // k-steps of S = Q K^T, and 16-dim row tiles of O^T
        const int t4 = lane & 3, r8 = lane >> 2;
        const int g = r8 & 3;
        const bool lo_row = r8 >= 4;
        uint32_t qa[KS][2];  // A fragments of Q: rows 0-3 hi parts, rows 4-7 remainders, rows 8-15 zero
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            float2 x0 = make_float2(0.f, 0.f), x1 = x0;
            if (g < GQ && warp < NW) {
                const float *qp = a.q + (size_t)row * a.Hq * DH + (size_t)(kvh * GQ + g) * DH + ks * 16 + 2 * t4;
                x0 = *reinterpret_cast<const float2 *>(qp);
                x1 = *reinterpret_cast<const float2 *>(qp + 8);
            }
            x0.x *= a.qscale; x0.y *= a.qscale; x1.x *= a.qscale; x1.y *= a.qscale;
            const uint32_t h0 = pack_bf16x2(x0.x, x0.y), h1 = pack_bf16x2(x1.x, x1.y);
            qa[ks][0] = lo_row ? pack_bf16x2(x0.x - bf16lo(h0), x0.y - bf16hi(h0)) : h0;
            qa[ks][1] = lo_row ? pack_bf16x2(x1.x - bf16lo(h1), x1.y - bf16hi(h1)) : h1;
        }
        float m = -CUDART_INF_F, l = 0.f;  // head g's state (held twice: by the lanes of row g and of row 4 + g)
        float acc[KS][4];                  // O^T: dims 16 mt + r8 (+ 8), columns 2 t4, 2 t4 + 1
#pragma unroll
        for (int mt = 0; mt < KS; ++mt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][e] = 0.f;
        if (warp == NW) {
            for (int t = kAttnStages; t < n_tiles; ++t)
                if (!issue_tile(t)) break;
        } else {
            // ldmatrix row of this lane: matrix lane / 8 -> positions 8 (lane / 16) .., 16-byte chunk parity (lane / 8) & 1
            const int lpos = (lane & 7) + 8 * (lane >> 4), lodd = (lane >> 3) & 1;
            for (int t = 0; t < n_tiles; ++t) {
                const int s = t % kAttnStages;
                if (!mbar_wait(smem_u32(&bars[s]), (t / kAttnStages) & 1, abortp, a.dev_err)) break;
                const int pos0 = p0 + t * kAttnTile + warp * kPage;  // first position of this warp's page
                // positions of this page that take part: inside the split, and (KV Mask) with an entry in this block
                uint32_t seen = 0u;
                if (pos0 < p1) {
                    seen = (1u << min(kPage, p1 - pos0)) - 1u;
                    if (a.pos_depth) {
                        const uint4 dv = *reinterpret_cast<const uint4 *>(a.pos_depth + (size_t)slot * a.depth_stride + pos0);
                        const uint32_t dw[4] = {dv.x, dv.y, dv.z, dv.w};
                        uint32_t ok = 0u;
#pragma unroll
                        for (int i = 0; i < kPage; ++i)
                            if ((int)((dw[i >> 2] >> (8 * (i & 3))) & 0xffu) >= a.layer1 || pos0 + i == pos) ok |= 1u << i;
                        seen &= ok;
                    }
                }
                if (seen) {
                    const uint32_t kpg = smem_u32(stages + s * STAGE_BYTES + warp * PAGE_BYTES);
                    const uint32_t vpg = kpg + kAttnConsumers * PAGE_BYTES;
                    float sc[2][4];  // S: row r8, positions 8 j + 2 t4 (+ 1) in [j][0..1]; rows 8-15 (unused) in [j][2..3]
#pragma unroll
                    for (int j = 0; j < 2; ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) sc[j][e] = 0.f;
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int cg = 2 * ks + lodd, box = cg >> 3, c = cg & 7;
                        uint32_t kf[4];
                        ldsm_x4(kf, kpg + box * (kPage * 128) + lpos * 128 + ((c ^ (lpos & 7)) << 4));
                        const uint32_t af[4] = {qa[ks][0], 0u, qa[ks][1], 0u};
                        mma_bf16_m16n8k16(sc[0], af, kf[0], kf[1]);
                        mma_bf16_m16n8k16(sc[1], af, kf[2], kf[3]);
                    }
                    float p[2][2], mx = -CUDART_INF_F;
#pragma unroll
                    for (int j = 0; j < 2; ++j)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            float v = sc[j][e] + __shfl_xor_sync(0xffffffffu, sc[j][e], 16);  // hi row + remainder row
                            v = ((seen >> (8 * j + 2 * t4 + e)) & 1u) ? v : -CUDART_INF_F;  // select: other rows may hold anything
                            p[j][e] = v;
                            mx = fmaxf(mx, v);
                        }
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float mn = fmaxf(m, mx);  // finite: at least one position of the page takes part
                    const float corr = ex2(m - mn);
                    m = mn;
                    float psum = 0.f;
                    uint32_t pb[2];
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const float e0 = ex2(p[j][0] - mn), e1 = ex2(p[j][1] - mn);  // masked positions: exactly 0
                        psum += e0 + e1;
                        const uint32_t h = pack_bf16x2(e0, e1);
                        pb[j] = lo_row ? pack_bf16x2(e0 - bf16lo(h), e1 - bf16hi(h)) : h;
                    }
                    l = fmaf(l, corr, psum);
                    // the accumulator columns 2 t4, 2 t4 + 1 belong to heads (2 t4) & 3 and (2 t4 + 1) & 3
                    const float c0 = __shfl_sync(0xffffffffu, corr, ((2 * t4) & 3) * 4);
                    const float c1 = __shfl_sync(0xffffffffu, corr, ((2 * t4 + 1) & 3) * 4);
                    const bool cut = seen != 0xffffu;
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        const int cg = 2 * mt + lodd, box = cg >> 3, c = cg & 7;
                        uint32_t vf[4];
                        ldsm_x4_trans(vf, vpg + box * (kPage * 128) + lpos * 128 + ((c ^ (lpos & 7)) << 4));
                        if (cut) {  // vf[0..1]: positions 2 t4, 2 t4 + 1; vf[2..3]: positions 8 + 2 t4, 9 + 2 t4
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int pp = 2 * t4 + 8 * (q >> 1);
                                if (!((seen >> pp) & 1u)) vf[q] &= 0xffff0000u;
                                if (!((seen >> (pp + 1)) & 1u)) vf[q] &= 0x0000ffffu;
                            }
                        }
                        acc[mt][0] *= c0; acc[mt][1] *= c1; acc[mt][2] *= c0; acc[mt][3] *= c1;
                        mma_bf16_m16n8k16(acc[mt], vf, pb[0], pb[1]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars[kAttnStages + s]));
            }
        }
        __syncthreads();
        if (warp < NW && !s_abort) {
            // column 4 + g holds the remainder part of head g: add it to column g, then lanes t4 < 2 own heads 2 t4, 2 t4 + 1
#pragma unroll
            for (int mt = 0; mt < KS; ++mt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[mt][e] += __shfl_xor_sync(0xffffffffu, acc[mt][e], 2);
            if (t4 < 2) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int hg = 2 * t4 + e;
                    if (hg < GQ) {
                        float *dst = sm + (warp * GQ + hg) * (DH + 2);
#pragma unroll
                        for (int mt = 0; mt < KS; ++mt) {
                            dst[mt * 16 + r8] = acc[mt][e];
                            dst[mt * 16 + r8 + 8] = acc[mt][2 + e];
                        }
                    }
                }
            }
            float lsum = l + __shfl_xor_sync(0xffffffffu, l, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            if (t4 == 0 && r8 < GQ) {
                float *dst = sm + (warp * GQ + r8) * (DH + 2);
                dst[DH] = m;
                dst[DH + 1] = lsum;
            }
        }
        __syncthreads();
    } else {
        // ---------------- consumers: warp w owns positions [8 (w / 4), + 8) of page w % 4 of every tile
        const int r8 = lane & 7, qtr = lane >> 3;
        const int pg = warp & (kAttnConsumers - 1), ph = warp / kAttnConsumers;
        const int r = ph * HP + r8;  // this lane's position inside the page
        float m[GQ], l[GQ], acc[GQ][VE];
    #pragma unroll
        for (int g = 0; g < GQ; ++g) {
            m[g] = -CUDART_INF_F;
            l[g] = 0.f;
    #pragma unroll
            for (int e = 0; e < VE; ++e) acc[g][e] = 0.f;
        }
        if (warp == NW) {
            for (int t = kAttnStages; t < n_tiles; ++t)
                if (!issue_tile(t)) break;
        } else {
            float *my_sp = sp + warp * HP * GQ;
            for (int t = 0; t < n_tiles; ++t) {
                const int s = t % kAttnStages;
                if (!mbar_wait(smem_u32(&bars[s]), (t / kAttnStages) & 1, abortp, a.dev_err)) break;
                const int pos0 = p0 + t * kAttnTile + pg * kPage + ph * HP;  // first position of this warp's half page
                if (pos0 < p1) {
                    const uint8_t *kpg = stages + s * STAGE_BYTES + pg * PAGE_BYTES;
                    const uint8_t *vpg = kpg + kAttnConsumers * PAGE_BYTES;
                    // q.K for position r, dims [qtr*DH/4, (qtr+1)*DH/4)
                    float sc[GQ];
    #pragma unroll
                    for (int g = 0; g < GQ; ++g) sc[g] = 0.f;
    #pragma unroll
                    for (int i = 0; i < NCH; ++i) {
                        const int cg = qtr * NCH + i, box = cg >> 3, c = cg & 7;
                        const uint4 kw = *reinterpret_cast<const uint4 *>(kpg + box * (kPage * 128) + r * 128 +
                                                                         ((c ^ (r & 7)) << 4));
                        const float k0 = bf16lo(kw.x), k1 = bf16hi(kw.x), k2 = bf16lo(kw.y), k3 = bf16hi(kw.y);
                        const float k4 = bf16lo(kw.z), k5 = bf16hi(kw.z), k6 = bf16lo(kw.w), k7 = bf16hi(kw.w);
    #pragma unroll
                        for (int g = 0; g < GQ; ++g) {
                            const float4 qa = *reinterpret_cast<const float4 *>(sq + g * DH + cg * 8);
                            const float4 qb = *reinterpret_cast<const float4 *>(sq + g * DH + cg * 8 + 4);
                            float v = sc[g];
                            v = fmaf(qa.x, k0, v); v = fmaf(qa.y, k1, v); v = fmaf(qa.z, k2, v); v = fmaf(qa.w, k3, v);
                            v = fmaf(qb.x, k4, v); v = fmaf(qb.y, k5, v); v = fmaf(qb.z, k6, v); v = fmaf(qb.w, k7, v);
                            sc[g] = v;
                        }
                    }
                    const bool live = pos0 + r8 < p1;
                    float corr[GQ];
    #pragma unroll
                    for (int g = 0; g < GQ; ++g) {
                        float v = sc[g] + __shfl_xor_sync(0xffffffffu, sc[g], 8);
                        v += __shfl_xor_sync(0xffffffffu, v, 16);
                        v = live ? v : -CUDART_INF_F;  // select, never arithmetic: stale cache rows may hold anything
                        float mx = v;
    #pragma unroll
                        for (int o = 4; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                        const float mn = fmaxf(m[g], mx);  // finite: position pos0 is live
                        corr[g] = ex2(m[g] - mn);
                        m[g] = mn;
                        const float p = live ? ex2(v - mn) : 0.f;
                        if (qtr == 0) my_sp[r8 * GQ + g] = p;
                        l[g] = fmaf(l[g], corr[g], qtr == 0 ? p : 0.f);  // this lane's share of the sum; added up at the end
    #pragma unroll
                        for (int e = 0; e < VE; ++e) acc[g][e] *= corr[g];
                    }
                    __syncwarp();
                    // P.V: lane owns dims [lane*VE, lane*VE + VE)
                    const int n_live = min(HP, p1 - pos0);
                    const int vbyte = lane * VE * 2, vbox = vbyte >> 7, vc = (vbyte & 127) >> 4, vo = vbyte & 15;
                    for (int j = 0; j < n_live; ++j) {
                        const int vr = ph * HP + j;
                        const uint8_t *vp = vpg + vbox * (kPage * 128) + vr * 128 + ((vc ^ (vr & 7)) << 4) + vo;
                        float vf[VE];
                        if (VE == 4) {
                            const uint2 w = *reinterpret_cast<const uint2 *>(vp);
                            vf[0] = bf16lo(w.x); vf[1] = bf16hi(w.x); vf[2 % VE] = bf16lo(w.y); vf[3 % VE] = bf16hi(w.y);
                        } else {
                            const uint32_t w = *reinterpret_cast<const uint32_t *>(vp);
                            vf[0] = bf16lo(w); vf[1] = bf16hi(w);
                        }
    #pragma unroll
                        for (int g = 0; g < GQ; ++g) {
                            const float p = my_sp[j * GQ + g];
    #pragma unroll
                            for (int e = 0; e < VE; ++e) acc[g][e] = fmaf(p, vf[e], acc[g][e]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars[kAttnStages + s]));
            }
        }
        // every tile that was requested has landed and has been read by every consumer warp (unless the CTA gave up): the
        // stages may now hold the warp states
        __syncthreads();
        if (warp < NW && !s_abort) {
    #pragma unroll
            for (int g = 0; g < GQ; ++g) {
                float *dst = sm + (warp * GQ + g) * (DH + 2);
    #pragma unroll
                for (int e = 0; e < VE; ++e) dst[lane * VE + e] = acc[g][e];
                const float lsum = warp_sum(l[g]);
                if (lane == 0) { dst[DH] = m[g]; dst[DH + 1] = lsum; }
            }
        }
        __syncthreads();
    }
    if (s_abort) {
        // give copies that are still in flight time to land before the CTA's shared memory is handed on
        for (int i = 0; i < 2000; ++i) __nanosleep(100);
        return;
    }
    // merge the warp states -> one result per head for this split
    const int ns = pos / chunk + 1;  // splits of this row
    for (int t = tid; t < GQ * DH; t += kAttnThreads) {
        const int g = t / DH, e = t % DH;
        float M = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < NW; ++w) M = fmaxf(M, sm[(w * GQ + g) * (DH + 2) + DH]);
        float num = 0.f, den = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float *src = sm + (w * GQ + g) * (DH + 2);
            const float c = (src[DH] == -CUDART_INF_F) ? 0.f : ex2(src[DH] - M);
            num = fmaf(c, src[e], num);
            den = fmaf(c, src[DH + 1], den);
        }
        if (ns == 1) {  // the only split of the row: this is the attention output
            a.out[((size_t)row * a.Hq + kvh * GQ + g) * DH + e] = num / den;
        } else {
            const size_t idx = ((size_t)row * a.Hq + kvh * GQ + g) * n_splits + split;
            a.part_o[idx * DH + e] = num;
            if (e == 0) a.part_ml[idx] = make_float2(M, den);
        }
    }
    if (ns == 1) return;
    // the last split of this (row, kv head) to finish merges all of them:
    // out = sum_s 2^(m_s - M) o_s / sum_s 2^(m_s - M) l_s  (atomic ticket, no spinning)
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(&a.tickets[row * a.Hkv + kvh], 1u) == (unsigned)(ns - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    float *wgt = sm;  // [GQ][ns] weights 2^(m_s - M) / sum, reusing the merge buffer (ns <= 64)
    const size_t base0 = ((size_t)row * a.Hq + kvh * GQ) * n_splits;
    for (int t = tid; t < GQ * ns; t += kAttnThreads) {
        const int g = t / ns, sidx = t % ns;
        const float2 ml = __ldcg(&a.part_ml[base0 + (size_t)g * n_splits + sidx]);
        wgt[g * 64 + sidx] = ml.x;
        wgt[GQ * 64 + g * 64 + sidx] = ml.y;
    }
    __syncthreads();
    if (tid < GQ) {
        float M = -CUDART_INF_F;
        for (int sidx = 0; sidx < ns; ++sidx) M = fmaxf(M, wgt[tid * 64 + sidx]);
        float den = 0.f;
        for (int sidx = 0; sidx < ns; ++sidx) {
            const float c = ex2(wgt[tid * 64 + sidx] - M);
            den = fmaf(c, wgt[GQ * 64 + tid * 64 + sidx], den);
            wgt[tid * 64 + sidx] = c;
        }
        const float inv = 1.f / den;
        for (int sidx = 0; sidx < ns; ++sidx) wgt[tid * 64 + sidx] *= inv;
    }
    __syncthreads();
    for (int t = tid; t < GQ * DH; t += kAttnThreads) {
        const int g = t / DH, e = t % DH;
        const float *po = a.part_o + (base0 + (size_t)g * n_splits) * DH + e;
        float num = 0.f;
#pragma unroll 8
        for (int sidx = 0; sidx < ns; ++sidx) num = fmaf(wgt[g * 64 + sidx], __ldcg(po + (size_t)sidx * DH), num);
        a.out[((size_t)row * a.Hq + kvh * GQ + g) * DH + e] = num;
    }
    if (tid == 0) a.tickets[row * a.Hkv + kvh] = 0;
}

inline size_t attn_smem_bytes(int DH, int GQ) {  // (both consumer kinds: the tensor-core one leaves sq / sp unused)
    const size_t stage = 2 * kAttnConsumers * (size_t)(kPage * DH * 2);  // the warp states reuse the stages
    return 1024 + kAttnStages * stage + sizeof(float) * ((size_t)GQ * DH + (size_t)kAttnWarps * (kPage / 2) * GQ) +
           2 * kAttnStages * sizeof(uint64_t) + 64;
}

}  // namespace river
