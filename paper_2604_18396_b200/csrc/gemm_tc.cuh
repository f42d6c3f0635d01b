// Batched backbone projections on the 5th-generation tensor cores (sm_100a): tcgen05.mma with TMEM accumulators.
//
// With more than a handful of activation rows the CUDA-core stream kernel becomes issue-bound, while the projection
// is still a weight stream: D[128 output features x N rows] = W[128 x K] . X^T[K x N] ("swap-AB": the weights are the
// M = 128 operand, the rows of the step the N operand, 16 <= N <= 256).  One CTA owns one 128-feature tile and one
// K-split of it.  A producer lane brings 128 x 64 weight tiles and N x 64 activation tiles into shared memory with
// 2-D TMA copies (128-byte swizzle, K-major: the canonical UMMA layout); one lane issues tcgen05.mma (kind::f16,
// bf16 x bf16 -> fp32) against the activations' bf16 high part and again against their low part (x = hi + lo, so the
// activations keep 16 mantissa bits although the tensor cores take bf16); tcgen05.commit releases the stage.  Four
// epilogue warps read the accumulator out of TMEM (tcgen05.ld) and park it in shared memory.  The K-splits of one
// tile form a thread-block cluster: after a cluster barrier every split CTA adds, in split order, its own slice of
// the tile's rows from all peers' shared memory (distributed shared memory: a reduce-scatter with no trip through
// HBM, no atomics, a fixed summation order) and runs the projection's epilogue on that slice (RoPE + KV-cache
// write, residual add, SwiGLU, logits + argmax partials).
// Weights do not depend on the previous kernel: their first tiles are requested before the grid dependency resolves.
#pragma once
#include <cuda_fp16.h>
#include "mbar_tma.cuh"

namespace river {

constexpr int kTcBM = 128;      // output features per tile (UMMA M)
constexpr int kTcBK = 64;       // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kTcThreads = 192; // warp 0: TMA, warp 1: MMA + TMEM allocation, warps 2..5: epilogue

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// K-major operand tile in shared memory, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t tc_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTcBM >> 4) << 24);
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// ---------------------------------------------------------------- activation rows -> bf16 hi / lo operand buffers
// CTA (i, j) writes inputs [1024 j, 1024 j + 1024) of operand row i < n_pad: the i-th row of the backbone list (zero
// beyond the list), optionally RMS-normalised (every CTA of a row sums the whole row's squares itself: the row is a
// few KB in L2), split as x = hi + lo with hi = bf16(x), lo = bf16(x - hi).  One 128-bit load per thread.
constexpr int kPrepChunk = 1024;
__device__ __forceinline__ float tc_prep_scale(const ProjIn &in, const float4 *src, int K, float *red) {
    if (!in.gain) return 1.f;
    float ss = 0.f;
    const int nv = K >> 2;
    for (int v0 = 0; v0 < nv; v0 += 4 * 256) {
        float4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int v = v0 + u * 256 + threadIdx.x;
            x[u] = v < nv ? __ldcg(src + v) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) ss += x[u].x * x[u].x + x[u].y * x[u].y + x[u].z * x[u].z + x[u].w * x[u].w;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    ss = 0.f;
    for (int w = 0; w < 8; ++w) ss += red[w];
    return rsqrtf(ss / (float)K + in.eps);
}
// (the body of CTA (i, by); `red`: eight floats of shared memory)
__device__ __forceinline__ void tc_prep_body(const ProjIn &in, const int32_t *idx, const int32_t *cnt, int K,
                                             __nv_bfloat16 *xhi, __nv_bfloat16 *xlo, int i, int by, float *red) {
    const int n = *cnt;
    if (n <= 0) return;  // no row in the backbone any more: the GEMM returns before it reads an operand
    const int v = by * (kPrepChunk / 4) + threadIdx.x;  // 4-input group of the row
    const bool mine = v < (K >> 2);
    uint2 *hi = reinterpret_cast<uint2 *>(xhi + (size_t)i * K), *lo = reinterpret_cast<uint2 *>(xlo + (size_t)i * K);
    if (i >= n) {
        if (mine) { hi[v] = make_uint2(0u, 0u); lo[v] = make_uint2(0u, 0u); }
        return;
    }
    const float4 *src = reinterpret_cast<const float4 *>(in.src + (size_t)idx[i] * K);
    float4 y = mine ? __ldcg(src + v) : make_float4(0.f, 0.f, 0.f, 0.f);
    uint2 gw = make_uint2(0u, 0u);
    if (in.gain && mine) gw = *reinterpret_cast<const uint2 *>(in.gain + 4 * v);
    const float scale = tc_prep_scale(in, src, K, red);
    if (!mine) return;
    if (in.gain) {
        y.x = y.x * scale * bf16lo(gw.x); y.y = y.y * scale * bf16hi(gw.x);
        y.z = y.z * scale * bf16lo(gw.y); y.w = y.w * scale * bf16hi(gw.y);
    }
    auto split2 = [](float a, float b, uint32_t &h, uint32_t &l) {
        const __nv_bfloat16 ha = __float2bfloat16_rn(a), hb = __float2bfloat16_rn(b);
        const __nv_bfloat16 la = __float2bfloat16_rn(a - __bfloat162float(ha)), lb = __float2bfloat16_rn(b - __bfloat162float(hb));
        h = (uint32_t)__bfloat16_as_ushort(ha) | ((uint32_t)__bfloat16_as_ushort(hb) << 16);
        l = (uint32_t)__bfloat16_as_ushort(la) | ((uint32_t)__bfloat16_as_ushort(lb) << 16);
    };
    uint2 h, l;
    split2(y.x, y.y, h.x, l.x);
    split2(y.z, y.w, h.y, l.y);
    hi[v] = h;
    lo[v] = l;
}
static __global__ void __launch_bounds__(256) tc_prep_kernel(const ProjIn in, const int32_t *idx, const int32_t *cnt, int K,
                                                      __nv_bfloat16 *xhi, __nv_bfloat16 *xlo) {
    __shared__ float red[8];
    pdl_launch();
    pdl_wait();
    tc_prep_body(in, idx, cnt, K, xhi, xlo, blockIdx.x, blockIdx.y, red);
}

// ---------------------------------------------------------------- epilogues on a finished 128 x N tile in smem
// tile(r, n) = sum over K of W[row0 + r] . x[n], stored column by column: tile[n * ld + r] (consecutive threads take
// consecutive features r: no bank conflicts, coalesced global writes); `rows` maps n to the step's row id; only
// n < n_live are real.  The 128 tile rows are handled as 64 pairs in 16 quads of four pairs; an epilogue call covers
// the pairs [pr0, pr1) (a K-split CTA finishes its own slice of the tile: whole quads), and quad_row(i, q0, nq) names
// the first of four consecutive tile rows behind item i of the 2 nq four-row runs that make up the quads [q0, q0 + nq).
constexpr int kTcLd = kTcBM + 4;  // column stride of the tile in floats (16-byte aligned columns)
struct TcResidEpi {  // out[row][row0 + r] = resid[row][row0 + r] + tile(r, n)
    const float *resid;
    float *out;
    int out_dim;
    __device__ int quad_row(int i, int q0, int) const { return 8 * q0 + 4 * i; }  // pairs (2 pr, 2 pr + 1): one range
    // Four consecutive features per access; the residual values of a batch are all requested before the first sum is
    // stored (`out` and `resid` never overlap, but the compiler cannot know: left alone it waits for every load).
    __device__ void run(const float *tile, int ld, int tile_idx, int n_live, const int32_t *rows, int tid, int nthr,
                        int pr0, int pr1, int = 0) const {
        constexpr int UB = 4;
        const int row0 = tile_idx * kTcBM, nr4 = (pr1 - pr0) / 2, total = n_live * nr4;  // slices are whole quads of pairs
        for (int t0 = tid; t0 < total; t0 += UB * nthr) {
            float4 res[UB];
            size_t o[UB];
            int src[UB];
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int t = t0 + u * nthr;
                res[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                o[u] = 0; src[u] = -1;
                if (t < total) {
                    const int n = t / nr4, r = 2 * pr0 + 4 * (t % nr4);
                    o[u] = (size_t)rows[n] * out_dim + row0 + r;
                    src[u] = n * ld + r;
                    res[u] = __ldcg(reinterpret_cast<const float4 *>(resid + o[u]));
                }
            }
#pragma unroll
            for (int u = 0; u < UB; ++u)
                if (src[u] >= 0) {
                    const float4 x = *reinterpret_cast<const float4 *>(tile + src[u]);
                    *reinterpret_cast<float4 *>(out + o[u]) =
                        make_float4(res[u].x + x.x, res[u].y + x.y, res[u].z + x.z, res[u].w + x.w);
                }
        }
    }
};
struct TcGateUpEpi {  // tile rows 0..63: gate features f0.., rows 64..127: up features f0..
    float *act;
    int F;
    // optional: the down projection's operand rows, so that it needs no operand kernel: row n of the list, split
    // v = hi + lo exactly as tc_prep_kernel (omode 1: bf16) or tc_prep_w4_kernel (omode 2: f16, the inputs of every
    // group of eight in the order (0,4,1,5,2,6,3,7)) would split act[rows[n]]
    uint16_t *ohi = nullptr, *olo = nullptr;
    int omode = 0;
    __device__ int quad_row(int i, int q0, int nq) const { return i < nq ? 4 * (q0 + i) : 64 + 4 * (q0 + i - nq); }
    __device__ void run(const float *tile, int ld, int tile_idx, int n_live, const int32_t *rows, int tid, int nthr,
                        int pr0, int pr1, int = 0) const {
        const int f0 = tile_idx * 64, np = pr1 - pr0;
        for (int t = tid; t < n_live * np; t += nthr) {
            const int n = t / np, r = pr0 + t % np;
            const float g = tile[n * ld + r], u = tile[n * ld + 64 + r];
            const float v = g / (1.f + __expf(-g)) * u;
            act[(size_t)rows[n] * F + f0 + r] = v;
            if (omode == 1) {
                const __nv_bfloat16 h = __float2bfloat16_rn(v);
                const size_t o = (size_t)n * F + f0 + r;
                ohi[o] = __bfloat16_as_ushort(h);
                olo[o] = __bfloat16_as_ushort(__float2bfloat16_rn(v - __bfloat162float(h)));
            } else if (omode == 2) {
                const __half h = __float2half_rn(v);
                const int f = f0 + r, j = f & 7;
                const size_t o = (size_t)n * F + (f & ~7) + (j < 4 ? 2 * j : 2 * (j - 4) + 1);
                ohi[o] = __half_as_ushort(h);
                olo[o] = __half_as_ushort(__float2half_rn(v - __half2float(h)));
            }
        }
    }
};
struct TcQkvEpi {  // tiles walk the concatenated [q heads | k heads | v heads] features, 128 at a time
    int Hq, Hkv, dh;
    const float2 *rope_cs;
    float *q_out;
    KvAddr kv;
    int *dev_err;
    __device__ int quad_row(int i, int q0, int nq) const {  // pair pr = rows (head * dh + j, head * dh + j + dh / 2)
        const int half = dh >> 1, pr = 4 * (q0 + (i < nq ? i : i - nq));
        return (pr / half) * dh + pr % half + (i < nq ? 0 : half);
    }
    __device__ void run(const float *tile, int ld, int tile_idx, int n_live, const int32_t *rows, int tid, int nthr,
                        int pr0, int pr1, int = 0) const {
        const int half = dh >> 1, heads_per_tile = kTcBM / dh;
        const int feat0 = tile_idx * kTcBM;
        const int qdim = Hq * dh, kvdim = Hkv * dh;
        const int which = feat0 < qdim ? 0 : (feat0 < qdim + kvdim ? 1 : 2);
        const int base = which == 0 ? feat0 : (which == 1 ? feat0 - qdim : feat0 - qdim - kvdim);  // inside its matrix
        const int np = pr1 - pr0, total = n_live * np;
        // batches of four (row, pair) items: everything an item reads from global memory (its rotation, its cache slot)
        // is requested for the whole batch before the first result is stored
        constexpr int UB = 4;
        for (int t0 = tid; t0 < total; t0 += UB * nthr) {
            int row[UB], src[UB], ii[UB], hl[UB], pos[UB], page[UB];
            float2 cs[UB];
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int t = t0 + u * nthr;
                src[u] = -1; row[u] = 0; ii[u] = 0; hl[u] = 0; pos[u] = 0; page[u] = 0;
                cs[u] = make_float2(1.f, 0.f);
                if (t >= total) continue;
                const int n = t / np, pr = pr0 + t % np;
                const int hh = pr / half, i = pr % half;  // head inside the tile, pair index
                if (hh >= heads_per_tile) continue;
                row[u] = rows[n];
                src[u] = n * ld + hh * dh + i;
                ii[u] = i;
                hl[u] = (base + hh * dh) / dh;
                if (which != 2) cs[u] = rope_cs[(size_t)row[u] * half + i];
                if (which != 0) { pos[u] = kv.row_pos[row[u]]; page[u] = kv.row_page[row[u]]; }
            }
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                if (src[u] < 0) continue;
                float lo = tile[src[u]], hi = tile[src[u] + half];
                if (which != 2) {
                    const float a = lo * cs[u].x - hi * cs[u].y, b = hi * cs[u].x + lo * cs[u].y;
                    lo = a; hi = b;
                }
                if (which == 0) {
                    float *q = q_out + (size_t)row[u] * qdim + (size_t)hl[u] * dh;
                    q[ii[u]] = lo;
                    q[ii[u] + half] = hi;
                } else {
                    if (page[u] < 0 || page[u] >= kv.n_pages) { atomicExch(dev_err, DEV_BAD_PAGE); continue; }
                    const size_t o = kv.base(page[u], which - 1, hl[u], pos[u] % kPage);
                    kv.pool[o + ii[u]] = __float2bfloat16_rn(lo);
                    kv.pool[o + ii[u] + half] = __float2bfloat16_rn(hi);
                }
            }
        }
    }
};
struct TcHeadEpi {  // logits (optional) and the tile's (max, lowest id) per row for the greedy token
    const StepMeta *meta;
    int V;
    float *part_val;
    int32_t *part_idx;
    int n_parts;
    __device__ int quad_row(int i, int q0, int) const { return 8 * q0 + 4 * i; }
    // (the LM head is never K-split: the argmax partial below needs all 128 rows of the tile)
    // n0: operand row behind column 0 of `tile` (a tile may be handed over in column chunks)
    __device__ void run(const float *tile, int ld, int tile_idx, int n_live, const int32_t *, int tid, int nthr, int,
                        int, int n0 = 0) const {
        float *logits = meta->logits;
        const int v0 = tile_idx * kTcBM;
        if (logits)
            for (int t = tid; t < n_live * kTcBM; t += nthr) {
                const int n = t / kTcBM, r = t % kTcBM;
                logits[(size_t)(n0 + n) * V + v0 + r] = tile[n * ld + r];
            }
        // one warp per column: a lane scans four consecutive features, then (max, lowest id) over the warp
        const int lane = tid & 31;
        for (int n = tid >> 5; n < n_live; n += nthr >> 5) {
            const float4 x = *reinterpret_cast<const float4 *>(tile + n * ld + 4 * lane);
            float bv = -CUDART_INF_F;
            int bi = 0x7fffffff;
            if (x.x > bv) { bv = x.x; bi = v0 + 4 * lane; }
            if (x.y > bv) { bv = x.y; bi = v0 + 4 * lane + 1; }
            if (x.z > bv) { bv = x.z; bi = v0 + 4 * lane + 2; }
            if (x.w > bv) { bv = x.w; bi = v0 + 4 * lane + 3; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) {
                part_val[(size_t)(n0 + n) * n_parts + tile_idx] = bv;
                part_idx[(size_t)(n0 + n) * n_parts + tile_idx] = bi;
            }
        }
    }
};

// ---------------------------------------------------------------- the GEMM kernel
struct TcArgs {
    int K;            // inner dimension (multiple of 64)
    int n_pad;        // N operand rows (multiple of 16, <= 256)
    int splits;       // K splits per tile = CTAs per cluster (<= 8)
    int n_stages;     // pipeline depth
    int late_release; // 1: dependent grids may start only once this grid's own dependency is met (see the kernel)
    int one_box;      // 1: map_bhi covers the hi rows AND the lo rows behind them: one copy of 2 n_pad rows per k-block
    int wide;         // 1: hi and lo operand rows as one operand of 2 n_pad rows (the host checks the TMEM budget)
    int a_rows_per_map;  // a tile's 128 rows come from map tile_idx / (rows_per_map / 128) ... see tile_map()
    int gateup;       // 1: a tile is 64 rows of map 0 + 64 rows of map 1
    int qkv_q_tiles, qkv_k_tiles;  // QKV: tiles per matrix (0 otherwise)
    const int32_t *rows;   // step row id of operand row n
    const int32_t *cnt;    // live operand rows (device)
    const int32_t *hint;   // a count of those rows that is never too low: 0 means there are certainly none
    int *dev_err;
};

// ---------------------------------------------------------------- the common tail of the tensor-core GEMM kernels
// Called by every thread once the accumulator is complete and the pipeline memory is free: moves the accumulator
// from TMEM to shared memory (column by column, see the epilogues), frees TMEM, adds up the K-split partial tiles over
// the cluster and runs the epilogue.
//
// Reduce-scatter over the cluster: CTA `split` owns whole quads of row pairs and adds them up, in split order, from
// every peer's shared memory with 128-bit distributed-shared-memory loads, all peers' loads in flight together; the
// sums replace its own partial values in place (peers only ever read the rows of THEIR slices).  A CTA may not
// exit while a peer still reads its tile: it arrives at the second cluster barrier right after its own reads and waits
// for it after its epilogue.  Even a CTA that gave up takes part in both barriers: a cluster barrier has no time-out.
// `wide`: the accumulator has 2 NP columns, W hi^T in [0, NP) and W lo^T in [NP, 2 NP), to be added up here.
template <class Epi>
__device__ __forceinline__ void tc_finish(const Epi &epi, float *tile, uint32_t tmem_d, uint32_t tmem_cols, int NP,
                                          int splits, int split, int tile_idx, int n_live, const int32_t *rows, bool ok,
                                          const int *s_abort, int nthr, bool wide = false) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (warp >= 2 && warp < 6 && ok && n_live > 0) {
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        float *col = tile + q * 32 + lane;
        for (int c0 = 0; c0 < NP; c0 += 16) {
            float v[16];
            tc_ld16(tmem_d + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
            if (wide) {
                float w[16];
                tc_ld16(tmem_d + ((uint32_t)(q * 32) << 16) + (uint32_t)(NP + c0), w);
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] += w[j];
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) col[(c0 + j) * kTcLd] = v[j];
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(tmem_cols));
    }
    if (n_live <= 0) return;  // uniform over the cluster: nobody waits for anybody
    const bool good = ok && !*reinterpret_cast<const volatile int *>(s_abort);
    int pr0 = 0, pr1 = kTcBM / 2;
    if (splits > 1) {
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        const int q0 = 16 * split / splits, nq = 16 * (split + 1) / splits - q0;
        pr0 = 4 * q0;
        pr1 = 4 * (q0 + nq);
        if (good) {
            const int per_col = 2 * nq;
            for (int t = tid; t < NP * per_col; t += nthr) {
                const int n = t / per_col, r = epi.quad_row(t % per_col, q0, nq);
                float *p = tile + n * kTcLd + r;
                const uint32_t laddr = smem_u32(p);
                float4 x[8];
#pragma unroll
                for (int sp = 0; sp < 8; ++sp) {
                    x[sp] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (sp < splits) {
                        uint32_t raddr;
                        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(laddr), "r"(sp));
                        asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(x[sp].x), "=f"(x[sp].y), "=f"(x[sp].z), "=f"(x[sp].w)
                                     : "r"(raddr)
                                     : "memory");
                    }
                }
                float4 v = x[0];
#pragma unroll
                for (int sp = 1; sp < 8; ++sp) { v.x += x[sp].x; v.y += x[sp].y; v.z += x[sp].z; v.w += x[sp].w; }
                *reinterpret_cast<float4 *>(p) = v;
            }
        }
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        __syncthreads();
    }
    if (good) epi.run(tile, kTcLd, tile_idx, n_live, rows, tid, nthr, pr0, pr1);
    if (splits > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <class Epi>
__global__ void __launch_bounds__(kTcThreads) tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a0,
                                                             const __grid_constant__ CUtensorMap map_a1,
                                                             const __grid_constant__ CUtensorMap map_a2,
                                                             const __grid_constant__ CUtensorMap map_bhi,
                                                             const __grid_constant__ CUtensorMap map_blo,
                                                             const TcArgs a, const Epi epi) {
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int NP = a.n_pad, S = a.n_stages;
    const uint32_t a_bytes = kTcBM * kTcBK * 2, b_bytes = (uint32_t)NP * kTcBK * 2;
    const uint32_t stage_bytes = a_bytes + 2 * b_bytes;  // multiples of 1024 (n_pad multiple of 16 -> b_bytes of 2048)
    uint8_t *stages = smem;
    float *tile = reinterpret_cast<float *>(stages);     // the finished tile reuses the pipeline memory
    uint64_t *bars = reinterpret_cast<uint64_t *>(stages + (size_t)S * stage_bytes);  // full[S], empty[S], acc
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort, s_some;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile_idx = blockIdx.x / a.splits, split = blockIdx.x % a.splits;
    const int kb_total = a.K / kTcBK;
    const int kb0 = (int)(((long long)kb_total * split) / a.splits), kb1 = (int)(((long long)kb_total * (split + 1)) / a.splits);
    const int nkb = kb1 - kb0;
    // Up to 128 operand rows the hi and the lo boxes (adjacent in a stage) are ONE operand of 2 NP rows: a single MMA per
    // 16 inputs, D = [W hi^T | W lo^T] in 2 NP columns, added up when the tile leaves TMEM.  (An instruction costs ~85
    // cycles or more whatever its N, and it reads the weight box from shared memory once instead of twice.)
    const bool wide = a.wide != 0;
    const int acc_n = wide ? 2 * NP : NP;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < acc_n) tmem_cols <<= 1;

    // `late_release`: the next grid in the stream is the dequantising kernel of the same projection, which runs beside
    // this one instead of behind it: it never waits for this grid at its start, so it may only start once everything
    // BOTH read (the operand kernels' output) is complete - that is when every CTA here is past its own wait.
    if (!a.late_release) pdl_launch();
    if (tid == 0) s_some = *reinterpret_cast<const volatile int32_t *>(a.hint) > 0;  // one read for the whole CTA
    __syncthreads();
    if (!s_some) {  // every row has left the backbone: nothing to fetch, nothing to compute (uniform over the cluster:
        pdl_wait();  // the hint only changes between layers); still order this grid behind its predecessor
        return;
    }
    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&bars[s]), 1); mbar_init(smem_u32(&bars[S + s]), 1); }
        mbar_init(smem_u32(&bars[2 * S]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {  // TMEM accumulator: 128 lanes x tmem_cols fp32 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(tmem_cols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = s_tmem;
    volatile int *abortp = &s_abort;

    // where this tile's weight rows live
    const CUtensorMap *ma = &map_a0, *ma2 = nullptr;
    int ay = tile_idx * kTcBM, ay2 = 0;
    if (a.gateup) { ma2 = &map_a1; ay = tile_idx * 64; ay2 = tile_idx * 64; }
    else if (a.qkv_q_tiles) {
        if (tile_idx >= a.qkv_q_tiles + a.qkv_k_tiles) { ma = &map_a2; ay = (tile_idx - a.qkv_q_tiles - a.qkv_k_tiles) * kTcBM; }
        else if (tile_idx >= a.qkv_q_tiles) { ma = &map_a1; ay = (tile_idx - a.qkv_q_tiles) * kTcBM; }
    }
    // The two issuing lanes advance their state incrementally (stage, parity, addresses: no division or multiplication
    // per k-block): a single thread retires an instruction every few cycles, and a k-block it handles late is 16 KB of
    // weights not streamed.
    const uint32_t stage0 = smem_u32(stages), full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[S]);
    int ax = kb0 * kTcBK;  // inner coordinate of the next weight tile to request
    auto load_a = [&](uint32_t s) {  // ... into stage s (expects the stage's whole byte count)
        const uint32_t full = full0 + 8 * s, dst = stage0 + s * stage_bytes;
        mbar_expect_tx(full, stage_bytes);
        if (ma2) {  // two 64-row boxes: gate rows then up rows (each box 64 x 64 bf16 = 8 KB, 1024-aligned)
            tma_load_2d(dst, ma, ax, ay, full);
            tma_load_2d(dst + a_bytes / 2, ma2, ax, ay2, full);
        } else {
            tma_load_2d(dst, ma, ax, ay, full);
        }
        ax += kTcBK;
    };
    auto load_b = [&](uint32_t s, int x) {
        const uint32_t full = full0 + 8 * s, dst = stage0 + s * stage_bytes + a_bytes;
        tma_load_2d(dst, &map_bhi, x, 0, full);
        if (!a.one_box) tma_load_2d(dst + b_bytes, &map_blo, x, 0, full);
    };

    // weights first: they depend on nothing
    const int pre = min(S, nkb);
    if (tid == 0)
        for (int i = 0; i < pre; ++i) load_a((uint32_t)i);
    pdl_wait();
    if (a.late_release) pdl_launch();
    const int n_live = *a.cnt;  // rows of the backbone list; the stream kernel serves the exit-layer rows
    // even with no live row the requested weight tiles must land before the CTA may exit: run the pipeline once
    const int nkb_run = n_live > 0 ? nkb : pre;

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < pre; ++i) load_b((uint32_t)i, (kb0 + i) * kTcBK);
            uint32_t s = 0, par = 0;  // (k-block `pre` is the first to reuse a stage: stage 0, first completion of its barrier)
            for (int i = pre; i < nkb_run; ++i) {
                if (!mbar_wait(empty0 + 8 * s, par, abortp, a.dev_err)) break;
                const int x = ax;
                load_a(s);
                load_b(s, x);
                if (++s == (uint32_t)S) { s = 0; par ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc_idesc(acc_n);
            const uint64_t dfix = tc_smem_desc(0);  // everything but the address field
            const uint32_t stage16 = stage_bytes >> 4, a16 = a_bytes >> 4, b16 = b_bytes >> 4;
            uint32_t s = 0, par = 0, addr16 = stage0 >> 4;
            for (int i = 0; i < nkb_run; ++i) {
                if (!mbar_wait(full0 + 8 * s, par, abortp, a.dev_err)) break;
                tc_fence_after();
                const uint64_t da = dfix | addr16, dhi = da + a16, dlo = dhi + b16;  // (addresses below 256 KB: no carry)
                tc_mma(tmem_d, da, dhi, idesc, i > 0 ? 1u : 0u);
                if (!wide) tc_mma(tmem_d, da, dlo, idesc, 1u);
#pragma unroll
                for (int k = 1; k < kTcBK / 16; ++k) {  // UMMA K = 16 bf16 = 32 bytes: +2 in the 16-byte address field
                    tc_mma(tmem_d, da + 2 * k, dhi + 2 * k, idesc, 1u);
                    if (!wide) tc_mma(tmem_d, da + 2 * k, dlo + 2 * k, idesc, 1u);
                }
                tc_commit(empty0 + 8 * s);  // frees the stage once these MMAs have read it
                if (++s == (uint32_t)S) { s = 0; par ^= 1u; addr16 = stage0 >> 4; } else addr16 += stage16;
            }
            tc_commit(smem_u32(&bars[2 * S]));      // accumulator complete
        }
    }
    // The other lanes of the two single-lane warps park at a warp barrier: a spinning (and possibly suspending)
    // mbarrier wait in the same warp would steal the issuing lane's cycles.
    __syncwarp();
    // everyone: wait for the accumulator (bounded; sleeping between polls, so that the waiting warps leave the issue slots
    // to the two issuing lanes), then move it out of TMEM
    bool ok = mbar_wait_sleepy(smem_u32(&bars[2 * S]), 0, abortp, a.dev_err);
    tc_fence_after();
    __syncthreads();  // all TMA writes and MMA reads of the pipeline memory are over: it now holds the tile
    tc_finish(epi, tile, tmem_d, tmem_cols, NP, a.splits, split, tile_idx, n_live, a.rows, ok, &s_abort, kTcThreads, wide);
}

inline size_t tc_smem_bytes(int n_pad, int n_stages) {
    const size_t stage = (size_t)kTcBM * kTcBK * 2 + 2 * (size_t)n_pad * kTcBK * 2;
    const size_t pipe = (size_t)n_stages * stage;  // the finished tile reuses it (the host checks the fit)
    return 1024 + pipe + sizeof(uint64_t) * (2 * n_stages + 1) + 64;
}

}  // namespace river
