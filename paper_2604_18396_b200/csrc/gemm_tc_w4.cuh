// Batched exit-layer projections on tcgen05 (sm_100a): the 4-bit weights are dequantised ONCE per weight into the
// A operand of the tensor cores, whatever the number of activation rows, and that operand lives in TENSOR MEMORY.
//
// The CUDA-core evaluation of the 4-bit copy costs about three instructions per weight AND activation row; from
// five rows on it is far from the HBM roofline.  Here a CTA owns one 128-feature tile (and one K-split) as in
// tc_gemm_kernel, but its A operand is made on the fly:
//   * a producer lane brings raw code tiles (128 rows x 128 bytes = 256 inputs, 128-byte swizzle) and the f16
//     activation tiles (hi and lo parts) into shared memory with 2-D TMA copies;
//   * eight dequantisation warps - thread = weight row = TMEM lane, two warps per lane quarter taking the even and
//     the odd k-blocks - turn each 32-byte run of codes (one 64-input k-block = one quantisation group) into 64 f16
//     weights (q - z) * s - a code word becomes four f16x2 registers with one logic op each (0x6400 | q = 1024 + q,
//     0x6400 | q << 4 = 1024 + 16 q), then exact f16 subtractions and one rounding multiply - and write them with
//     ONE tcgen05.st (32 columns of two f16) into a ring of A tiles next to the accumulator; tcgen05.wait::st, a
//     tcgen05 fence and an mbarrier hand the tile to the MMA lane.  (Against an operand tile in shared memory: no
//     swizzled stores, no proxy fence, half the shared-memory reads per MMA, and the shared memory a stage needs is
//     the activation tile alone, so four stages fit beside a second CTA on the SM.)
//   * inside every 8 inputs the weights come out in the order (0,4,1,5,2,6,3,7); the activation tiles are written
//     in the same order by tc_prep_w4_kernel, so no permutation is ever executed;
//   * tcgen05.mma (kind::f16, A from tensor memory, B from shared memory, fp32 accumulator in TMEM) runs against the
//     activations' hi and lo parts; epilogues, K-split clusters and the distributed-shared-memory reduction are those
//     of tc_gemm_kernel.
// Requires group == 64 (one scale / zero per weight row and k-block) and K a multiple of 256.
#pragma once
#include <cuda_fp16.h>

#include "gemm_tc.cuh"

namespace river {

constexpr int kW4DqWarps = 8;                         // dequantisation warps: two per TMEM lane quarter (even / odd k-blocks)
constexpr int kW4Threads = 64 + 32 * kW4DqWarps;      // warp 0: TMA, warp 1: MMA + TMEM, warps 2..9: dequant / epilogue
constexpr int kW4Super = 4;                           // k-blocks per raw code tile: 4 x 32 bytes of codes per row
constexpr int kW4RawBufs = 2;
constexpr uint32_t kW4RawBytes = kTcBM * 128;         // one raw code tile
constexpr uint32_t kW4ACols = kTcBK / 2;              // TMEM columns of one A tile: 64 f16 per row, two per column

// A from tensor memory (lane = tile row, column c = inputs 2 c and 2 c + 1 of the k-block), B from shared memory.
__device__ __forceinline__ void tc_mma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// 32 consecutive columns of this warp's 32 lanes: register i of lane t -> (lane base + t, column + i)
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
        "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ uint32_t tc_idesc_f16(int n) {  // D fp32, A and B f16, K-major, M = 128, N = n
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTcBM >> 4) << 24);
}

// ---------------------------------------------------------------- activation rows -> f16 hi / lo operand buffers
// As tc_prep_kernel (CTA (i, j): inputs [2048 j, 2048 j + 2048) of operand row i, eight per thread), but f16 and with
// the inputs of every group of eight in the order (0,4,1,5,2,6,3,7).
__device__ __forceinline__ void tc_prep_w4_body(const ProjIn &in, const int32_t *idx, const int32_t *cnt, int K,
                                                __half *xhi, __half *xlo, int i, int by, float *red) {
    const int n = *cnt;
    if (n <= 0) return;  // no row on the exit layers: the GEMM returns before it reads an operand
    const int v = by * (2 * kPrepChunk / 8) + threadIdx.x;  // 8-input group of the row
    const bool mine = v < (K >> 3);
    uint4 *hi = reinterpret_cast<uint4 *>(xhi + (size_t)i * K), *lo = reinterpret_cast<uint4 *>(xlo + (size_t)i * K);
    if (i >= n) {
        if (mine) { hi[v] = make_uint4(0u, 0u, 0u, 0u); lo[v] = make_uint4(0u, 0u, 0u, 0u); }
        return;
    }
    const float4 *src = reinterpret_cast<const float4 *>(in.src + (size_t)idx[i] * K);
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    uint4 gw = make_uint4(0u, 0u, 0u, 0u);
    if (mine) {
        a = __ldcg(src + 2 * v);
        b = __ldcg(src + 2 * v + 1);
        if (in.gain) gw = *reinterpret_cast<const uint4 *>(in.gain + 8 * v);
    }
    const float scale = tc_prep_scale(in, src, K, red);
    if (!mine) return;
    float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    if (in.gain) {
        const uint32_t g[4] = {gw.x, gw.y, gw.z, gw.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            x[2 * q] = x[2 * q] * scale * bf16lo(g[q]);
            x[2 * q + 1] = x[2 * q + 1] * scale * bf16hi(g[q]);
        }
    }
    unsigned short h[8], l[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const __half hv = __float2half_rn(x[q]);
        h[q] = __half_as_ushort(hv);
        l[q] = __half_as_ushort(__float2half_rn(x[q] - __half2float(hv)));
    }
    // storage position p holds input perm[p], perm = (0,4,1,5,2,6,3,7)
    hi[v] = make_uint4((uint32_t)h[0] | ((uint32_t)h[4] << 16), (uint32_t)h[1] | ((uint32_t)h[5] << 16),
                       (uint32_t)h[2] | ((uint32_t)h[6] << 16), (uint32_t)h[3] | ((uint32_t)h[7] << 16));
    lo[v] = make_uint4((uint32_t)l[0] | ((uint32_t)l[4] << 16), (uint32_t)l[1] | ((uint32_t)l[5] << 16),
                       (uint32_t)l[2] | ((uint32_t)l[6] << 16), (uint32_t)l[3] | ((uint32_t)l[7] << 16));
}
static __global__ void __launch_bounds__(256) tc_prep_w4_kernel(const ProjIn in, const int32_t *idx, const int32_t *cnt, int K,
                                                         __half *xhi, __half *xlo) {
    __shared__ float red[8];
    pdl_launch();
    pdl_wait();
    tc_prep_w4_body(in, idx, cnt, K, xhi, xlo, blockIdx.x, blockIdx.y, red);
}
// Both operand sets of a projection in one launch: CTAs (i, j < ya) are tc_prep_kernel's for the backbone list, CTAs
// (i, ya + j) tc_prep_w4_kernel's for the list of the rows on the exit layers.
struct PrepPair {
    const int32_t *idx_a, *cnt_a, *idx_r, *cnt_r;
    __nv_bfloat16 *ahi, *alo;
    __half *rhi, *rlo;
    int ya;
};
static __global__ void __launch_bounds__(256) tc_prep_pair_kernel(const ProjIn in, const PrepPair p, int K) {
    __shared__ float red[8];
    pdl_launch();
    pdl_wait();
    if ((int)blockIdx.y < p.ya) tc_prep_body(in, p.idx_a, p.cnt_a, K, p.ahi, p.alo, blockIdx.x, blockIdx.y, red);
    else tc_prep_w4_body(in, p.idx_r, p.cnt_r, K, p.rhi, p.rlo, blockIdx.x, (int)blockIdx.y - p.ya, red);
}

// ---------------------------------------------------------------- the kernel
struct TcW4Args {
    int K;             // inner dimension (multiple of 256)
    int n_pad;         // N operand rows (multiple of 16, <= 256)
    int splits;        // K splits per tile = CTAs per cluster (<= 8), in whole raw tiles
    int n_stages;      // stages: activation tiles in shared memory AND A tiles in tensor memory (even)
    int overlap;       // 1: runs beside the preceding grid (tc_gemm_kernel of the same projection, launched with
                       // late_release): no wait at the start, the wait for that grid comes before the CTA exits
    int one_box;       // 1: map_bhi covers the hi rows AND the lo rows behind them: one copy of 2 n_pad rows per k-block
    int wide;          // 1: hi and lo activation rows as one operand of 2 n_pad rows (the host checks the TMEM budget)
    int gateup;        // 1: a tile is 64 rows of matrix 0 + 64 rows of matrix 1
    int qkv_q_tiles, qkv_k_tiles;  // QKV: tiles per matrix (0 otherwise)
    const uint16_t *scale[3], *zero[3];  // bf16 [rows][K/64] of the up to three matrices behind the code maps
    const int32_t *rows;
    const int32_t *cnt;
    const int32_t *hint;  // a count of exit-layer rows that is never too high (an earlier layer's): > 0 means rows exist
    int *dev_err;
};

// (1024 + q0, 1024 + q4), (1024 + 16 q1, 1024 + 16 q5), ... -> ((q0 - z) s, (q4 - z) s), ((q1 - z) s, (q5 - z) s), ...
__device__ __forceinline__ uint4 w4_word_to_f16(uint32_t v, __half2 z2, __half2 s2) {
    const __half2 k1024 = __half2half2(__ushort_as_half((unsigned short)0x6400));
    const __half2 k16th = __half2half2(__ushort_as_half((unsigned short)0x2C00));  // 1/16
    const __half2 nz2 = __hneg2(z2);
    const uint32_t v8 = v >> 8;
    uint32_t e0 = (v & 0x000f000fu) | 0x64006400u, o0 = (v & 0x00f000f0u) | 0x64006400u;
    uint32_t e1 = (v8 & 0x000f000fu) | 0x64006400u, o1 = (v8 & 0x00f000f0u) | 0x64006400u;
    auto even = [&](uint32_t e) {
        const __half2 q = __hsub2(*reinterpret_cast<__half2 *>(&e), k1024);  // exact
        const __half2 w = __hmul2(__hadd2(q, nz2), s2);                        // q - z exact, one rounding
        return *reinterpret_cast<const uint32_t *>(&w);
    };
    auto odd = [&](uint32_t o) {
        const __half2 q16 = __hsub2(*reinterpret_cast<__half2 *>(&o), k1024);  // 16 q, exact
        const __half2 w = __hmul2(__hfma2(q16, k16th, nz2), s2);               // q - z exact, one rounding
        return *reinterpret_cast<const uint32_t *>(&w);
    };
    return make_uint4(even(e0), odd(o0), even(e1), odd(o1));
}

template <class Epi>
__global__ void __launch_bounds__(kW4Threads, 2) tc_gemm_w4_kernel(const __grid_constant__ CUtensorMap map_c0,
                                                                const __grid_constant__ CUtensorMap map_c1,
                                                                const __grid_constant__ CUtensorMap map_c2,
                                                                const __grid_constant__ CUtensorMap map_bhi,
                                                                const __grid_constant__ CUtensorMap map_blo,
                                                                const TcW4Args a, const Epi epi) {
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int NP = a.n_pad, S = a.n_stages;
    const uint32_t b_bytes = (uint32_t)NP * kTcBK * 2;
    const uint32_t stage_bytes = 2 * b_bytes;  // hi and lo activation tiles; the A tile of a stage is in tensor memory
    uint8_t *stages = smem;
    uint8_t *raw = stages + (size_t)S * stage_bytes;                 // kW4RawBufs raw code tiles, 1024-aligned
    float *tile = reinterpret_cast<float *>(stages);                 // the finished tile reuses stages + raw
    // barriers: full[S] (A tile written and activation tile landed), empty[S], raw_full[R], raw_empty[R], acc
    uint64_t *bars = reinterpret_cast<uint64_t *>(raw + (size_t)kW4RawBufs * kW4RawBytes);
    uint64_t *b_afull = bars, *b_empty = bars + S, *b_rfull = bars + 2 * S, *b_rempty = bars + 2 * S + kW4RawBufs,
             *b_acc = bars + 2 * S + 2 * kW4RawBufs;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort, s_early;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile_idx = blockIdx.x / a.splits, split = blockIdx.x % a.splits;
    const int sb_total = a.K / (kTcBK * kW4Super);
    const int sb0 = (int)(((long long)sb_total * split) / a.splits), sb1 = (int)(((long long)sb_total * (split + 1)) / a.splits);
    const int nsb = sb1 - sb0, kb0 = sb0 * kW4Super, nkb = nsb * kW4Super;
    const bool wide = a.wide != 0;  // as in tc_gemm_kernel: one MMA per 16 inputs, D = [W hi^T | W lo^T]
    const int acc_n = wide ? 2 * NP : NP;
    uint32_t tmem_cols = 32;  // accumulator in columns [0, acc_n), then S A tiles of 32 columns
    while (tmem_cols < (uint32_t)acc_n + (uint32_t)S * kW4ACols) tmem_cols <<= 1;

    pdl_launch();
    if (tid == 0) {
        s_abort = 0;
        s_early = *reinterpret_cast<const volatile int32_t *>(a.hint) > 0;  // one read for the whole CTA
        for (int s = 0; s < S; ++s) {
            // a stage is full when its A tile is written (one arrival per lane quarter) AND its activation tile has
            // landed (the producer's arrival with the byte count): ONE barrier, one poll per k-block for the MMA lane
            mbar_init(smem_u32(&b_afull[s]), 4 + 1);
            mbar_init(smem_u32(&b_empty[s]), 1);
        }
        for (int r = 0; r < kW4RawBufs; ++r) {
            mbar_init(smem_u32(&b_rfull[r]), 1);
            mbar_init(smem_u32(&b_rempty[r]), kW4DqWarps);
        }
        mbar_init(smem_u32(b_acc), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    volatile int *abortp = &s_abort;

    // where this tile's weight rows live: (matrix, first row) for tile rows 0.. and, for gate/up, for rows 64..
    int m0 = 0, ay = tile_idx * kTcBM, m1 = 0, ay1 = 0;
    if (a.gateup) { m1 = 1; ay = tile_idx * 64; ay1 = tile_idx * 64; }
    else if (a.qkv_q_tiles) {
        if (tile_idx >= a.qkv_q_tiles + a.qkv_k_tiles) { m0 = 2; ay = (tile_idx - a.qkv_q_tiles - a.qkv_k_tiles) * kTcBM; }
        else if (tile_idx >= a.qkv_q_tiles) { m0 = 1; ay = (tile_idx - a.qkv_q_tiles) * kTcBM; }
    }
    const CUtensorMap *maps[3] = {&map_c0, &map_c1, &map_c2};
    auto load_raw = [&](int sb) {  // raw code tile of super-block sb0 + sb into raw buffer sb % R
        const int r = sb % kW4RawBufs;
        const uint32_t full = smem_u32(&b_rfull[r]), dst = smem_u32(raw + (size_t)r * kW4RawBytes);
        mbar_expect_tx(full, kW4RawBytes);
        const int x = (sb0 + sb) * 128;  // byte offset inside a code row
        if (a.gateup) {
            tma_load_2d(dst, maps[0], x, ay, full);
            tma_load_2d(dst + kW4RawBytes / 2, maps[1], x, ay1, full);
        } else {
            tma_load_2d(dst, maps[m0], x, ay, full);
        }
    };
    // codes first: they depend on nothing - if an earlier layer already had rows on its exit layer (the count only
    // grows inside a step); otherwise wait for the real count and leave at once if it is zero
    const bool early = s_early != 0;
    const int pre = early ? min(kW4RawBufs, nsb) : 0;
    if (tid == 0)
        for (int sb = 0; sb < pre; ++sb) load_raw(sb);
    // Beside the backbone kernel of the same projection (`overlap`): that grid let this one start only after the
    // operand kernels of both had completed, the two write disjoint rows, and the row count dates from the previous
    // block - nothing here depends on it.  Whoever comes next in the stream waits for THIS grid, so this grid must not
    // complete before that one: every CTA waits for it just before it exits.
    if (!a.overlap) pdl_wait();
    const int n_live = *a.cnt;
    if (n_live <= 0 && pre == 0) {  // uniform over the CTA and the cluster (nobody reaches a cluster barrier)
        if (a.overlap) pdl_wait();
        return;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(tmem_cols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = s_tmem;
    // even with no live row the requested code tiles must land before the CTA may exit
    const int nsb_run = n_live > 0 ? nsb : pre;
    const int nkb_run = n_live > 0 ? nkb : 0;

    if (warp == 0) {
        if (lane == 0) {
            int rs = pre;  // next raw tile to request
            if (n_live <= 0) {
                for (int sb = 0; sb < nsb_run; ++sb)
                    if (!mbar_wait(smem_u32(&b_rfull[sb % kW4RawBufs]), 0, abortp, a.dev_err)) break;
            }
            // stage, parity and addresses advance incrementally (a single lane retires an instruction every few
            // cycles: divisions by the runtime stage count cost more here than the copies they address)
            const uint32_t bfull0 = smem_u32(b_afull), empty0 = smem_u32(b_empty), rempty0 = smem_u32(b_rempty);
            const uint32_t stage0 = smem_u32(stages);
            uint32_t s = 0, epar = 1, dst = stage0;  // epar: parity of `empty` to wait for from the second round on
            int x = kb0 * kTcBK;
            for (int i = 0; i < nkb_run; ++i) {
                // raw tiles as far ahead as buffers are free; the one this k-block needs with a blocking wait
                while (rs < nsb) {
                    const uint32_t eb = rempty0 + 8 * (uint32_t)(rs % kW4RawBufs);
                    const uint32_t par = ((rs / kW4RawBufs) - 1) & 1;
                    if (rs <= i / kW4Super) {
                        if (!mbar_wait(eb, par, abortp, a.dev_err)) break;
                    } else if (!mbar_test_wait(eb, par)) {  // (a probe: try_wait would suspend the lane)
                        break;
                    }
                    load_raw(rs);
                    ++rs;
                }
                if (*abortp) break;
                if (i >= S && !mbar_wait(empty0 + 8 * s, epar, abortp, a.dev_err)) break;
                const uint32_t full = bfull0 + 8 * s;
                mbar_expect_tx(full, 2 * b_bytes);
                tma_load_2d(dst, &map_bhi, x, 0, full);
                if (!a.one_box) tma_load_2d(dst + b_bytes, &map_blo, x, 0, full);
                x += kTcBK;
                if (++s == (uint32_t)S) { s = 0; epar ^= 1u; dst = stage0; } else dst += stage_bytes;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc_idesc_f16(acc_n);
            const uint64_t dfix = tc_smem_desc(0);  // everything but the address field
            const uint32_t stage16 = stage_bytes >> 4, b16 = b_bytes >> 4;
            const uint32_t afull0 = smem_u32(b_afull), empty0 = smem_u32(b_empty);
            const uint32_t ta0 = tmem_d + (uint32_t)acc_n;
            uint32_t s = 0, par = 0, addr16 = smem_u32(stages) >> 4, ta = ta0;  // incremental: no division per k-block
            for (int i = 0; i < nkb_run; ++i) {
                if (!mbar_wait(afull0 + 8 * s, par, abortp, a.dev_err)) break;
                tc_fence_after();
                const uint64_t dhi = dfix | addr16, dlo = dhi + b16;  // (addresses below 256 KB: no carry)
                tc_mma_ts(tmem_d, ta, dhi, idesc, i > 0 ? 1u : 0u);
                if (!wide) tc_mma_ts(tmem_d, ta, dlo, idesc, 1u);
#pragma unroll
                for (int k = 1; k < kTcBK / 16; ++k) {  // 16 inputs = 8 columns of A = 32 bytes of a B row
                    tc_mma_ts(tmem_d, ta + 8 * k, dhi + 2 * k, idesc, 1u);
                    if (!wide) tc_mma_ts(tmem_d, ta + 8 * k, dlo + 2 * k, idesc, 1u);
                }
                tc_commit(empty0 + 8 * s);
                if (++s == (uint32_t)S) { s = 0; par ^= 1u; addr16 = smem_u32(stages) >> 4; ta = ta0; }
                else { addr16 += stage16; ta += kW4ACols; }
            }
            tc_commit(smem_u32(b_acc));
        }
    } else if (nkb_run > 0) {
        // ---- dequantisation: this warp may write TMEM lanes 32 (warp % 4) .. + 31 = tile rows; the two warps of a
        // lane quarter take the even and the odd k-blocks (S is even: each keeps to its own stages)
        const int r = 32 * (warp & 3) + lane, grp = (warp - 2) >> 2;
        const uint32_t ta_lane = tmem_d + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)acc_n;
        int mi = m0;
        size_t grow = (size_t)ay + r;  // row inside its matrix
        if (a.gateup && r >= 64) { mi = m1; grow = (size_t)ay1 + (r - 64); }
        const int ng = a.K >> 6;
        const uint16_t *sp = a.scale[mi] + grow * ng + kb0, *zp = a.zero[mi] + grow * ng + kb0;
        uint2 s_next = *reinterpret_cast<const uint2 *>(sp), z_next = *reinterpret_cast<const uint2 *>(zp);
        uint2 s_cur = s_next, z_cur = z_next;
        bool alive = true;
        // one lane polls a barrier for its warp (256 polling threads would compete with the converting ones for issue
        // slots); the shuffle hands the outcome, and the ordering the wait established, to the other lanes
        auto warp_wait = [&](uint32_t bar, uint32_t parity) {
            int ok = 1;
            if (lane == 0) ok = mbar_wait(bar, parity, abortp, a.dev_err) ? 1 : 0;
            return __shfl_sync(0xffffffffu, ok, 0) != 0;
        };
        int s = grp;
        uint32_t epar = 1;  // parity of the stage's `empty` barrier to wait for from the second round on: ((i / S) - 1) & 1
        for (int i = grp; i < nkb_run && alive; i += 2) {
            const int kq = i & (kW4Super - 1), sb = i / kW4Super, rb = sb % kW4RawBufs;
            if (kq < 2) {  // this warp's first k-block of the raw tile
                s_cur = s_next; z_cur = z_next;
                if (sb + 1 < nsb) {  // the next raw tile's scales / zeros travel while this one is processed
                    s_next = *reinterpret_cast<const uint2 *>(sp + (sb + 1) * kW4Super);
                    z_next = *reinterpret_cast<const uint2 *>(zp + (sb + 1) * kW4Super);
                }
                if (!warp_wait(smem_u32(&b_rfull[rb]), (sb / kW4RawBufs) & 1)) { alive = false; break; }
            }
            if (i >= S) {  // the MMAs that read this stage's A tile are complete
                if (!warp_wait(smem_u32(&b_empty[s]), epar)) { alive = false; break; }
                tc_fence_after();
            }
            const uint32_t sw = (kq < 2 ? s_cur.x : s_cur.y), zw = (kq < 2 ? z_cur.x : z_cur.y);
            const float sf = (kq & 1) ? bf16hi(sw) : bf16lo(sw), zf = (kq & 1) ? bf16hi(zw) : bf16lo(zw);
            const __half2 s2 = __float2half2_rn(sf), z2 = __float2half2_rn(zf);  // bf16 values are exact in f16 range here
            const uint8_t *rawt = raw + (size_t)rb * kW4RawBytes + (size_t)r * 128;
            const uint4 c0 = *reinterpret_cast<const uint4 *>(rawt + (((2 * kq) ^ (r & 7)) * 16));
            const uint4 c1 = *reinterpret_cast<const uint4 *>(rawt + (((2 * kq + 1) ^ (r & 7)) * 16));
            const uint32_t cw[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
            uint32_t wv[32];  // column 4 j + t of the A tile: inputs 8 j + (t, t + 4) in the low / high half
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint4 w = w4_word_to_f16(cw[j], z2, s2);
                wv[4 * j] = w.x; wv[4 * j + 1] = w.y; wv[4 * j + 2] = w.z; wv[4 * j + 3] = w.w;
            }
            tc_st32(ta_lane + (uint32_t)s * kW4ACols, wv);  // returns when the stores are complete
            tc_fence_before();
            __syncwarp();  // every lane's stores are done (and its reads of the raw tile): one arrival per warp
            if (lane == 0) {
                mbar_arrive(smem_u32(&b_afull[s]));
                if (kq >= kW4Super - 2) mbar_arrive(smem_u32(&b_rempty[rb]));
            }
            s += 2;
            if (s >= S) { s -= S; epar ^= 1u; }
        }
    }
    __syncwarp();
    bool ok = n_live > 0 ? mbar_wait(smem_u32(b_acc), 0, abortp, a.dev_err) : true;
    tc_fence_after();
    __syncthreads();  // all copies into and MMA reads of the pipeline memory are over: it now holds the tile
    tc_finish(epi, tile, tmem_d, tmem_cols, NP, a.splits, split, tile_idx, n_live, a.rows, ok, &s_abort, kW4Threads, wide);
    if (a.overlap) pdl_wait();
}

inline size_t tc_w4_smem_bytes(int n_pad, int n_stages) {
    const size_t stage = 2 * (size_t)n_pad * kTcBK * 2;
    return 1024 + (size_t)n_stages * stage + (size_t)kW4RawBufs * kW4RawBytes +
           sizeof(uint64_t) * (2 * n_stages + 2 * kW4RawBufs + 1) + 64;
}

}  // namespace river
