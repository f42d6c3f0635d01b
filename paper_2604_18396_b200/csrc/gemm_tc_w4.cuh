// Batched exit-layer projections on tcgen05 (sm_100a): the 4-bit weights are dequantised ONCE per weight into the
// shared-memory operand tile of the tensor cores, whatever the number of activation rows.
//
// The CUDA-core evaluation of the 4-bit copy costs about three instructions per weight AND activation row; from
// five rows on it is far from the HBM roofline.  Here a CTA owns one 128-feature tile (and one K-split) as in
// tc_gemm_kernel, but its A operand is made on the fly:
//   * a producer lane brings raw code tiles (128 rows x 128 bytes = 256 inputs, 128-byte swizzle) and the f16
//     activation tiles (hi and lo parts) into shared memory with 2-D TMA copies;
//   * eight dequantisation warps (two threads per weight row) turn each 32-byte run of codes (one 64-input k-block =
//     one quantisation group) into 64 f16 weights (q - z) * s - a code word becomes four f16x2 registers with one
//     logic op each (0x6400 | q = 1024 + q, 0x6400 | q << 4 = 1024 + 16 q), then exact f16 subtractions and one
//     rounding multiply - and store them as the K-major, 128-byte-swizzled operand tile; a proxy fence and an
//     mbarrier hand the tile to the MMA lane;
//   * inside every 8 inputs the weights come out in the order (0,4,1,5,2,6,3,7); the activation tiles are written
//     in the same order by tc_prep_w4_kernel, so no permutation is ever executed;
//   * tcgen05.mma (kind::f16, f16 x f16 -> fp32 in TMEM) runs against the activations' hi and lo parts; epilogues,
//     K-split clusters and the distributed-shared-memory reduction are those of tc_gemm_kernel.
// Requires group == 64 (one scale / zero per weight row and k-block) and K a multiple of 256.
#pragma once
#include <cuda_fp16.h>

#include "gemm_tc.cuh"

namespace river {

constexpr int kW4DqWarps = 8;                         // dequantisation warps (two threads per tile row)
constexpr int kW4Threads = 64 + 32 * kW4DqWarps;      // warp 0: TMA, warp 1: MMA + TMEM, warps 2..9: dequant / epilogue
constexpr int kW4Super = 4;                           // k-blocks per raw code tile: 4 x 32 bytes of codes per row
constexpr int kW4RawBufs = 2;
constexpr uint32_t kW4RawBytes = kTcBM * 128;         // one raw code tile

__device__ __forceinline__ uint32_t tc_idesc_f16(int n) {  // D fp32, A and B f16, K-major, M = 128, N = n
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTcBM >> 4) << 24);
}

// ---------------------------------------------------------------- activation rows -> f16 hi / lo operand buffers
// As tc_prep_kernel (CTA (i, j): inputs [2048 j, 2048 j + 2048) of operand row i, eight per thread), but f16 and with
// the inputs of every group of eight in the order (0,4,1,5,2,6,3,7).
static __global__ void __launch_bounds__(256) tc_prep_w4_kernel(const ProjIn in, const int32_t *idx, const int32_t *cnt, int K,
                                                         __half *xhi, __half *xlo) {
    __shared__ float red[8];
    pdl_launch();
    pdl_wait();
    const int i = blockIdx.x, n = *cnt;
    if (n <= 0) return;  // no row on the exit layers: the GEMM returns before it reads an operand
    const int v = blockIdx.y * (2 * kPrepChunk / 8) + threadIdx.x;  // 8-input group of the row
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

// ---------------------------------------------------------------- the kernel
struct TcW4Args {
    int K;             // inner dimension (multiple of 256)
    int n_pad;         // N operand rows (multiple of 16, <= 256)
    int splits;        // K splits per tile = CTAs per cluster (<= 8), in whole raw tiles
    int n_stages;      // operand stages
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
__global__ void __launch_bounds__(kW4Threads) tc_gemm_w4_kernel(const __grid_constant__ CUtensorMap map_c0,
                                                                const __grid_constant__ CUtensorMap map_c1,
                                                                const __grid_constant__ CUtensorMap map_c2,
                                                                const __grid_constant__ CUtensorMap map_bhi,
                                                                const __grid_constant__ CUtensorMap map_blo,
                                                                const TcW4Args a, const Epi epi) {
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int NP = a.n_pad, S = a.n_stages;
    const uint32_t a_bytes = kTcBM * kTcBK * 2, b_bytes = (uint32_t)NP * kTcBK * 2;
    const uint32_t stage_bytes = a_bytes + 2 * b_bytes;
    uint8_t *stages = smem;
    uint8_t *raw = stages + (size_t)S * stage_bytes;                 // kW4RawBufs raw code tiles, 1024-aligned
    float *tile = reinterpret_cast<float *>(stages);                 // the finished tile reuses stages + raw
    // barriers: a_full[S], b_full[S], empty[S], raw_full[R], raw_empty[R], acc
    uint64_t *bars = reinterpret_cast<uint64_t *>(raw + (size_t)kW4RawBufs * kW4RawBytes);
    uint64_t *b_afull = bars, *b_bfull = bars + S, *b_empty = bars + 2 * S, *b_rfull = bars + 3 * S,
             *b_rempty = bars + 3 * S + kW4RawBufs, *b_acc = bars + 3 * S + 2 * kW4RawBufs;
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort, s_early;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile_idx = blockIdx.x / a.splits, split = blockIdx.x % a.splits;
    const int sb_total = a.K / (kTcBK * kW4Super);
    const int sb0 = (int)(((long long)sb_total * split) / a.splits), sb1 = (int)(((long long)sb_total * (split + 1)) / a.splits);
    const int nsb = sb1 - sb0, kb0 = sb0 * kW4Super, nkb = nsb * kW4Super;
    const bool wide = a.wide != 0;  // as in tc_gemm_kernel: one MMA per 16 inputs, D = [W hi^T | W lo^T]
    const int acc_n = wide ? 2 * NP : NP;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < acc_n) tmem_cols <<= 1;

    pdl_launch();
    if (tid == 0) {
        s_abort = 0;
        s_early = *reinterpret_cast<const volatile int32_t *>(a.hint) > 0;  // one read for the whole CTA
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&b_afull[s]), kW4DqWarps);  // one arrival per dequantisation warp
            mbar_init(smem_u32(&b_bfull[s]), 1);
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
    auto load_b = [&](int i) {
        const int s = i % S;
        const uint32_t full = smem_u32(&b_bfull[s]), dst = smem_u32(stages + (size_t)s * stage_bytes) + a_bytes;
        mbar_expect_tx(full, 2 * b_bytes);
        const int x = (kb0 + i) * kTcBK;
        tma_load_2d(dst, &map_bhi, x, 0, full);
        tma_load_2d(dst + b_bytes, &map_blo, x, 0, full);
    };

    // codes first: they depend on nothing - if an earlier layer already had rows on its exit layer (the count only
    // grows inside a step); otherwise wait for the real count and leave at once if it is zero
    const bool early = s_early != 0;
    const int pre = early ? min(kW4RawBufs, nsb) : 0;
    if (tid == 0)
        for (int sb = 0; sb < pre; ++sb) load_raw(sb);
    pdl_wait();
    const int n_live = *a.cnt;
    if (n_live <= 0 && pre == 0) return;  // uniform over the CTA and the cluster (nobody reaches a cluster barrier)
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
            for (int i = 0; i < nkb_run; ++i) {
                // raw tiles as far ahead as buffers are free; the one this k-block needs with a blocking wait
                while (rs < nsb) {
                    const uint32_t eb = smem_u32(&b_rempty[rs % kW4RawBufs]);
                    const uint32_t par = ((rs / kW4RawBufs) - 1) & 1;
                    if (rs <= i / kW4Super) {
                        if (!mbar_wait(eb, par, abortp, a.dev_err)) break;
                    } else if (!mbar_try_wait(eb, par)) {
                        break;
                    }
                    load_raw(rs);
                    ++rs;
                }
                if (*abortp) break;
                if (i >= S && !mbar_wait(smem_u32(&b_empty[i % S]), ((i / S) - 1) & 1, abortp, a.dev_err)) break;
                load_b(i);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc_idesc_f16(acc_n);
            const uint64_t dfix = tc_smem_desc(0);  // everything but the address field
            const uint32_t stage16 = stage_bytes >> 4, a16 = a_bytes >> 4, b16 = b_bytes >> 4;
            const uint32_t afull0 = smem_u32(b_afull), bfull0 = smem_u32(b_bfull), empty0 = smem_u32(b_empty);
            uint32_t s = 0, par = 0, addr16 = smem_u32(stages) >> 4;  // incremental: no division per k-block
            for (int i = 0; i < nkb_run; ++i) {
                if (!mbar_wait(afull0 + 8 * s, par, abortp, a.dev_err)) break;
                if (!mbar_wait(bfull0 + 8 * s, par, abortp, a.dev_err)) break;
                tc_fence_after();
                const uint64_t da = dfix | addr16, dhi = da + a16, dlo = dhi + b16;  // (addresses below 256 KB: no carry)
                tc_mma(tmem_d, da, dhi, idesc, i > 0 ? 1u : 0u);
                if (!wide) tc_mma(tmem_d, da, dlo, idesc, 1u);
#pragma unroll
                for (int k = 1; k < kTcBK / 16; ++k) {
                    tc_mma(tmem_d, da + 2 * k, dhi + 2 * k, idesc, 1u);
                    if (!wide) tc_mma(tmem_d, da + 2 * k, dlo + 2 * k, idesc, 1u);
                }
                tc_commit(empty0 + 8 * s);
                if (++s == (uint32_t)S) { s = 0; par ^= 1u; addr16 = smem_u32(stages) >> 4; } else addr16 += stage16;
            }
            tc_commit(smem_u32(b_acc));
        }
    } else if (nkb_run > 0) {
        // ---- dequantisation: thread d owns tile row d / 2, 16-byte chunks 4 (d % 2) .. + 3 of every k-block
        const int d = tid - 64, r = d >> 1, hsel = d & 1;
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
        int s = 0;
        uint32_t epar = 1;  // parity of the stage's `empty` barrier to wait for from the second round on: ((i / S) - 1) & 1
        for (int i = 0; i < nkb_run && alive; ++i) {
            const int kq = i & (kW4Super - 1), sb = i / kW4Super, rb = sb % kW4RawBufs;
            if (kq == 0) {
                s_cur = s_next; z_cur = z_next;
                if (sb + 1 < nsb) {  // the next raw tile's scales / zeros travel while this one is processed
                    s_next = *reinterpret_cast<const uint2 *>(sp + (sb + 1) * kW4Super);
                    z_next = *reinterpret_cast<const uint2 *>(zp + (sb + 1) * kW4Super);
                }
                if (!warp_wait(smem_u32(&b_rfull[rb]), (sb / kW4RawBufs) & 1)) { alive = false; break; }
            }
            if (i >= S && !warp_wait(smem_u32(&b_empty[s]), epar)) { alive = false; break; }
            const uint32_t sw = (kq < 2 ? s_cur.x : s_cur.y), zw = (kq < 2 ? z_cur.x : z_cur.y);
            const float sf = (kq & 1) ? bf16hi(sw) : bf16lo(sw), zf = (kq & 1) ? bf16hi(zw) : bf16lo(zw);
            const __half2 s2 = __float2half2_rn(sf), z2 = __float2half2_rn(zf);  // bf16 values are exact in f16 range here
            const uint8_t *rawt = raw + (size_t)rb * kW4RawBytes + (size_t)r * 128;
            const uint4 codes = *reinterpret_cast<const uint4 *>(rawt + (((2 * kq + hsel) ^ (r & 7)) * 16));
            uint8_t *arow = stages + (size_t)s * stage_bytes + (size_t)r * 128;
            const uint32_t cw[4] = {codes.x, codes.y, codes.z, codes.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int cc = hsel * 4 + j;  // 16-byte chunk of the operand row = 8 inputs
                *reinterpret_cast<uint4 *>(arow + ((cc ^ (r & 7)) * 16)) = w4_word_to_f16(cw[j], z2, s2);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy stores -> tensor-core reads
            __syncwarp();  // every lane's stores are fenced (and its reads of the raw tile done): one arrival per warp
            if (lane == 0) {
                mbar_arrive(smem_u32(&b_afull[s]));
                if (kq == kW4Super - 1) mbar_arrive(smem_u32(&b_rempty[rb]));
            }
            if (++s == S) { s = 0; epar ^= 1u; }
        }
    }
    __syncwarp();
    bool ok = n_live > 0 ? mbar_wait(smem_u32(b_acc), 0, abortp, a.dev_err) : true;
    tc_fence_after();
    __syncthreads();  // all copies into and MMA reads of the pipeline memory are over: it now holds the tile
    tc_finish(epi, tile, tmem_d, tmem_cols, NP, a.splits, split, tile_idx, n_live, a.rows, ok, &s_abort, kW4Threads, wide);
}

inline size_t tc_w4_smem_bytes(int n_pad, int n_stages) {
    const size_t stage = (size_t)kTcBM * kTcBK * 2 + 2 * (size_t)n_pad * kTcBK * 2;
    return 1024 + (size_t)n_stages * stage + (size_t)kW4RawBufs * kW4RawBytes +
           sizeof(uint64_t) * (3 * n_stages + 2 * kW4RawBufs + 1) + 64;
}

}  // namespace river
