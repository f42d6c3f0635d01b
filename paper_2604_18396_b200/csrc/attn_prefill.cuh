// Causal paged GQA attention for prefill chunks on the warp-level tensor cores (sm_100a, mma.sync m16n8k16 bf16).
//
// A prefill chunk holds consecutive prompt positions; as independent decode rows they would each walk their whole
// prefix on CUDA cores (cost ~ rows x context instructions).  Here a CTA owns a tile of up to 16 consecutive positions
// of one sequence and one KV head: warp g holds the 16 x DH query block of query head (kv head, g) as bf16 A fragments
// in registers - split q = hi + lo, so that the scores keep 16 mantissa bits although the tensor cores take bf16 - and
// walks the cached keys 64 at a time: K and V tiles come from the paged cache into padded shared memory with cp.async
// (double buffered, whole 16-byte pieces, bank-conflict-free for ldmatrix), S = (Q_hi + Q_lo) K^T and O += (P_hi + P_lo) V
// run as mma.sync with fp32 accumulators, the softmax is online in fp32 (base-2 exponentials, causal mask by position).
// The GQ query heads of the group share every K/V tile.  K and V are the cache's bf16 values, exactly.
#pragma once
#include "mma_sync.cuh"

namespace river {

constexpr int kPfBM = 16;       // query positions per tile
constexpr int kPfBN = 64;       // keys per shared-memory tile (four pages)
constexpr int kPfPad = 8;       // bf16 elements of padding per staged row (16 bytes: rotates the banks by four words)

struct PrefillAttnArgs {
    const StepMeta *meta;        // n_tiles
    const int32_t *tile_row0;    // first row of the chunk in the tile
    const int32_t *tile_rows;    // rows in the tile (1..16): same sequence, consecutive positions
    const float *q;              // [rows][Hq * DH] fp32
    float *out;                  // [rows][Hq * DH]
    KvAddr kv;                   // layer set by the host
    int Hq;
    float qscale;                // log2(e) / sqrt(DH)
    int *dev_err;
    const uint8_t *skip;         // a tile whose first row's flag is set does not attend (its rows have left), or null
};

__device__ __forceinline__ void pf_cp16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ float pf_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pf_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <int DH, int GQ>
__global__ void __launch_bounds__(32 * GQ) attn_prefill_kernel(const PrefillAttnArgs a) {
    constexpr int LD = DH + kPfPad;              // staged row stride in elements
    constexpr int KS = DH / 16;                  // k-steps of S = Q K^T
    constexpr int NT = kPfBN / 8;                // n-tiles (8 keys) of S per staged tile
    constexpr int DT = DH / 8;                   // n-tiles (8 dims) of O
    constexpr int NTHR = 32 * GQ;
    extern __shared__ __align__(16) unsigned char pf_smem[];
    __nv_bfloat16 *ks = reinterpret_cast<__nv_bfloat16 *>(pf_smem);   // [2][kPfBN][LD]
    __nv_bfloat16 *vs = ks + 2 * kPfBN * LD;                         // [2][kPfBN][LD]
    pdl_launch();
    pdl_wait();  // q and the chunk's own K/V come from the kernel before this one
    const int tile = blockIdx.x, kvh = blockIdx.y;
    if (tile >= a.meta->pad2[0]) return;
    const int row0 = a.tile_row0[tile], n_rows = a.tile_rows[tile];
    if (a.skip && a.skip[row0]) return;  // (the rows of a chunk leave together: prefill exits at one depth)
    const int slot = a.kv.row_slot[row0], pos0 = a.kv.row_pos[row0];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
    const int head = kvh * GQ + warp;
    const int qr = lane >> 2, qc = (lane & 3) * 2;  // fragment row and column pair of this lane

    // ---- Q block of this warp's head as A fragments, hi and lo parts (rows beyond the tile are zero)
    uint32_t qhi[KS][4], qlo[KS][4];
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int r = qr + (h & 1) * 8, c = kk * 16 + qc + (h >> 1) * 8;
            float2 v = make_float2(0.f, 0.f);
            if (r < n_rows) v = __ldcg(reinterpret_cast<const float2 *>(a.q + (size_t)(row0 + r) * a.Hq * DH + (size_t)head * DH + c));
            v.x *= a.qscale; v.y *= a.qscale;
            const __nv_bfloat16 hx = __float2bfloat16_rn(v.x), hy = __float2bfloat16_rn(v.y);
            qhi[kk][h] = (uint32_t)__bfloat16_as_ushort(hx) | ((uint32_t)__bfloat16_as_ushort(hy) << 16);
            qlo[kk][h] = pack_bf16x2(v.x - __bfloat162float(hx), v.y - __bfloat162float(hy));
        }
    }
    float o[DT][4], m[2], l[2];
#pragma unroll
    for (int d = 0; d < DT; ++d) { o[d][0] = o[d][1] = o[d][2] = o[d][3] = 0.f; }
    m[0] = m[1] = -1e30f;
    l[0] = l[1] = 0.f;

    const int last_pos = pos0 + n_rows - 1;
    const int n_kt = last_pos / kPfBN + 1;
    const int32_t *pt = a.kv.page_tbl + (size_t)slot * a.kv.max_pages_per_seq;
    // stage tile kt into buffer b: 16-byte pieces, one page (16 keys) per four rows of pieces
    auto stage = [&](int kt, int b) {
        constexpr int PIECES = kPfBN * (DH / 8);  // per matrix
        for (int i = tid; i < PIECES; i += NTHR) {
            const int key = i / (DH / 8), pc = i % (DH / 8);
            const int p = kt * kPfBN + key;
            const uint32_t dk = pf_smem_u32(ks + ((size_t)b * kPfBN + key) * LD + pc * 8);
            const uint32_t dv = pf_smem_u32(vs + ((size_t)b * kPfBN + key) * LD + pc * 8);
            if (p <= last_pos) {
                int page = pt[p / kPage];
                if (page < 0 || page >= a.kv.n_pages) {
                    atomicExch(a.dev_err, DEV_BAD_PAGE);
                    page = 0;
                }
                pf_cp16(dk, a.kv.pool + a.kv.base(page, 0, kvh, p % kPage) + pc * 8);
                pf_cp16(dv, a.kv.pool + a.kv.base(page, 1, kvh, p % kPage) + pc * 8);
            } else {  // beyond the causal range: zeros (masked anyway; keeps NaNs of unwritten cache out of P V)
                *reinterpret_cast<uint4 *>(ks + ((size_t)b * kPfBN + key) * LD + pc * 8) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4 *>(vs + ((size_t)b * kPfBN + key) * LD + pc * 8) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    stage(0, 0);
    for (int kt = 0; kt < n_kt; ++kt) {
        const int b = kt & 1;
        if (kt + 1 < n_kt) {
            stage(kt + 1, b ^ 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const __nv_bfloat16 *kb = ks + (size_t)b * kPfBN * LD, *vb = vs + (size_t)b * kPfBN * LD;
        // ---- S = (Q_hi + Q_lo) K^T for 16 query rows x 64 keys
        float s[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
            uint32_t kf[NT / 2][4];
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {  // two n-tiles (16 keys) per ldmatrix.x4
                const int key = np * 16 + (lane >> 4) * 8 + (lane & 7), dim = kk * 16 + ((lane >> 3) & 1) * 8;
                ldsm_x4(kf[np], pf_smem_u32(kb + (size_t)key * LD + dim));
            }
            // eight independent accumulators per round: no mma waits for the one issued just before it
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
                mma_bf16_m16n8k16(s[2 * np], qhi[kk], kf[np][0], kf[np][1]);
                mma_bf16_m16n8k16(s[2 * np + 1], qhi[kk], kf[np][2], kf[np][3]);
            }
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
                mma_bf16_m16n8k16(s[2 * np], qlo[kk], kf[np][0], kf[np][1]);
                mma_bf16_m16n8k16(s[2 * np + 1], qlo[kk], kf[np][2], kf[np][3]);
            }
        }
        // ---- causal mask, online softmax (rows qr and qr + 8 of the block; a quad of lanes shares a row)
        float mx[2] = {m[0], m[1]};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = kt * kPfBN + nt * 8 + qc + (e & 1), r = qr + (e >> 1) * 8;
                if (key > pos0 + r || r >= n_rows) s[nt][e] = -1e30f;
                mx[e >> 1] = fmaxf(mx[e >> 1], s[nt][e]);
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
        }
        const float corr[2] = {pf_ex2(m[0] - mx[0]), pf_ex2(m[1] - mx[1])};
        float rs[2] = {0.f, 0.f};
        uint32_t pa[NT / 2][4], pb[NT / 2][4];  // P = hi + lo as A fragments of the P V product (16 keys per k-step)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                p[e] = s[nt][e] <= -1e29f ? 0.f : pf_ex2(s[nt][e] - mx[e >> 1]);
                rs[e >> 1] += p[e];
            }
            float r[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) r[e] = p[e] - __bfloat162float(__float2bfloat16_rn(p[e]));
            pa[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16x2(p[0], p[1]);
            pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16x2(p[2], p[3]);
            pb[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16x2(r[0], r[1]);
            pb[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16x2(r[2], r[3]);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            rs[h] += __shfl_xor_sync(0xffffffffu, rs[h], 1);
            rs[h] += __shfl_xor_sync(0xffffffffu, rs[h], 2);
            l[h] = l[h] * corr[h] + rs[h];
            m[h] = mx[h];
        }
#pragma unroll
        for (int d = 0; d < DT; ++d) {
            o[d][0] *= corr[0]; o[d][1] *= corr[0];
            o[d][2] *= corr[1]; o[d][3] *= corr[1];
        }
        // ---- O += P V
#pragma unroll
        for (int j = 0; j < NT / 2; ++j) {  // 16 keys per k-step
#pragma unroll
            for (int d0 = 0; d0 < DT / 2; d0 += 4) {  // 64 dims per round: eight independent accumulators
                uint32_t vf[4][4];
#pragma unroll
                for (int dp = 0; dp < 4; ++dp) {  // two n-tiles (16 dims) per ldmatrix.x4.trans
                    const int key = j * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), dim = (d0 + dp) * 16 + (lane >> 4) * 8;
                    ldsm_x4_trans(vf[dp], pf_smem_u32(vb + (size_t)key * LD + dim));
                }
#pragma unroll
                for (int dp = 0; dp < 4; ++dp) {
                    mma_bf16_m16n8k16(o[2 * (d0 + dp)], pa[j], vf[dp][0], vf[dp][1]);
                    mma_bf16_m16n8k16(o[2 * (d0 + dp) + 1], pa[j], vf[dp][2], vf[dp][3]);
                }
#pragma unroll
                for (int dp = 0; dp < 4; ++dp) {
                    mma_bf16_m16n8k16(o[2 * (d0 + dp)], pb[j], vf[dp][0], vf[dp][1]);
                    mma_bf16_m16n8k16(o[2 * (d0 + dp) + 1], pb[j], vf[dp][2], vf[dp][3]);
                }
            }
        }
        __syncthreads();  // the buffer is free for the tile after next
    }
    // ---- write the block: rows qr and qr + 8, dims d * 8 + qc, + 1
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = qr + h * 8;
        if (r < n_rows) {
            const float inv = 1.f / l[h];
            float *dst = a.out + (size_t)(row0 + r) * a.Hq * DH + (size_t)head * DH + qc;
#pragma unroll
            for (int d = 0; d < DT; ++d)
                *reinterpret_cast<float2 *>(dst + d * 8) = make_float2(o[d][2 * h] * inv, o[d][2 * h + 1] * inv);
        }
    }
}

inline size_t attn_prefill_smem_bytes(int DH) { return (size_t)4 * kPfBN * (DH + kPfPad) * sizeof(__nv_bfloat16); }

}  // namespace river
