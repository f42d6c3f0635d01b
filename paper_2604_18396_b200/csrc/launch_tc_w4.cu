// Launches of the dequantising tensor-core kernel for exit-layer rows (5 <= rows <= 256) and its operand kernel.
#include <algorithm>

#include "launch_tc.h"
#include "gemm_tc_w4.cuh"

namespace river {

cudaError_t launch_tc_prep_pair(river_ctx *c, const ProjIn &in, int K, int n, const int32_t *rows_a, const int32_t *cnt_a,
                                const int32_t *rows_r, const int32_t *cnt_r) {
    const int np = (n + 15) / 16 * 16;
    const river_ctx::BMap *ba = tc_bmap(c, K, np, false);
    if (!ba) return cudaErrorInvalidValue;
    __nv_bfloat16 *alo = ba->lo_ptr;  // (the next call may move the map table)
    const river_ctx::BMap *br = tc_bmap(c, K, np, true);
    if (!br) return cudaErrorInvalidValue;
    PrepPair p{rows_a, cnt_a, rows_r, cnt_r, c->tc_xhi, alo, reinterpret_cast<__half *>(c->tc_x4),
               reinterpret_cast<__half *>(br->lo_ptr), (K + kPrepChunk - 1) / kPrepChunk};
    const int yr = (K + 2 * kPrepChunk - 1) / (2 * kPrepChunk);
    ++c->st.launches_last_step;
    return launch_k(tc_prep_pair_kernel, dim3(np, p.ya + yr), dim3(256), 0, c->stream, true, in, p, K);
}

template <class Epi>
cudaError_t launch_tc_w4(river_ctx *c, const ProjIn &in, const CUtensorMap *const (&m)[3], const river_w4 *const (&w)[3],
                         int K, int tiles, int n, int gateup, int q_tiles, int k_tiles, const int32_t *rows,
                         const int32_t *cnt, const int32_t *hint, const Epi &epi, int phase, bool overlap, bool alt_operand) {
    const int np = (n + 15) / 16 * 16;
    const river_ctx::BMap *bm = tc_bmap(c, K, np, true, alt_operand);
    if (alt_operand) phase &= ~kTcPrep;  // the operand rows are there already (the previous projection's epilogues)
    if (!bm) return cudaErrorInvalidValue;
    cudaError_t e = cudaSuccess;
    if (phase & kTcPrep) {
        e = launch_k(tc_prep_w4_kernel, dim3(np, (K + 2 * kPrepChunk - 1) / (2 * kPrepChunk)), dim3(256), 0, c->stream, true, in,
                     rows, cnt, K, reinterpret_cast<__half *>(c->tc_x4), reinterpret_cast<__half *>(bm->lo_ptr));
        if (e != cudaSuccess) return e;
        ++c->st.launches_last_step;
    }
    if (!(phase & kTcGemm)) return e;
    TcW4Args a{};
    a.K = K; a.n_pad = np; a.one_box = bm->one ? 1 : 0;
    const size_t stage = 2 * (size_t)np * kTcBK * 2;  // the activations' hi and lo tiles; the A tiles are in tensor memory
    const size_t raw = (size_t)kW4RawBufs * kW4RawBytes;
    // two CTAs per SM (16 dequantisation warps) when two stages fit in half of the shared memory; an even number of
    // stages (the two dequantisation warps of a lane quarter alternate)
    const bool two = 2 * stage + raw + 4096 <= 110 * 1024;
    a.n_stages = two ? (int)std::min<size_t>(4, (110 * 1024 - raw - 4096) / stage)
                     : (int)std::max<size_t>(2, std::min<size_t>(4, (214 * 1024 - raw) / stage));
    a.n_stages &= ~1;
    // in raw tiles of four k-blocks: at least four per split, two when K is so short that four would allow only two
    // splits (measured on the 1B shape, K = 2048: 2 -> 4 splits 35 -> 31 us per layer for QKV, 33 -> 27 us for O)
    const int raw_tiles = K / (kTcBK * kW4Super);
    a.splits = tc_pick_splits(c, tiles, raw_tiles, c->num_sms * (two ? 2 : 1), raw_tiles <= 8 ? 2 : 4);
    if (sizeof(float) * (size_t)np * kTcLd > (size_t)a.n_stages * stage + raw) return cudaErrorInvalidValue;
    // tensor memory: accumulator + A tiles, a power of two of columns; every CTA that can be resident on an SM must get
    // its columns at once (a CTA stuck in the allocation while its cluster waits for it could not be waited out), so
    // the shared-memory request is padded until no more than `occ` CTAs fit
    const int occ = two ? 2 : 1;
    auto cols_for = [&](int acc) { int cols = 32; while (cols < acc + a.n_stages * (int)kW4ACols) cols <<= 1; return cols; };
    a.wide = (2 * np <= 256 && occ * cols_for(2 * np) <= 512) ? 1 : 0;
    const int cols = cols_for(a.wide ? 2 * np : np);
    if (occ * cols > 512) return cudaErrorInvalidValue;
    const size_t sm_smem = 228 * 1024;
    size_t smem = std::max(tc_w4_smem_bytes(np, a.n_stages), sm_smem / (occ + 1) + 1024);
    // CTAs of tc_gemm_kernel share the SMs with this kernel (beside it when `overlap`, and the next projection's may
    // take their tensor memory while CTAs of this grid are still to come): whatever mix of the two fits into an SM's
    // shared memory must fit into its 512 columns as well - pad the request until it does
    TcFootprint fp[2];
    const int nfp = tc_footprints(np, fp);
    auto mix_ok = [&](size_t mine) {
        for (int f = 0; f < nfp; ++f)
            for (int i = 0; i <= 8; ++i)
                for (int j = 0; j <= occ; ++j)
                    if (i * fp[f].smem + j * mine <= sm_smem && i * fp[f].cols + j * cols > 512) return false;
        return true;
    };
    while (!mix_ok(smem) && smem + 4096 <= sm_smem / occ - 1024) smem += 4096;
    if (!mix_ok(smem)) return cudaErrorInvalidValue;
    a.overlap = overlap ? 1 : 0;
    a.gateup = gateup; a.qkv_q_tiles = q_tiles; a.qkv_k_tiles = k_tiles;
    for (int i = 0; i < 3; ++i) { a.scale[i] = (const uint16_t *)w[i]->scale; a.zero[i] = (const uint16_t *)w[i]->zero; }
    a.rows = rows; a.cnt = cnt; a.hint = hint; a.dev_err = c->dev_err;
    e = ensure_smem(c, tc_gemm_w4_kernel<Epi>, smem);
    if (e != cudaSuccess) return e;
    return launch_kc(tc_gemm_w4_kernel<Epi>, dim3(tiles * a.splits), dim3(kW4Threads), smem, c->stream, true, a.splits,
                     *m[0], *m[1], *m[2], bm->hi, bm->lo, a, epi);
}
#define RIVER_TCW4_INST(E) \
    template cudaError_t launch_tc_w4<E>(river_ctx *, const ProjIn &, const CUtensorMap *const (&)[3], const river_w4 *const (&)[3], \
                                         int, int, int, int, int, int, const int32_t *, const int32_t *, const int32_t *, const E &, \
                                         int, bool, bool);
RIVER_TCW4_INST(TcQkvEpi) RIVER_TCW4_INST(TcResidEpi) RIVER_TCW4_INST(TcGateUpEpi)
#undef RIVER_TCW4_INST

}  // namespace river
