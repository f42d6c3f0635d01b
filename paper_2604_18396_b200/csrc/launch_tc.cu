// Launches of the tensor-core projection kernel for backbone rows (5 <= rows <= 256) and its operand kernel.
#include <algorithm>

#include "launch_tc.h"
#include "tensor_maps.h"

namespace river {

const river_ctx::BMap *tc_bmap(river_ctx *c, int K, int np, bool w4, bool alt) {
    for (auto &b : c->tc_bmaps)
        if (b.K == K && b.np == np && b.w4 == w4 && b.alt == alt) return &b;
    river_ctx::BMap b{K, np, w4, alt, 2 * np <= 256, nullptr, nullptr, {}, {}};
    __nv_bfloat16 *base = alt ? (w4 ? c->tc_x4alt : c->tc_xalt) : (w4 ? c->tc_x4 : c->tc_xhi);
    b.base = base;
    b.lo_ptr = b.one ? base + (size_t)np * K : base + (size_t)c->tc_max_pad * c->tc_kmax;
    const int hi_rows = b.one ? 2 * np : np;  // a box holds at most 256 rows
    if (!make_map_bf16(&b.hi, base, K, hi_rows, hi_rows) || !make_map_bf16(&b.lo, b.lo_ptr, K, np, np)) return nullptr;
    c->tc_bmaps.push_back(b);
    return &c->tc_bmaps.back();
}

// K-splits per tile: fill whole waves of the CTA slots, keep at least four 64-wide k-blocks per split; no split at
// all when there is a tile for every SM.  The kernel is memory-bound, so what matters is that all CTAs are resident
// together and every SM slot streams.
int tc_pick_splits(const river_ctx *c, int tiles, int kb_total, int slots, int min_kb) {
    int best = 1;
    double best_eff = 0.0;
    if (tiles >= c->num_sms) return 1;  // every SM has a tile of its own: splitting only adds reductions
    for (int s = 1; s <= 8; ++s) {  // a cluster holds at most 8 CTAs
        if (s > 1 && kb_total / s < min_kb) break;
        const int ctas = tiles * s, waves = (ctas + slots - 1) / slots;
        const double eff = (double)ctas / ((double)waves * slots);
        if (eff > best_eff + 0.02) { best_eff = eff; best = s; }
    }
    return best;
}

namespace {

constexpr size_t kSmSmem = 228 * 1024;
constexpr size_t kCtaFixed = 1024 + 1024 + 256;  // per CTA: system reserve, alignment slack, barriers

size_t tc_stage_bytes(int np) { return (size_t)kTcBM * kTcBK * 2 + 2 * (size_t)np * kTcBK * 2; }
// pipeline stages with `occ` CTAs per SM (0: they do not fit)
int tc_stages_at(int np, int occ) {
    const size_t stage = tc_stage_bytes(np), room = std::min<size_t>(kSmSmem / occ, 227 * 1024);
    return room < kCtaFixed + 2 * stage ? 0 : (int)std::min<size_t>(occ == 1 ? 8 : occ == 2 ? 4 : 3, (room - kCtaFixed) / stage);
}
// hi | lo as one operand doubles the accumulator columns; all CTAs that can be resident on an SM must get their
// tensor memory at once (a CTA stuck in the allocation while its cluster waits for it could not be waited out)
int tc_cols(int np, int occ, int *wide) {
    int cols = 32;
    while (cols < 2 * np) cols <<= 1;
    *wide = (2 * np <= 256 && occ * cols <= 512) ? 1 : 0;
    if (!*wide) { cols = 32; while (cols < np) cols <<= 1; }
    return cols;
}

}  // namespace

int tc_footprints(int np, TcFootprint (&out)[2]) {
    int n = 0;
    for (int occ = tc_stages_at(np, 2) ? 2 : 1; occ <= 3; ++occ) {
        const int st = tc_stages_at(np, occ);
        if (!st) break;
        int wide;
        out[n].cols = tc_cols(np, occ, &wide);
        out[n].smem = tc_smem_bytes(np, st);
        if (++n == 2 || occ == 1) break;
    }
    return n;
}

template <class Epi>
cudaError_t launch_tc(river_ctx *c, const ProjIn &in, const CUtensorMap &a0, const CUtensorMap &a1, const CUtensorMap &a2,
                      int K, int tiles, int n, int gateup, int q_tiles, int k_tiles, const int32_t *rows,
                      const int32_t *cnt, const Epi &epi, bool allow_split, const int32_t *hint, int phase,
                      bool late_release, bool alt_operand) {
    const int np = (n + 15) / 16 * 16;
    const river_ctx::BMap *bm = tc_bmap(c, K, np, false, alt_operand);
    if (alt_operand) phase &= ~kTcPrep;  // the operand rows are there already (the previous projection's epilogues)
    if (!bm) return cudaErrorInvalidValue;
    cudaError_t e = cudaSuccess;
    if (phase & kTcPrep) {
        e = launch_k(tc_prep_kernel, dim3(np, (K + kPrepChunk - 1) / kPrepChunk), dim3(256), 0, c->stream, true, in, rows, cnt, K,
                     c->tc_xhi, bm->lo_ptr);
        if (e != cudaSuccess) return e;
        ++c->st.launches_last_step;
    }
    if (!(phase & kTcGemm)) return e;
    TcArgs a{};
    a.K = K; a.n_pad = np; a.one_box = bm->one ? 1 : 0; a.late_release = late_release ? 1 : 0;
    const size_t stage = tc_stage_bytes(np);
    // CTAs per SM: two with three stages each, or three with two when that puts more CTAs of one wave to work (while
    // one CTA drains its accumulator and takes part in the cluster reduction the others keep the weight stream going);
    // one with deep stages when the operand tiles are too large for that.
    int occ = tc_stages_at(np, 2) ? 2 : 1;
    a.splits = tc_pick_splits(c, tiles, K / kTcBK, c->num_sms * occ);
    if (occ == 2 && tc_stages_at(np, 3) && allow_split) {
        const int s3 = tc_pick_splits(c, tiles, K / kTcBK, c->num_sms * 3);
        if (tiles * s3 > tiles * a.splits && tiles * s3 <= c->num_sms * 3) { occ = 3; a.splits = s3; }
    }
    a.n_stages = tc_stages_at(np, occ);
    tc_cols(np, occ, &a.wide);
    // the finished tile lives in the pipeline memory
    if (sizeof(float) * (size_t)np * kTcLd > (size_t)a.n_stages * stage) return cudaErrorInvalidValue;
    if (!allow_split) a.splits = 1;
    a.gateup = gateup; a.qkv_q_tiles = q_tiles; a.qkv_k_tiles = k_tiles;
    a.rows = rows; a.cnt = cnt; a.dev_err = c->dev_err;
    a.hint = hint ? hint : cnt;
    const size_t smem = tc_smem_bytes(np, a.n_stages);
    e = ensure_smem(c, tc_gemm_kernel<Epi>, smem);
    if (e != cudaSuccess) return e;
    return launch_kc(tc_gemm_kernel<Epi>, dim3(tiles * a.splits), dim3(kTcThreads), smem, c->stream, true, a.splits, a0,
                     a1, a2, bm->hi, bm->lo, a, epi);
}
#define RIVER_TC_INST(E) \
    template cudaError_t launch_tc<E>(river_ctx *, const ProjIn &, const CUtensorMap &, const CUtensorMap &, const CUtensorMap &, \
                                      int, int, int, int, int, int, const int32_t *, const int32_t *, const E &, bool, const int32_t *, \
                                      int, bool, bool);
RIVER_TC_INST(TcQkvEpi) RIVER_TC_INST(TcResidEpi) RIVER_TC_INST(TcGateUpEpi) RIVER_TC_INST(TcHeadEpi)
#undef RIVER_TC_INST

}  // namespace river
