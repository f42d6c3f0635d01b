// Launches of the paged GQA decode attention kernels (a3): the TMA-fed split-KV kernel for steps of five and more rows
// and for prefill chunks, the small-step kernel for decode steps of one to four rows.
#include <algorithm>
#include <cmath>

#include "launch.h"
#include "attn_decode.cuh"
#include "attn_small.cuh"
#include "attn_prefill.cuh"

namespace river {

namespace {

template <int DH, int GQ>
cudaError_t launch_attn_split(river_ctx *c, int n, int layer0) {
    const river_config &g = c->cfg;
    AttnArgs a{};
    a.meta = c->meta(); a.q = c->qbuf; a.page_tbl = c->page_tbl_dev; a.row_slot = c->row_slot(); a.row_pos = c->row_pos();
    a.order = c->attn_order();
    a.n_pages = g.n_pages; a.max_pages_per_seq = g.max_pages_per_seq; a.Hkv = g.Hkv; a.Hq = g.Hq; a.layer0 = layer0;
    a.qscale = 1.4426950408889634f / std::sqrt((float)DH);
    a.part_o = c->part_o; a.part_ml = c->part_ml; a.tickets = c->attn_tickets; a.out = c->obuf; a.dev_err = c->dev_err;
    a.skip = c->attn_skip;
    a.pos_depth = c->attn_layer1 ? c->pos_depth : nullptr; a.depth_stride = g.max_pages_per_seq * kPage; a.layer1 = c->attn_layer1;
    a.early = (c->rows_distinct && !a.skip) ? 1 : 0;  // (the exit flags of a skipping strategy belong to this block: wait first)
    const size_t smem = attn_smem_bytes(DH, GQ);
    constexpr bool MMA = GQ <= 4;  // groups of up to four query heads: contractions on the warp-level tensor cores
    const cudaError_t e = ensure_smem(c, attn_split_kernel<DH, GQ, MMA>, smem);
    if (e != cudaSuccess) return e;
    return launch_k(attn_split_kernel<DH, GQ, MMA>, dim3(c->attn_splits_now, g.Hkv, n), dim3(attn_threads(MMA)), smem,
                    c->stream, true, c->kv_tmap, a);
}

// Steps of 1-4 rows: the split-KV kernel that fetches the cached positions before the grid dependency resolves.
template <int DH, int GQ>
cudaError_t launch_attn_small(river_ctx *c, int n, int layer0, int early) {
    const river_config &g = c->cfg;
    SmallAttnArgs a{};
    a.meta = c->meta();
    a.Hq = g.Hq; a.Hkv = g.Hkv;
    a.qscale = 1.4426950408889634f / std::sqrt((float)g.dh);
    a.qbuf = c->qbuf; a.obuf = c->obuf; a.kv = kv_addr(c, layer0);
    a.part_o = c->part_o; a.part_ml = c->part_ml; a.attn_tickets = c->attn_tickets; a.dev_err = c->dev_err;
    a.skip = c->attn_skip;
    a.pos_depth = c->attn_layer1 ? c->pos_depth : nullptr; a.depth_stride = g.max_pages_per_seq * kPage; a.layer1 = c->attn_layer1;
    if (a.skip) early = 0;  // the flags belong to this block: nothing may be fetched before the dependency resolves
    const int S = small_attn_splits(c->num_sms, n, g.Hkv);  // as the step metadata says
    const size_t smem = sizeof(float) * (size_t)kSmallAttnWarps * GQ * (DH + 2);
    const cudaError_t e = ensure_smem(c, attn_small_kernel<DH, GQ>, smem);
    if (e != cudaSuccess) return e;
    return launch_k(attn_small_kernel<DH, GQ>, dim3(n * g.Hkv * S), dim3(kSmallAttnThreads), smem, c->stream, true, a,
                    layer0, early);
}

}  // namespace

bool prefill_attn_supported(const river_ctx *c) {
    const int gq = c->cfg.Hq / c->cfg.Hkv;
    return (c->cfg.dh == 64 || c->cfg.dh == 128) && (gq == 1 || gq == 2 || gq == 4 || gq == 8);
}

namespace {
template <int DH, int GQ>
cudaError_t launch_attn_prefill_t(river_ctx *c, int n, int layer0) {
    const river_config &g = c->cfg;
    PrefillAttnArgs a{};
    a.meta = c->meta(); a.tile_row0 = c->tile_row0(); a.tile_rows = c->tile_rows();
    a.q = c->qbuf; a.out = c->obuf; a.kv = kv_addr(c, layer0); a.Hq = g.Hq;
    a.qscale = 1.4426950408889634f / std::sqrt((float)DH);
    a.dev_err = c->dev_err;
    a.skip = c->attn_skip;
    const size_t smem = attn_prefill_smem_bytes(DH);
    const cudaError_t e = ensure_smem(c, attn_prefill_kernel<DH, GQ>, smem);
    if (e != cudaSuccess) return e;
    // at most one tile per row; the kernel reads the tile count of the chunk from the step metadata
    return launch_k(attn_prefill_kernel<DH, GQ>, dim3(n, g.Hkv), dim3(32 * GQ), smem, c->stream, true, a);
}
}  // namespace

cudaError_t launch_attention_prefill(river_ctx *c, int n, int layer0) {
    const int gq = c->cfg.Hq / c->cfg.Hkv;
#define ATTP(DH_, GQ_) if (c->cfg.dh == DH_ && gq == GQ_) return launch_attn_prefill_t<DH_, GQ_>(c, n, layer0);
    ATTP(64, 1) ATTP(64, 2) ATTP(64, 4) ATTP(64, 8) ATTP(128, 1) ATTP(128, 2) ATTP(128, 4) ATTP(128, 8)
#undef ATTP
    return cudaErrorInvalidValue;
}

cudaError_t launch_attention(river_ctx *c, int n, int layer0) {
    const int gq = c->cfg.Hq / c->cfg.Hkv;
    if (c->attn_small_now) {
#define ATTS(DH_, GQ_) if (c->cfg.dh == DH_ && gq == GQ_) return launch_attn_small<DH_, GQ_>(c, n, layer0, c->rows_distinct ? 1 : 0);
        ATTS(64, 1) ATTS(64, 2) ATTS(64, 4) ATTS(64, 8) ATTS(128, 1) ATTS(128, 2) ATTS(128, 4) ATTS(128, 8)
#undef ATTS
    }
#define ATT(DH_, GQ_) if (c->cfg.dh == DH_ && gq == GQ_) return launch_attn_split<DH_, GQ_>(c, n, layer0);
    ATT(64, 1) ATT(64, 2) ATT(64, 4) ATT(64, 8) ATT(128, 1) ATT(128, 2) ATT(128, 4) ATT(128, 8)
#undef ATT
    return cudaErrorInvalidValue;
}

}  // namespace river
