// Host side of the C ABI declared in include/river.h: argument checks, the KV page table, the per-step
// metadata upload and the kernel launch sequence of one early-exit decode step.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "river_ctx.h"
#include "launch.h"
#include "launch_tc.h"
#include "tensor_maps.h"
#include "river_kernels.cuh"
#include "attn_decode.cuh"
#include "attn_small.cuh"
#include "attn_prefill.cuh"

using namespace river;

namespace {

thread_local std::string g_init_error;

const char *const kClassNames[kNumClasses] = {"step_begin", "qkv_rope_kv", "attn_decode", "o_proj_resid", "gateup_swiglu",
                                              "down_resid", "exit_score", "lm_head", "argmax_final", "prefill_attn"};

struct Carver {
    char *base;
    size_t off = 0;
    template <class T>
    T *take(size_t n) {
        off = (off + 255) & ~(size_t)255;
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

}  // namespace

namespace {

int fail(river_ctx *c, int code, const std::string &msg) {
    if (c) c->err = msg;
    else g_init_error = msg;
    return code;
}

#define CUDA_TRY(ctx, expr)                                                                             \
    do {                                                                                                \
        cudaError_t e_ = (expr);                                                                        \
        if (e_ != cudaSuccess)                                                                          \
            return fail(ctx, RIVER_E_DEVICE, std::string(#expr) + ": " + cudaGetErrorString(e_));       \
    } while (0)

const char *check_config(const river_config *c) {
    if (!c) return "null config";
    if (c->L <= 0 || c->d <= 0 || c->Hq <= 0 || c->Hkv <= 0 || c->F <= 0 || c->V <= 0) return "non-positive dimension";
    if (c->Hq % c->Hkv) return "Hq must be a multiple of Hkv";
    const int gq = c->Hq / c->Hkv;
    if (!(gq == 1 || gq == 2 || gq == 4 || gq == 8)) return "GQA group must be 1, 2, 4 or 8";
    if (!(c->dh == 64 || c->dh == 128)) return "head dim must be 64 or 128";
    if (!(c->group == 32 || c->group == 64 || c->group == 128)) return "quantisation group must be 32, 64 or 128";
    if (c->d % c->group || c->F % c->group || (c->Hq * c->dh) % c->group) return "input dims must be multiples of group";
    if (c->d % 32 || c->F % 32 || c->V % 4 || c->d % 4) return "d, F must be multiples of 32 and V of 4";
    if (c->page_size != kPage) return "page_size must be 16";
    if (c->entry_layer < 0 || c->entry_layer >= c->L) return "entry_layer out of range";
    if (c->max_batch <= 0 || c->max_batch > kMaxBatch) return "max_batch out of range";
    if (c->prefill_chunk < 0 || c->prefill_chunk > 256) return "prefill_chunk out of range (0 .. 256)";
    if (c->max_seqs <= 0 || c->max_pages_per_seq <= 0 || c->n_pages <= 0) return "bad cache geometry";
    if (!(c->exit_mode == RIVER_EXIT_PER_TOKEN || c->exit_mode == RIVER_EXIT_BATCH_MIN)) return "bad exit_mode";
    if (c->kv_strategy < RIVER_KV_RIVER || c->kv_strategy > RIVER_KV_MASK) return "bad kv_strategy";
    if (c->kv_strategy == RIVER_KV_MASK && (c->Hq / c->Hkv > 4 || c->L > 255))
        return "KV Mask needs groups of at most four query heads per KV head";
    return nullptr;
}

int head_grid_for(const river_config *c) { return 148 * 2 > c->V / 4 ? std::max(1, c->V / 4) : 148 * 2; }
int head_parts_for(const river_config *c) { return std::max(head_grid_for(c), c->V / 128 + 1); }  // argmax partials per row

// Row-indexed buffers are sized for the larger of a decode step and a prefill chunk; the logits staging only for the
// rows that can need logits at once (a decode step's rows, or as many prompt ends in a chunk).
river_config effective(const river_config *cfg, int *user_max_batch) {
    river_config e = *cfg;
    if (user_max_batch) *user_max_batch = cfg->max_batch;
    e.max_batch = std::max(cfg->max_batch, cfg->prefill_chunk);
    return e;
}

size_t carve(const river_config *c, river_ctx *x, char *base, int head_rows) {
    Carver cv{base};
    const size_t B = c->max_batch, d = c->d, L = c->L;
    float *h0 = cv.take<float>(B * d), *h1 = cv.take<float>(B * d), *h2 = cv.take<float>(B * d);
    float *qb = cv.take<float>(B * c->Hq * c->dh), *ob = cv.take<float>(B * c->Hq * c->dh);
    float *act = cv.take<float>(B * c->F);
    float *pv = cv.take<float>(B * (size_t)head_parts_for(c));
    int32_t *pi = cv.take<int32_t>(B * (size_t)head_parts_for(c));
    float *tau = cv.take<float>(B);
    float *lg = cv.take<float>((size_t)head_rows * (size_t)c->V);
    float *sc = cv.take<float>(B * L);
    float2 *cs = cv.take<float2>(B * (c->dh / 2));
    double *fr = cv.take<double>(c->dh / 2);
    int32_t *ai = cv.take<int32_t>((L + 1) * B), *ri = cv.take<int32_t>((L + 1) * B);
    int32_t *na = cv.take<int32_t>(L + 1), *nr = cv.take<int32_t>(L + 1);
    int32_t *pt = cv.take<int32_t>((size_t)c->max_seqs * c->max_pages_per_seq);
    int32_t *tk = cv.take<int32_t>(B), *fo = cv.take<int32_t>(B), *ex = cv.take<int32_t>(B), *nx = cv.take<int32_t>(B);
    int32_t *md = cv.take<int32_t>(kMetaHdr + 11 * B);
    int32_t *pff = cv.take<int32_t>((size_t)c->max_seqs * (L + 1));
    float *po = cv.take<float>((B + 600) * (size_t)c->Hq * c->dh);
    float2 *pml = cv.take<float2>((B + 600) * (size_t)c->Hq);
    const size_t sstride = (B + 15) / 16 * 16;
    uint8_t *exd = cv.take<uint8_t>((L + 1) * sstride), *ps = cv.take<uint8_t>(B);
    int *de = cv.take<int>(1);
    unsigned *atk = cv.take<unsigned>(B * (size_t)c->Hkv), *tk4 = cv.take<unsigned>(4);
    int32_t *hint = md ? md + 5 : nullptr;  // StepMeta::hint_act
    int32_t *scap = cv.take<int32_t>((size_t)c->max_seqs);
    uint8_t *pdep = cv.take<uint8_t>((size_t)c->max_seqs * c->max_pages_per_seq * kPage);
    unsigned long long *ehist = cv.take<unsigned long long>((size_t)c->L + 1);
    const size_t tc_pad = std::min<size_t>(256, (B + 15) / 16 * 16);
    const size_t tc_kmax = std::max<size_t>(std::max<size_t>(c->d, c->F), (size_t)c->Hq * c->dh);
    // one allocation: lo rows may start right behind the hi rows in use (launch_tc.cu: tc_bmap)
    __nv_bfloat16 *txh = cv.take<__nv_bfloat16>(2 * tc_pad * tc_kmax), *txl = txh ? txh + tc_pad * tc_kmax : nullptr;
    __nv_bfloat16 *tx4 = cv.take<__nv_bfloat16>(2 * tc_pad * tc_kmax);
    __nv_bfloat16 *txa = cv.take<__nv_bfloat16>(2 * tc_pad * tc_kmax), *tx4a = cv.take<__nv_bfloat16>(2 * tc_pad * tc_kmax);

    if (x) {
        x->h[0] = h0; x->h[1] = h1; x->h[2] = h2; x->qbuf = qb; x->obuf = ob; x->act = act;
        x->part_val = pv; x->part_idx = pi; x->tau_i = tau; x->logits_i = lg; x->scores_i = sc; x->rope_cs = cs;
        x->inv_freq = fr; x->act_idx = ai; x->riv_idx = ri; x->n_act = na; x->n_riv = nr; x->page_tbl_dev = pt;
        x->tok_i = tk; x->forced_i = fo; x->exit_i = ex; x->next_i = nx; x->meta_dev = md; x->state = exd; x->state_stride = (int)sstride; x->prefill_fail = pff;
        x->pass = ps; x->dev_err = de; x->part_o = po; x->part_ml = pml; x->attn_tickets = atk; x->tickets = tk4; x->hint_act = hint;
        x->slot_cap = scap; x->pos_depth = pdep; x->exit_hist = ehist;
        x->tc_xhi = txh; x->tc_xlo = txl; x->tc_x4 = tx4; x->tc_xalt = txa; x->tc_x4alt = tx4a; x->tc_max_pad = (int)tc_pad; x->tc_kmax = (int)tc_kmax;
    }
    return (cv.off + 255) & ~(size_t)255;
}

// KV split geometry of this step.  A (row, kv head, split) item costs its positions plus a fixed start and end worth
// about four 64-position tiles, and splitting at all adds the merge through global memory (about five tiles' time,
// once); items are handed to the CTA slots in launch order, rows longest first.  One wave of items lasts as long as its
// longest item; more waves last about (all positions / slots) + a quarter of the longest item (what a slot still
// holds when the others run dry), and with rows of equal length no less than whole waves of the mean item; every slot
// pays the fixed part once per item (constants fitted to measurements at 16, 64 and 128 rows with equal and with mixed
// lengths).  The split count that minimises this estimate is taken from a short list - one split when the rows are
// equally long and outnumber the slots, a few when the lengths are mixed, and with few rows enough to fill three
// quarters of the slots.  Splits are whole tiles, at least two.  The split count is part of a captured launch's key;
// the chunk length lives in the step metadata.
void set_attn_meta(river_ctx *c, int32_t *mh, int n) {
    const river_config &g = c->cfg;
    int max_pos = 0;
    double total = 0.0;
    for (int i = 0; i < n; ++i) {
        const int pos = mh[kMetaHdr + g.max_batch + i];
        max_pos = std::max(max_pos, pos);
        total += pos + 1;
    }
    // three CTAs of the attention kernel fit per SM (registers; shared memory at head dim 128)
    const double slots = 3.0 * c->num_sms, ovh = 250.0 * 128.0 / g.dh, merge = 350.0 * 128.0 / g.dh;
    const bool uniform = (max_pos + 1) <= 1.3 * total / n;  // whole waves of equal items bound the time only then
    const int s_cap = std::max(1, std::min(64, (g.max_batch + 600) / n));  // the partials hold max_batch + 600 (row, split) slots
    static const int cand[] = {1, 2, 3, 4, 5, 6, 8, 12, 16, 24, 32, 48, 64};
    int S = 1, chunk = 0;
    double best = 0.0;
    // fewer items than slots: at least fill three quarters of them (three CTAs share an SM: one wave that leaves some
    // slots empty beats a second, nearly empty wave)
    const int s_lo = std::max(1, std::min(s_cap, (int)std::ceil(0.75 * slots / (n * g.Hkv))));
    for (int k = -1; k < (int)(sizeof(cand) / sizeof(cand[0])); ++k) {
        const int s = k < 0 ? s_lo : cand[k];
        if (k >= 0 && (s <= s_lo || s > s_cap)) continue;
        int ch = (max_pos + 1 + s - 1) / s;
        ch = std::max(2 * kAttnTile, (ch + kAttnTile - 1) / kAttnTile * kAttnTile);
        double items = 0.0;
        for (int i = 0; i < n; ++i) items += (mh[kMetaHdr + g.max_batch + i] + ch) / ch;  // ceil((pos + 1) / ch)
        items *= g.Hkv;
        const int longest = std::min(ch, max_pos + 1);
        // whole waves of items of the mean length bound it from below as well (equal lengths: 1.3 waves cost 2)
        const double waves = std::ceil(items / slots), mean_item = total * g.Hkv / items;
        // one wave: the longest item; more: the slots' mean load plus a tail (the rows enter longest first, so what a
        // slot still holds at the end is a fraction of an item)
        const double body = items <= slots ? (double)longest
                                           : std::max(std::max(total * g.Hkv / slots + 0.25 * longest, uniform ? waves * mean_item : 0.0),
                                                      (double)longest);
        const double t = body + ovh * std::max(1.0, items / slots) + (s > 1 ? merge : 0.0);
        if (chunk == 0 || t < best * 0.97) { best = t; S = s; chunk = ch; }
        if (ch == 2 * kAttnTile) break;  // finer splits do not exist
    }
    mh[3] = chunk;
    mh[4] = S;
    mh[5] = n;  // hint_act: every row starts in the backbone
    // the attention grid takes its rows longest context first: CTA slots are handed out in launch order, and a long
    // item that starts last is what the step ends on
    int32_t *order = mh + kMetaHdr + 10 * g.max_batch;
    for (int i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order, order + n, [&](int32_t x, int32_t y) {
        return mh[kMetaHdr + g.max_batch + x] > mh[kMetaHdr + g.max_batch + y];
    });
    // the small-step kernel: one CTA per (row, kv head, split), chunks in whole pages
    const int Sc = small_attn_splits(c->num_sms, n, g.Hkv);
    int cchunk = (max_pos + 1 + Sc - 1) / Sc;
    cchunk = std::max(kPage, (cchunk + kPage - 1) / kPage * kPage);
    mh[6] = cchunk;  // StepMeta::pad[0]
    mh[7] = Sc;      // StepMeta::pad[1]
    // the small-step kernel walks a split in batches of 4 positions per warp without a load pipeline, but requests the
    // cache before the grid dependency resolves: in the replayed step it wins up to four batches per warp (contexts up
    // to ~4.6 K at one row: 3.84 -> 3.49 ms per step at 4 K), beyond that the TMA-fed kernel's staging pays
    c->attn_small_now = n <= 4 && cchunk <= 4 * 4 * kSmallAttnWarps && !(g.flags & RIVER_F_TMA_ATTN);
    c->attn_splits_now = S;
}

void set_io_meta(int32_t *mh, const int32_t *tok, const float *tau, const int32_t *forced, float *logits,
                 int32_t *next_tok, int32_t *exit_layer, float *scores) {
    StepMeta *m = reinterpret_cast<StepMeta *>(mh);
    m->tok = tok; m->tau = tau; m->forced = forced; m->logits = logits; m->next_tok = next_tok;
    m->exit_layer = exit_layer; m->scores = scores;
}

// ---- tensor maps of the weights for the tensor-core projections
// The shapes the tensor-core path takes: every output dimension in whole 128-feature tiles.
bool tc_shape_ok(const river_config &g) {
    return g.d % 128 == 0 && (g.Hq * g.dh) % 128 == 0 && (g.Hkv * g.dh) % 128 == 0 && g.F % 64 == 0 && g.V % 128 == 0 &&
           g.d % 64 == 0 && g.F % 64 == 0 && (g.Hq * g.dh) % 64 == 0;
}
bool make_tc_maps(river_ctx *c) {
    const river_config &g = c->cfg;
    const int qdim = g.Hq * g.dh, kvdim = g.Hkv * g.dh;
    c->tc_maps.resize(g.L);
    for (int l = 0; l < g.L; ++l) {
        const river_layer_weights &w = c->layers[l];
        river_ctx::LayerMaps &m = c->tc_maps[l];
        if (!make_map_bf16(&m.q, w.wq, g.d, qdim, 128) || !make_map_bf16(&m.k, w.wk, g.d, kvdim, 128) ||
            !make_map_bf16(&m.v, w.wv, g.d, kvdim, 128) || !make_map_bf16(&m.o, w.wo, qdim, g.d, 128) ||
            !make_map_bf16(&m.g, w.wg, g.d, g.F, 64) || !make_map_bf16(&m.u, w.wu, g.d, g.F, 64) ||
            !make_map_bf16(&m.d, w.wd, g.F, g.d, 128))
            return false;
    }
    return make_map_bf16(&c->tc_map_head, c->lm_head, g.d, g.V, 128);
}
// The exit layers' code matrices for the dequantising tensor-core kernel: one scale / zero per row and 64-input
// k-block, raw tiles of 256 inputs.
bool make_w4_maps(river_ctx *c) {
    const river_config &g = c->cfg;
    const int qdim = g.Hq * g.dh, kvdim = g.Hkv * g.dh;
    if (g.group != 64 || g.d % 256 || g.F % 256 || qdim % 256) return false;
    c->w4_maps.resize(g.L);
    for (int l = 0; l < g.L; ++l) {
        const river_layer_weights &w = c->layers[l];
        if (!w.rq.codes) continue;
        river_ctx::LayerMaps &m = c->w4_maps[l];
        if (!make_map_codes(&m.q, w.rq.codes, g.d / 2, qdim, 128) || !make_map_codes(&m.k, w.rk.codes, g.d / 2, kvdim, 128) ||
            !make_map_codes(&m.v, w.rv.codes, g.d / 2, kvdim, 128) || !make_map_codes(&m.o, w.ro.codes, qdim / 2, g.d, 128) ||
            !make_map_codes(&m.g, w.rg.codes, g.d / 2, g.F, 64) || !make_map_codes(&m.u, w.ru.codes, g.d / 2, g.F, 64) ||
            !make_map_codes(&m.d, w.rd.codes, g.F / 2, g.d, 128))
            return false;
    }
    return true;
}

// 2-D tiled tensor map over the KV pool seen as [all cache rows][dh] bf16, box = 16 rows x 64 elements (128 bytes),
// 128-byte swizzle: one box is the K (or V) of one page, one kv head, one half of the head dim.
int make_kv_tensor_map(river_ctx *c) {
    const river_config &g = c->cfg;
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn)
        return fail(nullptr, RIVER_E_DEVICE, "cuTensorMapEncodeTiled is not available");
    const cuuint64_t rows = (cuuint64_t)g.L * g.n_pages * 2 * g.Hkv * kPage;
    if (rows >= (1ull << 31)) return fail(nullptr, RIVER_E_SHAPE, "KV pool has too many cache rows for one tensor map");
    const cuuint64_t gdim[2] = {(cuuint64_t)g.dh, rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)g.dh * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kPage};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = ((EncodeFn)fn)(&c->kv_tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c->pool, gdim, gstride, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(nullptr, RIVER_E_DEVICE, "cuTensorMapEncodeTiled failed: " + std::to_string((int)r));
    return 0;
}

// Allocate the page that position `pos` of `slot` falls in, if it has none yet; queue the device update.
int ensure_page(river_ctx *c, int slot, int pos, int32_t *mh, int &n_upd) {
    const river_config &g = c->cfg;
    const int pi = pos / kPage;
    if (pi >= g.max_pages_per_seq) return fail(c, RIVER_E_NOPAGE, "sequence exceeds max_pages_per_seq");
    int32_t &e = c->page_tbl[(size_t)slot * g.max_pages_per_seq + pi];
    if (e >= 0) return 0;
    if (c->free_pages.empty()) return fail(c, RIVER_E_NOPAGE, "KV pool exhausted");
    if (n_upd >= g.max_batch) return fail(c, RIVER_E_NOPAGE, "too many new pages in one step");
    e = c->free_pages.back();
    c->free_pages.pop_back();
    int32_t *u = mh + kMetaHdr + 2 * g.max_batch;
    u[n_upd] = slot;
    u[g.max_batch + n_upd] = pi;
    u[2 * g.max_batch + n_upd] = e;
    ++n_upd;
    return 0;
}

int32_t *next_meta(river_ctx *c) {
    const int i = c->meta_next;
    c->meta_next = (i + 1) % kStaging;
    cudaEventSynchronize(c->meta_ev[i]);
    return c->meta_host[i];
}

int push_meta(river_ctx *c, int32_t *mh) {
    const int i = (int)((c->meta_next + kStaging - 1) % kStaging);
    CUDA_TRY(c, cudaMemcpyAsync(c->meta_dev, mh, sizeof(int32_t) * c->meta_ints(), cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaEventRecord(c->meta_ev[i], c->stream));
    return 0;
}

// Per-kernel timing support: an event before and after every launch while profiling is on.
struct LaunchScope {
    river_ctx *c;
    int idx = -1;
    LaunchScope(river_ctx *c_, int cls, double bytes_act, double bytes_riv, int list_idx) : c(c_) {
        ++c->st.launches_last_step;
        if (!c->profiling) return;
        idx = (int)c->prof_rec.size();
        if ((size_t)(2 * idx + 1) >= c->prof_ev.size()) { idx = -1; return; }
        c->prof_rec.push_back({cls, bytes_act, bytes_riv, list_idx});
        cudaEventRecord(c->prof_ev[2 * idx], c->stream);
    }
    ~LaunchScope() {
        if (idx >= 0) cudaEventRecord(c->prof_ev[2 * idx + 1], c->stream);
    }
};

int profile_collect(river_ctx *c) {
    const river_config &g = c->cfg;
    const int L = g.L;
    std::vector<int32_t> na(L + 1), nr(L + 1);
    CUDA_TRY(c, cudaMemcpyAsync(na.data(), c->n_act, sizeof(int32_t) * (L + 1), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(nr.data(), c->n_riv, sizeof(int32_t) * (L + 1), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (size_t i = 0; i < c->prof_rec.size(); ++i) {
        const auto &r = c->prof_rec[i];
        float ms = 0.f;
        CUDA_TRY(c, cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]));
        c->prof_ms[r.cls] += ms;
        c->prof_launches[r.cls] += 1;
        double bytes = 0.0;
        if (r.list_idx < 0) bytes = r.bytes_act;
        else bytes = (na[r.list_idx] > 0 ? r.bytes_act : 0.0) + (nr[r.list_idx] > 0 ? r.bytes_riv : 0.0);
        c->prof_bytes[r.cls] += bytes;
    }
    c->prof_rec.clear();
    return 0;
}

// ---- backbone offloading (Section 4.2, "Backbone Offloading")
// Stage block l's seven bf16 matrices from pinned host memory into the device slot its layer entry points at, unless
// the slot already holds them; the copy runs on its own stream, after the kernels that last used the slot.
int offload_fetch(river_ctx *c, int l) {
    const river_config &g = c->cfg;
    const int slot = (l - c->off_first) & 1;
    if (c->off_slot_layer[slot] == l) return RIVER_OK;
    const river_layer_weights &dst = c->layers[l - 1], &src = c->off_host[l - 1];
    const size_t qdim = (size_t)g.Hq * g.dh, kvdim = (size_t)g.Hkv * g.dh, d = g.d, F = g.F;
    const void *dp[7] = {dst.wq, dst.wk, dst.wv, dst.wo, dst.wg, dst.wu, dst.wd};
    const void *sp[7] = {src.wq, src.wk, src.wv, src.wo, src.wg, src.wu, src.wd};
    const size_t nb[7] = {qdim * d * 2, kvdim * d * 2, kvdim * d * 2, d * qdim * 2, F * d * 2, F * d * 2, d * F * 2};
    CUDA_TRY(c, cudaStreamWaitEvent(c->off_copy, c->off_freed[slot], 0));
    for (int i = 0; i < 7; ++i)
        CUDA_TRY(c, cudaMemcpyAsync(const_cast<void *>(dp[i]), sp[i], nb[i], cudaMemcpyHostToDevice, c->off_copy));
    CUDA_TRY(c, cudaEventRecord(c->off_ready[slot], c->off_copy));
    c->off_slot_layer[slot] = l;
    c->st.offload_fetches += 1;
    return RIVER_OK;
}

// Before block l >= off_first: are rows still in the backbone?  (A host decision: the one place where a step with
// offloading synchronises.)  If so the block's weights are staged and the next block's copy is started behind them.
int offload_before_layer(river_ctx *c, int l, bool *staged) {
    *staged = false;
    int32_t na = 0;
    CUDA_TRY(c, cudaMemcpyAsync(&na, c->n_act + (l - 1), sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    if (na <= 0) return RIVER_OK;
    if (int rc = offload_fetch(c, l)) return rc;
    CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->off_ready[(l - c->off_first) & 1], 0));
    if (l + 1 <= c->cfg.L)
        if (int rc = offload_fetch(c, l + 1)) return rc;
    *staged = true;
    return RIVER_OK;
}

// The tensor-core kernels of one projection: `backbone(phase, late_release)` launches tc_gemm_kernel's part,
// `river(phase, beside)` the dequantising kernel's.  With both, one operand kernel serves both lists and the two GEMMs
// share the device: the first lets the second start once the operands are complete, the second waits for the first
// before it ends (the kernels' comments say why that is enough); RIVER_F_SERIAL_TC keeps them one after the other.
// `operand_ready`: the operand rows of both lists were written by the previous projection's epilogues: no operand kernel.
template <class Bb, class Rv>
cudaError_t tc_pair(river_ctx *c, bool with_river, const ProjIn &in, int K, int n, const RowLists &rl, Bb &&backbone,
                    Rv &&river, bool operand_ready = false) {
    const int whole = operand_ready ? kTcGemm : kTcBoth;
    if (!with_river) return backbone(whole, false);
    cudaError_t e;
    if (c->cfg.flags & RIVER_F_SERIAL_TC) {
        if ((e = backbone(whole, false)) != cudaSuccess) return e;
        return river(whole, false);
    }
    if (!operand_ready &&
        (e = launch_tc_prep_pair(c, in, K, n, rl.act_idx, rl.n_act, rl.riv_idx, rl.n_riv)) != cudaSuccess)
        return e;
    if ((e = backbone(kTcGemm, true)) != cudaSuccess) return e;
    return river(kTcGemm, true);
}

// a2 of block l for the n rows of the step: attention norm + QKV + RoPE + KV write, on the weight set(s) the row
// lists name (small steps: from the exit flags).
cudaError_t launch_qkv(river_ctx *c, int l, int n, const float *h_in, const DecideArgs &dec, double kv_write) {
    const river_config &g = c->cfg;
    const int d = g.d, B = g.max_batch, qdim = g.Hq * g.dh, kvdim = g.Hkv * g.dh;
    const double w4f = 0.25 + 2.0 / g.group;
    const river_layer_weights &w = c->layers[l - 1];
    const int strat = g.kv_strategy;
    const int has_river = strat == RIVER_KV_RIVER && w.rq.codes != nullptr;
    const int32_t *ai = c->act_idx + (size_t)(l - 1) * B, *ri = c->riv_idx + (size_t)(l - 1) * B;
    const int32_t *na = c->n_act + (l - 1), *nr = c->n_riv + (l - 1);
    const RowLists rl{ai, na, ri, nr, c->hint_act, c->meta_dev /* StepMeta::n_rows */, c->state_at(l - 1)};
    const bool tc = c->tc_ok && n >= 5 && n <= c->tc_max_pad;
    const river_ctx::LayerMaps *tm = tc ? &c->tc_maps[l - 1] : nullptr;
    const river_ctx::LayerMaps *wm = (tc && c->w4tc_ok && has_river) ? &c->w4_maps[l - 1] : nullptr;
    const int32_t *nrh = c->n_riv + std::max(0, l - 2);  // never above the count entering this block
    cudaError_t err = cudaSuccess;
    auto note = [&](cudaError_t e) { if (err == cudaSuccess) err = e; };
    const double wb = 2.0 * (qdim + 2.0 * kvdim) * d;
    // bytes the rows that have left cost here: the 4-bit copy; the bf16 K and V matrices (State Propagation); nothing
    const double riv_bytes = strat == RIVER_KV_RIVER ? wb * w4f + kv_write
                           : strat == RIVER_KV_STATE_PROPAGATION ? 2.0 * 2.0 * kvdim * d + kv_write : 0.0;
    LaunchScope ls(c, K_QKV, wb + kv_write, riv_bytes, l - 1);
    QkvProblem p{};
    p.wq = (const uint16_t *)w.wq; p.wk = (const uint16_t *)w.wk; p.wv = (const uint16_t *)w.wv;
    p.rq = w4_of(w.rq); p.rk = w4_of(w.rk); p.rv = w4_of(w.rv);
    p.K = d; p.Hq = g.Hq; p.Hkv = g.Hkv; p.dh = g.dh; p.group = g.group;
    p.rope_cs = c->rope_cs; p.q_out = c->qbuf; p.kv = kv_addr(c, l - 1); p.dev_err = c->dev_err;
    const ProjIn in{h_in, (const uint16_t *)w.attn_norm, g.rms_eps};
    if (tc) {
        const TcQkvEpi e{g.Hq, g.Hkv, g.dh, c->rope_cs, c->qbuf, kv_addr(c, l - 1), c->dev_err};
        const CUtensorMap *const cm[3] = {wm ? &wm->q : nullptr, wm ? &wm->k : nullptr, wm ? &wm->v : nullptr};
        const river_w4 *const cw[3] = {&w.rq, &w.rk, &w.rv};
        note(tc_pair(c, wm != nullptr, in, d, n, rl,
                     [&](int phase, bool late) {
                         return launch_tc(c, in, tm->q, tm->k, tm->v, d, (qdim + 2 * kvdim) / kTcBM, n, 0, qdim / kTcBM,
                                          kvdim / kTcBM, ai, na, e, true, c->hint_act, phase, late);
                     },
                     [&](int phase, bool beside) {
                         return launch_tc_w4(c, in, cm, cw, d, (qdim + 2 * kvdim) / kTcBM, n, 0, qdim / kTcBM, kvdim / kTcBM,
                                             ri, nr, nrh, e, phase, beside);
                     }));
    }
    if (!wm && (!tc || has_river)) {
        note(launch_stream(c, p, in, rl, d, (g.Hq + 2 * g.Hkv) * (g.dh / 2), n, has_river, true, tc ? 1 : 0, dec));
    }
    if (strat == RIVER_KV_STATE_PROPAGATION) {
        // Section 3: K / V of this block for the rows that have left, from their hidden state at the exit (this block's
        // norm, the backbone's K and V matrices); the same kernels on a K / V-only problem (no query heads) and on the
        // list of the rows that left
        if (tc) {
            TcQkvEpi e{0, g.Hkv, g.dh, c->rope_cs, c->qbuf, kv_addr(c, l - 1), c->dev_err};
            // (the kernel's early-out hint must never under-count; the count of rows that left only grows, so the
            // hint is the step's row count: the kernel always waits for the real count)
            note(launch_tc(c, in, tm->k, tm->v, tm->v, d, 2 * kvdim / kTcBM, n, 0, kvdim / kTcBM, kvdim / kTcBM, ri, nr, e,
                           true, c->meta_dev /* StepMeta::n_rows */));
            ++c->st.launches_last_step;
        } else {
            QkvProblem pk = p;
            pk.Hq = 0;
            note(launch_stream(c, pk, in, rl, d, 2 * g.Hkv * (g.dh / 2), n, 2, true, 0, DecideArgs{}));
            ++c->st.launches_last_step;
        }
    }
    return err;
}

// The launch sequence of one step over the rows described in the device metadata (rows, positions, caller buffers).
//
// Steps of up to four rows: per block QKV, attention, O, gate/up, down - the exit decision of block l is taken by the
// QKV kernel of block l + 1 (every CTA computes Eq. 1 for itself while it stages the rows, see gemv_stream.cuh), so
// no kernel boundary is spent on it; one score kernel after the LM head records the last block's score and the final
// row lists.  Steps of five and more rows: backbone rows on the tensor-core GEMM, exit-layer rows on its dequantising
// variant, and the score / compaction kernel after every block.
int run_rows(river_ctx *c, int n, int n_head, const int32_t *row_pos_host, bool record_fail = false) {
    const river_config &g = c->cfg;
    const int L = g.L, d = g.d, B = g.max_batch;
    int32_t *fail_buf = record_fail ? c->prefill_fail : nullptr;
    c->st.launches_last_step = 0;
    Lists lists{c->act_idx, c->riv_idx, c->n_act, c->n_riv, B};
    const int qdim = g.Hq * g.dh, kvdim = g.Hkv * g.dh;
    const double w4f = 0.25 + 2.0 / g.group;  // bytes of a 4-bit copy relative to bf16: (1/2 + 4/G) / 2
    double kv_read = 0.0;
    for (int i = 0; i < n; ++i) kv_read += (double)(row_pos_host[i] + 1) * 2.0 * kvdim * 2.0;
    const double kv_write = (double)n * 2.0 * kvdim * 2.0;
    cudaError_t err = cudaSuccess;
    auto note = [&](cudaError_t e) { if (err == cudaSuccess) err = e; };
    const int strat = g.kv_strategy;
    // the decisions ride in the QKV kernels - unless the host has to see every decision before it stages a block
    // (offloading) or the rows that left take another route than the 4-bit copies (then: score kernel per block)
    const bool fold = n <= 4 && !c->off_first && strat == RIVER_KV_RIVER;
    const DecideArgs no_dec{};

    {
        LaunchScope ls(c, K_BEGIN, (double)n * d * 2.0, 0, -1);
        note(launch_k(step_begin_kernel, dim3(std::max(n, 1)), dim3(128), 0, c->stream, false, c->meta(), c->upd(),
                      c->page_tbl_dev, g.max_pages_per_seq, B, c->embed, d, g.V, c->h[0], c->row_pos(), c->inv_freq,
                      g.dh / 2, c->rope_cs, L, g.entry_layer, c->state_at(0), c->dev_err, lists, c->hint_act, c->tickets));
    }
    auto launch_score = [&](int l, const float *h_in, const float *h_out) {
        LaunchScope ls(c, K_SCORE, (double)n * d * 8.0, 0, -1);
        note(launch_k(score_compact_kernel, dim3(n), dim3(256), 0, c->stream, true, c->meta(), l, L, g.entry_layer,
                      g.exit_mode, h_in, h_out, d, c->pass, (const uint8_t *)c->state_at(l - 1), c->state_at(l), lists,
                      c->hint_act, c->tickets + 1, fail_buf, (const int32_t *)c->row_slot(),
                      strat == RIVER_KV_MONO_DECREASING ? c->slot_cap : (int32_t *)nullptr));
    };
    int hi = 0;                  // h[hi] = block input
    const float *prev_in = nullptr;  // input of the previous block (its output is h[hi])
    for (int l = 1; l <= L; ++l) {
        const river_layer_weights &w = c->layers[l - 1];
        const int has_river = strat == RIVER_KV_RIVER && w.rq.codes != nullptr;
        const int32_t *ai = c->act_idx + (size_t)(l - 1) * B, *ri = c->riv_idx + (size_t)(l - 1) * B;
        const int32_t *na = c->n_act + (l - 1), *nr = c->n_riv + (l - 1);
        const RowLists rl{ai, na, ri, nr, c->hint_act, c->meta_dev /* StepMeta::n_rows */, c->state_at(l - 1)};
        float *h_in = c->h[hi], *h_mid = c->h[(hi + 1) % 3], *h_out = c->h[(hi + 2) % 3];
        // With more rows than one CUDA-core pass takes, the backbone rows go to the tensor-core GEMM and the stream
        // kernel only serves the exit-layer rows of the same launch slot.
        const bool tc = c->tc_ok && n >= 5 && n <= c->tc_max_pad;
        const river_ctx::LayerMaps *tm = tc ? &c->tc_maps[l - 1] : nullptr;
        const river_ctx::LayerMaps *wm = (tc && c->w4tc_ok && has_river) ? &c->w4_maps[l - 1] : nullptr;
        const int32_t *nrh = c->n_riv + std::max(0, l - 2);  // never above the count entering this block
        const int skip_bb = tc ? 1 : 0;
        bool staged = false;
        if (c->off_first && l >= c->off_first)
            if (int rc = offload_before_layer(c, l, &staged)) return rc;
        // ---- a2: attention norm + QKV + RoPE + KV write (+ a6 / a7 of the previous block when the step is small)
        {
            DecideArgs dec{};
            if (fold && l >= 2) {
                dec.meta = c->meta(); dec.l = l - 1; dec.L = L; dec.entry_layer = g.entry_layer; dec.exit_mode = g.exit_mode;
                dec.h_prev = prev_in; dec.state_in = c->state_at(l - 2); dec.state_out = c->state_at(l - 1);
                dec.lists = lists; dec.hint_act = c->hint_act; dec.fail = fail_buf; dec.row_slot = c->row_slot();
            }
            note(launch_qkv(c, l, n, h_in, dec, kv_write));
        }
        // the other KV strategies (Section 3): a row that has left neither attends nor changes its hidden state
        c->attn_skip = strat == RIVER_KV_RIVER ? nullptr : c->state_at(l - 1);
        // (a prefill chunk needs no visibility test: a prompt starts in an empty slot and all its positions stop at one
        // depth, so whatever a row that still runs may look back at has an entry - and the chunk's own positions have
        // not been noted yet)
        c->attn_layer1 = (strat == RIVER_KV_MASK && c->rows_distinct) ? l : 0;
        if (strat != RIVER_KV_RIVER) {
            LaunchScope ls(c, K_SCORE, 0, 0, -1);
            note(launch_k(carry_rows_kernel, dim3(n, (d / 4 + 255) / 256), dim3(256), 0, c->stream, true, c->meta(),
                          (const uint8_t *)c->state_at(l - 1), (const float *)h_in, h_out, d));
        }
        // ---- a3: paged GQA decode attention
        if (c->prefill_attn_now) {
            LaunchScope ls(c, K_PREFILL_ATTN, kv_read, 0, -1);
            note(launch_attention_prefill(c, n, l - 1));
        } else {
            LaunchScope ls(c, K_ATTN, kv_read, 0, -1);
            note(launch_attention(c, n, l - 1));
        }
        // ---- a4: O projection + residual
        {
            const double wb = 2.0 * qdim * d;
            LaunchScope ls(c, K_OPROJ, wb, wb * w4f, l - 1);
            ResidProblem p{};
            p.w = (const uint16_t *)w.wo; p.rw = w4_of(w.ro); p.K = qdim; p.out_dim = d; p.group = g.group;
            p.resid = h_in; p.out = h_mid;
            const ProjIn in{c->obuf, nullptr, 0.f};
            if (tc) {
                const TcResidEpi e{h_in, h_mid, d};
                const CUtensorMap *const cm[3] = {wm ? &wm->o : nullptr, wm ? &wm->o : nullptr, wm ? &wm->o : nullptr};
                const river_w4 *const cw[3] = {&w.ro, &w.ro, &w.ro};
                note(tc_pair(c, wm != nullptr, in, qdim, n, rl,
                             [&](int phase, bool late) {
                                 return launch_tc(c, in, tm->o, tm->o, tm->o, qdim, d / kTcBM, n, 0, 0, 0, ai, na, e, true,
                                                  c->hint_act, phase, late);
                             },
                             [&](int phase, bool beside) {
                                 return launch_tc_w4(c, in, cm, cw, qdim, d / kTcBM, n, 0, 0, 0, ri, nr, nrh, e, phase, beside);
                             }));
            }
            if (!wm && (!tc || has_river))
                note(launch_stream(c, p, in, rl, qdim, d / 2, n, has_river, true, skip_bb, no_dec));
        }
        // ---- a5: FFN norm + gate/up + SwiGLU
        {
            const double wb = 2.0 * 2.0 * g.F * d;
            LaunchScope ls(c, K_GATEUP, wb, wb * w4f, l - 1);
            GateUpProblem p{};
            p.wg = (const uint16_t *)w.wg; p.wu = (const uint16_t *)w.wu; p.rg = w4_of(w.rg); p.ru = w4_of(w.ru);
            p.K = d; p.F = g.F; p.group = g.group; p.act = c->act;
            const ProjIn in{h_mid, (const uint16_t *)w.ffn_norm, g.rms_eps};
            if (tc) {
                // the epilogues also write the down projection's operand rows (second operand buffers: this
                // projection's own operand is still being read while they do)
                const int npad = (n + 15) / 16 * 16;
                TcGateUpEpi e{c->act, g.F}, e4{c->act, g.F};
                if (const river_ctx::BMap *bd = tc_bmap(c, g.F, npad, false, true)) {
                    e.ohi = reinterpret_cast<uint16_t *>(bd->base); e.olo = reinterpret_cast<uint16_t *>(bd->lo_ptr); e.omode = 1;
                } else note(cudaErrorInvalidValue);
                if (wm) {
                    if (const river_ctx::BMap *bd = tc_bmap(c, g.F, npad, true, true)) {
                        e4.ohi = reinterpret_cast<uint16_t *>(bd->base); e4.olo = reinterpret_cast<uint16_t *>(bd->lo_ptr); e4.omode = 2;
                    } else note(cudaErrorInvalidValue);
                }
                const CUtensorMap *const cm[3] = {wm ? &wm->g : nullptr, wm ? &wm->u : nullptr, wm ? &wm->u : nullptr};
                const river_w4 *const cw[3] = {&w.rg, &w.ru, &w.ru};
                note(tc_pair(c, wm != nullptr, in, d, n, rl,
                             [&](int phase, bool late) {
                                 return launch_tc(c, in, tm->g, tm->u, tm->u, d, g.F / 64, n, 1, 0, 0, ai, na, e, true,
                                                  c->hint_act, phase, late);
                             },
                             [&](int phase, bool beside) {
                                 return launch_tc_w4(c, in, cm, cw, d, g.F / 64, n, 1, 0, 0, ri, nr, nrh, e4, phase, beside);
                             }));
            }
            if (!wm && (!tc || has_river)) note(launch_stream(c, p, in, rl, d, g.F, n, has_river, true, skip_bb, no_dec));
        }
        // ---- a5: down projection + residual
        {
            const double wb = 2.0 * g.F * d;
            LaunchScope ls(c, K_DOWN, wb, wb * w4f, l - 1);
            ResidProblem p{};
            p.w = (const uint16_t *)w.wd; p.rw = w4_of(w.rd); p.K = g.F; p.out_dim = d; p.group = g.group;
            p.resid = h_mid; p.out = h_out;
            const ProjIn in{c->act, nullptr, 0.f};
            if (tc) {
                const TcResidEpi e{h_mid, h_out, d};
                const CUtensorMap *const cm[3] = {wm ? &wm->d : nullptr, wm ? &wm->d : nullptr, wm ? &wm->d : nullptr};
                const river_w4 *const cw[3] = {&w.rd, &w.rd, &w.rd};
                note(tc_pair(c, wm != nullptr, in, g.F, n, rl,
                             [&](int phase, bool late) {
                                 return launch_tc(c, in, tm->d, tm->d, tm->d, g.F, d / kTcBM, n, 0, 0, 0, ai, na, e, true,
                                                  c->hint_act, phase, late, true);
                             },
                             [&](int phase, bool beside) {
                                 return launch_tc_w4(c, in, cm, cw, g.F, d / kTcBM, n, 0, 0, 0, ri, nr, nrh, e, phase, beside, true);
                             },
                             true));  // operand rows: written by the gate/up epilogues
            }
            if (!wm && (!tc || has_river))
                note(launch_stream(c, p, in, rl, g.F, d / 2, n, has_river, true, skip_bb, no_dec));
        }
        // ---- a6 + a7: exit score, decision, compaction -> row lists entering block l+1
        if (!fold) launch_score(l, h_in, h_out);
        if (staged) note(cudaEventRecord(c->off_freed[(l - c->off_first) & 1], c->stream));  // the slot may be refilled
        prev_in = h_in;
        hi = (hi + 2) % 3;
    }
    if (n_head > 0) {
        HeadArgs a{};
        a.w = c->lm_head;
        a.in = ProjIn{c->h[hi], c->final_norm, g.rms_eps};
        a.d = d; a.V = g.V; a.rows = c->head_rows(); a.meta = c->meta();
        a.part_val = c->part_val; a.part_idx = c->part_idx;
        int n_parts = c->head_grid;
        if (c->tc_ok && n_head >= 5 && n_head <= c->tc_max_pad) {
            LaunchScope ls(c, K_HEAD, 2.0 * g.V * d + 4.0 * n_head * g.V, 0, -1);
            n_parts = g.V / kTcBM;
            TcHeadEpi e{c->meta(), g.V, c->part_val, c->part_idx, n_parts};
            note(launch_tc(c, a.in, c->tc_map_head, c->tc_map_head, c->tc_map_head, d, n_parts, n_head, 0, 0, 0,
                           c->head_rows(), c->meta_dev + 2 /* StepMeta::n_head_rows */, e, false, nullptr));
        } else {
            LaunchScope ls(c, K_HEAD, 2.0 * g.V * d + 4.0 * n_head * g.V, 0, -1);
            note(launch_head_stream(c, a, n_head));
        }
        {
            LaunchScope ls(c, K_ARGMAX, 0, 0, -1);
            note(launch_argmax_final(c, n_head, n_parts));
        }
    }
    // small steps: the last block's score (a diagnostic: no exit is taken after block L) and the final row lists
    if (fold) launch_score(L, prev_in, c->h[hi]);
    if (strat == RIVER_KV_MASK) {  // what the later tokens' attention may see of this step's positions
        LaunchScope ls(c, K_SCORE, 0, 0, -1);
        note(launch_k(depth_note_kernel, dim3((n + 127) / 128), dim3(128), 0, c->stream, true, c->meta(),
                      (const int32_t *)c->row_slot(), (const int32_t *)c->row_pos(), c->pos_depth, g.max_pages_per_seq * kPage));
    }
    if (err == cudaSuccess) err = cudaGetLastError();
    if (err != cudaSuccess) return fail(c, RIVER_E_DEVICE, std::string("kernel launch failed: ") + cudaGetErrorString(err));
    c->st.launches_total += c->st.launches_last_step;
    if (c->profiling) return profile_collect(c);
    return 0;
}

// One decode step through a CUDA graph of the launch sequence (captured the second time a row count is seen; the
// per-step inputs live in device memory, so the graph never needs new parameters).
int run_step(river_ctx *c, int n, const int32_t *row_pos_host) {
    const bool use_graph = (c->cfg.flags & RIVER_F_GRAPH) && !c->profiling && !c->off_first;
    if (!use_graph) return run_rows(c, n, n, row_pos_host);
    const int key_splits = c->attn_small_now ? 0 : c->attn_splits_now;  // the attention grid of the captured launches
    for (auto &ge : c->graphs)
        if (ge.n == n && ge.small_attn == c->attn_small_now && ge.attn_splits == key_splits) {
            if (!ge.exec) {  // second use: capture
                cudaGraph_t graph = nullptr;
                CUDA_TRY(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
                const int rc = run_rows(c, n, n, row_pos_host);
                const cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
                if (rc) { if (graph) cudaGraphDestroy(graph); return rc; }
                if (e != cudaSuccess) return fail(c, RIVER_E_DEVICE, std::string("graph capture failed: ") + cudaGetErrorString(e));
                const cudaError_t e2 = cudaGraphInstantiate(&ge.exec, graph, 0);
                cudaGraphDestroy(graph);
                if (e2 != cudaSuccess) { ge.exec = nullptr; return fail(c, RIVER_E_DEVICE, std::string("graph instantiate failed: ") + cudaGetErrorString(e2)); }
                ge.launches = c->st.launches_last_step;
                c->st.launches_total -= ge.launches;  // capturing launched nothing
            }
            CUDA_TRY(c, cudaGraphLaunch(ge.exec, c->stream));
            c->st.launches_last_step = ge.launches;
            c->st.launches_total += ge.launches;
            return 0;
        }
    c->graphs.push_back({n, c->attn_small_now, key_splits, nullptr, 0});
    return run_rows(c, n, n, row_pos_host);  // first use: plain launches (also sets the kernels' attributes)
}

// Device error word -> return code.  The word is sticky on the device; once the host has seen it, the context
// refuses further steps with the same code until river_clear_device_error.
int note_device_error(river_ctx *c, int de) {
    c->st.device_error = de;
    if (de == 0) return RIVER_OK;
    static const char *const names[] = {"", "forced exit layer out of range", "token id out of range",
                                        "page id out of range", "a bounded device-side wait ran out", "internal"};
    const std::string what = de > 0 && de < 6 ? names[de] : "unknown";
    return fail(c, de == DEV_WAIT_TIMEOUT ? RIVER_E_TIMEOUT : RIVER_E_DEVICE,
                "a kernel flagged an error (" + std::to_string(de) + ": " + what + "); river_clear_device_error resets it");
}
int refuse_if_flagged(river_ctx *c) {
    if (c->st.device_error == 0) return RIVER_OK;
    return note_device_error(c, c->st.device_error);
}

// Give back the pages a failed call took: the host table entries return to -1 and the pages to the free list, in
// reverse order, so that the retry finds the state it would have found at first.
void rollback_pages(river_ctx *c, const int32_t *mh, int n_upd) {
    const river_config &g = c->cfg;
    const int32_t *u = mh + kMetaHdr + 2 * g.max_batch;
    for (int i = n_upd - 1; i >= 0; --i) {
        const int slot = u[i], pi = u[g.max_batch + i], page = u[2 * g.max_batch + i];
        c->page_tbl[(size_t)slot * g.max_pages_per_seq + pi] = -1;
        c->free_pages.push_back(page);
    }
}


// One pass of the prompts through the decode kernels in chunks of rows (slot, position): rows of a chunk are
// consecutive prompt positions, possibly of several sequences; K/V of the whole chunk are written before its attention
// runs, and a row attends to positions <= its own, so causality holds inside a chunk.  depth[s]: the unified exit depth
// of sequence s (L = the whole backbone).  record_fail: note per (sequence, block) whether some position failed Eq. 1.
int prefill_pass(river_ctx *c, int n_seqs, const int32_t *slots, const int32_t *tok, const int32_t *offsets,
                 const int32_t *depth, float tau, bool record_fail, float *logits_last, int32_t *next_tok) {
    const river_config &g = c->cfg;
    {
        std::vector<float> ta(g.max_batch, tau);
        CUDA_TRY(c, cudaMemcpyAsync(c->tau_i, ta.data(), sizeof(float) * ta.size(), cudaMemcpyHostToDevice, c->stream));
        CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    }
    int s = 0, p = 0;  // next (sequence, position) to schedule
    while (s < n_seqs) {
        int32_t *mh = next_meta(c);
        int n = 0, n_upd = 0, n_head = 0;
        const int tok0 = offsets[s] + p;
        int head_seq[kMaxBatch];
        while (s < n_seqs && n < g.max_batch && n_head < c->user_max_batch) {
            const int len = offsets[s + 1] - offsets[s];
            if (offsets[s] + p != tok0 + n) break;  // token ids of a chunk must be contiguous in tok
            if (int rc = ensure_page(c, slots[s], p, mh, n_upd)) { rollback_pages(c, mh, n_upd); return rc; }
            mh[kMetaHdr + n] = slots[s];
            mh[kMetaHdr + g.max_batch + n] = p;
            mh[kMetaHdr + 6 * g.max_batch + n] = c->page_tbl[(size_t)slots[s] * g.max_pages_per_seq + p / kPage];
            mh[kMetaHdr + 7 * g.max_batch + n] = depth[s];
            if (p == len - 1) {
                mh[kMetaHdr + 5 * g.max_batch + n_head] = n;
                head_seq[n_head++] = s;
            }
            ++n;
            if (++p == len) { c->seq_len[slots[s]] = len; ++s; p = 0; }
        }
        mh[0] = n; mh[1] = n_upd; mh[2] = n_head;
        set_attn_meta(c, mh, n);
        // query tiles for the tensor-core prefill attention: up to 16 consecutive positions of one sequence each
        int n_tiles = 0;
        for (int i = 0; i < n;) {
            int j = i + 1;
            while (j < n && j - i < kPfBM && mh[kMetaHdr + j] == mh[kMetaHdr + i] &&
                   mh[kMetaHdr + g.max_batch + j] == mh[kMetaHdr + g.max_batch + i] + (j - i))
                ++j;
            mh[kMetaHdr + 8 * g.max_batch + n_tiles] = i;
            mh[kMetaHdr + 9 * g.max_batch + n_tiles] = j - i;
            ++n_tiles;
            i = j;
        }
        reinterpret_cast<StepMeta *>(mh)->pad2[0] = n_tiles;
        c->prefill_attn_now = n >= 5 && prefill_attn_supported(c);
        const bool want_logits = logits_last && n_head > 0;
        set_io_meta(mh, tok + tok0, c->tau_i, c->row_forced(), want_logits ? c->logits_i : nullptr, c->next_i, c->exit_i,
                    nullptr);
        if (int rc = push_meta(c, mh)) return rc;
        c->rows_distinct = false;  // consecutive positions of one sequence share a chunk
        const int rc_rows = run_rows(c, n, n_head, mh + kMetaHdr + g.max_batch, record_fail);
        c->rows_distinct = true;
        c->prefill_attn_now = false;
        if (rc_rows) return rc_rows;
        for (int i = 0; i < n_head; ++i) {
            if (logits_last)
                CUDA_TRY(c, cudaMemcpyAsync(logits_last + (size_t)head_seq[i] * g.V, c->logits_i + (size_t)i * g.V,
                                            sizeof(float) * g.V, cudaMemcpyDeviceToDevice, c->stream));
            if (next_tok)
                CUDA_TRY(c, cudaMemcpyAsync(next_tok + head_seq[i], c->next_i + i, sizeof(int32_t), cudaMemcpyDeviceToDevice, c->stream));
        }
    }
    return RIVER_OK;
}

int check_slot(const river_ctx *c, int slot) { return slot >= 0 && slot < c->cfg.max_seqs; }

}  // namespace

extern "C" {

size_t river_workspace_bytes(const river_config *cfg) {
    if (check_config(cfg)) return 0;
    int mb = 0;
    const river_config e = effective(cfg, &mb);
    return carve(&e, nullptr, nullptr, mb);
}

size_t river_kv_pool_bytes(const river_config *cfg) {
    if (check_config(cfg)) return 0;
    return (size_t)cfg->L * cfg->n_pages * 2 * cfg->Hkv * kPage * cfg->dh * sizeof(__nv_bfloat16);
}

int river_init(const river_config *cfg, const river_weights *w, void *kv_pool, size_t kv_pool_bytes, void *workspace,
               size_t workspace_bytes, void *cuda_stream, river_ctx **out) {
    if (!out) return fail(nullptr, RIVER_E_BADARG, "out is null");
    *out = nullptr;
    if (const char *m = check_config(cfg)) return fail(nullptr, RIVER_E_SHAPE, m);
    if (!w || !w->embed || !w->lm_head || !w->final_norm || !w->layers) return fail(nullptr, RIVER_E_BADARG, "null weights");
    if (!kv_pool || !workspace) return fail(nullptr, RIVER_E_BADARG, "null kv_pool / workspace");
    if (((uintptr_t)kv_pool | (uintptr_t)workspace) & 255) return fail(nullptr, RIVER_E_BADARG, "kv_pool / workspace must be 256-byte aligned");
    if (kv_pool_bytes < river_kv_pool_bytes(cfg)) return fail(nullptr, RIVER_E_NOMEM, "kv_pool too small");
    if (workspace_bytes < river_workspace_bytes(cfg)) return fail(nullptr, RIVER_E_NOMEM, "workspace too small");
    for (int l = 0; l < cfg->L; ++l) {
        const river_layer_weights &y = w->layers[l];
        if (!y.attn_norm || !y.wq || !y.wk || !y.wv || !y.wo || !y.ffn_norm || !y.wg || !y.wu || !y.wd)
            return fail(nullptr, RIVER_E_BADARG, "null backbone weight in layer " + std::to_string(l + 1));
        const river_w4 *r[7] = {&y.rq, &y.rk, &y.rv, &y.ro, &y.rg, &y.ru, &y.rd};
        int have = 0;
        for (auto p : r) have += (p->codes && p->scale && p->zero) ? 1 : 0;
        if (have != 0 && have != 7) return fail(nullptr, RIVER_E_BADARG, "partial exit-layer weights in layer " + std::to_string(l + 1));
        if (have == 0 && l + 1 > cfg->entry_layer)
            return fail(nullptr, RIVER_E_BADARG, "layer " + std::to_string(l + 1) + " is above entry_layer but has no exit-layer copy");
    }
    river_ctx *c = new river_ctx();
    c->cfg = effective(cfg, &c->user_max_batch);
    cfg = &c->cfg;  // from here on max_batch means rows per launch sequence (a decode step or a prefill chunk)
    c->layers.assign(w->layers, w->layers + cfg->L);
    c->embed = (const uint16_t *)w->embed;
    c->lm_head = (const uint16_t *)w->lm_head;
    c->final_norm = (const uint16_t *)w->final_norm;
    c->stream = (cudaStream_t)cuda_stream;
    if ((cfg->flags & RIVER_F_GRAPH) && (c->stream == nullptr || c->stream == cudaStreamLegacy)) {
        delete c;
        return fail(nullptr, RIVER_E_BADARG, "RIVER_F_GRAPH needs a stream other than the default stream");
    }
    c->pool = (__nv_bfloat16 *)kv_pool;
    c->ws_bytes = carve(cfg, c, (char *)workspace, c->user_max_batch);
    c->head_grid = head_grid_for(cfg);
    auto bail = [&](const std::string &m) {
        g_init_error = m;
        river_destroy(c);
        return RIVER_E_DEVICE;
    };
    int dev = 0, cc_major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return bail("cudaGetDevice failed (no CUDA device?)");
    if (cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return bail("cudaDeviceGetAttribute failed");
    if (cc_major != 10) return bail("this library is built for sm_100a (B200) only");
    c->device = dev;
    if (make_kv_tensor_map(c)) { river_destroy(c); return RIVER_E_DEVICE; }
    c->tc_ok = !(cfg->flags & RIVER_F_NO_TC) && tc_shape_ok(*cfg) && make_tc_maps(c);
    c->w4tc_ok = c->tc_ok && !(cfg->flags & RIVER_F_NO_W4TC) && make_w4_maps(c);
    for (int i = 0; i < kStaging; ++i) {
        if (cudaMallocHost((void **)&c->meta_host[i], sizeof(int32_t) * c->meta_ints()) != cudaSuccess) return bail("cudaMallocHost failed");
        std::memset(c->meta_host[i], 0, sizeof(int32_t) * c->meta_ints());  // entries past a step's rows stay valid row ids
        if (cudaEventCreateWithFlags(&c->meta_ev[i], cudaEventDisableTiming) != cudaSuccess) return bail("cudaEventCreate failed");
    }
    c->pin_io_bytes = (size_t)cfg->max_batch * (4 * sizeof(int32_t) + sizeof(float)) + sizeof(int32_t);
    if (cudaMallocHost(&c->pin_io, c->pin_io_bytes) != cudaSuccess) return bail("cudaMallocHost failed");
    c->page_tbl.assign((size_t)cfg->max_seqs * cfg->max_pages_per_seq, -1);
    c->seq_len.assign(cfg->max_seqs, 0);
    c->free_pages.resize(cfg->n_pages);
    for (int i = 0; i < cfg->n_pages; ++i) c->free_pages[i] = cfg->n_pages - 1 - i;  // pop_back hands out 0, 1, 2, ...
    if (cfg->page_shuffle_seed) {
        uint64_t s = cfg->page_shuffle_seed * 0x9E3779B97F4A7C15ull + 1;
        for (int i = cfg->n_pages - 1; i > 0; --i) {
            s ^= s >> 12; s ^= s << 25; s ^= s >> 27;
            const uint64_t r = (s * 0x2545F4914F6CDD1Dull) >> 33;
            std::swap(c->free_pages[i], c->free_pages[(size_t)(r % (uint64_t)(i + 1))]);
        }
    }
    std::vector<double> fr(cfg->dh / 2);
    for (int i = 0; i < cfg->dh / 2; ++i) fr[i] = std::pow((double)cfg->rope_theta, -2.0 * i / cfg->dh);
    cudaError_t e = cudaMemcpyAsync(c->inv_freq, fr.data(), sizeof(double) * fr.size(), cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->page_tbl_dev, 0xff, sizeof(int32_t) * c->page_tbl.size(), c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->dev_err, 0, sizeof(int), c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->state, 0, (size_t)(cfg->L + 1) * c->state_stride, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->attn_tickets, 0, sizeof(unsigned) * (size_t)cfg->max_batch * cfg->Hkv, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->tickets, 0, sizeof(unsigned) * 4, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->exit_hist, 0, sizeof(unsigned long long) * (cfg->L + 1), c->stream);
    {
        const std::vector<int32_t> caps((size_t)cfg->max_seqs, cfg->L);  // Mono-Decreasing Exit: every sequence starts at L
        if (e == cudaSuccess) e = cudaMemcpy(c->slot_cap, caps.data(), sizeof(int32_t) * caps.size(), cudaMemcpyHostToDevice);
    }

    if (e == cudaSuccess) e = cudaMemsetAsync(c->n_act, 0, sizeof(int32_t) * (cfg->L + 1), c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->n_riv, 0, sizeof(int32_t) * (cfg->L + 1), c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) return bail(std::string("init copies failed: ") + cudaGetErrorString(e));
    *out = c;
    return RIVER_OK;
}

int river_decode_step(river_ctx *c, int batch, const int32_t *slots, const int32_t *tok, const float *tau,
                      const int32_t *forced_exit, float *logits, int32_t *next_tok, int32_t *exit_layer,
                      float *scores) {
    if (!c) return RIVER_E_BADARG;
    const river_config &g = c->cfg;
    if (int rc = refuse_if_flagged(c)) return rc;
    if (batch <= 0 || batch > c->user_max_batch) return fail(c, RIVER_E_BADARG, "batch out of range");
    if (!slots || !tok || !tau || !next_tok || !exit_layer) return fail(c, RIVER_E_BADARG, "null argument");
    // everything that can fail is checked before any page is taken: slots, lengths, and the pages the whole batch needs
    int new_pages = 0;
    for (int b = 0; b < batch; ++b) {
        if (!check_slot(c, slots[b])) return fail(c, RIVER_E_BADSLOT, "slot out of range");
        for (int b2 = 0; b2 < b; ++b2)
            if (slots[b2] == slots[b]) return fail(c, RIVER_E_BADSLOT, "a slot appears twice in one step");
        const int pos = c->seq_len[slots[b]];
        if (pos >= g.max_pages_per_seq * kPage) return fail(c, RIVER_E_NOPAGE, "sequence full");
        if (c->page_tbl[(size_t)slots[b] * g.max_pages_per_seq + pos / kPage] < 0) ++new_pages;
    }
    if (new_pages > (int)c->free_pages.size()) return fail(c, RIVER_E_NOPAGE, "KV pool exhausted");
    int32_t *mh = next_meta(c);
    int n_upd = 0;
    c->last_pos.resize(batch);
    for (int b = 0; b < batch; ++b) {
        const int pos = c->seq_len[slots[b]];
        if (int rc = ensure_page(c, slots[b], pos, mh, n_upd)) { rollback_pages(c, mh, n_upd); return rc; }
        mh[kMetaHdr + b] = slots[b];
        mh[kMetaHdr + g.max_batch + b] = pos;
        mh[kMetaHdr + 5 * g.max_batch + b] = b;
        mh[kMetaHdr + 6 * g.max_batch + b] = c->page_tbl[(size_t)slots[b] * g.max_pages_per_seq + pos / kPage];
        c->last_pos[b] = pos;
    }
    mh[0] = batch; mh[1] = n_upd; mh[2] = batch;
    set_attn_meta(c, mh, batch);
    set_io_meta(mh, tok, tau, forced_exit, logits, next_tok, exit_layer, scores);
    if (int rc = push_meta(c, mh)) { rollback_pages(c, mh, n_upd); return rc; }
    if (int rc = run_step(c, batch, c->last_pos.data())) return rc;
    for (int b = 0; b < batch; ++b) c->seq_len[slots[b]] += 1;
    c->st.steps += 1;
    c->st.batch_last = batch;
    return RIVER_OK;
}

int river_decode_step_host(river_ctx *c, int batch, const int32_t *slots, const int32_t *tok, const float *tau,
                           const int32_t *forced_exit, float *logits, int32_t *next_tok, int32_t *exit_layer,
                           float *scores) {
    if (!c) return RIVER_E_BADARG;
    const river_config &g = c->cfg;
    if (batch <= 0 || batch > c->user_max_batch) return fail(c, RIVER_E_BADARG, "batch out of range");
    if (!slots || !tok || !tau || !next_tok || !exit_layer) return fail(c, RIVER_E_BADARG, "null argument");
    if (forced_exit)
        for (int b = 0; b < batch; ++b)
            if (forced_exit[b] >= 0 && (forced_exit[b] > g.L || forced_exit[b] < g.entry_layer))
                return fail(c, RIVER_E_BADARG, "forced_exit out of range");
    const size_t B = g.max_batch;
    int32_t *p_tok = (int32_t *)c->pin_io, *p_forced = p_tok + B, *p_next = p_forced + B, *p_exit = p_next + B;
    float *p_tau = (float *)(p_exit + B);
    int32_t *p_err = (int32_t *)(p_tau + B);  // pin_io holds 5 arrays of max_batch entries and this word
    std::memcpy(p_tok, tok, sizeof(int32_t) * batch);
    std::memcpy(p_tau, tau, sizeof(float) * batch);
    if (forced_exit) std::memcpy(p_forced, forced_exit, sizeof(int32_t) * batch);
    CUDA_TRY(c, cudaMemcpyAsync(c->tok_i, p_tok, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(c->tau_i, p_tau, sizeof(float) * batch, cudaMemcpyHostToDevice, c->stream));
    if (forced_exit)
        CUDA_TRY(c, cudaMemcpyAsync(c->forced_i, p_forced, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, c->stream));
    if (int rc = river_decode_step(c, batch, slots, c->tok_i, c->tau_i, forced_exit ? c->forced_i : nullptr,
                                   logits ? c->logits_i : nullptr, c->next_i, c->exit_i, scores ? c->scores_i : nullptr))
        return rc;
    CUDA_TRY(c, cudaMemcpyAsync(p_next, c->next_i, sizeof(int32_t) * batch, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(p_exit, c->exit_i, sizeof(int32_t) * batch, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(p_err, c->dev_err, sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    if (logits)
        CUDA_TRY(c, cudaMemcpyAsync(logits, c->logits_i, sizeof(float) * (size_t)batch * g.V, cudaMemcpyDeviceToHost, c->stream));
    if (scores)
        CUDA_TRY(c, cudaMemcpyAsync(scores, c->scores_i, sizeof(float) * (size_t)batch * g.L, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    std::memcpy(next_tok, p_next, sizeof(int32_t) * batch);
    std::memcpy(exit_layer, p_exit, sizeof(int32_t) * batch);
    return note_device_error(c, *p_err);
}

int river_prefill(river_ctx *c, int n_seqs, const int32_t *slots, const int32_t *tok, const int32_t *offsets,
                  int prefill_exit_layer, float tau, float *logits_last, int32_t *next_tok, int32_t *depth_out) {
    if (!c) return RIVER_E_BADARG;
    const river_config &g = c->cfg;
    if (int rc = refuse_if_flagged(c)) return rc;
    if (n_seqs <= 0 || !slots || !tok || !offsets) return fail(c, RIVER_E_BADARG, "null / empty argument");
    const bool auto_depth = prefill_exit_layer == -1;
    if (!auto_depth && (prefill_exit_layer < std::max(g.entry_layer, 0) || prefill_exit_layer > g.L))
        return fail(c, RIVER_E_BADARG, "prefill_exit_layer must be -1 or lie in [entry_layer, L]");
    long long new_pages = 0;
    for (int s = 0; s < n_seqs; ++s) {
        if (!check_slot(c, slots[s])) return fail(c, RIVER_E_BADSLOT, "slot out of range");
        if (c->seq_len[slots[s]] != 0) return fail(c, RIVER_E_BADSLOT, "prefill needs an empty slot");
        for (int s2 = 0; s2 < s; ++s2)
            if (slots[s2] == slots[s]) return fail(c, RIVER_E_BADSLOT, "a slot appears twice");
        const int n = offsets[s + 1] - offsets[s];
        if (n <= 0) return fail(c, RIVER_E_BADARG, "empty prompt");
        if (n > g.max_pages_per_seq * kPage) return fail(c, RIVER_E_NOPAGE, "prompt longer than the page table");
        for (int pi = 0; pi < (n + kPage - 1) / kPage; ++pi)
            if (c->page_tbl[(size_t)slots[s] * g.max_pages_per_seq + pi] < 0) ++new_pages;
    }
    if (new_pages > (long long)c->free_pages.size()) return fail(c, RIVER_E_NOPAGE, "KV pool exhausted");
    // Unified depth (Section 4.2, "Prefill Phase": all tokens of a prompt leave at one depth).  -1: per sequence, the
    // first block l in [max(entry_layer, 1), L - 1] after which EVERY position of the prompt passes Eq. 1 (s > tau),
    // else L.  Scores up to that block only involve backbone blocks, so a first pass runs the whole backbone over the
    // prompts and notes per (sequence, block) whether some position failed; if some depth is below L a second pass
    // redoes the prompts with the exit layers above each sequence's depth (the cache entries are simply rewritten).
    std::vector<int32_t> depth(n_seqs, auto_depth ? g.L : prefill_exit_layer);
    if (auto_depth) {
        CUDA_TRY(c, cudaMemsetAsync(c->prefill_fail, 0, sizeof(int32_t) * (size_t)g.max_seqs * (g.L + 1), c->stream));
        if (int rc = prefill_pass(c, n_seqs, slots, tok, offsets, depth.data(), tau, true, logits_last, next_tok)) return rc;
        std::vector<int32_t> failed((size_t)g.max_seqs * (g.L + 1));
        CUDA_TRY(c, cudaMemcpyAsync(failed.data(), c->prefill_fail, sizeof(int32_t) * failed.size(), cudaMemcpyDeviceToHost, c->stream));
        CUDA_TRY(c, cudaStreamSynchronize(c->stream));
        bool again = false;
        for (int s = 0; s < n_seqs; ++s)
            for (int l = std::max(g.entry_layer, 1); l < g.L; ++l)
                if (!failed[(size_t)slots[s] * (g.L + 1) + l]) { depth[s] = l; again = true; break; }
        if (depth_out) std::memcpy(depth_out, depth.data(), sizeof(int32_t) * n_seqs);
        if (!again) return RIVER_OK;  // the first pass is the result
        for (int s = 0; s < n_seqs; ++s) c->seq_len[slots[s]] = 0;  // the pages stay; every position is rewritten
    } else if (depth_out) {
        std::memcpy(depth_out, depth.data(), sizeof(int32_t) * n_seqs);
    }
    return prefill_pass(c, n_seqs, slots, tok, offsets, depth.data(), tau, false, logits_last, next_tok);
}

// Common front of the single-stage entry points: rows (slot, last cached position) into the step metadata.
static int stage_rows(river_ctx *c, int layer, int n_rows, const int32_t *slots, int on_exit_layer) {
    const river_config &g = c->cfg;
    if (int rc = refuse_if_flagged(c)) return rc;
    if (layer < 1 || layer > g.L) return fail(c, RIVER_E_BADARG, "layer out of range");
    if (n_rows <= 0 || n_rows > c->user_max_batch || !slots) return fail(c, RIVER_E_BADARG, "rows out of range");
    if (on_exit_layer && !c->layers[layer - 1].rq.codes) return fail(c, RIVER_E_BADARG, "this block has no exit-layer copy");
    for (int b = 0; b < n_rows; ++b) {
        if (!check_slot(c, slots[b])) return fail(c, RIVER_E_BADSLOT, "slot out of range");
        if (c->seq_len[slots[b]] <= 0) return fail(c, RIVER_E_BADSLOT, "empty sequence");
        for (int b2 = 0; b2 < b; ++b2)
            if (slots[b2] == slots[b]) return fail(c, RIVER_E_BADSLOT, "a slot appears twice");
    }
    int32_t *mh = next_meta(c);
    c->last_pos.resize(n_rows);
    for (int b = 0; b < n_rows; ++b) {
        const int pos = c->seq_len[slots[b]] - 1;
        mh[kMetaHdr + b] = slots[b];
        mh[kMetaHdr + g.max_batch + b] = pos;
        mh[kMetaHdr + 6 * g.max_batch + b] = c->page_tbl[(size_t)slots[b] * g.max_pages_per_seq + pos / kPage];
        c->last_pos[b] = pos;
    }
    mh[0] = n_rows; mh[1] = 0; mh[2] = 0;
    set_attn_meta(c, mh, n_rows);
    set_io_meta(mh, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr);
    if (int rc = push_meta(c, mh)) return rc;
    Lists lists{c->act_idx, c->riv_idx, c->n_act, c->n_riv, g.max_batch};
    stage_begin_kernel<<<n_rows, 64, 0, c->stream>>>(c->meta(), c->row_pos(), c->inv_freq, g.dh / 2, c->rope_cs,
                                                      c->state_at(layer - 1), lists, layer - 1, on_exit_layer, c->hint_act);
    CUDA_TRY(c, cudaGetLastError());
    c->st.launches_total += 1;
    return RIVER_OK;
}

int river_attention(river_ctx *c, int layer, int n_rows, const int32_t *slots, const float *q, float *out) {
    if (!c) return RIVER_E_BADARG;
    if (!q || !out) return fail(c, RIVER_E_BADARG, "null argument");
    if (int rc = stage_rows(c, layer, n_rows, slots, 0)) return rc;
    float *q_keep = c->qbuf, *o_keep = c->obuf;
    c->qbuf = const_cast<float *>(q);
    c->obuf = out;
    c->attn_skip = nullptr;  // every listed row attends
    c->attn_layer1 = 0;      // ... to every cached position
    c->st.launches_last_step = 0;
    cudaError_t e;
    {
        double kv_read = 0.0;
        for (int b = 0; b < n_rows; ++b) kv_read += (double)(c->last_pos[b] + 1) * 4.0 * c->cfg.Hkv * c->cfg.dh;
        LaunchScope ls(c, K_ATTN, kv_read, 0, -1);
        e = launch_attention(c, n_rows, layer - 1);
    }
    c->qbuf = q_keep;
    c->obuf = o_keep;
    if (e != cudaSuccess) return fail(c, RIVER_E_DEVICE, std::string("kernel launch failed: ") + cudaGetErrorString(e));
    c->st.launches_total += c->st.launches_last_step;
    if (c->profiling) return profile_collect(c);
    return RIVER_OK;
}

int river_project_kv(river_ctx *c, int layer, int use_exit_layer, int n_rows, const int32_t *slots, const float *h,
                     float *q_out) {
    if (!c) return RIVER_E_BADARG;
    if (!h) return fail(c, RIVER_E_BADARG, "null argument");
    if (int rc = stage_rows(c, layer, n_rows, slots, use_exit_layer ? 1 : 0)) return rc;
    if (!use_exit_layer && c->off_first && layer >= c->off_first) {  // an offloaded backbone block: stage it first
        if (int rc = offload_fetch(c, layer)) return rc;
        CUDA_TRY(c, cudaStreamWaitEvent(c->stream, c->off_ready[(layer - c->off_first) & 1], 0));
    }
    float *q_keep = c->qbuf;
    if (q_out) c->qbuf = q_out;
    c->st.launches_last_step = 0;
    const cudaError_t e = launch_qkv(c, layer, n_rows, h, DecideArgs{}, (double)n_rows * 4.0 * c->cfg.Hkv * c->cfg.dh);
    c->qbuf = q_keep;
    if (e != cudaSuccess) return fail(c, RIVER_E_DEVICE, std::string("kernel launch failed: ") + cudaGetErrorString(e));
    if (!use_exit_layer && c->off_first && layer >= c->off_first)
        CUDA_TRY(c, cudaEventRecord(c->off_freed[(layer - c->off_first) & 1], c->stream));
    c->st.launches_total += c->st.launches_last_step;
    if (c->profiling) return profile_collect(c);
    return RIVER_OK;
}

int river_generate(river_ctx *c, int batch, const int32_t *slots, const int32_t *tok0, const float *tau, int n_steps,
                   int32_t *out_tok, int32_t *out_exit) {
    if (!c) return RIVER_E_BADARG;
    if (!tok0 || !tau || !out_tok || n_steps <= 0) return fail(c, RIVER_E_BADARG, "null argument / no steps");
    for (int t = 0; t < n_steps; ++t) {
        const int32_t *tok = t == 0 ? tok0 : out_tok + (size_t)(t - 1) * batch;  // fed back on the device
        int32_t *ex = out_exit ? out_exit + (size_t)t * batch : c->exit_i;
        if (int rc = river_decode_step(c, batch, slots, tok, tau, nullptr, nullptr, out_tok + (size_t)t * batch, ex, nullptr))
            return rc;
    }
    return RIVER_OK;
}

int river_offload(river_ctx *c, int first_offloaded_layer, const river_layer_weights *host_layers) {
    if (!c) return RIVER_E_BADARG;
    const river_config &g = c->cfg;
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    if (first_offloaded_layer == 0) { c->off_first = 0; return RIVER_OK; }
    if (g.kv_strategy == RIVER_KV_STATE_PROPAGATION)
        return fail(c, RIVER_E_BADARG, "State Propagation projects K / V with every skipped block's backbone matrices: they cannot be offloaded");
    if (first_offloaded_layer < 2 || first_offloaded_layer > g.L || !host_layers)
        return fail(c, RIVER_E_BADARG, "first_offloaded_layer must be 0 or lie in [2, L], with the host copies given");
    for (int l = first_offloaded_layer; l <= g.L; ++l) {
        const river_layer_weights &h = host_layers[l - 1], &dv = c->layers[l - 1];
        if (!h.wq || !h.wk || !h.wv || !h.wo || !h.wg || !h.wu || !h.wd)
            return fail(c, RIVER_E_BADARG, "null host copy in an offloaded layer");
        if (l + 2 <= g.L) {  // blocks two apart must share a device slot
            const river_layer_weights &d2 = c->layers[l + 1];
            if (dv.wq != d2.wq || dv.wk != d2.wk || dv.wv != d2.wv || dv.wo != d2.wo || dv.wg != d2.wg || dv.wu != d2.wu || dv.wd != d2.wd)
                return fail(c, RIVER_E_BADARG, "offloaded blocks l and l + 2 must be given the same device matrices (two staging slots)");
        }
    }
    if (!c->off_copy) {
        CUDA_TRY(c, cudaStreamCreateWithFlags(&c->off_copy, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CUDA_TRY(c, cudaEventCreateWithFlags(&c->off_ready[i], cudaEventDisableTiming));
            CUDA_TRY(c, cudaEventCreateWithFlags(&c->off_freed[i], cudaEventDisableTiming));
        }
    }
    c->off_host.assign(host_layers, host_layers + g.L);
    c->off_first = first_offloaded_layer;
    c->off_slot_layer[0] = c->off_slot_layer[1] = -1;
    return RIVER_OK;
}

int river_exit_histogram(river_ctx *c, int64_t *counts, int reset) {
    if (!c || !counts) return RIVER_E_BADARG;
    const int n = c->cfg.L + 1;
    CUDA_TRY(c, cudaMemcpyAsync(counts, c->exit_hist, sizeof(int64_t) * n, cudaMemcpyDeviceToHost, c->stream));
    if (reset) CUDA_TRY(c, cudaMemsetAsync(c->exit_hist, 0, sizeof(unsigned long long) * n, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    return RIVER_OK;
}

int river_suggest_offload(river_ctx *c, double max_deep_fraction) {
    if (!c || !(max_deep_fraction >= 0.0)) return RIVER_E_BADARG;
    const int L = c->cfg.L;
    std::vector<int64_t> h((size_t)L + 1);
    if (int rc = river_exit_histogram(c, h.data(), 0)) return rc;
    int64_t total = 0;
    for (int64_t v : h) total += v;
    if (total == 0) return 0;  // nothing decoded yet: no advice
    // tokens that reach block l are those whose exit layer is >= l; the first block (>= 2) that at most the given
    // fraction of the tokens reaches
    int64_t reach = total - h[0];  // exit layer >= 1
    for (int l = 1; l <= L; ++l) {
        if (l >= 2 && (double)reach <= max_deep_fraction * (double)total) return l;
        reach -= h[l];
    }
    return 0;  // every block is reached too often
}

int river_clear_device_error(river_ctx *c) {
    if (!c) return RIVER_E_BADARG;
    CUDA_TRY(c, cudaMemsetAsync(c->dev_err, 0, sizeof(int), c->stream));
    // a launch that gave up may have left tickets of unfinished attention merges behind
    CUDA_TRY(c, cudaMemsetAsync(c->attn_tickets, 0, sizeof(unsigned) * (size_t)c->cfg.max_batch * c->cfg.Hkv, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    c->st.device_error = 0;
    return RIVER_OK;
}

int river_selftest_wait_timeout(river_ctx *c, int poll_limit) {
    if (!c) return RIVER_E_BADARG;
    if (poll_limit < 1 || poll_limit > (1 << 20)) return fail(c, RIVER_E_BADARG, "poll_limit out of range");
    wait_timeout_probe_kernel<<<1, 32, 0, c->stream>>>(c->dev_err, (uint32_t)poll_limit);
    CUDA_TRY(c, cudaGetLastError());
    int de = 0;
    CUDA_TRY(c, cudaMemcpyAsync(&de, c->dev_err, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    return note_device_error(c, de);
}

static int kv_copy(river_ctx *c, int slot, int layer, int pos0, int n, void *k, void *v, int to_cache) {
    if (!c) return RIVER_E_BADARG;
    const river_config &g = c->cfg;
    if (!check_slot(c, slot)) return fail(c, RIVER_E_BADSLOT, "slot out of range");
    if (layer < 1 || layer > g.L || pos0 < 0 || n <= 0 || !k || !v) return fail(c, RIVER_E_BADARG, "bad range");
    if (!to_cache && pos0 + n > c->seq_len[slot]) return fail(c, RIVER_E_BADARG, "range beyond the cached length");
    if (to_cache) {
        if (pos0 + n > g.max_pages_per_seq * kPage) return fail(c, RIVER_E_NOPAGE, "range beyond the page table");
        std::vector<int32_t> u;
        for (int p = pos0; p < pos0 + n; ++p) {
            int32_t &e = c->page_tbl[(size_t)slot * g.max_pages_per_seq + p / kPage];
            if (e >= 0) continue;
            if (c->free_pages.empty()) return fail(c, RIVER_E_NOPAGE, "KV pool exhausted");
            e = c->free_pages.back();
            c->free_pages.pop_back();
            CUDA_TRY(c, cudaMemcpyAsync(c->page_tbl_dev + (size_t)slot * g.max_pages_per_seq + p / kPage, &e,
                                        sizeof(int32_t), cudaMemcpyHostToDevice, c->stream));
            CUDA_TRY(c, cudaStreamSynchronize(c->stream));
        }
        c->seq_len[slot] = std::max(c->seq_len[slot], pos0 + n);
    }
    kv_copy_kernel<<<n, 128, 0, c->stream>>>(kv_addr(c, layer - 1), slot, pos0, n, (__nv_bfloat16 *)k,
                                             (__nv_bfloat16 *)v, to_cache);
    CUDA_TRY(c, cudaGetLastError());
    c->st.launches_total += 1;
    return RIVER_OK;
}

int river_read_kv(river_ctx *c, int slot, int layer, int pos0, int n, void *k_out, void *v_out) {
    return kv_copy(c, slot, layer, pos0, n, k_out, v_out, 0);
}
int river_write_kv(river_ctx *c, int slot, int layer, int pos0, int n, const void *k_in, const void *v_in) {
    return kv_copy(c, slot, layer, pos0, n, const_cast<void *>(k_in), const_cast<void *>(v_in), 1);
}

int river_last_lists(river_ctx *c, int32_t *act_idx, int32_t *n_act, int32_t *riv_idx, int32_t *n_riv) {
    if (!c || !act_idx || !n_act || !riv_idx || !n_riv) return RIVER_E_BADARG;
    const river_config &g = c->cfg;
    const int B = c->st.batch_last, L = g.L;
    if (B <= 0) return fail(c, RIVER_E_BADARG, "no decode step has run");
    std::vector<int32_t> a((size_t)(L + 1) * g.max_batch), r((size_t)(L + 1) * g.max_batch);
    CUDA_TRY(c, cudaMemcpyAsync(a.data(), c->act_idx, sizeof(int32_t) * a.size(), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(r.data(), c->riv_idx, sizeof(int32_t) * r.size(), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(n_act, c->n_act, sizeof(int32_t) * (L + 1), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(n_riv, c->n_riv, sizeof(int32_t) * (L + 1), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (int l = 0; l <= L; ++l)
        for (int i = 0; i < B; ++i) {
            act_idx[(size_t)l * B + i] = i < n_act[l] ? a[(size_t)l * g.max_batch + i] : -1;
            riv_idx[(size_t)l * B + i] = i < n_riv[l] ? r[(size_t)l * g.max_batch + i] : -1;
        }
    return RIVER_OK;
}

int river_seq_len(const river_ctx *c, int slot) {
    if (!c || !check_slot(c, slot)) return RIVER_E_BADSLOT;
    return c->seq_len[slot];
}

int river_release(river_ctx *c, int slot) {
    if (!c) return RIVER_E_BADARG;
    if (!check_slot(c, slot)) return fail(c, RIVER_E_BADSLOT, "slot out of range");
    const river_config &g = c->cfg;
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (int i = g.max_pages_per_seq - 1; i >= 0; --i) {
        int32_t &e = c->page_tbl[(size_t)slot * g.max_pages_per_seq + i];
        if (e >= 0) { c->free_pages.push_back(e); e = -1; }
    }
    c->seq_len[slot] = 0;
    CUDA_TRY(c, cudaMemsetAsync(c->page_tbl_dev + (size_t)slot * g.max_pages_per_seq, 0xff,
                                sizeof(int32_t) * g.max_pages_per_seq, c->stream));
    const int32_t cap0 = g.L;  // a new sequence in this slot may go to full depth again
    CUDA_TRY(c, cudaMemcpyAsync(c->slot_cap + slot, &cap0, sizeof(int32_t), cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    return RIVER_OK;
}

int river_stats(river_ctx *c, river_stats_t *out) {
    if (!c || !out) return RIVER_E_BADARG;
    const river_config &g = c->cfg;
    const int L = g.L, B = c->st.batch_last;
    std::vector<int32_t> na(L + 1), nr(L + 1);
    int de = 0;
    CUDA_TRY(c, cudaMemcpyAsync(na.data(), c->n_act, sizeof(int32_t) * (L + 1), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(nr.data(), c->n_riv, sizeof(int32_t) * (L + 1), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(&de, c->dev_err, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    c->st.pages_in_use = g.n_pages - (int)c->free_pages.size();
    // algorithmic bytes of the last decode step from its actual exit pattern
    double bytes = 0.0, layers_run = 0.0;
    if (B > 0 && c->st.steps > 0) {
        const double P = (double)g.d * g.Hq * g.dh + 2.0 * g.d * g.Hkv * g.dh + (double)g.Hq * g.dh * g.d + 3.0 * g.d * g.F;
        const double kv_tok = 2.0 * g.Hkv * g.dh * 2.0;
        for (int l = 0; l < L; ++l) {
            if (na[l] > 0) bytes += 2.0 * P;
            if (nr[l] > 0) bytes += P / 2.0 + 4.0 * P / g.group;
            layers_run += na[l];
        }
        for (int b = 0; b < B; ++b) bytes += (double)L * ((c->last_pos[b] + 1) * kv_tok + kv_tok);
        bytes += 2.0 * g.V * g.d + (double)B * g.d * 2.0;
        c->st.layers_executed_last = layers_run / ((double)B * L);
    }
    c->st.alg_bytes_last_step = bytes;
    const int rc = note_device_error(c, de);
    *out = c->st;
    return rc;
}

int river_profile(river_ctx *c, int enable) {
    if (!c) return RIVER_E_BADARG;
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    if (enable && c->prof_ev.empty()) {
        c->prof_ev.resize(2 * (size_t)(8 * c->cfg.L + 8));
        for (auto &e : c->prof_ev) CUDA_TRY(c, cudaEventCreate(&e));
    }
    if (enable) {
        for (int i = 0; i < kNumClasses; ++i) { c->prof_ms[i] = 0; c->prof_bytes[i] = 0; c->prof_launches[i] = 0; }
        c->prof_rec.clear();
    }
    c->profiling = enable != 0;
    return RIVER_OK;
}

int river_profile_read(river_ctx *c, river_kernel_time *out, int cap, int *n_out) {
    if (!c || !out || !n_out) return RIVER_E_BADARG;
    int n = 0;
    for (int i = 0; i < kNumClasses && n < cap; ++i) {
        if (!c->prof_launches[i]) continue;
        std::memset(&out[n], 0, sizeof(out[n]));
        std::strncpy(out[n].name, kClassNames[i], sizeof(out[n].name) - 1);
        out[n].launches = c->prof_launches[i];
        out[n].ms_total = c->prof_ms[i];
        out[n].alg_bytes_total = c->prof_bytes[i];
        ++n;
    }
    *n_out = n;
    return RIVER_OK;
}

void river_destroy(river_ctx *c) {
    if (!c) return;
    cudaStreamSynchronize(c->stream);
    for (auto &e : c->prof_ev) cudaEventDestroy(e);
    for (auto &ge : c->graphs) if (ge.exec) cudaGraphExecDestroy(ge.exec);
    for (int i = 0; i < kStaging; ++i) {
        if (c->meta_host[i]) { cudaFreeHost(c->meta_host[i]); cudaEventDestroy(c->meta_ev[i]); }
    }
    if (c->pin_io) cudaFreeHost(c->pin_io);
    if (c->off_copy) {
        cudaStreamSynchronize(c->off_copy);
        for (int i = 0; i < 2; ++i) { cudaEventDestroy(c->off_ready[i]); cudaEventDestroy(c->off_freed[i]); }
        cudaStreamDestroy(c->off_copy);
    }
    delete c;
}

const char *river_last_error(const river_ctx *c) { return c ? c->err.c_str() : g_init_error.c_str(); }

}  // extern "C"
