// Launches of the CUDA-core streaming kernels: projections of steps of up to four rows per pass, the LM head and
// the merge of its argmax partials.
#include <algorithm>
#include <cmath>

#include "launch.h"

namespace river {

namespace {

// Launch geometry: warps per CTA and CTAs per SM such that every warp gets the same number of tasks (a task is R
// weight rows) and at least 16 warps per SM have loads in flight; searched once per (kernel, task count, K).
struct StreamGeom { int threads, grid; };

template <class Kern>
StreamGeom pick_geometry(river_ctx *c, Kern kern, int tasks, size_t smem) {
    StreamGeom best{256, c->num_sms};
    double best_cost = 1e30;
    int best_w = 0;
    for (int w = 4; w <= 16; ++w) {
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, w * 32, smem) != cudaSuccess || occ < 1) continue;
        occ = std::min(occ, 64 / w);
        for (int o = 1; o <= occ; ++o) {
            const int ctas = c->num_sms * o;
            const int per_cta = (tasks + ctas - 1) / ctas;
            const int rounds = (per_cta + w - 1) / w;
            const int W = w * o;
            const double cost = rounds * (W < 16 ? 16.0 / W : 1.0) * (1.0 + 0.002 * o);  // few large CTAs share x loads
            if (cost < best_cost - 1e-9 || (std::fabs(cost - best_cost) < 1e-9 && W > best_w)) {
                best_cost = cost; best_w = W; best = StreamGeom{w * 32, ctas};
            }
        }
    }
    return best;
}

template <class P, int N, int R>
cudaError_t launch_stream_t(river_ctx *c, const P &p, const ProjIn &in, const RowLists &rl, int K, int tasks,
                            int has_river, bool pdl, int skip_backbone, const DecideArgs &dec) {
    const size_t smem = stream_smem_bytes(N, K);
    auto kern = stream_proj_kernel<P, N, R>;
    const void *fn = reinterpret_cast<const void *>(kern);
    const river_ctx::Geom *geom = nullptr;
    for (auto &e : c->geoms)
        if (e.fn == fn && e.tasks == tasks && e.K == K) geom = &e;
    if (!geom) {
        const cudaError_t e = ensure_smem(c, kern, smem);
        if (e != cudaSuccess) return e;
        const StreamGeom g = pick_geometry(c, kern, tasks, smem);
        c->geoms.push_back({fn, tasks, K, g.threads, g.grid});
        geom = &c->geoms.back();
    }
    return launch_k(kern, dim3(geom->grid), dim3(geom->threads), smem, c->stream, pdl, p, in, rl, has_river,
                    xs_stride(K, 32), skip_backbone, dec);
}

}  // namespace

template <class P>
cudaError_t launch_stream(river_ctx *c, const P &p, const ProjIn &in, const RowLists &rl, int K, int tasks_r2, int n,
                          int has_river, bool pdl, int skip_backbone, const DecideArgs &dec) {
    int n_sel = 1;
    while (n_sel < n && n_sel < 4 && stream_smem_bytes(n_sel * 2, K) <= 200 * 1024) n_sel *= 2;
    const int r = K >= 4096 ? 2 : 4;  // weight rows per task
    const int tasks = tasks_r2 * 2 / r;
#define STREAM_CASE(N_, R_) if (n_sel == N_ && r == R_) return launch_stream_t<P, N_, R_>(c, p, in, rl, K, tasks, has_river, pdl, skip_backbone, dec);
    STREAM_CASE(1, 2) STREAM_CASE(2, 2) STREAM_CASE(4, 2)
    STREAM_CASE(1, 4) STREAM_CASE(2, 4) STREAM_CASE(4, 4)
#undef STREAM_CASE
    return cudaErrorInvalidValue;
}
template cudaError_t launch_stream<QkvProblem>(river_ctx *, const QkvProblem &, const ProjIn &, const RowLists &, int, int, int, int, bool, int, const DecideArgs &);
template cudaError_t launch_stream<ResidProblem>(river_ctx *, const ResidProblem &, const ProjIn &, const RowLists &, int, int, int, int, bool, int, const DecideArgs &);
template cudaError_t launch_stream<GateUpProblem>(river_ctx *, const GateUpProblem &, const ProjIn &, const RowLists &, int, int, int, int, bool, int, const DecideArgs &);

cudaError_t launch_head_stream(river_ctx *c, const HeadArgs &a, int n_head) {
    int n_sel = 1;
    while (n_sel < n_head && n_sel < 4) n_sel *= 2;
    const int xstride = xs_stride(a.d, 8);
    const size_t smem = sizeof(float) * (32 + (size_t)n_sel * xstride);
#define HEAD_CASE(N_)                                                                                              \
    if (n_sel == N_) {                                                                                             \
        const cudaError_t e = ensure_smem(c, lm_head_kernel<N_, 4>, smem);                                         \
        if (e != cudaSuccess) return e;                                                                            \
        return launch_k(lm_head_kernel<N_, 4>, dim3(c->head_grid), dim3(256), smem, c->stream, true, a, xstride); \
    }
    HEAD_CASE(1) HEAD_CASE(2) HEAD_CASE(4)
#undef HEAD_CASE
    return cudaErrorInvalidValue;
}

cudaError_t launch_argmax_final(river_ctx *c, int n_head, int n_parts) {
    return launch_k(argmax_final_kernel, dim3(n_head), dim3(128), 0, c->stream, true, c->meta(),
                    (const float *)c->part_val, (const int32_t *)c->part_idx, n_parts,
                    c->rows_distinct ? c->exit_hist : (unsigned long long *)nullptr);  // (not for prefill chunks)
}

}  // namespace river
