// Launch functions of the kernel families, one translation unit each (internal).
#pragma once
#include "river_ctx.h"
#include "gemv_stream.cuh"

namespace river {

// launch_stream.cu: projections on CUDA cores (rows <= 4 per pass), LM head, argmax merge
template <class P>
cudaError_t launch_stream(river_ctx *c, const P &p, const ProjIn &in, const RowLists &rl, int K, int tasks_r2, int n,
                          int has_river, bool pdl, int skip_backbone, const DecideArgs &dec);
extern template cudaError_t launch_stream<QkvProblem>(river_ctx *, const QkvProblem &, const ProjIn &, const RowLists &, int, int, int, int, bool, int, const DecideArgs &);
extern template cudaError_t launch_stream<ResidProblem>(river_ctx *, const ResidProblem &, const ProjIn &, const RowLists &, int, int, int, int, bool, int, const DecideArgs &);
extern template cudaError_t launch_stream<GateUpProblem>(river_ctx *, const GateUpProblem &, const ProjIn &, const RowLists &, int, int, int, int, bool, int, const DecideArgs &);
cudaError_t launch_head_stream(river_ctx *c, const HeadArgs &a, int n_head);
cudaError_t launch_argmax_final(river_ctx *c, int n_head, int n_parts);

// launch_attn.cu: paged GQA decode attention (TMA-fed split-KV kernel; small-step kernel for 1-4 rows)
cudaError_t launch_attention(river_ctx *c, int n, int layer0);
bool prefill_attn_supported(const river_ctx *c);
cudaError_t launch_attention_prefill(river_ctx *c, int n, int layer0);  // tensor-core causal attention of a prefill chunk

}  // namespace river
