// Launch functions of the tensor-core projection kernels (internal).
#pragma once
#include "river_ctx.h"
#include "gemm_tc.cuh"

namespace river {

const river_ctx::BMap *tc_bmap(river_ctx *c, int K, int np, bool w4 = false, bool alt = false);

// Both kernels of a projection (backbone rows, exit-layer rows) are in flight together: `phase` says which part of a
// launch function runs - the operand kernel, the GEMM, or both in a row.
enum : int { kTcPrep = 1, kTcGemm = 2, kTcBoth = 3 };
// Shared memory and tensor-memory columns per CTA of the configurations tc_gemm_kernel may run in for `np` operand
// rows (two or three CTAs per SM): what a kernel that shares the SMs with it must budget against.
struct TcFootprint { size_t smem; int cols; };
int tc_footprints(int np, TcFootprint (&out)[2]);
int tc_pick_splits(const river_ctx *c, int tiles, int kb_total, int slots, int min_kb = 4);

// launch_tc.cu: backbone rows, 5 <= rows <= 256
template <class Epi>
cudaError_t launch_tc(river_ctx *c, const ProjIn &in, const CUtensorMap &a0, const CUtensorMap &a1, const CUtensorMap &a2,
                      int K, int tiles, int n, int gateup, int q_tiles, int k_tiles, const int32_t *rows,
                      const int32_t *cnt, const Epi &epi, bool allow_split, const int32_t *hint, int phase = kTcBoth,
                      bool late_release = false, bool alt_operand = false);
#define RIVER_TC_DECL(E) \
    extern template cudaError_t launch_tc<E>(river_ctx *, const ProjIn &, const CUtensorMap &, const CUtensorMap &, const CUtensorMap &, \
                                             int, int, int, int, int, int, const int32_t *, const int32_t *, const E &, bool, const int32_t *, \
                                             int, bool, bool);
RIVER_TC_DECL(TcQkvEpi) RIVER_TC_DECL(TcResidEpi) RIVER_TC_DECL(TcGateUpEpi) RIVER_TC_DECL(TcHeadEpi)
#undef RIVER_TC_DECL

// launch_tc_w4.cu: the operand kernels of both lists as one launch (then launch_tc / launch_tc_w4 with kTcGemm)
cudaError_t launch_tc_prep_pair(river_ctx *c, const ProjIn &in, int K, int n, const int32_t *rows_a, const int32_t *cnt_a,
                                const int32_t *rows_r, const int32_t *cnt_r);

// launch_tc_w4.cu: exit-layer rows through the dequantising kernel: m[0..2] are the code maps, w[0..2] the matching
// scale / zero arrays (one matrix, gate + up, or q + k + v)
template <class Epi>
cudaError_t launch_tc_w4(river_ctx *c, const ProjIn &in, const CUtensorMap *const (&m)[3], const river_w4 *const (&w)[3],
                         int K, int tiles, int n, int gateup, int q_tiles, int k_tiles, const int32_t *rows,
                         const int32_t *cnt, const int32_t *hint, const Epi &epi, int phase = kTcBoth, bool overlap = false,
                         bool alt_operand = false);
#define RIVER_TCW4_DECL(E) \
    extern template cudaError_t launch_tc_w4<E>(river_ctx *, const ProjIn &, const CUtensorMap *const (&)[3], const river_w4 *const (&)[3], \
                                                int, int, int, int, int, int, const int32_t *, const int32_t *, const int32_t *, const E &, \
                                                int, bool, bool);
RIVER_TCW4_DECL(TcQkvEpi) RIVER_TCW4_DECL(TcResidEpi) RIVER_TCW4_DECL(TcGateUpEpi)
#undef RIVER_TCW4_DECL

}  // namespace river
