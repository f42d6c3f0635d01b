// Host-side state of one decode context and the launch helpers shared by the translation units of the library.
// (Internal: the public interface is include/river.h.)
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <string>
#include <utility>
#include <vector>

#include "../../include/river.h"
#include "river_common.cuh"

constexpr int kStaging = 4;  // pinned metadata buffers in flight
enum KernelClass { K_BEGIN, K_QKV, K_ATTN, K_OPROJ, K_GATEUP, K_DOWN, K_SCORE, K_HEAD, K_ARGMAX, K_PREFILL_ATTN, kNumClasses };

struct river_ctx {
    river_config cfg;        // as given, except max_batch = max(max_batch, prefill_chunk): rows per launch sequence
    int user_max_batch = 0;  // rows per decode step the caller asked for
    std::vector<river_layer_weights> layers;
    const uint16_t *embed, *lm_head, *final_norm;
    cudaStream_t stream;
    int device = 0, num_sms = 0;
    __nv_bfloat16 *pool = nullptr;

    // workspace
    float *h[3], *qbuf, *obuf, *act, *part_val, *tau_i, *logits_i, *scores_i;
    float2 *rope_cs, *part_ml;
    float *part_o;
    CUtensorMap kv_tmap;
    int attn_splits_now = 1;
    bool attn_small_now = false;  // this step's attention runs on the small-step kernel (short contexts, 1-4 rows)
    unsigned *attn_tickets, *tickets;  // [max_batch*Hkv], [4]
    // tensor-core path: operand buffers, tensor maps of every weight matrix
    __nv_bfloat16 *tc_xhi = nullptr, *tc_xlo = nullptr;
    __nv_bfloat16 *tc_x4 = nullptr;  // the same pair for the exit-layer rows (f16 bits): both kernels of a projection run at once
    __nv_bfloat16 *tc_xalt = nullptr, *tc_x4alt = nullptr;  // second set: operand rows written by the PREVIOUS projection's
                                                            // epilogues (gate/up -> down) while that projection still reads its own
    int tc_max_pad = 0, tc_kmax = 0;
    bool tc_ok = false;
    struct LayerMaps { CUtensorMap q, k, v, o, g, u, d; };
    std::vector<LayerMaps> tc_maps;
    std::vector<LayerMaps> w4_maps;  // code matrices of the exit layers (u8 [rows][K/2], 128-byte boxes)
    bool w4tc_ok = false;
    CUtensorMap tc_map_head;
    // operand maps of the tensor-core projections for (K, padded rows): up to 128 rows the lo rows follow the hi rows
    // in one buffer (`lo_ptr` = tc_xhi + np K) and `hi` covers both (one copy per k-block); beyond, two buffers
    struct BMap { int K, np; bool w4, alt, one; __nv_bfloat16 *base, *lo_ptr; CUtensorMap hi, lo; };
    std::vector<BMap> tc_bmaps;
    int32_t *hint_act;
    const uint8_t *attn_skip = nullptr;  // exit flags of the block whose attention is being launched (strategies that run nothing for rows that left), else null
    uint8_t *pos_depth = nullptr;  // [max_seqs][max_pages_per_seq * 16] KV Mask: backbone blocks the token at each position ran
    int attn_layer1 = 0;           // block (1-based) whose attention is being launched (KV Mask: the visibility test)
    unsigned long long *exit_hist = nullptr;  // [L + 1] exit layers of all decoded tokens so far (river_exit_histogram)
    int32_t *slot_cap = nullptr;  // [max_seqs] Mono-Decreasing Exit: the depth the sequence's last token reached
    bool prefill_attn_now = false;  // this chunk's attention runs on the tensor-core prefill kernel
    bool rows_distinct = true;  // every row of the current step is a different sequence (decode), not a prefill chunk
    struct GraphEntry { int n; bool small_attn; int attn_splits; cudaGraphExec_t exec; int launches; };
    std::vector<GraphEntry> graphs;
    double *inv_freq;
    int32_t *act_idx, *riv_idx, *n_act, *n_riv, *page_tbl_dev, *part_idx, *tok_i, *forced_i, *exit_i, *next_i;
    int32_t *meta_dev;  // [kMetaHdr + 11*max_batch]: StepMeta, row_slot, row_pos, upd[3], head_rows, row_page, row_forced,
                        // tile_row0, tile_rows (query tiles of a prefill chunk), attn_order
    int32_t *prefill_fail;  // [max_seqs][L+1]: 1 where some prompt position of the sequence failed Eq. 1 after block l
    uint8_t *state;     // [(L+1)][state_stride]: sticky exit flags of the rows entering block l + 1 (entry L: at the LM head)
    int state_stride = 0;
    uint8_t *pass;
    int *dev_err;
    size_t ws_bytes = 0;

    // host state
    std::vector<int32_t> page_tbl, seq_len, free_pages;
    int32_t *meta_host[kStaging] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t meta_ev[kStaging];
    int meta_next = 0;
    void *pin_io = nullptr;  // pinned staging for the *_host entry point
    size_t pin_io_bytes = 0;
    std::vector<int32_t> last_pos;  // positions of the rows of the last decode step
    int head_grid = 0;

    river_stats_t st{};
    std::string err;

    // backbone offloading: blocks >= off_first keep their bf16 matrices in pinned host memory and are staged, on
    // demand, into the two device slots their layer entries alias
    int off_first = 0;  // 0 = off
    std::vector<river_layer_weights> off_host;
    cudaStream_t off_copy = nullptr;
    cudaEvent_t off_ready[2] = {nullptr, nullptr}, off_freed[2] = {nullptr, nullptr};
    int off_slot_layer[2] = {-1, -1};

    // per-context launch bookkeeping: the largest dynamic shared memory size set per kernel, and the launch geometry
    // of the streaming kernels per (kernel, task count, K)
    struct SmemAttr { const void *fn; size_t bytes; };
    std::vector<SmemAttr> smem_attr;
    struct Geom { const void *fn; int tasks, K, threads, grid; };
    std::vector<Geom> geoms;

    // optional per-kernel timing (river_profile): events around every launch of a step
    bool profiling = false;
    std::vector<cudaEvent_t> prof_ev;
    struct ProfRec { int cls; double bytes_act, bytes_riv; int list_idx; };
    std::vector<ProfRec> prof_rec;
    double prof_ms[kNumClasses] = {0}, prof_bytes[kNumClasses] = {0};
    int64_t prof_launches[kNumClasses] = {0};

    int meta_ints() const { return river::kMetaHdr + 11 * cfg.max_batch; }
    river::StepMeta *meta() const { return reinterpret_cast<river::StepMeta *>(meta_dev); }
    int32_t *row_slot() const { return meta_dev + river::kMetaHdr; }
    int32_t *row_pos() const { return meta_dev + river::kMetaHdr + cfg.max_batch; }
    int32_t *upd() const { return meta_dev + river::kMetaHdr + 2 * cfg.max_batch; }
    int32_t *head_rows() const { return meta_dev + river::kMetaHdr + 5 * cfg.max_batch; }
    int32_t *row_page() const { return meta_dev + river::kMetaHdr + 6 * cfg.max_batch; }  // page of each row's new position
    int32_t *row_forced() const { return meta_dev + river::kMetaHdr + 7 * cfg.max_batch; }  // prefill: forced exit per row
    int32_t *tile_row0() const { return meta_dev + river::kMetaHdr + 8 * cfg.max_batch; }
    int32_t *tile_rows() const { return meta_dev + river::kMetaHdr + 9 * cfg.max_batch; }
    int32_t *attn_order() const { return meta_dev + river::kMetaHdr + 10 * cfg.max_batch; }  // rows, longest context first
    uint8_t *state_at(int l) const { return state + (size_t)l * state_stride; }
};

namespace river {

// Launch with the programmatic-dependent-launch attribute: the kernel may start while its predecessor in the
// stream is still running and orders itself with griddepcontrol.wait.  Every kernel launched this way calls
// griddepcontrol.wait before it touches anything a predecessor writes.
template <class... KArgs, class... Args>
cudaError_t launch_kc(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                      int cluster_x, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    int na = 0;
    if (pdl) {
        at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (cluster_x > 1) {  // consecutive CTAs along x form a thread-block cluster
        at[na].id = cudaLaunchAttributeClusterDimension;
        at[na].val.clusterDim.x = cluster_x;
        at[na].val.clusterDim.y = 1;
        at[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = at;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(std::forward<Args>(args))...);
}
template <class... KArgs, class... Args>
cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                     Args &&...args) {
    return launch_kc(kern, grid, block, smem, st, pdl, 1, std::forward<Args>(args)...);
}

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to the context's device: remembered per context, raised when
// a launch needs more than any earlier one.
template <class Kern>
cudaError_t ensure_smem(river_ctx *c, Kern kern, size_t bytes) {
    const void *fn = reinterpret_cast<const void *>(kern);
    for (auto &a : c->smem_attr)
        if (a.fn == fn) {
            if (a.bytes >= bytes) return cudaSuccess;
            a.bytes = bytes;
            return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        }
    c->smem_attr.push_back({fn, bytes});
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

inline KvAddr kv_addr(const river_ctx *c, int layer0) {
    KvAddr k;
    k.pool = c->pool;
    k.page_tbl = c->page_tbl_dev;
    k.row_slot = c->row_slot();
    k.row_pos = c->row_pos();
    k.row_page = c->row_page();
    k.n_pages = c->cfg.n_pages;
    k.max_pages_per_seq = c->cfg.max_pages_per_seq;
    k.Hkv = c->cfg.Hkv;
    k.dh = c->cfg.dh;
    k.layer0 = layer0;
    return k;
}

inline W4 w4_of(const river_w4 &r) {
    return W4{(const uint8_t *)r.codes, (const uint16_t *)r.scale, (const uint16_t *)r.zero};
}

}  // namespace river
