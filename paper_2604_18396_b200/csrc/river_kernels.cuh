// The small kernels of the decode step that are not projections or attention (sm_100a): the step prologue (a0, a1, a9),
// the exit score / decision / compaction kernel (a6, a7) and the cache copy behind river_read_kv / river_write_kv.
#pragma once
#include "mbar_tma.cuh"

namespace river {

// ---------------------------------------------------------------- step prologue
// Applies the page-table updates of this step, embeds the tokens (a0), resets the per-row exit state and the
// score diagnostics, and tabulates cos/sin of the rotary angles of every row's position.
__global__ void step_begin_kernel(const StepMeta *meta, const int32_t *upd, /* [3][max_batch]: slot, idx, page */
                                  int32_t *page_tbl, int max_pages_per_seq, int max_batch,
                                  const uint16_t *embed, int d, int V, float *h0, const int32_t *row_pos,
                                  const double *inv_freq, int half_dh, float2 *rope_cs,
                                  int L, int entry_layer, uint8_t *exited /* flags entering block 1 */,
                                  int *dev_err, Lists lists, int32_t *hint_act, unsigned *ticket) {
    __shared__ int s_cnt[66];
    __shared__ bool s_last;
    pdl_launch();
    pdl_wait();
    const int b = blockIdx.x;
    const int n_rows = meta->n_rows;
    const int32_t *tok = meta->tok, *forced = meta->forced;
    int32_t *exit_layer = meta->exit_layer;
    float *scores = meta->scores;
    if (b == 0) {
        for (int i = threadIdx.x; i < meta->n_updates; i += blockDim.x)
            page_tbl[(size_t)upd[i] * max_pages_per_seq + upd[max_batch + i]] = upd[2 * max_batch + i];
    }
    if (b < n_rows) {
        int t = tok[b];
        if (t < 0 || t >= V) {
            if (threadIdx.x == 0) atomicExch(dev_err, DEV_BAD_TOKEN);
            t = 0;
        }
        const uint16_t *e = embed + (size_t)t * d;
        for (int i = threadIdx.x; i < d; i += blockDim.x) h0[(size_t)b * d + i] = bf16f(e[i]);
        const int pos = row_pos[b];
        for (int i = threadIdx.x; i < half_dh; i += blockDim.x) {
            double s, c;
            sincos((double)pos * inv_freq[i], &s, &c);
            rope_cs[(size_t)b * half_dh + i] = make_float2((float)c, (float)s);
        }
        if (scores)
            for (int i = threadIdx.x; i < L; i += blockDim.x) scores[(size_t)b * L + i] = CUDART_NAN_F;
        if (threadIdx.x == 0) {
            int f = forced ? forced[b] : -1;
            if (f >= 0 && (f > L || f < entry_layer)) {
                atomicExch(dev_err, DEV_BAD_FORCED);
                f = L;
            }
            const bool gone = (f == 0);
            exited[b] = gone ? 1 : 0;
            exit_layer[b] = gone ? 0 : L;
        }
    }
    // the last CTA to finish builds the row lists entering block 1 (a7)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (s_last) {
        __threadfence();
        build_lists(n_rows, exited, 0, lists, hint_act, s_cnt);
        if (threadIdx.x == 0) *ticket = 0;
    }
}

// ---------------------------------------------------------------- a6 + a7: exit score, decision, compaction
// (Steps of five and more rows after every block; steps of up to four rows only after the last block - their
// decisions are folded into the kernel that consumes the block output, see gemv_stream.cuh.)
// One CTA per row of the step.  state_in / state_out: the sticky exit flags entering block l / block l + 1.  A row
// still in the backbone gets s = <h_in, h_out> / (|h_in| |h_out|) (Eq. 1) in
// fp32 with a fixed reduction order and the flag s > tau (strict; NaN fails; a zero norm gives s = 0).  The last
// CTA to finish (atomic ticket, no spinning) applies the eligibility window entry_layer <= l < L, the forced-exit
// hook and the batch mode to the flags, updates the sticky exit state and emits the two ascending row lists
// (a stable partition, bit-exact) and their counts for block l+1.
__global__ void __launch_bounds__(256) score_compact_kernel(const StepMeta *meta, int l, int L, int entry_layer,
                                                            int exit_mode, const float *h_in, const float *h_out,
                                                            int d, uint8_t *pass, const uint8_t *state_in,
                                                            uint8_t *state_out, Lists lists, int32_t *hint_act,
                                                            unsigned *ticket, int32_t *fail, const int32_t *row_slot,
                                                            int32_t *slot_cap) {
    // slot_cap (Mono-Decreasing Exit only, else null): per sequence the depth its previous token reached; a row leaves
    // at that depth at the latest, and its own exit layer becomes the sequence's new cap
    __shared__ float red[3][8];
    __shared__ int s_cnt[66];
    __shared__ bool s_last;
    __shared__ int s_allpass;
    pdl_launch();
    // per-step constants (uploaded before the step's first kernel): fetched while the predecessor still runs, so the
    // decision below waits for nothing but the scores
    const int n = meta->n_rows;
    const float *tau = meta->tau;
    const int32_t *forced = meta->forced;
    int32_t *exit_layer = meta->exit_layer;
    float *scores = meta->scores;
    const int row = blockIdx.x;
    const float tau_row = row < n ? tau[row] : 0.f;
    int forced_mine = -1;  // thread b of the deciding CTA keeps row b's forced exit layer (rows beyond blockDim: read later)
    if (forced && (int)threadIdx.x < n) forced_mine = forced[threadIdx.x];
    pdl_wait();
    const bool eligible = (l >= 1) && (l >= entry_layer) && (l < L);
    if (n == 1 && gridDim.x == 1) {
        // A step of one row: its exit flag and both state vectors are requested together (one round trip), and one
        // thread takes the decision and writes the two one-element lists - no ballots, no second pass over flags.
        const int gone_before = state_in[0];
        float ab = 0.f, aa = 0.f, bb = 0.f;
        if (eligible || scores) {
            const float4 *a = reinterpret_cast<const float4 *>(h_in);
            const float4 *b = reinterpret_cast<const float4 *>(h_out);
            for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
                const float4 x = __ldcg(a + i), y = __ldcg(b + i);
                ab += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
                aa += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
                bb += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
            }
            ab = warp_sum(ab); aa = warp_sum(aa); bb = warp_sum(bb);
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            if (lane == 0) { red[0][warp] = ab; red[1][warp] = aa; red[2][warp] = bb; }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            bool pass1 = false;
            if (gone_before == 0 && (eligible || scores)) {
                ab = aa = bb = 0.f;
                for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { ab += red[0][w]; aa += red[1][w]; bb += red[2][w]; }
                float sc = 0.f;
                if (aa > 0.f && bb > 0.f) sc = ab / (sqrtf(aa) * sqrtf(bb));
                pass1 = sc > tau_row;
                if (scores) scores[l - 1] = sc;
                if (fail && !pass1) fail[(size_t)row_slot[0] * (L + 1) + l] = 1;
            }
            bool gone = gone_before != 0;
            if (!gone) {
                bool leave = eligible && pass1;  // with one row the batch minimum is the row itself
                if (forced_mine >= 0) leave = (forced_mine == l) && (l < L);
                if (slot_cap && l < L && l >= slot_cap[row_slot[0]]) leave = true;
                if (leave) {
                    exit_layer[0] = l;
                    if (slot_cap) slot_cap[row_slot[0]] = l;
                    gone = true;
                }
            }
            state_out[0] = gone ? 1 : 0;
            (gone ? lists.riv_idx : lists.act_idx)[(size_t)l * lists.max_batch] = 0;
            lists.n_act[l] = gone ? 0 : 1;
            lists.n_riv[l] = gone ? 1 : 0;
            *hint_act = gone ? 0 : 1;
        }
        return;
    }
    if (row < n && state_in[row] == 0 && (eligible || scores)) {
        const float4 *a = reinterpret_cast<const float4 *>(h_in + (size_t)row * d);
        const float4 *b = reinterpret_cast<const float4 *>(h_out + (size_t)row * d);
        float ab = 0.f, aa = 0.f, bb = 0.f;
        const int nv = d / 4;
        for (int i0 = 0; i0 < nv; i0 += 4 * 256) {  // four loads of each vector in flight per thread
            float4 x[4], y[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * 256 + threadIdx.x;
                x[u] = i < nv ? __ldcg(a + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                y[u] = i < nv ? __ldcg(b + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                ab += x[u].x * y[u].x + x[u].y * y[u].y + x[u].z * y[u].z + x[u].w * y[u].w;
                aa += x[u].x * x[u].x + x[u].y * x[u].y + x[u].z * x[u].z + x[u].w * x[u].w;
                bb += y[u].x * y[u].x + y[u].y * y[u].y + y[u].z * y[u].z + y[u].w * y[u].w;
            }
        }
        ab = warp_sum(ab); aa = warp_sum(aa); bb = warp_sum(bb);
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        if (lane == 0) { red[0][warp] = ab; red[1][warp] = aa; red[2][warp] = bb; }
        __syncthreads();
        if (threadIdx.x == 0) {
            ab = aa = bb = 0.f;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { ab += red[0][w]; aa += red[1][w]; bb += red[2][w]; }
            float s = 0.f;
            if (aa > 0.f && bb > 0.f) s = ab / (sqrtf(aa) * sqrtf(bb));
            pass[row] = (s > tau_row) ? 1 : 0;
            if (scores) scores[(size_t)row * L + (l - 1)] = s;
            if (fail && !(s > tau_row)) fail[(size_t)row_slot[row] * (L + 1) + l] = 1;
        }
    }
    if (gridDim.x > 1) {  // a single CTA is its own last arriver
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    } else {
        __syncthreads();
    }
    // ---- decision for every row still in the backbone
    if (threadIdx.x == 0) s_allpass = 1;
    __syncthreads();
    if (exit_mode == 1) {
        for (int b = threadIdx.x; b < n; b += blockDim.x)
            if (state_in[b] == 0 && !(eligible && pass[b])) atomicAnd(&s_allpass, 0);
        __syncthreads();
    }
    for (int b = threadIdx.x; b < n; b += blockDim.x) {
        if (state_in[b] != 0) { state_out[b] = 1; continue; }
        bool leave = eligible && (exit_mode == 1 ? (s_allpass != 0) : (pass[b] != 0));
        const int f = forced ? (b == (int)threadIdx.x ? forced_mine : forced[b]) : -1;
        if (f >= 0) leave = (f == l) && (l < L);
        if (slot_cap && l < L && l >= slot_cap[row_slot[b]]) leave = true;
        if (leave) {
            exit_layer[b] = l;
            if (slot_cap) slot_cap[row_slot[b]] = l;  // (rows of one prefill chunk share a slot: they all write l)
        }
        state_out[b] = leave ? 1 : 0;
    }
    __syncthreads();
    build_lists(n, state_out, l, lists, hint_act, s_cnt);
    if (threadIdx.x == 0 && gridDim.x > 1) *ticket = 0;
}

// ---------------------------------------------------------------- skipped blocks of the other KV strategies
// State Propagation and Mono-Decreasing Exit (Section 3): a row that has left runs nothing that changes its hidden
// state, so the block's output row is its input row.  CTA (b, j): floats [1024 j, 1024 j + 1024) of row b.
static __global__ void __launch_bounds__(256) carry_rows_kernel(const StepMeta *meta, const uint8_t *state, const float *h_in,
                                                                float *h_out, int d) {
    pdl_launch();
    pdl_wait();
    const int b = blockIdx.x;
    if (b >= meta->n_rows || state[b] == 0) return;
    const int i = blockIdx.y * 256 + threadIdx.x;
    if (i < d / 4)
        reinterpret_cast<float4 *>(h_out + (size_t)b * d)[i] = __ldcg(reinterpret_cast<const float4 *>(h_in + (size_t)b * d) + i);
}

// KV Mask (Section 3): at the end of a step, note for every row's position how many backbone blocks its token ran -
// the later tokens' attention in block l sees a position only if that number is at least l.
static __global__ void depth_note_kernel(const StepMeta *meta, const int32_t *row_slot, const int32_t *row_pos,
                                         uint8_t *pos_depth, int stride) {
    pdl_launch();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < meta->n_rows) pos_depth[(size_t)row_slot[b] * stride + row_pos[b]] = (uint8_t)meta->exit_layer[b];
}

// ---------------------------------------------------------------- prologue of the single-stage entry points
// river_attention / river_project_kv run one stage of the path for a caller-given list of rows: this kernel tabulates
// the rotary angles of the rows' positions and puts all rows on one weight set of block `l0 + 1` (exit flags, row
// lists, counts, prefetch hint), as the step prologue and the compaction would have.
static __global__ void stage_begin_kernel(const StepMeta *meta, const int32_t *row_pos, const double *inv_freq, int half_dh,
                                          float2 *rope_cs, uint8_t *state, Lists lists, int l0, int on_exit_layer,
                                          int32_t *hint_act) {
    const int b = blockIdx.x, n = meta->n_rows;
    if (b >= n) return;
    const int pos = row_pos[b];
    for (int i = threadIdx.x; i < half_dh; i += blockDim.x) {
        double s, c;
        sincos((double)pos * inv_freq[i], &s, &c);
        rope_cs[(size_t)b * half_dh + i] = make_float2((float)c, (float)s);
    }
    if (threadIdx.x == 0) {
        state[b] = on_exit_layer ? 1 : 0;
        (on_exit_layer ? lists.riv_idx : lists.act_idx)[(size_t)l0 * lists.max_batch + b] = b;
        if (b == 0) {
            lists.n_act[l0] = on_exit_layer ? 0 : n;
            lists.n_riv[l0] = on_exit_layer ? n : 0;
            *hint_act = on_exit_layer ? 0 : n;
        }
    }
}

// ---------------------------------------------------------------- self-test of the bounded waits
// Runs the library's bounded mbarrier wait on a barrier that nobody completes: after `limit` polls the wait gives up,
// records DEV_WAIT_TIMEOUT in the error word and the kernel returns normally (no trap, no endless loop).
static __global__ void wait_timeout_probe_kernel(int *dev_err, uint32_t limit) {
    __shared__ uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(smem_u32(&bar), 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &s_abort, dev_err, limit);
    __syncthreads();
}

// ---------------------------------------------------------------- cache copy in / out (bf16 [n][Hkv][dh])
__global__ void kv_copy_kernel(KvAddr kv, int slot, int pos0, int n, __nv_bfloat16 *k_io, __nv_bfloat16 *v_io,
                               int to_cache) {
    const int i = blockIdx.x;  // position index
    if (i >= n) return;
    const int pos = pos0 + i;
    const int page = kv.page_tbl[(size_t)slot * kv.max_pages_per_seq + pos / kPage];
    const int w = kv.Hkv * kv.dh;
    for (int t = threadIdx.x; t < w; t += blockDim.x) {
        const int kvh = t / kv.dh, e = t % kv.dh;
        const size_t ok = kv.base(page, 0, kvh, pos % kPage) + e, ov = kv.base(page, 1, kvh, pos % kPage) + e;
        if (to_cache) {
            kv.pool[ok] = k_io[(size_t)i * w + t];
            kv.pool[ov] = v_io[(size_t)i * w + t];
        } else {
            k_io[(size_t)i * w + t] = kv.pool[ok];
            v_io[(size_t)i * w + t] = kv.pool[ov];
        }
    }
}

}  // namespace river
