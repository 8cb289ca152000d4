// Vocabulary-sharded verification: every rank holds the columns [v_begin, v_begin + V_local) of all
// logit rows (a tensor-parallel output projection leaves them like that) and the full-vocabulary
// logits are never gathered.  What crosses the ranks is small:
//   1. sweep of the local slice          -> one merged state per logit row and shard (16 bytes each)
//   2. row epilogue on all shards' states -> signals, controller, acceptance, stop position (every
//      rank computes the same, from the same gathered bytes)
//   3. weight of the stop position's residual (or target) distribution over the local slice
//      -> two doubles per batch row and shard
//   4. the shard whose slice holds the threshold u * W draws the token.
// The statistics are those of the unsharded path: the online-softmax states merge associatively
// (Sec. 3.1 fixes only the distributions, not how their normalisers are summed), and the inverse
// CDF runs over the vocabulary in index order, shard after shard.
#pragma once

#include "speckv_kernels.cuh"

namespace speckv {

// Phase 1 for short slice rows: one warp per (batch row, logit row), every warp on its own row with
// U loads of 16 bytes in flight per lane; the warp's merged state is the shard's state of that row.
// No partials, no tickets.  (Wider slices use sweep_kernel with export_state set.)
template <typename T, bool ALIGNED, int U>
__global__ void __launch_bounds__(kThreads, kSweepCtasPerSm) shard_rows_kernel(const __grid_constant__ KParams P) {
    const int lane = threadIdx.x & 31;
    const long long w = static_cast<long long>(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    if (w >= static_cast<long long>(P.B) * P.J) return;
    const int b = static_cast<int>(w / P.J), j = static_cast<int>(w - static_cast<long long>(b) * P.J);
    const int gam = P.gamma ? P.gamma[b] : P.G;
    const float Tf = P.temp ? P.temp[b] : P.temp_scalar;
    const bool row_ok = (gam >= 1 && gam <= P.G) && (Tf >= 0.f) && (Tf != __int_as_float(0x7f800000));
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    const bool is_target = j <= P.G;
    const int pos = is_target ? j : j - (P.G + 1);
    const bool active = row_ok && (is_target ? pos <= gam : pos < gam);
    float4 st = make_float4(0.f, 0.f, 0.f, 0.f);
    if (active) {
        if (is_target) {
            const T* row = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(pos) * P.tsp;
            if (greedy) {
                st = sweep_warp<T, ALIGNED, PATH_ARGMAX, U, 32, false>(row, 0, P.V, lane, scale, nullptr);
                const int idx = __float_as_int(st.y);
                if (idx != 0x7fffffff) st.y = __int_as_float(idx + P.v_begin);
            } else {
                st = sweep_warp<T, ALIGNED, PATH_TARGET, U, 32, false>(row, 0, P.V, lane, scale, nullptr);
            }
        } else {
            const T* row = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(pos) * P.dsp;
            if (lane == 0 && !greedy) {
                // both logits at the draft token, if it falls into this slice
                const int x = __ldg(P.tok + static_cast<long long>(b) * P.G + pos) - P.v_begin;
                if (x >= 0 && x < P.V) {
                    const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(pos) * P.tsp;
                    SPECKV_ST(P.tokl[static_cast<long long>(b) * P.G + pos], make_float2(elem_to_float(row, x), elem_to_float(trow, x)));
                }
            }
            st = sweep_warp<T, ALIGNED, PATH_DRAFT, U, 32, false>(row, 0, P.V, lane, scale, nullptr);
        }
    }
    if (lane == 0) P.state[static_cast<long long>(b) * P.J + j] = st;
}

// Phase 2: one warp per batch row; the partials of a logit row are the n_shards gathered states.
template <typename T>
__global__ void __launch_bounds__(kThreads) shard_finish_kernel(const __grid_constant__ KParams P) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b >= P.B) return;
    const int gam = P.gamma ? P.gamma[b] : P.G;
    const float Tf = P.temp ? P.temp[b] : P.temp_scalar;
    const float4* row = P.part + static_cast<long long>(b) * P.J;
    row_epilogue<T>(P, b, gam, Tf, row + P.G + 1 + lane, P.n_shards, row + lane, P.n_shards);
}

// Phase 3: grid B * R.  Chunk sums of the stop position over the local slice: of the row's own
// weights and, for a residual draw, of p as well (the draw falls back to p when the residual is
// numerically empty, and whether it is shows only once all shards' masses are known).  The last
// CTA of a row adds them up.
template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(kThreads, 4) shard_sums_kernel(const __grid_constant__ KParams P) {
    __shared__ int sh_flag;
    __shared__ float sh_cs[kRsStage];
    const int b = blockIdx.x / P.R;
    const int share = blockIdx.x - b * P.R;
    const RowInfo ri = P.info[b];
    if (ri.mode == RS_NONE) {
        if (share == 0 && threadIdx.x < 2) P.weight[2 * static_cast<long long>(b) + threadIdx.x] = 0.0;
        return;
    }
    const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(ri.n) * P.tsp;
    const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(ri.n) * P.dsp;
    float* csum = P.csum + static_cast<long long>(b) * P.nchunk;
    float* csum_p = P.csum2 + static_cast<long long>(b) * P.nchunk;
    RsConst c = rs_const(ri, ri.mode);
    const int c0 = share * P.chunks_per_cta;
    const int c1 = min(P.nchunk, c0 + P.chunks_per_cta);
    if (ri.mode == RS_RESIDUAL) rs_chunk_sums<T, ALIGNED>(c, trow, drow, c0, c1, P.V, csum);
    c.mode = RS_BONUS;
    rs_chunk_sums<T, ALIGNED>(c, trow, drow, c0, c1, P.V, csum_p);

    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        sh_flag = (atomicAdd(P.tick2 + b, 1) == P.R - 1);
    }
    __syncthreads();
    if (!sh_flag) return;
    __threadfence();
    const int per_lane = (P.nchunk + 31) / 32;
    double own, W_res = 0.0;
    if (ri.mode == RS_RESIDUAL) {
        RsSums cs = rs_stage_sums(sh_cs, csum, P.nchunk);
        if (threadIdx.x < 32) W_res = rs_total(cs, P.nchunk, per_lane, &own);
        __syncthreads();
    }
    RsSums cp = rs_stage_sums(sh_cs, csum_p, P.nchunk);
    if (threadIdx.x < 32) {
        const double W_p = rs_total(cp, P.nchunk, per_lane, &own);
        if (threadIdx.x == 0) {
            P.weight[2 * static_cast<long long>(b)] = W_res;
            P.weight[2 * static_cast<long long>(b) + 1] = W_p;
        }
    }
}

// Phase 4: one CTA per batch row.  Every rank finds the owning shard from the gathered masses; the
// owner searches its own chunk sums and writes the token into out_tokens[b, n]; the others leave the
// -1 that the row epilogue put there, so an element-wise maximum over the ranks completes the row.
template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(kThreads) shard_pick_kernel(const __grid_constant__ KParams P) {
    __shared__ float sh_cs[kRsStage];
    __shared__ int sh_go;
    __shared__ int sh_mode;
    __shared__ double sh_tau;
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const RowInfo ri = P.info[b];
    if (ri.mode == RS_NONE) return;
    if (warp == 0) {
        // lane r holds shard r's masses (n_shards <= 32)
        double wr = 0.0, wp = 0.0;
        if (lane < P.n_shards) {
            const double* w = P.all_weight + (static_cast<long long>(lane) * P.B + b) * 2;
            wr = w[0];
            wp = w[1];
        }
        // shards are added in index order on every rank, so all ranks see the same totals
        double tot_r = 0.0, tot_p = 0.0;
        for (int r = 0; r < P.n_shards; ++r) {
            tot_r += __shfl_sync(0xffffffffu, wr, r);
            tot_p += __shfl_sync(0xffffffffu, wp, r);
        }
        const bool use_res = (ri.mode == RS_RESIDUAL) && (tot_r > 1e-6);
        const double tot = use_res ? tot_r : tot_p;
        const double tau = static_cast<double>(ri.u2) * tot;
        double run = 0.0, before = 0.0;
        int owner = -1, last_pos = -1;
        double last_before = 0.0;
        for (int r = 0; r < P.n_shards; ++r) {
            const double w = __shfl_sync(0xffffffffu, use_res ? wr : wp, r);
            if (w > 0.0) { last_pos = r; last_before = run; }
            if (owner < 0 && w > 0.0 && run + w > tau) { owner = r; before = run; }
            run += w;
        }
        if (owner < 0) { owner = last_pos; before = last_before; }
        if (lane == 0) {
            sh_go = (owner == P.rank);
            sh_mode = use_res ? RS_RESIDUAL : RS_BONUS;
            sh_tau = tau - before;
            // no shard has any mass: cannot happen for a finite row; same answer as the unsharded path
            if (owner < 0 && P.rank == 0) P.out_tok[static_cast<long long>(b) * (P.G + 1) + ri.n] = 0;
        }
    }
    __syncthreads();
    if (!sh_go) return;
    const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(ri.n) * P.tsp;
    const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(ri.n) * P.dsp;
    const RsConst c = rs_const(ri, sh_mode);
    const float* csum = (sh_mode == RS_RESIDUAL ? P.csum : P.csum2) + static_cast<long long>(b) * P.nchunk;
    const RsSums cs = rs_stage_sums(sh_cs, csum, P.nchunk);
    if (warp != 0) return;
    const int per_lane = (P.nchunk + 31) / 32;
    double own;
    (void)rs_total(cs, P.nchunk, per_lane, &own);
    const int tok = rs_search<T, ALIGNED>(c, trow, drow, cs, P.nchunk, P.V, sh_tau, own, per_lane);
    if (lane == 0) P.out_tok[static_cast<long long>(b) * (P.G + 1) + ri.n] = tok + P.v_begin;
}

}  // namespace speckv
