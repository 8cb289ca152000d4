// Draft-side sampling in one pass over the logits (tokens[b,i] ~ softmax(d_i / T_b) by inverse CDF,
// argmax for T_b = 0; the drafting step of Sec. 3.1).
//
// The inverse CDF needs the running sum of exp((x_v - M) / T) in vocabulary order, and M, the row
// maximum, is known only at the end of the row.  Instead of a second pass, every 256-element chunk
// keeps a pair (m_c, Z_c = sum over the chunk of exp((x_v - m_c) / T)) with a reference m_c at or above
// its elements: rescaled by exp((m_c - M) / T) these are the chunk sums the search needs, 8 bytes per
// 256 logits.  The CTA that
// completes a row stages the rescaled sums in shared memory, finds the chunk that holds u * Z and
// reads that one chunk again.
#pragma once

#include "speckv_kernels.cuh"

namespace speckv {

// grid: B * G * S CTAs, S = P.R shares per logit row; P.csum2 holds the (m_c, Z_c) pairs
// [B*G, nchunk] as float2, P.tick2 one counter per draw, P.tick1 one per batch row, P.rdone
// (here: a per-row status word) zeroed by the host.
template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(kThreads, 4) sample_onepass_kernel(const __grid_constant__ KParams P) {
    __shared__ int sh_flag;
    __shared__ float sh_red[kWarps];
    __shared__ int sh_redi[kWarps];
    __shared__ float sh_cs[kRsStage];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = blockIdx.x / P.R;  // draw: batch row b, drafted position i
    const int share = blockIdx.x - r * P.R;
    const int b = r / P.G, i = r - b * P.G;
    const int gam = P.gamma ? P.gamma[b] : P.G;
    const float Tf = P.temp ? P.temp[b] : P.temp_scalar;
    int bits = 0;
    if (gam < 1 || gam > P.G) bits |= 1;
    if (!(Tf >= 0.f) || Tf == __int_as_float(0x7f800000)) bits |= 8;
    if (bits || i >= gam) {  // nothing to draw at this position
        if (share == 0 && threadIdx.x == 0) {
            P.out_tok[r] = -1;
            if (i == 0 && bits && P.status) P.status[b] = bits;
        }
        return;
    }
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    const T* row = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(i) * P.dsp;
    float2* cz = reinterpret_cast<float2*>(P.csum2) + static_cast<long long>(r) * P.nchunk;
    const float ninf = __int_as_float(0xff800000);

    // ---- this CTA's chunks: KU per warp at a time, the next KU requested before the current ones are used ----
    const int c0 = share * P.chunks_per_cta;
    const int c1 = min(P.nchunk, c0 + P.chunks_per_cta);
    constexpr int KU = sizeof(T) == 2 ? 4 : 2;  // chunks per batch: 16 registers of loads in flight per lane
    int base = c0 + warp;
    float ref_m = ninf;  // sampled rows: the largest element this warp has met (the same in every lane)
    Raw<T> cur[KU];
#pragma unroll
    for (int u = 0; u < KU; ++u)
        cur[u] = (base + u * kWarps < c1) ? rs_load_lane<T, ALIGNED>(row, base + u * kWarps, P.V, ninf) : raw_fill<T>(ninf);
    while (base < c1) {
        const int next = base + KU * kWarps;
        Raw<T> nxt[KU];
#pragma unroll
        for (int u = 0; u < KU; ++u)
            nxt[u] = (next + u * kWarps < c1) ? rs_load_lane<T, ALIGNED>(row, next + u * kWarps, P.V, ninf) : raw_fill<T>(ninf);
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            const int ch = base + u * kWarps;
            if (ch >= c1) break;  // uniform across the warp
            float x[kVec];
            unpack<T>(cur[u], x);
            bool bad = false;
            float lm = ninf;
#pragma unroll
            for (int j = 0; j < kVec; ++j) {
                bad |= (x[j] != x[j]) || (x[j] == __int_as_float(0x7f800000));
                if (x[j] < kFloor) x[j] = ninf;  // below the floor counts as -inf
                lm = fmaxf(lm, x[j]);
            }
            bad = __any_sync(0xffffffffu, bad);
            // The reference of a chunk's sum need not be the chunk's own maximum: any common value at or
            // above it will do.  Sampled rows keep the warp's running maximum and raise it only when a lane
            // sees a larger element (one vote per chunk instead of a five-step reduction); greedy rows need
            // the chunk's maximum itself.
            float mc;
            if (greedy) {
                mc = warp_maxf(lm);
            } else {
                if (__any_sync(0xffffffffu, lm > ref_m)) ref_m = fmaxf(ref_m, warp_maxf(lm));
                mc = ref_m;
            }
            float second;
            if (greedy) {
                int idx = 0x7fffffff;
#pragma unroll
                for (int j = kVec - 1; j >= 0; --j)
                    if (x[j] == mc) idx = min(idx, rs_elem<T>(ch, lane, j));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) idx = min(idx, __shfl_xor_sync(0xffffffffu, idx, o));
                second = __int_as_float(bad ? -2 : idx);
            } else {
                float z = 0.f;
                if (mc > ninf) {
                    const float ref = mc * scale;
#pragma unroll
                    for (int j = 0; j < kVec; ++j) z += ex2f(__fmaf_rn(x[j], scale, -ref));
                }
                z = warp_sumf(z);
                second = bad ? __int_as_float(0x7fc00000) : z;
            }
            if (lane == 0) SPECKV_ST(cz[ch], make_float2(mc, second));
        }
#pragma unroll
        for (int u = 0; u < KU; ++u) cur[u] = nxt[u];
        base = next;
    }

    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        sh_flag = (atomicAdd(P.tick2 + r, 1) == P.R - 1);
    }
    __syncthreads();
    if (!sh_flag) return;
    __threadfence();

    // ---- the row's last CTA: maximum over the chunks, rescaled sums, search ----
    float M = ninf;
    int bad_i = 0, best_idx = 0x7fffffff;
    for (int c = threadIdx.x; c < P.nchunk; c += kThreads) {
        const float2 v = __ldcg(cz + c);
        if (greedy) {
            const int idx = __float_as_int(v.y);
            if (idx == -2) bad_i = 1;
            else if (v.x > M || (v.x == M && idx < best_idx)) { M = v.x; best_idx = idx; }
        } else {
            if (v.y != v.y) bad_i = 1;
            M = fmaxf(M, v.x);
        }
    }
    // block-wide maximum (and, for greedy rows, the lowest index attaining it)
    float wm = warp_maxf(M);
    if (greedy) {
        int cand = (M == wm) ? best_idx : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cand = min(cand, __shfl_xor_sync(0xffffffffu, cand, o));
        if (lane == 0) sh_redi[warp] = cand;
    }
    bad_i = __any_sync(0xffffffffu, bad_i) ? 1 : 0;
    if (lane == 0) sh_red[warp] = wm;
    __syncthreads();
    float Mall = sh_red[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) Mall = fmaxf(Mall, sh_red[w]);
    int tok_greedy = 0x7fffffff;
    if (greedy) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w)
            if (sh_red[w] == Mall) tok_greedy = min(tok_greedy, sh_redi[w]);
    }
    const int any_bad = __syncthreads_or(bad_i);
    int status = 0;
    if (any_bad || !(Mall > kFloor)) status = 4;

    int tok = -1;
    if (!status) {
        if (greedy) {
            tok = tok_greedy;
        } else {
            for (int c = threadIdx.x; c < P.nchunk; c += kThreads) {
                const float2 v = __ldcg(cz + c);
                sh_cs[c] = (v.y > 0.f) ? v.y * ex2f((v.x - Mall) * scale) : 0.f;
            }
            __syncthreads();
            if (warp == 0) {
                RsSums cs;
                cs.sh = sh_cs;
                cs.glob = nullptr;
                const int per_lane = (P.nchunk + 31) / 32;
                double own;
                const double W = rs_total(cs, P.nchunk, per_lane, &own);
                RsConst c;
                c.mode = RS_BONUS;
                c.scale = scale;
                c.lp_hi = Mall * scale; c.lp_lo = 0.f; c.lq_hi = 0.f; c.lq_lo = 0.f;
                const double tau = static_cast<double>(__ldg(P.u + r)) * W;
                tok = rs_search<T, ALIGNED>(c, row, row, cs, P.nchunk, P.V, tau, own, per_lane);
            }
        }
    }
    if (warp != 0) return;
    // per-row bookkeeping: the row's status is the OR over its positions; a flagged row gives -1 everywhere
    int last = 0;
    if (lane == 0) {
        P.out_tok[r] = status ? -1 : tok;
        if (status) atomicOr(P.rdone + b, status);
        __threadfence();
        last = (atomicAdd(P.tick1 + b, 1) == gam - 1);
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) return;
    __threadfence();
    const int st = __ldcg(P.rdone + b);
    if (st && lane < P.G) P.out_tok[static_cast<long long>(b) * P.G + lane] = -1;
    if (lane == 0 && P.status) P.status[b] = st;
}

}  // namespace speckv
