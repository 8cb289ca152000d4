// Staged sweep for sm_100a: persistent CTAs stream the logit rows through a shared-memory ring
// filled by bulk asynchronous copies (cp.async.bulk, completion counted on an mbarrier); consumer
// warps fold each staged 512-byte block into the online softmax statistics behind the Sec. 4.2
// signals and the verification normalisers.  The bytes in flight live in shared memory instead of
// registers, so the memory pipeline stays full while the warps spend their registers on arithmetic.
//
// Work layout.  The logit rows a step needs (for batch row b: target positions 0..gamma_b, then
// draft positions 0..gamma_b-1) are laid end to end in one virtual stream, each row padded to a
// whole number of ring stages.  The stream is cut into equal quanta which the CTAs take in stream
// order from a shared counter, so the load balances itself and batch rows complete progressively.
// A quantum that crosses a row end is a short list of segments (row, granule range); every segment
// ends in one partial.  A batch row is complete when the stages posted for it add up to its padded
// size.
//
// Warp roles in a CTA: 8 consumer warps; one producer warp (a single thread issues the copies); one
// epilogue warp that merges and publishes the segments' partials, so that no consumer ever waits
// for global memory, and that runs row epilogues taken from a global queue of completed rows.
//
// Every wait in this file is bounded: when a limit runs out the thread raises the CTA's error
// flag, the row being worked on gets SPECKV_ROW_TIMEOUT, and all warps of the CTA leave their
// loops at the next check.  No CTA ever waits for another CTA.
#pragma once

#include "speckv_kernels.cuh"

namespace speckv {

constexpr int kPipeWarpsCfg = 8;
constexpr int kPipeWarps = kPipeWarpsCfg;        // consumer warps per CTA
constexpr int kPipeThreads = (kPipeWarps + 2) * 32;  // + one producer warp + one epilogue warp
constexpr int kStageGranCfg = 1024;  // 16-byte granules per ring stage (16 KB)
constexpr int kStagesCfg = 6;
constexpr int kQuantumStages = 16;  // target quantum: 256 KB
constexpr int kStageGran = kStageGranCfg;
constexpr int kStageBytes = kStageGran * 16;
constexpr int kStages = kStagesCfg;
constexpr int kSegSlotsCfg = 32;
constexpr int kPipeMaxBCfg = 1024;
constexpr int kPipeCtasPerSm = 2;  // CTAs per SM
constexpr int kSegSlots = kSegSlotsCfg;          // segments between the consumers and the epilogue warp
constexpr int kPipeMaxB = kPipeMaxBCfg;          // batch rows whose per-row tables fit the CTA
constexpr int kMaxSeg = 32;                          // partial slots per logit row
constexpr int kWaitLimit = 1 << 22;

enum : int { ST_FIRST = 1, ST_LAST = 2, ST_END = 4 };

struct SegInfo {      // one per segment, written by the producer
    int b;            // batch row
    int path;         // PATH_*
    int pos;          // position within the batch row
    int stages;       // padded ring stages of this segment (ticket increment)
    long long part;   // index of this segment's partial in the workspace
    float scale;      // log2(e) / T of the row
    int jrows;        // logit rows of the batch row (ticket total = jrows * stages per row)
};
struct StageDesc {
    int seg;     // running segment number within the CTA
    int n_gran;  // valid granules in the stage
    int gran0;   // granule of the logit row where the stage starts
    int flags;   // ST_*
};

struct PipeShared {
    unsigned long long full[kStages];         // stage filled (bulk copy landed)
    unsigned long long empty[kStages];        // stage released by all consumer warps
    unsigned long long seg_bar[kSegSlots];    // all consumer warps posted their partial of the segment
    unsigned long long slot_free[kSegSlots];  // the epilogue warp is done with the segment slot
    StageDesc desc[kStages];
    SegInfo seg[kSegSlots];
    float4 part[kSegSlots][kPipeWarps];
    int error;
    int total_segs;                           // -1 until the producer has issued its last segment
    int published;                            // set once the epilogue warp has published them all
    long long Q, Tg;                          // quantum and stream length, in granules
    int prefix[kPipeMaxB + 1];                // logit rows of the stream before each batch row
    float temp[kPipeMaxB];                    // the rows' temperature and gamma, read once
    unsigned char gam[kPipeMaxB];             // (0 for a row that contributes nothing)
    int warp_tot[kPipeThreads / 32];
};

// ---- mbarrier and bulk-copy primitives -----------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(unsigned long long* bar, uint32_t parity) {  // non-blocking
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait for the phase with the given parity; false when the limit ran out or the CTA's
// error flag is up.  The bound is a time (about two seconds on the GPU's nanosecond clock), not a number of
// tries: one try may come back at once or only when the hardware's own limit for a try is up.
constexpr unsigned long long kWaitNs = 2000000000ull;
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, volatile int* error) {
    unsigned long long t0 = 0;
    for (int it = 0; it < kWaitLimit; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
        if (ok) return true;
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (t0 == 0) t0 = now;
        else if (now - t0 > kWaitNs) break;
        if ((it & 63) == 63 && *error) return false;
    }
    *error = 1;
    return false;
}
// global -> shared bulk copy of `bytes` (multiple of 16, both addresses 16-byte aligned); completion
// is counted on `bar`.  No multicast: the destination is this CTA's own shared memory.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
#ifdef SPECKV_DEBUG
    // the consumers wait for these bytes, so a copy that fails the check is not dropped but redirected to
    // the start of the draft logits (registered range 0), which is always there and large enough here
    if (!dbg_ok(src, bytes, DBG_COPY)) src = reinterpret_cast<const void*>(g_dbg_ranges.lo[0]);
#endif
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// warp-wide maximum in one instruction (sm_100a); NaN wins
__device__ __forceinline__ float warp_max_nan(float v) {
    float r;
    asm volatile("redux.sync.max.NaN.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ int ld_volatile(const int* p) { return *reinterpret_cast<const volatile int*>(p); }

// How many logit rows a batch row contributes to the stream.
__device__ __forceinline__ int pipe_rows_of(const KParams& P, int gam, float Tf) {
    const bool ok = (gam >= 1 && gam <= P.G) && (Tf >= 0.f) && (Tf != __int_as_float(0x7f800000));
    if (!ok) return 0;
    return (P.mode & MODE_VERIFY) ? 2 * gam + 1 : gam;
}

// ---- staged data -> raw register images -----------------------------------------------------
// A "unit" is what one warp folds in one step: kVec elements per lane.  bf16: one 512-byte block
// (lane l owns granule l).  fp32: two consecutive blocks (lane l owns granule l of each), so that
// every shared-memory read is a conflict-free 16 bytes per lane.
template <typename T> struct PipeUnit {
    static constexpr int kGran = sizeof(T) == 2 ? 32 : 64;               // granules per unit
    static constexpr int kPerWarp = kStageGran / kGran / kPipeWarps;     // units per warp and stage
    static_assert(kPerWarp * kGran * kPipeWarps == kStageGran, "a stage must split evenly over the consumer warps");
};

template <typename T, bool FULL>
__device__ __forceinline__ Raw<T> stage_raw(const uint4* stage, int unit, int lane, int n_gran, float pad) {
    Raw<T> r;
    if constexpr (sizeof(T) == 2) {
        const int g = unit * 32 + lane;
        if (FULL || g < n_gran) r.a = stage[g];
        else r = raw_fill<T>(pad);
    } else {
        const int g = unit * 64 + lane;
        const uint32_t w = __float_as_uint(pad);
        r.a = (FULL || g < n_gran) ? stage[g] : make_uint4(w, w, w, w);
        r.b = (FULL || g + 32 < n_gran) ? stage[g + 32] : make_uint4(w, w, w, w);
    }
    return r;
}

// element index (within the logit row) of the first element of each half of a lane's unit
template <typename T>
__device__ __forceinline__ void unit_elems(int gran0, int unit, int lane, int& ea, int& eb) {
    if constexpr (sizeof(T) == 2) {
        ea = (gran0 + unit * 32 + lane) * 8;
        eb = ea + 4;
    } else {
        ea = (gran0 + unit * 64 + lane) * 4;
        eb = ea + 128;
    }
}

// argmax step whose two halves of kVec/2 elements start at element ea and eb
template <typename T>
__device__ __forceinline__ void argmax_step_split(ArgmaxState& as, const Raw<T>& raw, int ea, int eb) {
    if (!raw_exceeds<false>(raw, as.best)) return;
    float x[kVec];
    unpack<T>(raw, x);
#pragma unroll
    for (int j = 0; j < kVec; ++j) {
        const int idx = (j < kVec / 2) ? ea + j : eb + j - kVec / 2;
        as.bad |= (x[j] != x[j]) || (x[j] == __int_as_float(0x7f800000));
        if (x[j] > as.best || (x[j] == as.best && idx < as.idx)) { as.best = x[j]; as.idx = idx; }
    }
}

// ---- per-warp sweep state -------------------------------------------------------------------
// The running maximum M is the same in all 32 lanes of a warp, so a stage is checked once (one
// warp-wide maximum over everything the warp holds of the stage) instead of once per vector, no
// warm start is needed, and the merge of the lanes at the end of a segment is a plain sum.
//
// DRAFT   M (logit units); cnt = elements equal to M, kept out of the sums so that a dominant
//         token never absorbs the tail; Zx = sum over the others of 2^((x-M)*scale);
//         S = sum of 2^((x-M)*scale) * (x-M).  Partial = (M, cnt, Zx, S); cnt = NaN marks NaN/+inf.
// TARGET  M, r = M*scale; Z = sum 2^(x*scale - r).  Partial = (r, Z).
// ARGMAX  per-lane best value and lowest index.  Partial = (best, index, bad).
struct PipeState {
    float M, r, cnt;
    f2 za, zb, sa, sb;
    bool bad;
    ArgmaxState as;
    __device__ __forceinline__ void init(float scale) {
        M = kFloor; r = kFloor * scale; cnt = 0.f; bad = false;
        za = zb = sa = sb = pack2(0.f, 0.f);
        as.init(kFloor);
    }
    __device__ __forceinline__ float zsum() const { return hsum2(za) + hsum2(zb); }
    __device__ __forceinline__ float ssum() const { return hsum2(sa) + hsum2(sb); }
};

// fast draft unit: every element is below M
template <typename T>
__device__ __forceinline__ void draft_unit_fast(PipeState& st, Raw<T> raw, f2 m2, f2 sc2) {
    raw_floor(raw);
    f2 x[4];
    unpack_pairs(raw, x);
    const f2 d0 = sub2(x[0], m2), d1 = sub2(x[1], m2), d2 = sub2(x[2], m2), d3 = sub2(x[3], m2);
    const f2 e0 = ex2_2(mul2(d0, sc2)), e1 = ex2_2(mul2(d1, sc2));
    const f2 e2 = ex2_2(mul2(d2, sc2)), e3 = ex2_2(mul2(d3, sc2));
    st.za = add2(st.za, e0); st.zb = add2(st.zb, e1);
    st.sa = fma2(e0, d0, st.sa); st.sb = fma2(e1, d1, st.sb);
    st.za = add2(st.za, e2); st.zb = add2(st.zb, e3);
    st.sa = fma2(e2, d2, st.sa); st.sb = fma2(e3, d3, st.sb);
}

// careful draft unit: elements equal to M are counted, the rest summed
template <typename T>
__device__ __forceinline__ void draft_unit_careful(PipeState& st, const Raw<T>& raw, float scale) {
    float x[kVec];
    unpack<T>(raw, x);
    float z = 0.f, sv = 0.f;
#pragma unroll
    for (int j = 0; j < kVec; ++j) {
        const float xj = fmaxf(x[j], kFloor);
        const bool top = (xj == st.M);
        const float dx = xj - st.M;
        const float e = top ? 0.f : ex2f(dx * scale);
        st.cnt += top ? 1.f : 0.f;
        z += e;
        sv = fmaf(e, dx, sv);
    }
    st.za = add2(st.za, pack2(z, 0.f));
    st.sa = add2(st.sa, pack2(sv, 0.f));
}

template <typename T>
__device__ __forceinline__ void target_unit(PipeState& st, const Raw<T>& raw, f2 sc2, f2 nr2) {
    f2 x[4];
    unpack_pairs(raw, x);
    const f2 e0 = ex2_2(fma2(x[0], sc2, nr2)), e1 = ex2_2(fma2(x[1], sc2, nr2));
    const f2 e2 = ex2_2(fma2(x[2], sc2, nr2)), e3 = ex2_2(fma2(x[3], sc2, nr2));
    st.za = add2(st.za, e0); st.zb = add2(st.zb, e1);
    st.za = add2(st.za, e2); st.zb = add2(st.zb, e3);
}

// a new maximum wm (finite, > M) moves everything gathered so far below it
__device__ __forceinline__ void draft_rescale(PipeState& st, float wm, float scale) {
    const float dm = st.M - wm;
    const float f = ex2f(dm * scale);
    const float zall = st.cnt + st.zsum();
    st.sa = pack2(fmaf(dm, zall, st.ssum()) * f, 0.f); st.sb = pack2(0.f, 0.f);
    st.za = pack2(zall * f, 0.f); st.zb = pack2(0.f, 0.f);
    st.cnt = 0.f;
    st.M = wm;
}
__device__ __forceinline__ void target_rescale(PipeState& st, float wm, float scale) {
    const float rn = wm * scale;
    st.za = pack2(st.zsum() * ex2f(st.r - rn), 0.f); st.zb = pack2(0.f, 0.f);
    st.r = rn;
    st.M = wm;
}

// ---- folding one stage ------------------------------------------------------------------------
// full stage, draft or target path: one check per stage, then units without any check
template <typename T, int PATH>
__device__ __forceinline__ void pipe_fold_full(const uint4* stage, int warp, int lane, float scale, PipeState& st) {
    constexpr int kPerWarp = PipeUnit<T>::kPerWarp;
    Raw<T> raw[kPerWarp];
    float um[kPerWarp];
    float lm = __int_as_float(0xff800000);
#pragma unroll
    for (int v = 0; v < kPerWarp; ++v) {
        raw[v] = stage_raw<T, true>(stage, warp + v * kPipeWarps, lane, 0, 0.f);
        um[v] = raw_max(raw[v]);
        lm = max_nan(lm, um[v]);
    }
    const float wm = warp_max_nan(lm);  // NaN propagates
    if constexpr (PATH == PATH_DRAFT) {
        if (!(wm < st.M)) {  // a new maximum, a tie with it, NaN or +inf
            if (!(wm < __int_as_float(0x7f800000))) { st.bad = true; return; }  // the row gets flagged
            if (wm > st.M) draft_rescale(st, wm, scale);
            const f2 m2 = pack2(st.M, st.M), sc2 = pack2(scale, scale);
#pragma unroll
            for (int v = 0; v < kPerWarp; ++v) {  // only units holding an element equal to M take the careful path
                if (__any_sync(0xffffffffu, um[v] == st.M)) draft_unit_careful<T>(st, raw[v], scale);
                else draft_unit_fast<T>(st, raw[v], m2, sc2);
            }
            return;
        }
        const f2 m2 = pack2(st.M, st.M), sc2 = pack2(scale, scale);
#pragma unroll
        for (int v = 0; v < kPerWarp; ++v) draft_unit_fast<T>(st, raw[v], m2, sc2);
    } else {
        if (!(wm <= st.M)) {
            if (!(wm < __int_as_float(0x7f800000))) { st.bad = true; return; }
            target_rescale(st, wm, scale);
        }
        const f2 sc2 = pack2(scale, scale), nr2 = pack2(-st.r, -st.r);
#pragma unroll
        for (int v = 0; v < kPerWarp; ++v) target_unit<T>(st, raw[v], sc2, nr2);
    }
}

// everything else: a partial stage (the end of a logit row) or a greedy row's target (argmax);
// one unit at a time, each with its own check
template <typename T>
__device__ __forceinline__ void pipe_fold_rare(const uint4* stage, int n_gran, int gran0, int path, int warp, int lane,
                                               float scale, PipeState& st) {
    const float pad = (path == PATH_DRAFT) ? kFloor : __int_as_float(0xff800000);
#pragma unroll 1
    for (int v = 0; v < PipeUnit<T>::kPerWarp; ++v) {
        const int unit = warp + v * kPipeWarps;
        if (unit * PipeUnit<T>::kGran >= n_gran) break;
        const Raw<T> raw = stage_raw<T, false>(stage, unit, lane, n_gran, pad);
        if (path == PATH_ARGMAX) {
            int ea, eb;
            unit_elems<T>(gran0, unit, lane, ea, eb);
            argmax_step_split<T>(st.as, raw, ea, eb);
            continue;
        }
        const float um = raw_max(raw);
        const float wm = warp_max_nan(um);
        if (!(wm < __int_as_float(0x7f800000))) { st.bad = true; continue; }
        if (path == PATH_DRAFT) {
            if (wm > st.M) draft_rescale(st, wm, scale);
            if (__any_sync(0xffffffffu, um == st.M)) draft_unit_careful<T>(st, raw, scale);
            else draft_unit_fast<T>(st, raw, pack2(st.M, st.M), pack2(scale, scale));
        } else {
            if (wm > st.M) target_rescale(st, wm, scale);
            target_unit<T>(st, raw, pack2(scale, scale), pack2(-st.r, -st.r));
        }
    }
}

// ---- producer: takes quanta from the shared counter and feeds the ring -----------------------
template <typename T>
__device__ __forceinline__ void pipe_producer(const KParams& P, PipeShared& sh, unsigned char* ring) {
    const long long Lp = P.Lp, Lg = P.Lg, Q = sh.Q, Tg = sh.Tg;
    const bool verify = (P.mode & MODE_VERIFY) != 0;
    volatile int* error = &sh.error;
    int k = 0;      // stages issued
    int sigma = 0;  // segments issued
    // Quanta are handed out in stream order: the first one by CTA index, the rest from a global
    // counter, fetched one quantum ahead so that the round trip never stalls the copies.  A CTA
    // that falls behind simply takes fewer quanta.
    long long q = blockIdx.x;
    while (q * Q < Tg) {
        const long long q_next = static_cast<long long>(gridDim.x) + atomicAdd(P.qcount, 1);
        long long beta = q * Q;
        const long long beta_end = min(Tg, beta + Q);
        long long r = beta / Lp;      // logit row of the stream
        long long o = beta - r * Lp;  // granule within it (a multiple of the stage size, below Lg)
        int lo = 0, hi = P.B;         // batch row holding stream row r: prefix[b] <= r < prefix[b+1]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (sh.prefix[mid] <= r) lo = mid; else hi = mid;
        }
        int b = lo;
        while (beta < beta_end) {
            while (sh.prefix[b + 1] <= r) ++b;  // batch rows without logit rows are skipped
            const int a = static_cast<int>(r - sh.prefix[b]);
            const int gam = sh.gam[b];
            const float Tf = sh.temp[b];
            const bool greedy = (Tf == 0.f);
            const bool is_target = verify && a <= gam;
            const int pos = is_target ? a : (verify ? a - gam - 1 : a);
            const T* row = is_target
                ? static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(pos) * P.tsp
                : static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(pos) * P.dsp;
            const long long seg_end = min(Lp, o + (beta_end - beta));  // padded coordinates
            const long long g_hi = min(Lg, seg_end);
            // the segment's slot must have been released by the epilogue warp
            const int slot = sigma % kSegSlots;
            if (sigma >= kSegSlots && !mbar_wait(&sh.slot_free[slot], ((sigma / kSegSlots) - 1) & 1, error)) return;
            SegInfo si;
            si.b = b;
            si.path = is_target ? (greedy ? PATH_ARGMAX : PATH_TARGET) : PATH_DRAFT;
            si.pos = pos;
            si.stages = static_cast<int>((seg_end - o) / kStageGran);
            si.part = r * kMaxSeg + (q - (r * Lp) / Q);
            si.scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
            si.jrows = sh.prefix[b + 1] - sh.prefix[b];
            sh.seg[slot] = si;
            for (long long g = o; g < g_hi; g += kStageGran) {
                const int n = static_cast<int>(min(static_cast<long long>(kStageGran), g_hi - g));
                const int s = k % kStages;
                if (k >= kStages && !mbar_wait(&sh.empty[s], ((k / kStages) - 1) & 1, error)) return;
                StageDesc d;
                d.seg = sigma;
                d.n_gran = n;
                d.gran0 = static_cast<int>(g);
                d.flags = (g == o ? ST_FIRST : 0) | (g + n >= g_hi ? ST_LAST : 0);
                sh.desc[s] = d;
                mbar_expect_tx(&sh.full[s], static_cast<uint32_t>(n) * 16u);
                bulk_load(ring + static_cast<size_t>(s) * kStageBytes,
                          reinterpret_cast<const unsigned char*>(row) + g * 16, static_cast<uint32_t>(n) * 16u,
                          &sh.full[s]);
                ++k;
            }
            ++sigma;
            beta += seg_end - o;
            ++r;
            o = 0;
        }
        q = q_next;
    }
    // segment total for the epilogue warp, end marker for the consumers
    *reinterpret_cast<volatile int*>(&sh.total_segs) = sigma;
    const int s = k % kStages;
    if (k >= kStages && !mbar_wait(&sh.empty[s], ((k / kStages) - 1) & 1, error)) return;
    StageDesc d;
    d.seg = sigma; d.n_gran = 0; d.gran0 = 0; d.flags = ST_END;
    sh.desc[s] = d;
    mbar_arrive(&sh.full[s]);
}

// ---- epilogue warp --------------------------------------------------------------------------
// It keeps every dependent global-memory round trip off the consumer warps.  Two duties:
//   1. for each finished segment of its own CTA, in order: merge the consumer warps' partials,
//      publish the result, add the segment's stages to the batch row's ticket; whoever completes
//      a batch row puts it on a global queue;
//   2. whenever it has nothing to publish, it takes a completed batch row off that queue (any
//      CTA's) and runs the row epilogue.
// A warp leaves when its own segments are all published and it has seen the queue empty; a row
// put on the queue is therefore always taken by a warp that is still running (its pusher at the
// latest).
template <typename T>
__device__ __forceinline__ void pipe_row_job(const KParams& P, PipeShared& sh, int b, int lane) {
    const bool verify = (P.mode & MODE_VERIFY) != 0;
    const int gam = sh.gam[b];
    const long long Lp = P.Lp, Q = sh.Q;
    const float4 *pd = nullptr, *pt = nullptr;
    int nd = 0, nt = 0;
    if (lane < gam) {  // lane i gathers draft position i and target position i
        const long long r = sh.prefix[b] + (verify ? gam + 1 + lane : lane);
        pd = P.part + r * kMaxSeg;
        nd = static_cast<int>(((r + 1) * Lp - 1) / Q - (r * Lp) / Q) + 1;
    }
    if (verify && lane <= gam) {
        const long long r = sh.prefix[b] + lane;
        pt = P.part + r * kMaxSeg;
        nt = static_cast<int>(((r + 1) * Lp - 1) / Q - (r * Lp) / Q) + 1;
    }
    row_epilogue<T>(P, b, gam, sh.temp[b], pd, nd, pt, nt);
}

// Take a completed batch row off the global queue (whole warp; the answer is the same in all lanes):
// the row, or -1: queue empty, or -2: lost the claim to another warp, look again.
__device__ __forceinline__ int pipe_pop_row(const KParams& P, volatile int* error, int lane) {
    int b = -1;
    if (lane == 0) {
        const int h = ld_volatile(P.qhead);
        if (h < ld_volatile(P.qtail)) {
            b = -2;
            if (atomicCAS(P.qhead, h, h + 1) == h) {
                int v = 0;
                for (int it = 0; it < kWaitLimit && v == 0; ++it) v = ld_volatile(P.rowq + h);  // filled right after the push
                if (v == 0) *error = 1;
                b = v - 1;
                __threadfence();
            }
        }
    }
    return __shfl_sync(0xffffffffu, b, 0);
}

template <typename T>
__device__ __forceinline__ void pipe_epilogue_warp(const KParams& P, PipeShared& sh, int lane) {
    volatile int* error = &sh.error;
    // batch rows that contribute no logit rows (bad gamma / temperature): defaults and status
    for (int b = blockIdx.x; b < P.B; b += gridDim.x)
        if (sh.prefix[b + 1] == sh.prefix[b])
            row_epilogue<T>(P, b, P.gamma ? P.gamma[b] : P.G, sh.temp[b], nullptr, 0, nullptr, 0);

    int sigma = 0;
    bool own_done = false;
    for (int idle = 0; idle < kWaitLimit;) {
        if (__shfl_sync(0xffffffffu, *error, 0)) return;
        // ---- duty 1: the next finished segment of this CTA
        if (!own_done) {
            const int slot = sigma % kSegSlots;
            const int ready = __shfl_sync(0xffffffffu, mbar_test(&sh.seg_bar[slot], (sigma / kSegSlots) & 1) ? 1 : 0, 0);
            if (ready) {
                const SegInfo si = sh.seg[slot];
                // lanes beyond the consumer warps start from an empty partial of the segment's kind
                float4 acc = (si.path == PATH_TARGET) ? make_float4(-3.0e38f, 0.f, 0.f, 0.f)
                           : (si.path == PATH_DRAFT) ? make_float4(kFloor, 0.f, 0.f, 0.f)
                                                     : make_float4(kFloor, __int_as_float(0x7fffffff), 0.f, 0.f);
                if (lane < kPipeWarps) acc = sh.part[slot][lane];
                static_assert(kPipeWarps <= 16, "the merge tree below spans 16 lanes");
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) {
                    const float4 other = shfl_xor4(acc, o);
                    acc = (si.path == PATH_DRAFT) ? merge_draft(acc, other, si.scale)
                        : (si.path == PATH_TARGET) ? merge_target(acc, other) : merge_argmax(acc, other);
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&sh.slot_free[slot]);
                    SPECKV_ST(P.part[si.part], acc);
                    __threadfence();
                    const int total = si.jrows * (P.Lp / kStageGran);
                    if (atomicAdd(P.tick1 + si.b, si.stages) + si.stages == total) {  // row complete: enqueue it
                        const int at = atomicAdd(P.qtail, 1);
                        __threadfence();
                        *reinterpret_cast<volatile int*>(P.rowq + at) = si.b + 1;
                    }
                }
                ++sigma;
                idle = 0;
                continue;
            }
            if (__shfl_sync(0xffffffffu, *reinterpret_cast<volatile int*>(&sh.total_segs), 0) == sigma) own_done = true;
        }
        // ---- duty 2: a completed batch row from the global queue.  Once the producer has issued
        // everything, publishing must not be held up any more: the consumer warps, idle by then,
        // take the remaining rows.
        if (own_done) {
            if (lane == 0) *reinterpret_cast<volatile int*>(&sh.published) = 1;
            return;
        }
        const bool tail = __shfl_sync(0xffffffffu, *reinterpret_cast<volatile int*>(&sh.total_segs), 0) >= 0;
        const int b = tail ? -1 : pipe_pop_row(P, error, lane);
        if (b >= 0) {
            pipe_row_job<T>(P, sh, b, lane);
            idle = 0;
            continue;
        }
        ++idle;
    }
    *error = 1;
}

// ---- the kernel -------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kPipeThreads, kPipeCtasPerSm) pipe_sweep_kernel(const __grid_constant__ KParams P) {
    extern __shared__ __align__(128) unsigned char pipe_smem[];
    PipeShared& sh = *reinterpret_cast<PipeShared*>(pipe_smem);
    unsigned char* ring = pipe_smem + (sizeof(PipeShared) + 127) / 128 * 128;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], kPipeWarps); }
        for (int s = 0; s < kSegSlots; ++s) { mbar_init(&sh.seg_bar[s], kPipeWarps); mbar_init(&sh.slot_free[s], 1); }
        sh.error = 0;
        sh.total_segs = -1;
        sh.published = 0;
        sh.prefix[0] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }

    // per-row tables (every CTA computes the same ones): gamma, temperature, prefix sums of the logit rows
    {
        const int per = (P.B + kPipeThreads - 1) / kPipeThreads;
        const int b0 = min(P.B, static_cast<int>(threadIdx.x) * per), b1 = min(P.B, b0 + per);
        int sum = 0;
        for (int b = b0; b < b1; ++b) {
            const int gam = P.gamma ? P.gamma[b] : P.G;
            const float Tf = P.temp ? P.temp[b] : P.temp_scalar;
            const int j = pipe_rows_of(P, gam, Tf);
            sh.gam[b] = static_cast<unsigned char>(j ? gam : 0);
            sh.temp[b] = Tf;
            sh.prefix[b + 1] = j;
            sum += j;
        }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) sh.warp_tot[warp] = incl;
        __syncthreads();
        int run = incl - sum;
        for (int w = 0; w < warp; ++w) run += sh.warp_tot[w];
        for (int b = b0; b < b1; ++b) {
            run += sh.prefix[b + 1];
            sh.prefix[b + 1] = run;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const long long Lp = P.Lp;
        const long long Tg = static_cast<long long>(sh.prefix[P.B]) * Lp;
        const long long G = gridDim.x;
        const long long qt = static_cast<long long>(kQuantumStages) * kStageGran;
        long long K = (Tg + G * qt / 2) / (G * qt);  // quanta per CTA, rounded
        if (K < 1) K = 1;
        long long Q = (Tg + G * K - 1) / (G * K);
        const long long q_min = (Lp + 27) / 28;      // at most 30 segments per logit row
        if (Q < q_min) Q = q_min;
        Q = (Q + kStageGran - 1) / kStageGran * kStageGran;
        sh.Q = Q;
        sh.Tg = Tg;
    }
    __syncthreads();

    if (warp == kPipeWarps) {
        if (lane == 0) pipe_producer<T>(P, sh, ring);
        return;
    }
    if (warp == kPipeWarps + 1) {
        pipe_epilogue_warp<T>(P, sh, lane);
        return;
    }

    volatile int* error = &sh.error;
    PipeState st;
    st.init(1.f);
    int path = PATH_DRAFT, cur_b = -1;
    float scale = 1.f;
    for (int k = 0;; ++k) {
        const int s = k % kStages;
        if (!mbar_wait(&sh.full[s], (k / kStages) & 1, error)) {
            if (lane == 0 && cur_b >= 0 && P.status) atomicOr(P.status + cur_b, 16);
            return;
        }
        const StageDesc d = sh.desc[s];
        if (d.flags & ST_END) break;
        const uint4* stage = reinterpret_cast<const uint4*>(ring + static_cast<size_t>(s) * kStageBytes);
        if (d.flags & ST_FIRST) {
            const SegInfo& si = sh.seg[d.seg % kSegSlots];
            path = si.path; scale = si.scale; cur_b = si.b;
            st.init(scale);
        }
        if (d.n_gran == kStageGran && path == PATH_DRAFT) pipe_fold_full<T, PATH_DRAFT>(stage, warp, lane, scale, st);
        else if (d.n_gran == kStageGran && path == PATH_TARGET) pipe_fold_full<T, PATH_TARGET>(stage, warp, lane, scale, st);
        else pipe_fold_rare<T>(stage, d.n_gran, d.gran0, path, warp, lane, scale, st);
        if (d.flags & ST_LAST) {  // post this warp's partial of the segment; nobody waits here
            const float nan = __int_as_float(0x7fc00000);
            float4 part;
            if (path == PATH_DRAFT)
                part = make_float4(st.M, warp_sumf(st.bad ? nan : st.cnt), warp_sumf(st.zsum()), warp_sumf(st.ssum()));
            else if (path == PATH_TARGET)
                part = make_float4(st.r, warp_sumf(st.bad ? nan : st.zsum()), 0.f, 0.f);
            else
                part = warp_merge<PATH_ARGMAX>(st.as.partial(), scale);
            if (lane == 0) {
                const int slot = d.seg % kSegSlots;
                sh.part[slot][warp] = part;
                mbar_arrive(&sh.seg_bar[slot]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[s]);
    }
    // The stream is used up: this warp now runs row epilogues from the global queue until its
    // CTA has published all its segments and the queue is empty.  A row is queued by the warp that
    // publishes its last segment, so the consumer warps of that CTA are still here to take it.
    // (Two warps per CTA are plenty for the few rows left at that point, and keep the queue's
    // counters from being polled by thousands of warps.)
    if (warp >= 2) return;
    for (int idle = 0; idle < kWaitLimit; ++idle) {
        if (__shfl_sync(0xffffffffu, *error, 0)) return;
        int published = 0;
        if (lane == 0) {
            published = *reinterpret_cast<volatile int*>(&sh.published);
            __threadfence();  // the flag is read before the queue: whatever was queued before it was set is seen
        }
        published = __shfl_sync(0xffffffffu, published, 0);
        const int b = pipe_pop_row(P, error, lane);
        if (b >= 0) { pipe_row_job<T>(P, sh, b, lane); idle = 0; }
        else if (b == -1 && published) return;
        else __nanosleep(b == -2 ? 50 : 200);
    }
}

}  // namespace speckv
