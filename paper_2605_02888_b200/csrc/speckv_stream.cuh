// Stream sweep for sm_100a: one persistent CTA per SM walks the logit rows of a verification step in
// position-major order, decides every drafted position as soon as its draft and target rows are in,
// and draws the fresh token from rows that are still in L2.
//
// Order of work.  The rows a step needs are laid out as a stream of items: phase p = 0, 1, ... holds,
// for every batch row b with gamma_b >= p, the target row t[b,p] and (for p < gamma_b) the draft row
// d[b,p], each cut into n_slice slices.  CTAs take items from one global counter, so at any moment
// the whole GPU works on a window of a few dozen megabytes of the stream.  Two things follow:
//   * early exit (Sec. 3.1: what the target produced behind the first mismatch is discarded): when
//     phase p of a batch row comes up, the decisions of its positions < p are usually known; a target
//     row behind a known rejection is not read at all;
//   * the second look at the stop position (residual max(0, p - q), or p for the bonus token) starts
//     a few microseconds after the first, while both rows are still in L2.
//
// Inside a CTA the 32 warps are independent.  An item is cut into warp quanta of 16 vector steps; the
// quanta of successive items are numbered through and quantum g belongs to warp g mod 32, so every
// warp knows its own sequence and nothing is handed out at run time.  A warp keeps 4 sixteen-byte
// loads per lane in flight and requests the first loads of its next quantum before it merges the
// current one.  Partials meet in shared memory; the warp that completes an item publishes one
// partial per (logit row, slice) and takes the pair's ticket; the warp that completes a pair runs
// the position's epilogue (normalisers, entropy, confidence, acceptance) and ORs its decision into
// the batch row's state word; whoever completes the decided prefix queues the row's draw, whoever
// completes the row runs the signals and the controller, and the later of the two writes the tokens.
//
// No warp ever waits for another warp's work except (a) for a free slot in the CTA's item ring and
// (b) at the very end, for the draws of the last rows; both polls are bounded, and when a bound runs
// out the CTA marks its unfinished rows with SPECKV_ROW_TIMEOUT and leaves.
#pragma once

#include "speckv_kernels.cuh"
#include "speckv_pipeline.cuh"

namespace speckv {

constexpr int kSWarps = 32;                   // warps per CTA; one CTA per SM
constexpr int kSThreads = kSWarps * 32;
constexpr int kSSteps = 16;                   // vector steps (kChunk elements each) per warp quantum
constexpr int kSQElems = kSSteps * kChunk;    // elements per warp quantum
constexpr int kSRing = 8;                     // items queued per CTA
constexpr int kSFillBatch = 4;                // stream items taken per fill at most
constexpr int kSMaxQ = 64;                    // warp quanta per item at most
constexpr int kSMaxB = 4096;                  // batch rows the per-CTA tables hold
constexpr int kSMaxSlice = 16;                // slices per logit row at most
constexpr int kSMaxPhase = 17;                // gamma_max + 1 at most
constexpr int kSRsSub = 8;                    // 256-element chunks per resample warp job
constexpr int kSRsShareQ = 16;                // warp jobs per resample share
constexpr int kSRsShare = kSRsSub * kSRsShareQ;  // chunks per share
constexpr int kSPollLimit = 1 << 20;

// ---- batch-row state word (64 bits, OR-ed into by the position epilogues) --------------------------
//   bits  0..16  position p decided
//   bits 17..33  the walk over the positions ends at p (rejected token, unusable token, non-finite target row)
//   bits 34..50  target row p is non-finite
//   bit  51      some draft row is non-finite          bit 52  some draft token is out of range
//   bit  53      fresh token known (or not needed)     bit 54  signals and controller written
constexpr int kStRej = 17, kStTbad = 34;
constexpr unsigned long long kStDbad = 1ull << 51, kStBadTok = 1ull << 52, kStDraw = 1ull << 53, kStEpi = 1ull << 54;

__device__ __forceinline__ int st_stop(unsigned long long s, int gam, bool* known) {
    const unsigned dec = static_cast<unsigned>(s & 0x1ffffu);
    const unsigned rej = static_cast<unsigned>((s >> kStRej) & 0x1ffffu);
    const int r = rej ? (__ffs(rej) - 1) : gam;
    const unsigned need = (2u << r) - 1u;
    *known = (dec & need) == need;
    return r;
}
__device__ __forceinline__ bool st_complete(unsigned long long s, int gam) {
    const unsigned need = (2u << gam) - 1u;
    return (static_cast<unsigned>(s & 0x1ffffu) & need) == need;
}
// status bits of a batch row whose positions are all decided (or whose stop position is known, for
// the bits known so far)
__device__ __forceinline__ int st_status(unsigned long long s, int n) {
    int status = 0;
    if (s & kStBadTok) status |= 2;
    if ((s & kStDbad) || ((s >> (kStTbad + n)) & 1ull)) status |= 4;
    return status;
}

struct PosRec {  // what a position's epilogue leaves for the row's draw and final epilogue (32 bytes)
    float H, c;
    double lse2_q, lse2_p;
    int amax, pad;
};
static_assert(sizeof(PosRec) == 32, "position record");

struct SCtrl {  // global counters of one launch (cleared by the host before the launch)
    int item_next;   // items handed out beyond the first one per CTA
    int rs_tail;     // batch rows queued for a draw
    int rs_next;     // resample shares handed out
    int resolved;    // batch rows whose outputs are complete
    int error;
    int pad[3];
};

struct SParams {  // stream-kernel extras beside KParams
    int n_slice, slice_elems, rs_shares, read_all;
    SCtrl* ctrl;
    unsigned long long* state;  // [B]
    int* ptick;                 // [B*(G+1)] pair tickets
    int* rsq;                   // [B] queue of rows to draw for (b+1)
    PosRec* pos;                // [B*(G+1)]
    int* fresh;                 // [B]
    int poll_limit;
};

struct SItem {
    int type;      // 1 sweep, 2 resample
    int path;      // PATH_* (sweep)
    int b, p;
    int n_q;       // warp quanta of the item
    int done;      // quanta finished
    int busy;      // 1 from the fill until the item's last quantum has been merged; the slot is refilled after that
    int absent;    // a quantum of a target row was left out behind a known rejection
    float scale;
    int pair;      // b*(G+1)+p
    int part_idx;  // where the item's partial goes
    int pair_total;
    int elem0, n_elem;  // slice of the logit row (sweep); chunk range c0, c1 (resample)
    int rs_mode;
    float Tf;      // the batch row's temperature
    unsigned long long ctr;  // (item's sequence number << 32) | (its quanta << 16) | quanta handed out: one atomic add
                             // claims a quantum and tells whose it is, whatever has happened to the slot meanwhile
    const void* row;    // sweep: the logit row; resample: the target row of the stop position
    const void* drow;   // resample: the draft row of the stop position
    RowInfo ri;         // resample: the row's constants
    float4 part[kSMaxQ];
};

// Bookkeeping that needs global round trips (publishing an item's partial and taking the pair's ticket,
// with the position epilogue behind it; the token search of a finished draw) is not done by the warp that
// found it due: that warp is the last of its item, so already behind, and everybody else's progress is
// bounded by the slowest warp.  It leaves a job in this queue instead, and warps that are ahead of the
// ring and have nothing to sweep take the jobs.
struct SJob {
    float4 merged;
    int type;      // 1 publish a partial, 2 search a finished draw
    int b, p, part_idx, pair, pair_total;
    float Tf;
    int ready;     // 0: free; job number + 1 once the entry is written
};
constexpr int kSJobs = 32;

struct SShared {
    int tail;        // items filled so far
    int lock;        // one warp fills at a time
    int exhausted;   // nothing will be filled any more
    int stream_done; // the global item counter has run out
    int error;
    int n_items;     // items of the whole stream
    int idle_polls;
    int first_taken; // the CTA's first item is its own index in the stream, no counter involved
    int pend_share;  // a share number taken before its row was queued; -1: none
    int n_blk;
    int phase0[kSMaxPhase + 2];
    unsigned short pre[kSMaxPhase][kSMaxB / 32 + 1];
    unsigned char gam[kSMaxB];
    int job_head, job_tail;
    unsigned long long wake;  // mbarrier the idle warps sleep on; whoever adds work to the ring or the queue arrives on it
    int wake_gen;             // arrivals so far (the parity an idle warp waits for)
    SJob jobs[kSJobs];
    SItem ring[kSRing];
};


// ---- one warp quantum ---------------------------------------------------------------------------------
// The bytes in flight live in shared memory, not in registers: every lane copies its own 16-byte pieces
// with cp.async into a ring of slots private to its warp and reads the same pieces back when their
// group has landed, so no lane ever waits for another lane's copy and nothing needs a barrier.  A warp
// keeps kInFlight vector steps (5.5 KB) on their way, across quantum boundaries, and they keep coming
// in while the warp does bookkeeping.
template <typename T> struct SStage {
    static constexpr int kSlots = sizeof(T) == 2 ? 12 : 6;   // vector steps the warp's ring holds
    static constexpr int kInFlight = kSlots - 1;             // a slot is refilled one step after it was read
    static constexpr int kSlotBytes = 32 * kVec * sizeof(T);
    static constexpr int kWarpBytes = kSlots * kSlotBytes;
};
constexpr int kSDynBytes = kSWarps * SStage<float>::kWarpBytes;
static_assert(SStage<float>::kWarpBytes == SStage<__nv_bfloat16>::kWarpBytes, "one dynamic size for both types");

__device__ __forceinline__ void cp_async16(uint32_t saddr, const void* g) {
    if (!dbg_ok(g, 16, DBG_LOGIT16)) return;  // the slot keeps stale bytes: wrong numbers, counted, no fault
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(saddr), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr) : "memory");
    return v;
}

// Vector step `step` of an item that starts at `base` and has n_valid elements (a multiple of the
// 16-byte granule: the rows this kernel takes are 16-byte aligned and a whole number of granules long)
// goes into ring slot `slot` of the warp whose ring starts at shared address `ring`.  Pieces beyond
// the end are not copied; sq_read gives -inf for them, which no path counts.
//
// Which steps make up a quantum: quantum q of an item of n_q quanta takes the item's steps q, q + n_q,
// q + 2 n_q, ...  The warps of a CTA work on the quanta of one item at about the same pace, so what
// they request at any moment is one contiguous stretch of the logit row (32 warps x 512 bytes), and
// DRAM sees long sequential bursts instead of thousands of interleaved 512-byte streams.
template <typename T>
__device__ __forceinline__ void sq_issue(uint32_t ring, int slot, const T* base, int step, int n_valid, int lane) {
    const int e = step * kChunk + lane * kVec;  // `step` counts the item's vector steps
    const uint32_t at = ring + slot * SStage<T>::kSlotBytes + lane * 16;
    if constexpr (sizeof(T) == 2) {
        if (e + kVec <= n_valid) cp_async16(at, base + e);
    } else {
        if (e + 4 <= n_valid) cp_async16(at, base + e);
        if (e + 8 <= n_valid) cp_async16(at + 512, base + e + 4);
    }
}
template <typename T>
__device__ __forceinline__ Raw<T> sq_read(uint32_t ring, int slot, int step, int n_valid, int lane) {
    const int e = step * kChunk + lane * kVec;
    const uint32_t at = ring + slot * SStage<T>::kSlotBytes + lane * 16;
    const uint32_t ninf = 0xff800000u;
    Raw<T> r;
    if constexpr (sizeof(T) == 2) {
        if (e + kVec <= n_valid) r.a = lds128(at);
        else r.a = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
    } else {
        if (e + 4 <= n_valid) r.a = lds128(at);
        else r.a = make_uint4(ninf, ninf, ninf, ninf);
        if (e + 8 <= n_valid) r.b = lds128(at + 512);
        else r.b = make_uint4(ninf, ninf, ninf, ninf);
    }
    return r;
}
template <typename T> __device__ __forceinline__ int sq_next_slot(int s) { return s + 1 == SStage<T>::kSlots ? 0 : s + 1; }

// The first kInFlight steps of a quantum go out (a warp that could not chain from its previous quantum).
template <typename T>
__device__ __forceinline__ void sq_prime(uint32_t ring, int& wslot, const T* base, int q, int nq, int n_valid, int lane) {
#pragma unroll
    for (int k = 0; k < SStage<T>::kInFlight; ++k) {
        sq_issue<T>(ring, wslot, base, q + k * nq, n_valid, lane);
        cp_commit();
        wslot = sq_next_slot<T>(wslot);
    }
}

// Sweeps one quantum whose first kInFlight steps are on their way (or here); rslot = the slot of its
// step 0, wslot = the slot the next copy goes to.  While it runs, the first kInFlight steps of the
// quantum qn of the item at nbase (n_next valid elements; nbase == nullptr: none) are requested.  e_row =
// index of the item's first element within its logit row (the argmax path reports row indices).  Returns the
// warp's merged partial in every lane.
//
// The running maximum is the same in all lanes of the warp (one warp-wide maximum per vector step), so
// a new maximum is handled by all lanes together, elements equal to it are counted by the lanes that
// hold them, and the lanes' sums add up without any rescaling at the end of the quantum.  What a
// quantum returns depends on its own elements only, whichever warp sweeps it and whenever.
// (Not inlined: the loop below gets the whole register budget to itself, and what the caller keeps
// across the call is saved once per quantum instead of spilling inside the loop.  The caller advances
// its two slot numbers by the kSSteps steps a call consumes and issues.)
template <typename T, int PATH>
__device__ __noinline__ float4 sq_sweep(uint32_t ring, int rslot, int wslot, const T* base, int q, int nq, int n_valid,
                                        int e_row, float scale, const T* nbase, int qn, int nqn, int n_next) {
    constexpr int F = SStage<T>::kInFlight;
    const int lane = threadIdx.x & 31;
    PipeState st;
    st.init(scale);
    if constexpr (PATH != PATH_ARGMAX) {
        // start from the largest finite element of the first steps (they are read again below): fewer new
        // maxima on the way
        constexpr int kWarm = F < 4 ? F : 4;
        cp_wait<F - kWarm>();
        float m0 = kFloor;
        int sl = rslot;
#pragma unroll
        for (int k = 0; k < kWarm; ++k) {
            const float v = raw_max(sq_read<T>(ring, sl, q + k * nq, n_valid, lane));
            if (v >= kFloor && v < __int_as_float(0x7f800000)) m0 = fmaxf(m0, v);
            sl = sq_next_slot<T>(sl);
        }
        m0 = warp_maxf(m0);
        st.M = m0;
        st.r = m0 * scale;
    }
    const f2 sc2 = pack2(scale, scale);
    // (a short loop body: every warp of the SM runs this loop at its own place, and what they run has to
    // stay in the instruction cache)
#pragma unroll 2
    for (int step = 0; step < kSSteps; ++step) {
        cp_wait<F - 1>();
        const Raw<T> cur = sq_read<T>(ring, rslot, q + step * nq, n_valid, lane);
        rslot = sq_next_slot<T>(rslot);
        if (step + F < kSSteps) sq_issue<T>(ring, wslot, base, q + (step + F) * nq, n_valid, lane);
        else if (nbase) sq_issue<T>(ring, wslot, nbase, qn + (step + F - kSSteps) * nqn, n_next, lane);
        cp_commit();
        wslot = sq_next_slot<T>(wslot);
        if constexpr (PATH == PATH_ARGMAX) {
            st.as.template step<T>(cur, e_row + (q + step * nq) * kChunk + lane * kVec);
        } else {
            const float um = raw_max(cur);
            const float wm = warp_max_nan(um);  // NaN wins
            if (!(wm < __int_as_float(0x7f800000))) {
                st.bad = true;  // NaN or +inf: the row gets flagged
            } else if constexpr (PATH == PATH_DRAFT) {
                if (wm > st.M) draft_rescale(st, wm, scale);
                if (__any_sync(0xffffffffu, um == st.M)) draft_unit_careful<T>(st, cur, scale);
                else draft_unit_fast<T>(st, cur, pack2(st.M, st.M), sc2);
            } else {
                if (wm > st.M) target_rescale(st, wm, scale);
                target_unit<T>(st, cur, sc2, pack2(-st.r, -st.r));
            }
        }
    }
    const float nan = __int_as_float(0x7fc00000);
    if constexpr (PATH == PATH_DRAFT)
        return make_float4(st.M, warp_sumf(st.bad ? nan : st.cnt), warp_sumf(st.zsum()), warp_sumf(st.ssum()));
    else if constexpr (PATH == PATH_TARGET)
        return make_float4(st.r, warp_sumf(st.bad ? nan : st.zsum()), 0.f, 0.f);
    else
        return warp_merge<PATH_ARGMAX>(st.as.partial(), scale);
}

__device__ __forceinline__ float4 s_neutral(int path) {
    return path == PATH_DRAFT ? make_float4(kFloor, 0.f, 0.f, 0.f)
         : path == PATH_TARGET ? make_float4(-3.0e38f, 0.f, 0.f, 0.f)
                               : make_float4(kFloor, __int_as_float(0x7fffffff), 0.f, 0.f);
}
__device__ __forceinline__ float4 s_merge(int path, float4 a, float4 b, float scale) {
    return path == PATH_DRAFT ? merge_draft(a, b, scale) : path == PATH_TARGET ? merge_target(a, b) : merge_argmax(a, b);
}
__device__ __forceinline__ float4 s_warp_merge(int path, float4 v, float scale) {
    return path == PATH_DRAFT ? warp_merge<PATH_DRAFT>(v, scale)
         : path == PATH_TARGET ? warp_merge<PATH_TARGET>(v, scale) : warp_merge<PATH_ARGMAX>(v, scale);
}

__device__ __forceinline__ unsigned long long ld_state(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}


// ---- what happens when things complete ---------------------------------------------------------------
// Every function below is run by one whole warp; the lanes compute the same values and lane 0 writes.

// Tokens, accepted length: written by whichever of (draw finished, signals written) comes second.
__device__ __noinline__ void s_finalize_tokens(const KParams& P, const SParams& S, int b, int gam, unsigned long long st) {
    const int lane = threadIdx.x & 31;
    bool known;
    const int n = st_stop(st, gam, &known);
    const int status = st_status(st, n);
    const int G = P.G;
    int v = -1;
    if (status == 0 && lane <= G) {
        if (lane < n) v = __ldg(P.tok + static_cast<long long>(b) * G + lane);
        else if (lane == n) v = __ldcg(S.fresh + b);
    }
    if (lane <= G) P.out_tok[static_cast<long long>(b) * (G + 1) + lane] = v;
    if (lane == 0) {
        P.n_acc[b] = status == 0 ? n : 0;
        atomicAdd(&S.ctrl->resolved, 1);
    }
}

// The fresh token is known (fresh[b] written) or the row needs none.
__device__ __forceinline__ void s_draw_done(const KParams& P, const SParams& S, int b, int gam) {
    const int lane = threadIdx.x & 31;
    unsigned long long old = 0;
    if (lane == 0) {
        __threadfence();
        old = atomicOr(S.state + b, kStDraw);
    }
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old & kStEpi) {
        __threadfence();
        s_finalize_tokens(P, S, b, gam, old | kStDraw);
    }
}

// The stop position of batch row b has just become known: queue the draw, or settle rows that need none.
__device__ __noinline__ void s_resolve_stop(const KParams& P, const SParams& S, int b, int gam, float Tf,
                                            unsigned long long st) {
    const int lane = threadIdx.x & 31;
    bool known;
    const int n = st_stop(st, gam, &known);
    const bool greedy = (Tf == 0.f);
    const PosRec* pr = S.pos + static_cast<long long>(b) * (P.G + 1) + n;
    if (st_status(st, n) != 0 || greedy) {
        // flagged as far as is known (nothing to draw), or greedy: the target's argmax at the stop position
        if (lane == 0) S.fresh[b] = (st_status(st, n) == 0) ? __ldcg(&pr->amax) : -1;
        s_draw_done(P, S, b, gam);
        return;
    }
    if (lane == 0) {
        RowInfo ri;
        ri.mode = n < gam ? RS_RESIDUAL : RS_BONUS;
        ri.n = n;
        ri.u2 = __ldg(P.u + (static_cast<long long>(b) * (P.G + 1) + n) * 2 + 1);
        ri.scale = static_cast<float>(kLog2e / static_cast<double>(Tf));
        ri.lse2_p = __ldcg(&pr->lse2_p);
        ri.lse2_q = n < gam ? __ldcg(&pr->lse2_q) : 0.0;
        SPECKV_ST(P.info[b], ri);
        __threadfence();
        const int at = atomicAdd(&S.ctrl->rs_tail, 1);
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(S.rsq + at), "r"(b + 1) : "memory");
    }
    __syncwarp();
}

// All positions of batch row b are decided: signals (Sec. 4.2), controller (Sec. 4.3, Eq. 1), status.
__device__ __noinline__ void s_row_final(const KParams& P, const SParams& S, int b, int gam, unsigned long long st) {
    const int lane = threadIdx.x & 31;
    const int G = P.G;
    bool known;
    const int n = st_stop(st, gam, &known);
    const int status = st_status(st, n);
    CtlRegs ctl;
    if ((P.mode & MODE_MLP) && !status) ctl = ctl_load(P, b, lane);
    float Hi = 0.f, ci = 0.f;
    if (status == 0 && lane < gam) {
        const PosRec* pr = S.pos + static_cast<long long>(b) * (G + 1) + lane;
        Hi = __ldcg(&pr->H);
        ci = __ldcg(&pr->c);
    }
    const float in_bits = P.bits ? static_cast<float>(kLog2e) : 1.f;
    const float Hout = Hi * in_bits, Cout = ci;
    float f4[4] = {0.f, 0.f, 0.f, 0.f};
    if (status == 0) {
        f4[0] = warp_sumf(Hout) / static_cast<float>(gam);
        f4[1] = warp_sumf(Cout) / static_cast<float>(gam);
        f4[2] = warp_maxf(Hout);
        f4[3] = -warp_maxf(lane < gam ? -Cout : -2.f);
    }
    if (lane < G) {
        if (P.H) P.H[static_cast<long long>(b) * G + lane] = Hout;
        if (P.C) P.C[static_cast<long long>(b) * G + lane] = Cout;
    }
    if (P.feat && lane < 4)
        P.feat[static_cast<long long>(b) * 4 + lane] = lane == 0 ? f4[0] : lane == 1 ? f4[1] : lane == 2 ? f4[2] : f4[3];
    if (P.mode & MODE_MLP) {
        if (status == 0) {
            ctl_eval(P, ctl, f4, P.scores ? P.scores + static_cast<long long>(b) * P.n_out : nullptr, P.gamma_next + b);
        } else {
            if (P.scores && lane < P.n_out) P.scores[static_cast<long long>(b) * P.n_out + lane] = 0.f;
            if (lane == 0) P.gamma_next[b] = 0;
        }
    }
    if (P.status && lane == 0) P.status[b] = status;
    unsigned long long old = 0;
    if (lane == 0) {
        __threadfence();
        old = atomicOr(S.state + b, kStEpi);
    }
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old & kStDraw) {
        __threadfence();
        s_finalize_tokens(P, S, b, gam, old | kStEpi);
    }
}

// Both logit rows of position p of batch row b are in (or the target row was left out behind a known
// rejection): normalisers, entropy and confidence (Sec. 4.2), the acceptance test, and the decision
// OR-ed into the row's state.
template <typename T>
__device__ __noinline__ void s_pair_epilogue(const KParams& P, const SParams& S, int b, int p, int gam, float Tf) {
    const int lane = threadIdx.x & 31;
    const int G = P.G, ns = S.n_slice;
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    const double sd = static_cast<double>(scale);
    const bool have_draft = p < gam;
    const long long pair = static_cast<long long>(b) * (G + 1) + p;
    const float4* pp = P.part + pair * 2 * ns;
    const int tpath = greedy ? PATH_ARGMAX : PATH_TARGET;

    // everything that does not depend on another load goes out first
    float4 qt = lane < ns ? ldcg4(pp + lane) : s_neutral(tpath);
    float4 qd = (have_draft && lane < ns) ? ldcg4(pp + ns + lane) : s_neutral(PATH_DRAFT);
    const int x = have_draft ? __ldg(P.tok + static_cast<long long>(b) * G + p) : -1;
    const float u_acc = have_draft ? __ldg(P.u + pair * 2) : 0.f;
    const bool badtok = have_draft && (x < 0 || x >= P.V);
    const bool absent = __any_sync(0xffffffffu, lane < ns && qt.w != 0.f);
    float dxf = 0.f, txf = 0.f;
    if (have_draft && !badtok && !greedy && !absent) {
        const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(p) * P.dsp;
        const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(p) * P.tsp;
        dxf = elem_to_float(drow, x);
        txf = elem_to_float(trow, x);
    }
    if (absent && lane < ns) qt = s_neutral(tpath);
    const float4 at = s_warp_merge(tpath, qt, scale);
    const float4 ad = warp_merge<PATH_DRAFT>(qd, scale);

    float Hi = 0.f, ci = 0.f;
    double lse2_q = 0.0, lse2_p = 0.0;
    int amax = -1;
    bool dbad = false, tbad = false, accept = true;
    if (have_draft) {
        const float m = ad.x, cnt = ad.y, Zx = ad.z, Sx = ad.w;
        const float Z = cnt + Zx;
        if (!(cnt >= 1.f) || !(Z < 3e38f) || !(m > kFloor)) {
            dbad = true;
        } else {
            const float lnZ = (cnt == 1.f) ? log1pf(Zx) : logf(cnt) + log1pf(Zx / cnt);
            const float rZ = 1.f / Z;
            Hi = fmaxf(lnZ - static_cast<float>(kLn2) * scale * Sx * rZ, 0.f);
            ci = rZ;
            lse2_q = static_cast<double>(m) * sd + log2_split(static_cast<double>(cnt) + static_cast<double>(Zx));
        }
    }
    if (!absent) {
        if (greedy) {
            const int bi = __float_as_int(at.y);
            if (at.z != 0.f || bi == 0x7fffffff || !(at.x > kFloor)) tbad = true;
            amax = bi;
        } else {
            if (!(at.y > 0.f) || !(at.y < 3e38f)) tbad = true;
            else lse2_p = static_cast<double>(at.x) + log2_split(static_cast<double>(at.y));
        }
    }
    if (have_draft && !absent && !tbad && !dbad && !badtok) {
        if (greedy) {
            accept = (x == amax);
        } else {
            const double lq = static_cast<double>(dxf) * sd - lse2_q;
            const double lp = static_cast<double>(txf) * sd - lse2_p;
            const double l2u = (u_acc > 0.f) ? log2_split(static_cast<double>(u_acc)) : -__longlong_as_double(0x7ff0000000000000LL);
            accept = (l2u + lq) < lp;  // u * q(x) < p(x)
        }
    }
    const bool stopper = !absent && (tbad || (have_draft && (badtok || !accept)));
    unsigned long long bits = 1ull << p;
    if (stopper) bits |= 1ull << (kStRej + p);
    if (tbad) bits |= 1ull << (kStTbad + p);
    if (dbad) bits |= kStDbad;
    if (badtok) bits |= kStBadTok;
    unsigned long long old = 0;
    if (lane == 0) {
        PosRec r;
        r.H = Hi; r.c = ci; r.lse2_q = lse2_q; r.lse2_p = lse2_p; r.amax = amax; r.pad = 0;
        SPECKV_ST(S.pos[pair], r);
        __threadfence();
        old = atomicOr(S.state + b, bits);
    }
    old = __shfl_sync(0xffffffffu, old, 0);
    const unsigned long long now = old | bits;
    bool k_old, k_new;
    st_stop(old, gam, &k_old);
    st_stop(now, gam, &k_new);
    if (k_new && !k_old) {
        __threadfence();
        s_resolve_stop(P, S, b, gam, Tf, now);
    }
    if (st_complete(now, gam) && !st_complete(old, gam)) {
        // every other position's OR came before this one, so `now` holds all their bits
        __threadfence();
        s_row_final(P, S, b, gam, now);
    }
}


// ---- the draw ---------------------------------------------------------------------------------------
// One warp sums the residual (or bonus) weights of chunks [a, e) of the stop position, KU chunks at a
// time with the next KU requested before the current ones are evaluated.  Same loads, operations and
// roundings per element as rs_chunk_weights, which rescans the located chunk.
template <typename T, int MODE, int KU>
__device__ __forceinline__ void s_warp_sums(const RsConst& c0, const T* trow, const T* drow, int a, int e, int V, float* csum) {
    const int lane = threadIdx.x & 31;
    const float ninf = __int_as_float(0xff800000);
    RsConst c = c0;
    c.mode = MODE;
    Raw<T> rt[KU], rd[KU];
    auto load = [&](int base, Raw<T> (&xt)[KU], Raw<T> (&xd)[KU]) {
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            if (base + u < e) {
                xt[u] = rs_load_lane<T, true>(trow, base + u, V, ninf);
                if (MODE == RS_RESIDUAL) xd[u] = rs_load_lane<T, true>(drow, base + u, V, ninf);
            } else {
                xt[u] = raw_fill<T>(ninf);
                if (MODE == RS_RESIDUAL) xd[u] = xt[u];
            }
        }
    };
    load(a, rt, rd);
    for (int base = a; base < e; base += KU) {
        Raw<T> nt[KU], nd[KU];
        if (base + KU < e) load(base + KU, nt, nd);
        float sm[KU];
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            float w[kVec];
            rs_weights<T>(c, rt[u], rd[u], w);
            sm[u] = 0.f;
#pragma unroll
            for (int j = 0; j < kVec; ++j) sm[u] = __fadd_rn(sm[u], w[j]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int u = 0; u < KU; ++u) sm[u] = __fadd_rn(sm[u], __shfl_xor_sync(0xffffffffu, sm[u], o));
        }
#pragma unroll
        for (int u = 0; u < KU; ++u)
            if (lane == 0 && base + u < e) SPECKV_ST(csum[base + u], sm[u]);
        if (base + KU < e) {
#pragma unroll
            for (int u = 0; u < KU; ++u) {
                rt[u] = nt[u];
                if (MODE == RS_RESIDUAL) rd[u] = nd[u];
            }
        }
    }
}

template <typename T>
__device__ __forceinline__ void s_warp_sums_any(const RsConst& c, const T* trow, const T* drow, int a, int e, int V, float* csum) {
    constexpr int kResidual = sizeof(T) == 2 ? 2 : 1;
    if (c.mode == RS_BONUS) s_warp_sums<T, RS_BONUS, 2>(c, trow, drow, a, e, V, csum);
    else s_warp_sums<T, RS_RESIDUAL, kResidual>(c, trow, drow, a, e, V, csum);
}

// All chunk sums of batch row b's stop position are written: locate the threshold, write the fresh token.
template <typename T>
__device__ __noinline__ void s_search(const KParams& P, const SParams& S, int b, int gam, const RowInfo& ri,
                                      const T* trow, const T* drow) {
    const int lane = threadIdx.x & 31;
    __threadfence();
    RsConst c = rs_const(ri, ri.mode);
    float* csum = P.csum + static_cast<long long>(b) * P.nchunk;
    const int per_lane = (P.nchunk + 31) / 32;
    RsSums cs;
    cs.sh = nullptr;
    cs.glob = csum;
    double own = 0.0;
    double W = rs_total(cs, P.nchunk, per_lane, &own);
    int tok = 0;
    bool have = true;
    if (!(W > (c.mode == RS_RESIDUAL ? 1e-6 : 0.0))) {
        if (c.mode != RS_RESIDUAL) {
            have = false;  // p itself without mass: cannot happen for a finite row
        } else {
            // numerically empty residual (p == q at the stop position): the token comes from p
            c.mode = RS_BONUS;
            s_warp_sums_any<T>(c, trow, drow, 0, P.nchunk, P.V, csum);
            __threadfence();
            __syncwarp();
            W = rs_total(cs, P.nchunk, per_lane, &own);
        }
    }
    if (have) {
        const double tau = static_cast<double>(ri.u2) * W;
        tok = rs_search<T, true>(c, trow, drow, cs, P.nchunk, P.V, tau, own, per_lane);
    }
    if (lane == 0) S.fresh[b] = tok;
    s_draw_done(P, S, b, gam);
}


// ---- the CTA's item ring -------------------------------------------------------------------------------
__device__ __forceinline__ int s_vol(const int* p) { return *reinterpret_cast<const volatile int*>(p); }

// Stream item i -> batch row, position, slot (0 target row, 1 draft row), slice.  Whole warp.
__device__ __forceinline__ void s_decode(const KParams& P, const SParams& S, const SShared& sh, int i, int& b, int& p,
                                         int& slot, int& slice) {
    const int lane = threadIdx.x & 31;
    const int u = i / S.n_slice;
    slice = i - u * S.n_slice;
    // phase: the last p with phase0[p] <= u
    const unsigned ph = __ballot_sync(0xffffffffu, lane <= P.G && sh.phase0[lane] <= u);
    p = 31 - __clz(ph);
    const int ul = u - sh.phase0[p];
    // block of 32 batch rows: the last one whose prefix is <= ul
    int cnt = 0;
    for (int c = 0; c < sh.n_blk; c += 32) {
        const int k = c + lane;
        cnt += __popc(__ballot_sync(0xffffffffu, k < sh.n_blk && static_cast<int>(sh.pre[p][k]) <= ul));
    }
    const int blk = cnt - 1;
    const int r = ul - static_cast<int>(sh.pre[p][blk]);
    const int bb = blk * 32 + lane;
    const int gam = bb < P.B ? sh.gam[bb] : 0;
    const unsigned A = __ballot_sync(0xffffffffu, gam > p);
    const unsigned E = __ballot_sync(0xffffffffu, gam == p && gam >= 1);
    const unsigned below = (1u << lane) - 1u;
    const int before = 2 * __popc(A & below) + __popc(E & below);
    const int w = gam > p ? 2 : (gam == p && gam >= 1) ? 1 : 0;
    const unsigned hit = __ballot_sync(0xffffffffu, w > 0 && before <= r && r < before + w);
    const int j = __ffs(hit) - 1;
    b = blk * 32 + j;
    slot = r - __shfl_sync(0xffffffffu, before, j);
}

// One partial per (logit row, slice) goes out, the pair's ticket is taken, and the warp that completes the
// pair runs the position's epilogue.
template <typename T>
__device__ __noinline__ void s_publish(const KParams& P, const SParams& S, const SShared& sh, float4 merged, int b, int p,
                                          int part_idx, int pair, int pair_total, float Tf) {
    const int lane = threadIdx.x & 31;
    int t = 0;
    if (lane == 0) {
        SPECKV_ST(P.part[part_idx], merged);
        __threadfence();
        t = atomicAdd(S.ptick + pair, 1);
    }
    t = __shfl_sync(0xffffffffu, t, 0);
    if (t == pair_total - 1) {
        __threadfence();
        s_pair_epilogue<T>(P, S, b, p, sh.gam[b], Tf);
    }
}

template <typename T>
__device__ __noinline__ void s_do_job(const KParams& P, const SParams& S, SShared& sh, const SJob& j) {
    if (j.type == 1) {
        s_publish<T>(P, S, sh, j.merged, j.b, j.p, j.part_idx, j.pair, j.pair_total, j.Tf);
    } else {
        const int4* ip = reinterpret_cast<const int4*>(P.info + j.b);
        const RowInfo ri = row_info_from(__ldcg(ip), __ldcg(ip + 1));
        const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(j.b) * P.tsb + static_cast<long long>(ri.n) * P.tsp;
        const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(j.b) * P.dsb + static_cast<long long>(ri.n) * P.dsp;
        s_search<T>(P, S, j.b, sh.gam[j.b], ri, trow, drow);
    }
}

// Leave a job in the queue (whole warp calls; every lane holds the same job).  When the entry it would go
// to is still occupied the caller does the job itself.
template <typename T>
__device__ __forceinline__ void s_job_push(const KParams& P, const SParams& S, SShared& sh, const SJob& j) {
    const int lane = threadIdx.x & 31;
    int at = -1;
    if (lane == 0) {
        for (;;) {
            const int t = s_vol(&sh.job_tail);
            if (s_vol(&sh.jobs[t % kSJobs].ready) != 0) break;  // the entry of 32 jobs ago has not been taken yet
            if (atomicCAS(&sh.job_tail, t, t + 1) == t) { at = t; break; }
        }
        if (at >= 0) {
            SJob* e = &sh.jobs[at % kSJobs];
            e->merged = j.merged; e->type = j.type; e->b = j.b; e->p = j.p; e->part_idx = j.part_idx;
            e->pair = j.pair; e->pair_total = j.pair_total; e->Tf = j.Tf;
            __threadfence_block();
            *reinterpret_cast<volatile int*>(&e->ready) = at + 1;
            atomicAdd(&sh.wake_gen, 1);
            mbar_arrive(&sh.wake);
        }
    }
    at = __shfl_sync(0xffffffffu, at, 0);
    if (at < 0) s_do_job<T>(P, S, sh, j);
}

// Reserve the oldest job nobody has reserved yet: its number, or -1.  The warp that holds a number runs
// that job (s_job_run) as soon as it has no quantum in hand.
__device__ __forceinline__ int s_job_reserve(SShared& sh) {
    int r = -1;
    if ((threadIdx.x & 31) == 0) {
        const int have = s_vol(&sh.job_head);
        if (have < s_vol(&sh.job_tail) && atomicCAS(&sh.job_head, have, have + 1) == have) r = have;
    }
    return __shfl_sync(0xffffffffu, r, 0);
}
template <typename T>
__device__ __forceinline__ void s_job_run(const KParams& P, const SParams& S, SShared& sh, int r) {
    const int lane = threadIdx.x & 31;
    SJob j;
    if (lane == 0) {
        SJob* e = &sh.jobs[r % kSJobs];
        for (int k = 0; k < S.poll_limit && s_vol(&e->ready) != r + 1; ++k) {}  // being written by its pusher right now
        __threadfence_block();
        const volatile SJob* v = e;
        j.merged = make_float4(v->merged.x, v->merged.y, v->merged.z, v->merged.w);
        j.type = v->type; j.b = v->b; j.p = v->p; j.part_idx = v->part_idx; j.pair = v->pair;
        j.pair_total = v->pair_total; j.Tf = v->Tf;
        __threadfence_block();
        *reinterpret_cast<volatile int*>(&e->ready) = 0;  // the entry may be used again
    }
    j.merged.x = __shfl_sync(0xffffffffu, j.merged.x, 0); j.merged.y = __shfl_sync(0xffffffffu, j.merged.y, 0);
    j.merged.z = __shfl_sync(0xffffffffu, j.merged.z, 0); j.merged.w = __shfl_sync(0xffffffffu, j.merged.w, 0);
    j.type = __shfl_sync(0xffffffffu, j.type, 0); j.b = __shfl_sync(0xffffffffu, j.b, 0);
    j.p = __shfl_sync(0xffffffffu, j.p, 0); j.part_idx = __shfl_sync(0xffffffffu, j.part_idx, 0);
    j.pair = __shfl_sync(0xffffffffu, j.pair, 0); j.pair_total = __shfl_sync(0xffffffffu, j.pair_total, 0);
    j.Tf = __shfl_sync(0xffffffffu, j.Tf, 0);
    s_do_job<T>(P, S, sh, j);
}

template <typename T>
__device__ __forceinline__ void s_finish_sweep(const KParams& P, const SParams& S, SShared& sh, SItem& it, int q, float4 part) {
    const int lane = threadIdx.x & 31;
    int d = 0;
    if (lane == 0) {
        volatile float4* dst = &it.part[q];
        dst->x = part.x; dst->y = part.y; dst->z = part.z; dst->w = part.w;
        __threadfence_block();
        d = atomicAdd(&it.done, 1);
    }
    d = __shfl_sync(0xffffffffu, d, 0);
    const int nq = it.n_q;
    if (d != nq - 1) return;
    __threadfence_block();
    const int path = it.path;
    const float scale = it.scale;
    const volatile float4* vp = it.part;
    float4 v = s_neutral(path);
    if (lane < nq) v = make_float4(vp[lane].x, vp[lane].y, vp[lane].z, vp[lane].w);
    if (lane + 32 < nq) v = s_merge(path, v, make_float4(vp[lane + 32].x, vp[lane + 32].y, vp[lane + 32].z, vp[lane + 32].w), scale);
    SJob j;
    j.merged = s_warp_merge(path, v, scale);
    if (s_vol(&it.absent)) j.merged = make_float4(0.f, 0.f, 0.f, 1.f);  // part of the row was left out: the row counts as not read
    j.type = 1; j.b = it.b; j.p = it.p; j.part_idx = it.part_idx; j.pair = it.pair; j.pair_total = it.pair_total; j.Tf = it.Tf;
    __syncwarp();
    if (lane == 0) { __threadfence_block(); *reinterpret_cast<volatile int*>(&it.busy) = 0; }  // the slot may be refilled
    s_job_push<T>(P, S, sh, j);
}

template <typename T>
__device__ __forceinline__ void s_resample_job(const KParams& P, const SParams& S, SShared& sh, SItem& it, int q) {
    const int lane = threadIdx.x & 31;
    const int b = it.b;
    const T* trow = static_cast<const T*>(it.row);
    const T* drow = static_cast<const T*>(it.drow);
    const RowInfo ri = it.ri;
    const int a = it.elem0 + q * kSRsSub;
    const int e = min(it.n_elem, a + kSRsSub);
    const RsConst c = rs_const(ri, ri.mode);
    s_warp_sums_any<T>(c, trow, drow, a, e, P.V, P.csum + static_cast<long long>(b) * P.nchunk);
    __threadfence();
    __syncwarp();
    int last = 0;
    if (lane == 0) {
        const int d = atomicAdd(&it.done, 1);
        if (d == it.n_q - 1) {
            *reinterpret_cast<volatile int*>(&it.busy) = 0;  // the slot may be refilled
            __threadfence();
            last = (atomicAdd(P.tick2 + b, 1) == S.rs_shares - 1);
        }
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
        SJob j;
        j.merged = make_float4(0.f, 0.f, 0.f, 0.f);
        j.type = 2; j.b = b; j.p = 0; j.part_idx = 0; j.pair = 0; j.pair_total = 0; j.Tf = 0.f;
        s_job_push<T>(P, S, sh, j);
    }
}

// Idle warps do not spin: they block on an mbarrier phase (the hardware parks the warp) until somebody
// has added work, or for about two microseconds at most.
__device__ __forceinline__ void s_wake(SShared& sh) {
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&sh.wake_gen, 1);
        mbar_arrive(&sh.wake);
    }
}
__device__ __forceinline__ void s_nap(SShared& sh, int gen) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(smem_u32(&sh.wake)), "r"(static_cast<uint32_t>(gen & 1)), "r"(2000u)
        : "memory");
    (void)ok;
}

// One step of filling, by whichever warp gets the lock: a resample share if one is waiting (its rows
// are the freshest in L2), else the next item of the stream.
// `starving`: the caller has nothing to do until the ring grows (it may sleep a little); otherwise it
// is filling ahead of need and returns at once when another warp holds the lock.
template <typename T>
__device__ __noinline__ void s_try_fill(const KParams& P, const SParams& S, SShared& sh, bool starving) {
    const int lane = threadIdx.x & 31;
    int got = 0;
    if (lane == 0) got = (atomicCAS(&sh.lock, 0, 1) == 0);
    got = __shfl_sync(0xffffffffu, got, 0);
    if (!got) return;
    auto unlock = [&]() {
        __syncwarp();
        if (lane == 0) { __threadfence_block(); atomicExch(&sh.lock, 0); }
    };
    const int tail = s_vol(&sh.tail);
    SItem& it = sh.ring[tail % kSRing];
    const bool slot_free = tail < kSRing || s_vol(&it.busy) == 0;
    if (!slot_free || s_vol(&sh.exhausted)) { unlock(); return; }

    // A share of a queued draw comes first (its rows are the freshest in L2).  The counter is a plain
    // atomic add, so nobody retries; a share number beyond the rows queued so far (another CTA was quicker)
    // is kept until its row arrives.
    int share = -1, brow = -1;
    if (lane == 0) {
        share = sh.pend_share;
        if (share < 0) {
            const int nx = ld_relaxed(&S.ctrl->rs_next);
            const int tq = ld_relaxed(&S.ctrl->rs_tail);
            if (nx < tq * S.rs_shares) share = atomicAdd(&S.ctrl->rs_next, 1);
        }
        int v = 0;
        if (share >= 0) {
            const int qpos = share / S.rs_shares;
            if (qpos >= P.B) share = -1;                 // beyond anything that can ever be queued
            else v = ld_acquire(S.rsq + qpos);
        }
        if (share >= 0 && v == 0) { sh.pend_share = share; share = -1; }
        else sh.pend_share = -1;
        brow = v - 1;
    }
    share = __shfl_sync(0xffffffffu, share, 0);
    brow = __shfl_sync(0xffffffffu, brow, 0);
    if (share >= 0) {
        const int part = share % S.rs_shares;
        const int b = brow;
        if (lane == 0) {
            const int4* ip = reinterpret_cast<const int4*>(P.info + b);
            const RowInfo ri = row_info_from(__ldcg(ip), __ldcg(ip + 1));
            it.type = 2; it.path = 0; it.b = b; it.p = ri.n;
            it.elem0 = part * kSRsShare;
            it.n_elem = min(P.nchunk, it.elem0 + kSRsShare);
            it.n_q = (it.n_elem - it.elem0 + kSRsSub - 1) / kSRsSub;
            it.done = 0; it.busy = 1; it.absent = 0;
            it.ri = ri;
            it.row = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(ri.n) * P.tsp;
            it.drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(ri.n) * P.dsp;
            sh.idle_polls = 0;
            __threadfence_block();
            *reinterpret_cast<volatile unsigned long long*>(&it.ctr) =
                (static_cast<unsigned long long>(tail) << 32) | (static_cast<unsigned long long>(it.n_q) << 16);
            __threadfence_block();
            *reinterpret_cast<volatile int*>(&sh.tail) = tail + 1;
        }
        unlock();
        s_wake(sh);
        return;
    }

    // The stream's next items: as many as there are free slots in a row (at most kSFillBatch) for one
    // atomic add, so that a fill's global round trips are shared by several items.
    if (!s_vol(&sh.stream_done)) {
        int i0 = -1, k = 0;
        if (lane == 0) {
            int kfree = 1;
            while (kfree < kSFillBatch && (tail + kfree < kSRing || s_vol(&sh.ring[(tail + kfree) % kSRing].busy) == 0)) ++kfree;
            if (!sh.first_taken) { sh.first_taken = 1; i0 = blockIdx.x; k = 1; }
            else { k = kfree; i0 = static_cast<int>(gridDim.x) + atomicAdd(&S.ctrl->item_next, k); }
            if (i0 >= sh.n_items) k = 0;
            else if (i0 + k > sh.n_items) k = sh.n_items - i0;
            if (i0 + k >= sh.n_items) sh.stream_done = 1;
        }
        i0 = __shfl_sync(0xffffffffu, i0, 0);
        k = __shfl_sync(0xffffffffu, k, 0);
        if (k > 0) {
            int bb[kSFillBatch], pp[kSFillBatch], sl[kSFillBatch], sc[kSFillBatch];
            float Tfs[kSFillBatch];
#pragma unroll
            for (int j = 0; j < kSFillBatch; ++j) {
                bb[j] = 0; pp[j] = 0; sl[j] = 0; sc[j] = 0; Tfs[j] = 1.f;
                if (j < k) {
                    s_decode(P, S, sh, i0 + j, bb[j], pp[j], sl[j], sc[j]);
                    Tfs[j] = P.temp ? __ldg(P.temp + bb[j]) : P.temp_scalar;
                }
            }
            if (lane == 0) {
#pragma unroll
                for (int j = 0; j < kSFillBatch; ++j) {
                    if (j >= k) break;
                    SItem& x = sh.ring[(tail + j) % kSRing];
                    const int b = bb[j], p = pp[j], slot = sl[j], slice = sc[j];
                    const float Tf = Tfs[j];
                    const bool greedy = (Tf == 0.f);
                    x.type = 1;
                    x.path = slot == 1 ? PATH_DRAFT : (greedy ? PATH_ARGMAX : PATH_TARGET);
                    x.b = b; x.p = p;
                    x.elem0 = slice * S.slice_elems;
                    x.n_elem = min(P.V - x.elem0, S.slice_elems);
                    x.n_q = (x.n_elem + kSQElems - 1) / kSQElems;
                    x.done = 0; x.busy = 1; x.absent = 0;
                    x.scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
                    x.Tf = Tf;
                    x.pair = b * (P.G + 1) + p;
                    x.part_idx = (x.pair * 2 + slot) * S.n_slice + slice;
                    x.pair_total = S.n_slice * (p < sh.gam[b] ? 2 : 1);
                    x.row = slot == 1
                        ? static_cast<const void*>(static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb + static_cast<long long>(p) * P.dsp)
                        : static_cast<const void*>(static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb + static_cast<long long>(p) * P.tsp);
                    __threadfence_block();
                    *reinterpret_cast<volatile unsigned long long*>(&x.ctr) =
                        (static_cast<unsigned long long>(tail + j) << 32) | (static_cast<unsigned long long>(x.n_q) << 16);
                }
                sh.idle_polls = 0;
                __threadfence_block();
                *reinterpret_cast<volatile int*>(&sh.tail) = tail + k;
            }
        }
        unlock();
        if (k > 0) s_wake(sh);
        return;
    }

    // nothing to hand out: done once every batch row has its outputs
    if (lane == 0) {
        if (ld_relaxed(&S.ctrl->resolved) >= P.B) sh.exhausted = 1;
        else if (++sh.idle_polls > S.poll_limit) { sh.error = 1; sh.exhausted = 1; }
    }
    unlock();
    if (sh.exhausted) s_wake(sh);
}

// Claims the next quantum of the CTA's ring for this warp: one atomic add on the item's counter, which
// carries the item's sequence number, so a warp whose cursor has fallen behind a refilled slot simply
// finds itself holding a quantum of the newer item.  A quantum of a target row behind a rejection that
// has become known since the item was filled is settled on the spot (Sec. 3.1: such a row is not part
// of the step).  `blocking`: with nothing in the ring the warp does queued jobs, fills, or naps, until
// there is a quantum or the step is over; otherwise it returns false at once.
template <typename T>
__device__ __forceinline__ bool s_claim(const KParams& P, const SParams& S, SShared& sh, int& cursor, SItem*& out_it,
                                        int& out_q, bool blocking) {
    const int lane = threadIdx.x & 31;
    for (;;) {
        const int gen = s_vol(&sh.wake_gen);  // read before looking for work: work added after this ends the nap at once
        if (blocking) {  // a warp without a quantum in hand takes queued bookkeeping first
            const int r = s_job_reserve(sh);
            if (r >= 0) { s_job_run<T>(P, S, sh, r); continue; }
        }
        if (cursor >= s_vol(&sh.tail)) {
            if (!blocking) return false;
            if (s_vol(&sh.exhausted)) return false;
            const int before = s_vol(&sh.tail);
            s_try_fill<T>(P, S, sh, true);
            if (s_vol(&sh.tail) == before && !s_vol(&sh.exhausted)) s_nap(sh, gen);  // nothing came of it
            continue;
        }
        SItem* it = &sh.ring[cursor % kSRing];
        unsigned long long v = 0;
        if (lane == 0) v = atomicAdd(&it->ctr, 1ull);
        v = __shfl_sync(0xffffffffu, v, 0);
        const int seq = static_cast<int>(v >> 32), q = static_cast<int>(v & 0xffffu);
        if (seq > cursor) cursor = seq;
        if (q >= static_cast<int>((v >> 16) & 0xffffu)) { cursor = seq + 1; continue; }
        if (it->type == 1 && it->path != PATH_DRAFT && it->p >= 1 && !S.read_all) {
            unsigned long long st = 0;
            if (lane == 0) st = ld_state(S.state + it->b);
            st = __shfl_sync(0xffffffffu, st, 0);
            if (((st >> kStRej) & ((1ull << it->p) - 1ull)) != 0) {
                if (lane == 0) *reinterpret_cast<volatile int*>(&it->absent) = 1;
                s_finish_sweep<T>(P, S, sh, *it, q, s_neutral(it->path));
                continue;
            }
        }
        out_it = it;
        out_q = q;
        return true;
    }
}

// ---- the kernel -------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kSThreads, 1) stream_kernel(const __grid_constant__ KParams P, const __grid_constant__ SParams S) {
    __shared__ SShared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = P.G;

    // per-CTA tables: gamma of every usable batch row, and for every phase the number of row slots
    // (2 for a drafted position, 1 for the bonus position) in front of every block of 32 batch rows
    const int n_blk = (P.B + 31) / 32;
    if (threadIdx.x == 0) {
        sh.tail = 0; sh.lock = 0; sh.exhausted = 0; sh.stream_done = 0; sh.error = 0;
        sh.idle_polls = 0; sh.first_taken = 0; sh.n_blk = n_blk;
        sh.job_head = 0; sh.job_tail = 0; sh.pend_share = -1; sh.wake_gen = 0;
        mbar_init(&sh.wake, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < kSJobs) sh.jobs[threadIdx.x].ready = 0;  // shared memory keeps what the last launch left
    for (int blk = warp; blk < n_blk; blk += kSWarps) {
        const int b = blk * 32 + lane;
        int gam = 0;
        if (b < P.B) {
            const int g = P.gamma ? P.gamma[b] : G;
            const float Tf = P.temp ? P.temp[b] : P.temp_scalar;
            const bool ok = (g >= 1 && g <= G) && (Tf >= 0.f) && (Tf != __int_as_float(0x7f800000));
            gam = ok ? g : 0;
            sh.gam[b] = static_cast<unsigned char>(gam);
        }
        for (int p = 0; p <= G; ++p) {
            const unsigned A = __ballot_sync(0xffffffffu, gam > p);
            const unsigned E = __ballot_sync(0xffffffffu, gam == p && gam >= 1);
            if (lane == 0) sh.pre[p][blk] = static_cast<unsigned short>(2 * __popc(A) + __popc(E));
        }
    }
    __syncthreads();
    if (threadIdx.x <= G) {
        const int p = threadIdx.x;
        int run = 0;
        for (int blk = 0; blk < n_blk; ++blk) {
            const int w = sh.pre[p][blk];
            sh.pre[p][blk] = static_cast<unsigned short>(run);
            run += w;
        }
        sh.pre[p][n_blk] = static_cast<unsigned short>(run);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int p = 0; p <= G; ++p) { sh.phase0[p] = run; run += sh.pre[p][n_blk]; }
        sh.phase0[G + 1] = run;
        sh.n_items = run * S.n_slice;
    }
    __syncthreads();

    // batch rows that take no part (gamma or temperature out of range): neutral outputs and their status
    for (int b = blockIdx.x + warp * gridDim.x; b < P.B; b += gridDim.x * kSWarps) {
        if (sh.gam[b] != 0) continue;
        const int g = P.gamma ? P.gamma[b] : G;
        const float Tf = P.temp ? P.temp[b] : P.temp_scalar;
        int status = 0;
        if (g < 1 || g > G) status |= 1;
        if (!(Tf >= 0.f) || Tf == __int_as_float(0x7f800000)) status |= 8;
        if (lane < G) {
            if (P.H) P.H[static_cast<long long>(b) * G + lane] = 0.f;
            if (P.C) P.C[static_cast<long long>(b) * G + lane] = 0.f;
        }
        if (P.feat && lane < 4) P.feat[static_cast<long long>(b) * 4 + lane] = 0.f;
        if (P.mode & MODE_MLP) {
            if (P.scores && lane < P.n_out) P.scores[static_cast<long long>(b) * P.n_out + lane] = 0.f;
            if (lane == 0) P.gamma_next[b] = 0;
        }
        if (lane <= G) P.out_tok[static_cast<long long>(b) * (G + 1) + lane] = -1;
        if (lane == 0) {
            P.n_acc[b] = 0;
            if (P.status) P.status[b] = status;
            atomicAdd(&S.ctrl->resolved, 1);
        }
    }

    // ---- every warp: claim a quantum, sweep it (with the next one's first loads already out), post it ----
    extern __shared__ __align__(128) unsigned char s_dyn[];
    const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(s_dyn)) + warp * SStage<T>::kWarpBytes;
    int cursor = 0, rslot = 0, wslot = 0;
    SItem* it = nullptr;
    int q = 0;
    bool have = s_claim<T>(P, S, sh, cursor, it, q, true);
    while (have) {
        if (it->type == 2) {
            s_resample_job<T>(P, S, sh, *it, q);
            have = s_claim<T>(P, S, sh, cursor, it, q, true);
            continue;
        }
        const T* base = static_cast<const T*>(it->row) + it->elem0;
        int n_valid = it->n_elem, nq = it->n_q;
        rslot = wslot;  // nothing of this warp is in flight: the ring starts afresh wherever the write slot stands
        sq_prime<T>(ring, wslot, base, q, nq, n_valid, lane);
        for (;;) {
            // whoever passes here while the ring has a free slot fills it (a fill is a chain of global round
            // trips; paid here, with this warp's copies in flight, it is hidden)
            if (!s_vol(&sh.lock) && !s_vol(&sh.exhausted) &&
                (s_vol(&sh.tail) < kSRing || s_vol(&sh.ring[s_vol(&sh.tail) % kSRing].busy) == 0) &&
                !(s_vol(&sh.stream_done) && ld_relaxed(&S.ctrl->rs_next) >= ld_relaxed(&S.ctrl->rs_tail) * S.rs_shares))
                s_try_fill<T>(P, S, sh, false);
            // the quantum after this one, if the ring has one: its first copies go out while this one is swept
            // (unless bookkeeping is queued: then this warp reserves a job and runs it after this quantum)
            SItem* nit = nullptr;
            int qn = 0;
            const int job = s_job_reserve(sh);
            const bool ahead = job < 0 && s_claim<T>(P, S, sh, cursor, nit, qn, false);
            const bool chain = ahead && nit->type == 1;
            const T* nbase = nullptr;
            int n_next = 0, nqn = 1;
            if (chain) {
                nbase = static_cast<const T*>(nit->row) + nit->elem0;
                n_next = nit->n_elem;
                nqn = nit->n_q;
            }
            const int e_row = it->elem0;
            const float scale = it->scale;
            const int path = it->path;
            float4 part;
            if (path == PATH_DRAFT) part = sq_sweep<T, PATH_DRAFT>(ring, rslot, wslot, base, q, nq, n_valid, e_row, scale, nbase, qn, nqn, n_next);
            else if (path == PATH_TARGET) part = sq_sweep<T, PATH_TARGET>(ring, rslot, wslot, base, q, nq, n_valid, e_row, scale, nbase, qn, nqn, n_next);
            else part = sq_sweep<T, PATH_ARGMAX>(ring, rslot, wslot, base, q, nq, n_valid, e_row, scale, nbase, qn, nqn, n_next);
            rslot = (rslot + kSSteps) % SStage<T>::kSlots;
            wslot = (wslot + kSSteps) % SStage<T>::kSlots;
            s_finish_sweep<T>(P, S, sh, *it, q, part);
            if (job >= 0) s_job_run<T>(P, S, sh, job);
            have = ahead;
            it = nit; q = qn; base = nbase; n_valid = n_next; nq = nqn;
            if (!chain) break;
        }
        if (!have) have = s_claim<T>(P, S, sh, cursor, it, q, true);
    }

    // a poll limit ran out somewhere: the batch rows this CTA answers for and that are not complete get
    // SPECKV_ROW_TIMEOUT and neutral tokens
    if (s_vol(&sh.error)) {
        if (threadIdx.x == 0) atomicExch(&S.ctrl->error, 1);
        for (int b = blockIdx.x + warp * gridDim.x; b < P.B; b += gridDim.x * kSWarps) {
            if (sh.gam[b] == 0) continue;
            unsigned long long st = 0;
            if (lane == 0) st = ld_state(S.state + b);
            st = __shfl_sync(0xffffffffu, st, 0);
            if ((st & kStDraw) && (st & kStEpi)) continue;
            if (lane <= G) P.out_tok[static_cast<long long>(b) * (G + 1) + lane] = -1;
            if (lane == 0) {
                P.n_acc[b] = 0;
                if (P.status) {
                    if (st & kStEpi) atomicOr(P.status + b, 16);
                    else P.status[b] = 16;
                }
            }
        }
    }
}

}  // namespace speckv
