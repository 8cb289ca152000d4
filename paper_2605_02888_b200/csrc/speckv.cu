// Host side of libspeckv: argument checks, workspace plan and kernel launches behind the
// C ABI declared in include/speckv.h.  No allocation, no synchronisation.  The only state the
// library keeps between calls is a handful of per-device constants (SM count, kernel attributes set,
// the address of the built-in scratch array), each published with release/acquire atomics; none of
// them survives cudaDeviceReset.
#include "speckv.h"
#include "speckv_internal.h"

#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdint>

#include "speckv_kernels.cuh"
#include "speckv_pipeline.cuh"
#include "speckv_shard.cuh"
#include "speckv_sample.cuh"

namespace {

using namespace speckv;

constexpr int kSliceBytes = 262144;  // bytes of one logit row that one sweep CTA streams
constexpr size_t kAlign = 256;

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Plan {
    int J_full;      // logit rows per batch row with verification: 2*G + 1
    int nvec;        // kVec-element vectors per logit row
    int nchunk;      // 256-element chunks per logit row
    int R;           // resample CTAs per batch row
    int chunks_per_cta;
    size_t off_tick, off_info, off_part, off_csum, off_tokl, total;
};

inline int esize(speckv_dtype dt) { return dt == SPECKV_BF16 ? 2 : 4; }

// Bounds-checked build: the extents a call's kernels may touch, registered on the call's stream before
// its first kernel.  Range 0: draft logits, 1: target logits, 2: workspace, 3..: further caller arrays.
struct DbgExtra { const void* p; size_t bytes; };
cudaError_t dbg_register(cudaStream_t cs, const speckv_batch* bt, bool target, const void* ws, size_t ws_bytes,
                         const DbgExtra* extra = nullptr, int n_extra = 0) {
#ifdef SPECKV_DEBUG
    DbgRanges r{};
    auto span = [&](const void* base, int64_t sb, int64_t sp, int n_pos) -> unsigned long long {
        const long long last = static_cast<long long>(bt->B - 1) * sb + static_cast<long long>(n_pos - 1) * sp + bt->V;
        return reinterpret_cast<unsigned long long>(base) + static_cast<unsigned long long>(last) * esize(bt->dtype);
    };
    if (bt->B > 0 && bt->draft_logits) {
        r.lo[0] = reinterpret_cast<unsigned long long>(bt->draft_logits);
        r.hi[0] = span(bt->draft_logits, bt->draft_stride_b, bt->draft_stride_pos, bt->gamma_max);
    }
    if (bt->B > 0 && target && bt->target_logits) {
        r.lo[1] = reinterpret_cast<unsigned long long>(bt->target_logits);
        r.hi[1] = span(bt->target_logits, bt->target_stride_b, bt->target_stride_pos, bt->gamma_max + 1);
    }
    r.lo[2] = reinterpret_cast<unsigned long long>(ws);
    r.hi[2] = r.lo[2] + ws_bytes;
    for (int k = 0; k < n_extra && 3 + k < kDbgRanges; ++k) {
        r.lo[3 + k] = reinterpret_cast<unsigned long long>(extra[k].p);
        r.hi[3 + k] = r.lo[3 + k] + extra[k].bytes;
    }
    return cudaMemcpyToSymbolAsync(g_dbg_ranges, &r, sizeof r, 0, cudaMemcpyHostToDevice, cs);
#else
    (void)cs; (void)bt; (void)target; (void)ws; (void)ws_bytes; (void)extra; (void)n_extra;
    return cudaSuccess;
#endif
}

// vocabulary slices per logit row for a sweep over J logit rows per batch row
int choose_nsplit(int B, int J, int V, speckv_dtype dt) {
    const int nvec = (V + kVec - 1) / kVec;
    const double row_bytes = static_cast<double>(V) * esize(dt);
    int ns = static_cast<int>(std::lround(row_bytes / static_cast<double>(kSliceBytes)));
    if (ns < 1) ns = 1;
    // small batches: enough CTAs to put a few on every SM
    const long long rows = static_cast<long long>(B) * J;
    const long long want = (1184 + rows - 1) / (rows > 0 ? rows : 1);
    if (want > ns) ns = static_cast<int>(want > kMaxSplit ? kMaxSplit : want);
    if (ns > kMaxSplit) ns = kMaxSplit;
    // at least one vector per thread in a slice
    int cap = nvec / kThreads;
    if (cap < 1) cap = 1;
    if (ns > cap) ns = cap;
    return ns;
}

constexpr int kEarlyPositions = 2;   // positions whose acceptance tests the sliced sweep takes ahead of the rest of the row
constexpr int kRsChunksPerCta = 64;  // 256-element chunks of the stop position that one resample CTA sums

Plan make_plan(const speckv_batch* bt) {
    Plan p;
    const size_t B = static_cast<size_t>(bt->B);
    p.J_full = 2 * bt->gamma_max + 1;
    p.nvec = (bt->V + kVec - 1) / kVec;
    p.nchunk = (bt->V + kChunk - 1) / kChunk;
    p.R = (p.nchunk + kRsChunksPerCta - 1) / kRsChunksPerCta;
    if (p.R > 32) p.R = 32;
    if (p.R < 1) p.R = 1;
    p.chunks_per_cta = (p.nchunk + p.R - 1) / p.R;
    size_t off = 0;
    p.off_tick = off; off = align_up(off + (6 * B + 4) * sizeof(int));  // tickets, counters, row queue, row flags, first-generation tickets, early stops
    p.off_info = off; off = align_up(off + B * sizeof(RowInfo));
    p.off_part = off; off = align_up(off + B * p.J_full * kMaxSplit * sizeof(float4));
    p.off_csum = off; off = align_up(off + B * p.nchunk * sizeof(float));
    p.off_tokl = off; off = align_up(off + B * static_cast<size_t>(bt->gamma_max) * sizeof(float2));
    p.total = off < kAlign ? kAlign : off;
    return p;
}

// what the caller must provide
size_t workspace_total(const speckv_batch* bt) { return make_plan(bt).total; }

// polls a waiting CTA spends before it gives a row up (SPECKV_ROW_TIMEOUT); lowered by tests only
std::atomic<int> g_wait_limit{1 << 20};

speckv_status check_batch(const speckv_batch* bt, bool need_target) {
    if (!bt) return SPECKV_ERR_INVALID_ARG;
    if (bt->B < 0 || bt->gamma_max < 1 || bt->V < 1) return SPECKV_ERR_INVALID_ARG;
    if (bt->dtype != SPECKV_F32 && bt->dtype != SPECKV_BF16) return SPECKV_ERR_UNSUPPORTED;
    if (bt->gamma_max > SPECKV_MAX_GAMMA) return SPECKV_ERR_UNSUPPORTED;
    if (bt->V > (1 << 30) || bt->B > (1 << 24)) return SPECKV_ERR_UNSUPPORTED;
    if (bt->B == 0) return SPECKV_OK;
    if (!bt->draft_logits) return SPECKV_ERR_INVALID_ARG;
    // a stride of 0 broadcasts one row; anything else must step over whole rows
    auto stride_ok = [&](int64_t s) { return s == 0 || s >= bt->V; };
    if (!stride_ok(bt->draft_stride_b) || !stride_ok(bt->draft_stride_pos)) return SPECKV_ERR_INVALID_ARG;
    if (need_target) {
        if (!bt->target_logits || !bt->draft_tokens || !bt->uniforms) return SPECKV_ERR_INVALID_ARG;
        if (!stride_ok(bt->target_stride_b) || !stride_ok(bt->target_stride_pos)) return SPECKV_ERR_INVALID_ARG;
    }
    if (!(bt->temperature) && !(bt->temperature_scalar >= 0.f)) return SPECKV_ERR_INVALID_ARG;
    if (bt->flags & ~(SPECKV_READ_ALL_TARGET_ROWS | SPECKV_SCHEDULE_SLICED)) return SPECKV_ERR_INVALID_ARG;
    return SPECKV_OK;
}

speckv_status check_mlp(const speckv_mlp* m) {
    if (!m || !m->W2 || !m->b2) return SPECKV_ERR_INVALID_ARG;
    if (m->feature_layout < 0 || m->feature_layout > 2) return SPECKV_ERR_INVALID_ARG;
    const int min_hidden = m->feature_layout == 2 ? 0 : 1;  // the paper-form predictor may be linear
    if (m->n_hidden < min_hidden || m->n_out < 1 || m->n_in < 1) return SPECKV_ERR_INVALID_ARG;
    if (m->n_hidden > 0 && (!m->W1 || !m->b1)) return SPECKV_ERR_INVALID_ARG;
    if (m->n_hidden > SPECKV_MAX_HIDDEN || m->n_out > 8 || m->n_in > 8) return SPECKV_ERR_UNSUPPORTED;
    if (m->score_transform != 0 && m->score_transform != 1) return SPECKV_ERR_INVALID_ARG;
    if (m->n_in < (m->feature_layout == 0 ? 3 : m->feature_layout == 1 ? 4 : 5)) return SPECKV_ERR_INVALID_ARG;
    return SPECKV_OK;
}

bool rows_aligned(const void* base, int64_t sb, int64_t sp, int es) {
    return (reinterpret_cast<uintptr_t>(base) % 16 == 0) && ((sb * es) % 16 == 0) && ((sp * es) % 16 == 0);
}

void fill_mlp(KParams& P, const speckv_mlp* m, const float* comp) {
    P.n_in = m->n_in; P.n_hidden = m->n_hidden; P.n_out = m->n_out;
    P.layout = m->feature_layout; P.transform = m->score_transform;
    P.n_comp = m->n_in - (m->feature_layout == 0 ? 3 : m->feature_layout == 1 ? 4 : 5);
    P.W1 = m->W1; P.b1 = m->b1; P.W2 = m->W2; P.b2 = m->b2; P.comp = comp;
    for (int j = 0; j < 8; ++j) P.gch[j] = m->gamma_choices[j];
}

struct Events {  // optional timing events around the kernels of a step
    cudaEvent_t before_sweep = nullptr, after_sweep = nullptr, after_resample = nullptr;
};

// Staged sweep: persistent CTAs, two per SM.  Needs 16-byte aligned rows whose byte length is a
// multiple of 16, and a batch whose per-row tables fit in shared memory.
// SM count of the current device, looked up once per device (0 in the slot = not yet known).
cudaError_t sm_count(int* out) {
    static std::atomic<int> cached[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool slot = dev >= 0 && dev < 64;
    int sms = slot ? cached[dev].load(std::memory_order_acquire) : 0;
    if (sms == 0) {
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        if (slot) cached[dev].store(sms, std::memory_order_release);
    }
    *out = sms;
    return cudaSuccess;
}

template <typename T>
cudaError_t launch_pipe(const KParams& P, cudaStream_t st) {
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const size_t smem = (sizeof(PipeShared) + 127) / 128 * 128 + static_cast<size_t>(kStages) * kStageBytes;
    const bool slot = dev >= 0 && dev < 64;
    if (!slot || !configured[dev].load(std::memory_order_acquire)) {
        e = cudaFuncSetAttribute(pipe_sweep_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        if (slot) configured[dev].store(true, std::memory_order_release);
    }
    int sms = 0;
    e = sm_count(&sms);
    if (e != cudaSuccess) return e;
    pipe_sweep_kernel<T><<<kPipeCtasPerSm * sms, kPipeThreads, smem, st>>>(P);
    return cudaGetLastError();
}

// After the register-staged sweep the fresh tokens are drawn by extra CTAs of the same launch; the rows swept last have their fresh tokens drawn by more, shorter CTAs (see resample_body)
constexpr int kRsTailRows = 32;  // b256, same box, builds in turn: 16 rows 158.7 us, 32 rows 156.6 us, 64 rows 156.7 us, 128 rows 157.2 us
constexpr int kRsTailMult = 2;
constexpr int kRsSmallCtas = 1184;  // resample CTAs wanted in flight for a small batch (two per CTA slot)

template <typename T, bool ALIGNED>
cudaError_t launch_all(KParams P, cudaStream_t st, const Events& ev, bool staged) {
    constexpr int U = sizeof(T) == 2 ? kSweepLoads : (kSweepLoads + 1) / 2;
    const bool verify = (P.mode & MODE_VERIFY) != 0;
    const bool ring = ALIGNED && staged;
    P.rs_tail = 0; P.R2 = P.R; P.chunks_per_cta2 = P.chunks_per_cta;
    bool merged = verify && !ring && P.rdone;
    if (merged && P.B >= 4 * kRsTailRows && P.R * kRsTailMult <= 32 && kRsTailMult > 1) {
        P.rs_tail = kRsTailRows;
        P.R2 = P.R * kRsTailMult;
        P.chunks_per_cta2 = (P.nchunk + P.R2 - 1) / P.R2;
    }
    const long long n_draw = static_cast<long long>(P.B - P.rs_tail) * P.R + static_cast<long long>(P.rs_tail) * P.R2;
    merged = merged && P.n_sweep + n_draw <= 0x7fffffffLL;
    if (ev.before_sweep) cudaEventRecord(ev.before_sweep, st);
    cudaError_t e;
    if (ring) {
        e = launch_pipe<T>(P, st);
    } else {
        const long long grid = P.n_sweep + (merged ? n_draw : 0);
        sweep_kernel<T, ALIGNED, U><<<static_cast<unsigned>(grid), kThreads, 0, st>>>(P);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return e;
    if (ev.after_sweep) cudaEventRecord(ev.after_sweep, st);
    if (verify && !merged) {
        // programmatic dependent launch: the kernel's CTAs are scheduled while the sweep drains and
        // wait inside the kernel for the sweep's results
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(n_draw));
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, resample_kernel<T, ALIGNED>, P);
    }
    if (ev.after_resample) cudaEventRecord(ev.after_resample, st);
    return e;
}

// Shared driver of signals / verify / step.
speckv_status run(const speckv_batch* bt, int mode, const float* comp, const speckv_mlp* mlp, float* H,
                  float* C, float* feat, float* scores, int32_t* gamma_next, int32_t* n_accepted,
                  int32_t* out_tokens, int32_t* row_status, void* ws, size_t ws_bytes, void* stream,
                  const Events& ev = Events()) {
    const bool verify = (mode & MODE_VERIFY) != 0;
    speckv_status st = check_batch(bt, verify);
    if (st != SPECKV_OK) return st;
    if (mode & MODE_MLP) {
        st = check_mlp(mlp);
        if (st != SPECKV_OK) return st;
        if (!gamma_next || !feat) return SPECKV_ERR_INVALID_ARG;
    }
    if (verify && (!n_accepted || !out_tokens)) return SPECKV_ERR_INVALID_ARG;
    if (bt->B == 0) return SPECKV_OK;
    const Plan pl = make_plan(bt);
    if (!ws || reinterpret_cast<uintptr_t>(ws) % kAlign != 0) return SPECKV_ERR_INVALID_ARG;
    if (ws_bytes < workspace_total(bt)) return SPECKV_ERR_WORKSPACE;

    KParams P{};
    P.B = bt->B; P.G = bt->gamma_max; P.V = bt->V;
    P.J = verify ? pl.J_full : bt->gamma_max;
    P.nsplit = choose_nsplit(P.B, P.J, P.V, bt->dtype);
    P.nvec = pl.nvec;
    P.per_split = (pl.nvec + P.nsplit - 1) / P.nsplit;
    P.nchunk = pl.nchunk; P.R = pl.R; P.chunks_per_cta = pl.chunks_per_cta;
    {
        // small batches: more, shorter shares per row, so that the draw of a handful of rows still spreads
        // over the SMs (the draw of a row is a chain of dependent round trips, shorter with fewer chunks per CTA)
        const int want = (kRsSmallCtas + P.B - 1) / P.B;
        int cap = (P.nchunk + 7) / 8;  // at least one chunk per warp
        if (cap > 32) cap = 32;
        if (want > P.R && cap > P.R) {
            P.R = want < cap ? want : cap;
            P.chunks_per_cta = (P.nchunk + P.R - 1) / P.R;
        }
    }
    P.mode = mode; P.bits = bt->entropy_in_bits ? 1 : 0;
    P.wait_limit = g_wait_limit.load(std::memory_order_relaxed);
    P.d = bt->draft_logits; P.dsb = bt->draft_stride_b; P.dsp = bt->draft_stride_pos;
    P.t = bt->target_logits; P.tsb = bt->target_stride_b; P.tsp = bt->target_stride_pos;
    P.tok = bt->draft_tokens; P.gamma = bt->gamma; P.temp = bt->temperature;
    P.temp_scalar = bt->temperature_scalar; P.u = bt->uniforms;
    if (mode & MODE_MLP) fill_mlp(P, mlp, comp);
    P.H = H; P.C = C; P.feat = feat; P.scores = scores; P.gamma_next = gamma_next;
    P.n_acc = n_accepted; P.out_tok = out_tokens; P.status = row_status;
    char* w = static_cast<char*>(ws);
    P.tick1 = reinterpret_cast<int*>(w + pl.off_tick);
    P.tick2 = P.tick1 + P.B;
    P.qcount = P.tick1 + 2 * P.B;
    P.qhead = P.qcount + 1;
    P.qtail = P.qcount + 2;
    P.rowq = P.qcount + 4;
    P.info = reinterpret_cast<RowInfo*>(w + pl.off_info);
    P.part = reinterpret_cast<float4*>(w + pl.off_part);
    P.csum = reinterpret_cast<float*>(w + pl.off_csum);

    if (static_cast<long long>(P.B) * P.J * P.nsplit > 0x7fffffffLL) return SPECKV_ERR_UNSUPPORTED;
    P.n_sweep = P.B * P.J * P.nsplit;

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (dbg_register(cs, bt, verify, ws, ws_bytes) != cudaSuccess) return SPECKV_ERR_CUDA;
    const int es = esize(bt->dtype);
    bool aligned = rows_aligned(bt->draft_logits, bt->draft_stride_b, bt->draft_stride_pos, es);
    if (verify) aligned = aligned && rows_aligned(bt->target_logits, bt->target_stride_b, bt->target_stride_pos, es);
    const long long row_bytes = static_cast<long long>(P.V) * es;

    if (cudaMemsetAsync(P.tick1, 0, (6 * static_cast<size_t>(P.B) + 4) * sizeof(int), cs) != cudaSuccess)
        return SPECKV_ERR_CUDA;

    // the staged sweep wants whole 16-byte granules per row and a batch its per-row tables can hold
    // Which sweep.  Measured on B200 (full-size workloads, same inputs): fp32 logits are bound by
    // memory and the bulk-copy ring is faster (6.7-6.9 against 6.4 TB/s); bf16 logits need one
    // exponential per two bytes, and hiding that latency next to the memory latency takes the 32
    // warps per SM of the register-staged kernel (4.95 against 4.6 TB/s), whose draining tail the
    // resample CTAs of the same grid then fill.
    // Below a few hundred rows the ring's fixed costs (per-CTA tables, one epilogue warp per CTA, a
    // resample kernel that cannot overlap) outweigh its streaming rate: b512_mixed cut to 128 / 256 /
    // 512 rows takes 178 / 317 / 564 us with the ring and 166 / 307 / 581 us without.
constexpr int kPipeMinB = 384;
    const bool staged = bt->dtype == SPECKV_F32 && aligned && row_bytes % 16 == 0 && P.B <= kPipeMaxB && P.B >= kPipeMinB &&
                        !(bt->flags & SPECKV_SCHEDULE_SLICED);
    // completion flags per batch row and the logits at the draft tokens: only the register-staged sweep
    // overlaps the resample work with its own tail; after the ring sweep the resample kernel starts when
    // everything is done and a flag would only cost it a round trip
    P.rdone = (verify && !staged) ? P.rowq + P.B : nullptr;
    P.tokl = (verify && !staged) ? reinterpret_cast<float2*>(static_cast<char*>(ws) + pl.off_tokl) : nullptr;
    if (verify && !staged) {
        // generation order: positions 0..k of every batch row first, so that their acceptance tests are in
        // before the CTAs of the later target rows start (most walks that stop early stop at the first two
        // positions, and a later position's test would come too late for the CTAs behind it anyway)
        P.k_early = P.G >= 2 ? kEarlyPositions - 1 : 0;
        P.read_all = (bt->flags & SPECKV_READ_ALL_TARGET_ROWS) ? 1 : 0;
        P.tick_early = P.rowq + 2 * P.B;
        P.early = P.rowq + 3 * P.B;
    }
    P.rs_reverse = staged ? 1 : 0;  // the ring sweep ends all at once: no drain for the resample kernel to fill
    P.Lg = static_cast<int>(row_bytes / 16);
    P.Lp = (P.Lg + kStageGran - 1) / kStageGran * kStageGran;
    cudaError_t e;
    if (bt->dtype == SPECKV_BF16)
        e = aligned ? launch_all<__nv_bfloat16, true>(P, cs, ev, staged) : launch_all<__nv_bfloat16, false>(P, cs, ev, false);
    else
        e = aligned ? launch_all<float, true>(P, cs, ev, staged) : launch_all<float, false>(P, cs, ev, false);
    return e == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

// Draft-side sampling: its own workspace plan (one resample slot per drafted position).
struct SamplePlan {
    int nchunk, R, chunks_per_cta;
    size_t off_tick, off_info, off_part, off_csum, off_cz, total;
};
SamplePlan make_sample_plan(const speckv_batch* bt) {
    SamplePlan p;
    const size_t B = static_cast<size_t>(bt->B), G = static_cast<size_t>(bt->gamma_max);
    p.nchunk = (bt->V + kChunk - 1) / kChunk;
    p.R = (p.nchunk + 63) / 64;
    if (p.R > 32) p.R = 32;
    if (p.R < 1) p.R = 1;
    p.chunks_per_cta = (p.nchunk + p.R - 1) / p.R;
    size_t off = 0;
    p.off_tick = off; off = align_up(off + (2 * B + B * G) * sizeof(int));  // sweep tickets, resample tickets, row flags
    p.off_info = off; off = align_up(off + B * G * sizeof(RowInfo));
    p.off_part = off; off = align_up(off + B * G * kMaxSplit * sizeof(float4));
    p.off_csum = off; off = align_up(off + B * G * p.nchunk * sizeof(float));
    p.off_cz = off; off = align_up(off + B * G * p.nchunk * sizeof(float2));  // per-chunk (maximum, sum) of the one-pass kernel
    p.total = off < kAlign ? kAlign : off;
    return p;
}

speckv_status run_sample(const speckv_batch* bt, const float* uniforms, int32_t* tokens, int32_t* row_status,
                         void* ws, size_t ws_bytes, void* stream) {
    speckv_status st = check_batch(bt, false);
    if (st != SPECKV_OK) return st;
    if (bt->B == 0) return SPECKV_OK;
    if (!uniforms || !tokens) return SPECKV_ERR_INVALID_ARG;
    if (static_cast<long long>(bt->B) * bt->gamma_max > (1 << 24)) return SPECKV_ERR_UNSUPPORTED;
    const SamplePlan pl = make_sample_plan(bt);
    if (!ws || reinterpret_cast<uintptr_t>(ws) % kAlign != 0) return SPECKV_ERR_INVALID_ARG;
    if (ws_bytes < pl.total) return SPECKV_ERR_WORKSPACE;

    KParams P{};
    P.B = bt->B; P.G = bt->gamma_max; P.V = bt->V;
    P.J = bt->gamma_max;
    P.nsplit = choose_nsplit(P.B, P.J, P.V, bt->dtype);
    P.nvec = (bt->V + kVec - 1) / kVec;
    P.per_split = (P.nvec + P.nsplit - 1) / P.nsplit;
    P.nchunk = pl.nchunk; P.R = pl.R; P.chunks_per_cta = pl.chunks_per_cta;
    P.mode = MODE_SAMPLE; P.sample = 1; P.rs_reverse = 1;
    P.wait_limit = g_wait_limit.load(std::memory_order_relaxed);
    // the drafted positions are swept and drawn from as if they were target rows
    P.d = bt->draft_logits; P.dsb = bt->draft_stride_b; P.dsp = bt->draft_stride_pos;
    P.t = bt->draft_logits; P.tsb = bt->draft_stride_b; P.tsp = bt->draft_stride_pos;
    P.gamma = bt->gamma; P.temp = bt->temperature; P.temp_scalar = bt->temperature_scalar;
    P.u = uniforms;
    P.out_tok = tokens; P.status = row_status;
    char* w = static_cast<char*>(ws);
    P.tick1 = reinterpret_cast<int*>(w + pl.off_tick);
    P.tick2 = P.tick1 + P.B;
    P.rdone = P.tick2 + static_cast<size_t>(P.B) * P.G;
    P.info = reinterpret_cast<RowInfo*>(w + pl.off_info);
    P.part = reinterpret_cast<float4*>(w + pl.off_part);
    P.csum = reinterpret_cast<float*>(w + pl.off_csum);
    if (static_cast<long long>(P.B) * P.J * P.nsplit > 0x7fffffffLL) return SPECKV_ERR_UNSUPPORTED;
    P.n_sweep = P.B * P.J * P.nsplit;

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (dbg_register(cs, bt, false, ws, ws_bytes) != cudaSuccess) return SPECKV_ERR_CUDA;
    const size_t n_tick = static_cast<size_t>(P.B) * (2 + static_cast<size_t>(P.G));
    if (cudaMemsetAsync(P.tick1, 0, n_tick * sizeof(int), cs) != cudaSuccess) return SPECKV_ERR_CUDA;
    const int es = esize(bt->dtype);
    const bool aligned = rows_aligned(bt->draft_logits, bt->draft_stride_b, bt->draft_stride_pos, es);
constexpr int kSampleCtas = 2368;
    // One pass (speckv_sample.cuh) whenever a row's chunk records fit the searching CTA's shared memory.
    if (P.nchunk <= kRsStage &&
        static_cast<long long>(P.B) * P.G * P.R <= 0x7fffffffLL) {
        P.csum2 = reinterpret_cast<float*>(w + pl.off_cz);
        // shares per logit row: enough CTAs to fill the SMs a few times over, no more (a CTA costs a few
        // microseconds before its first load returns)
        {
            const long long draws = static_cast<long long>(P.B) * P.G;
            long long S = (kSampleCtas + draws - 1) / draws;
            if (S > P.R) S = P.R;
            if (S < 1) S = 1;
            P.R = static_cast<int>(S);
            P.chunks_per_cta = (P.nchunk + P.R - 1) / P.R;
        }
        const unsigned g1 = static_cast<unsigned>(P.B) * P.G * P.R;
        if (bt->dtype == SPECKV_BF16) {
            if (aligned) sample_onepass_kernel<__nv_bfloat16, true><<<g1, kThreads, 0, cs>>>(P);
            else sample_onepass_kernel<__nv_bfloat16, false><<<g1, kThreads, 0, cs>>>(P);
        } else {
            if (aligned) sample_onepass_kernel<float, true><<<g1, kThreads, 0, cs>>>(P);
            else sample_onepass_kernel<float, false><<<g1, kThreads, 0, cs>>>(P);
        }
        return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
    }
    // one launch: the draws' CTAs sit behind the sweep CTAs of the same grid and wait for their batch
    // row's flag (as in the verification step); two launches when the grid would not fit
    const long long n_draw = static_cast<long long>(P.B) * P.G * P.R;
    const bool merged = P.n_sweep + n_draw <= 0x7fffffffLL;
    if (merged) P.rs_reverse = 0; else P.rdone = nullptr;
    const unsigned grid1 = static_cast<unsigned>(P.n_sweep + (merged ? n_draw : 0));
    const unsigned grid2 = static_cast<unsigned>(n_draw);
    constexpr int Ub = kSweepLoads, Uf = (kSweepLoads + 1) / 2;
    if (bt->dtype == SPECKV_BF16) {
        if (aligned) { sweep_kernel<__nv_bfloat16, true, Ub><<<grid1, kThreads, 0, cs>>>(P); if (!merged) resample_kernel<__nv_bfloat16, true><<<grid2, kThreads, 0, cs>>>(P); }
        else { sweep_kernel<__nv_bfloat16, false, Ub><<<grid1, kThreads, 0, cs>>>(P); if (!merged) resample_kernel<__nv_bfloat16, false><<<grid2, kThreads, 0, cs>>>(P); }
    } else {
        if (aligned) { sweep_kernel<float, true, Uf><<<grid1, kThreads, 0, cs>>>(P); if (!merged) resample_kernel<float, true><<<grid2, kThreads, 0, cs>>>(P); }
        else { sweep_kernel<float, false, Uf><<<grid1, kThreads, 0, cs>>>(P); if (!merged) resample_kernel<float, false><<<grid2, kThreads, 0, cs>>>(P); }
    }
    return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

// Scratch for speckv_signals_static: lives in the library image, one copy per device that loads it.
static __device__ __align__(256) unsigned char g_static_scratch[SPECKV_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device.  In host code the array's name only
// stands for the symbol; the address a kernel can use has to be asked for, once per device.
cudaError_t static_scratch_address(void** out) {
    static std::atomic<void*> cached[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool slot = dev >= 0 && dev < 64;
    void* p = slot ? cached[dev].load(std::memory_order_acquire) : nullptr;
    if (!p) {
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (slot) cached[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return cudaSuccess;
}

// ---- vocabulary-sharded verification (speckv_shard.cuh) ----
struct ShardPlan {
    int nvec, nchunk, R, chunks_per_cta;
    size_t off_tick, off_part, off_csum, off_csum2, total;
};
ShardPlan make_shard_plan(const speckv_batch* bt) {
    ShardPlan p;
    const size_t B = static_cast<size_t>(bt->B), J = 2 * static_cast<size_t>(bt->gamma_max) + 1;
    p.nvec = (bt->V + kVec - 1) / kVec;
    p.nchunk = (bt->V + kChunk - 1) / kChunk;
    p.R = (p.nchunk + kRsChunksPerCta - 1) / kRsChunksPerCta;
    if (p.R > 32) p.R = 32;
    if (p.R < 1) p.R = 1;
    p.chunks_per_cta = (p.nchunk + p.R - 1) / p.R;
    size_t off = 0;
    p.off_tick = off; off = align_up(off + (3 * B + 4) * sizeof(int));  // sweep tickets, draw tickets, counters, row queue
    p.off_part = off; off = align_up(off + B * J * kMaxSplit * sizeof(float4));
    p.off_csum = off; off = align_up(off + B * p.nchunk * sizeof(float));
    p.off_csum2 = off; off = align_up(off + B * p.nchunk * sizeof(float));
    p.total = off < kAlign ? kAlign : off;
    return p;
}

constexpr int kShardWarpRowBytes = 65536;  // slice rows up to this size are swept by one warp each

// what every shard call needs from the local batch
speckv_status shard_params(const speckv_batch* bt, void* ws, size_t ws_bytes, KParams& P, ShardPlan& pl) {
    speckv_status st = check_batch(bt, true);
    if (st != SPECKV_OK) return st;
    pl = make_shard_plan(bt);
    if (bt->B == 0) return SPECKV_OK;
    if (!ws || reinterpret_cast<uintptr_t>(ws) % kAlign != 0) return SPECKV_ERR_INVALID_ARG;
    if (ws_bytes < pl.total) return SPECKV_ERR_WORKSPACE;
    P.B = bt->B; P.G = bt->gamma_max; P.V = bt->V; P.J = 2 * bt->gamma_max + 1;
    P.nvec = pl.nvec; P.nchunk = pl.nchunk; P.R = pl.R; P.chunks_per_cta = pl.chunks_per_cta;
    P.mode = MODE_VERIFY; P.bits = bt->entropy_in_bits ? 1 : 0;
    P.d = bt->draft_logits; P.dsb = bt->draft_stride_b; P.dsp = bt->draft_stride_pos;
    P.t = bt->target_logits; P.tsb = bt->target_stride_b; P.tsp = bt->target_stride_pos;
    P.tok = bt->draft_tokens; P.gamma = bt->gamma; P.temp = bt->temperature;
    P.temp_scalar = bt->temperature_scalar; P.u = bt->uniforms;
    char* w = static_cast<char*>(ws);
    P.tick1 = reinterpret_cast<int*>(w + pl.off_tick);
    P.tick2 = P.tick1 + P.B;
    P.qcount = P.tick1 + 2 * P.B;
    P.qhead = P.qcount + 1;
    P.qtail = P.qcount + 2;
    P.rowq = P.qcount + 4;
    P.part = reinterpret_cast<float4*>(w + pl.off_part);
    P.csum = reinterpret_cast<float*>(w + pl.off_csum);
    P.csum2 = reinterpret_cast<float*>(w + pl.off_csum2);
    return SPECKV_OK;
}
bool shard_aligned(const speckv_batch* bt) {
    const int es = esize(bt->dtype);
    return rows_aligned(bt->draft_logits, bt->draft_stride_b, bt->draft_stride_pos, es) &&
           rows_aligned(bt->target_logits, bt->target_stride_b, bt->target_stride_pos, es);
}

// Kernels of speckv_internal_wait_probe: arbitrary status words and empty token slots before the draw
// kernel runs, and afterwards a row epilogue that arrives late and raises each row's completion flag.
__global__ void wait_probe_fill(KParams P) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= P.B) return;
    P.status[b] = 0x5a5a;
    P.out_tok[2 * b] = -1;
    P.out_tok[2 * b + 1] = -1;
}
__global__ void wait_probe_late_epilogue(KParams P) {
    const int b = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b >= P.B) return;
    if ((threadIdx.x & 31) == 0) P.status[b] = 0;
    __syncwarp();
    row_done_signal(P, b, RS_BONUS, 1);
}

}  // namespace

extern "C" {

speckv_status speckv_workspace_size(const speckv_batch* batch, size_t* bytes) {
    if (!bytes) return SPECKV_ERR_INVALID_ARG;
    if (!batch || batch->B < 0 || batch->gamma_max < 1 || batch->V < 1) return SPECKV_ERR_INVALID_ARG;
    if (batch->gamma_max > SPECKV_MAX_GAMMA || batch->V > (1 << 30) || batch->B > (1 << 24))
        return SPECKV_ERR_UNSUPPORTED;
    *bytes = workspace_total(batch);
    return SPECKV_OK;
}

speckv_status speckv_signals(const speckv_batch* batch, float* H, float* C, float* feat,
                             int32_t* row_status, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
    return run(batch, MODE_SIGNALS, nullptr, nullptr, H, C, feat, nullptr, nullptr, nullptr, nullptr,
               row_status, workspace, workspace_bytes, cuda_stream);
}

speckv_status speckv_signals_static(const speckv_batch* batch, float* H, float* C, float* feat,
                                    int32_t* row_status, void* cuda_stream) {
    speckv_status st = check_batch(batch, false);
    if (st != SPECKV_OK) return st;
    if (batch->B == 0) return SPECKV_OK;
    if (make_plan(batch).total > SPECKV_STATIC_SCRATCH_BYTES) return SPECKV_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess || !scratch) return SPECKV_ERR_CUDA;
    // run() clears the ticket counters on the caller's stream; nothing else needs a known start
    return run(batch, MODE_SIGNALS, nullptr, nullptr, H, C, feat, nullptr, nullptr, nullptr, nullptr,
               row_status, scratch, SPECKV_STATIC_SCRATCH_BYTES, cuda_stream);
}

speckv_status speckv_sample_workspace_size(const speckv_batch* batch, size_t* bytes) {
    if (!bytes) return SPECKV_ERR_INVALID_ARG;
    if (!batch || batch->B < 0 || batch->gamma_max < 1 || batch->V < 1) return SPECKV_ERR_INVALID_ARG;
    if (batch->gamma_max > SPECKV_MAX_GAMMA || batch->V > (1 << 30) || batch->B > (1 << 24))
        return SPECKV_ERR_UNSUPPORTED;
    *bytes = make_sample_plan(batch).total;
    return SPECKV_OK;
}

speckv_status speckv_sample_draft(const speckv_batch* batch, const float* uniforms, int32_t* tokens,
                                  int32_t* row_status, void* workspace, size_t workspace_bytes,
                                  void* cuda_stream) {
    return run_sample(batch, uniforms, tokens, row_status, workspace, workspace_bytes, cuda_stream);
}

speckv_status speckv_select_gamma(int32_t B, const float* feat, const float* comp,
                                  const speckv_mlp* mlp, float* scores, int32_t* gamma_next,
                                  void* cuda_stream) {
    if (B < 0) return SPECKV_ERR_INVALID_ARG;
    speckv_status st = check_mlp(mlp);
    if (st != SPECKV_OK) return st;
    if (B == 0) return SPECKV_OK;
    if (!feat || !gamma_next) return SPECKV_ERR_INVALID_ARG;
    KParams P{};
    P.B = B;
    fill_mlp(P, mlp, comp);
    P.scores = scores; P.gamma_next = gamma_next;
    const int grid = (B + kWarps - 1) / kWarps;
    select_gamma_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(P, feat);
    return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

speckv_status speckv_verify(const speckv_batch* batch, int32_t* n_accepted, int32_t* out_tokens,
                            int32_t* row_status, void* workspace, size_t workspace_bytes,
                            void* cuda_stream) {
    return run(batch, MODE_VERIFY, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
               n_accepted, out_tokens, row_status, workspace, workspace_bytes, cuda_stream);
}

speckv_status speckv_step(const speckv_batch* batch, const float* comp, const speckv_mlp* mlp,
                          float* H, float* C, float* feat, float* scores, int32_t* gamma_next,
                          int32_t* n_accepted, int32_t* out_tokens, int32_t* row_status,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return run(batch, MODE_SIGNALS | MODE_VERIFY | MODE_MLP, comp, mlp, H, C, feat, scores, gamma_next,
               n_accepted, out_tokens, row_status, workspace, workspace_bytes, cuda_stream);
}

speckv_status speckv_step_profiled(const speckv_batch* batch, const float* comp, const speckv_mlp* mlp,
                                   float* H, float* C, float* feat, float* scores,
                                   int32_t* gamma_next, int32_t* n_accepted, int32_t* out_tokens,
                                   int32_t* row_status, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream, void* ev_before_sweep, void* ev_after_sweep,
                                   void* ev_after_resample) {
    Events ev;
    ev.before_sweep = static_cast<cudaEvent_t>(ev_before_sweep);
    ev.after_sweep = static_cast<cudaEvent_t>(ev_after_sweep);
    ev.after_resample = static_cast<cudaEvent_t>(ev_after_resample);
    return run(batch, MODE_SIGNALS | MODE_VERIFY | MODE_MLP, comp, mlp, H, C, feat, scores, gamma_next,
               n_accepted, out_tokens, row_status, workspace, workspace_bytes, cuda_stream, ev);
}

#ifdef SPECKV_DEBUG
namespace {
__global__ void dbg_selftest_kernel() {
    // addresses that no call has registered: looked at, never dereferenced
    dbg_ok(reinterpret_cast<const void*>(0x10ull), 16, DBG_LOGIT16);
    dbg_ok(reinterpret_cast<const void*>(0x20ull), 4, DBG_WS_STORE);
}
}  // namespace
#endif

speckv_status speckv_internal_debug_report(unsigned long long* out4, int reset, int selftest) {
#ifdef SPECKV_DEBUG
    if (!out4) return SPECKV_ERR_INVALID_ARG;
    if (selftest) dbg_selftest_kernel<<<1, 1>>>();
    if (cudaDeviceSynchronize() != cudaSuccess) return SPECKV_ERR_CUDA;
    if (cudaMemcpyFromSymbol(out4, g_dbg_report, sizeof(unsigned long long) * 4) != cudaSuccess) return SPECKV_ERR_CUDA;
    if (reset) {
        const unsigned long long zero[4] = {0, 0, 0, 0};
        if (cudaMemcpyToSymbol(g_dbg_report, zero, sizeof zero) != cudaSuccess) return SPECKV_ERR_CUDA;
    }
    return SPECKV_OK;
#else
    (void)out4; (void)reset; (void)selftest;
    return SPECKV_ERR_UNSUPPORTED;
#endif
}

int speckv_internal_set_wait_limit(int polls) {
    if (polls < 1) polls = 1;
    return g_wait_limit.exchange(polls);
}

speckv_status speckv_internal_wait_probe(int32_t B, int32_t* row_status, int32_t* out_tokens, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream) {
    if (B < 1 || B > 4096 || !row_status || !out_tokens || !workspace) return SPECKV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign != 0 || workspace_bytes < 2 * static_cast<size_t>(B) * sizeof(int))
        return SPECKV_ERR_WORKSPACE;
    // the draw kernel on its own, one CTA per batch row, with completion flags that nothing raises
    KParams P{};
    P.B = B; P.G = 1; P.V = kChunk; P.J = 3; P.nchunk = 1; P.R = 1; P.chunks_per_cta = 1;
    P.R2 = 1; P.chunks_per_cta2 = 1; P.mode = MODE_VERIFY;
    P.wait_limit = g_wait_limit.load(std::memory_order_relaxed);
    P.status = row_status; P.out_tok = out_tokens;
    P.rdone = static_cast<int*>(workspace);
    P.tick2 = P.rdone + B;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    {
        speckv_batch none{};
        if (dbg_register(cs, &none, false, workspace, workspace_bytes) != cudaSuccess) return SPECKV_ERR_CUDA;
    }
    if (cudaMemsetAsync(workspace, 0, 2 * static_cast<size_t>(B) * sizeof(int), cs) != cudaSuccess) return SPECKV_ERR_CUDA;
    wait_probe_fill<<<(B + 255) / 256, 256, 0, cs>>>(P);
    resample_kernel<float, true><<<static_cast<unsigned>(B), kThreads, 0, cs>>>(P);
    wait_probe_late_epilogue<<<(B + kWarps - 1) / kWarps, kThreads, 0, cs>>>(P);
    return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

speckv_status speckv_shard_workspace_size(const speckv_batch* local, size_t* bytes) {
    if (!bytes) return SPECKV_ERR_INVALID_ARG;
    if (!local || local->B < 0 || local->gamma_max < 1 || local->V < 1) return SPECKV_ERR_INVALID_ARG;
    if (local->gamma_max > SPECKV_MAX_GAMMA || local->V > (1 << 30) || local->B > (1 << 24))
        return SPECKV_ERR_UNSUPPORTED;
    *bytes = make_shard_plan(local).total;
    return SPECKV_OK;
}

speckv_status speckv_shard_sweep(const speckv_batch* local, int64_t v_begin, float* shard_state, float* shard_tokl,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
    KParams P{};
    ShardPlan pl;
    speckv_status st = shard_params(local, workspace, workspace_bytes, P, pl);
    if (st != SPECKV_OK || local->B == 0) return st;
    if (!shard_state || !shard_tokl || v_begin < 0 || v_begin > (1LL << 30)) return SPECKV_ERR_INVALID_ARG;
    P.nsplit = choose_nsplit(P.B, P.J, P.V, local->dtype);
    P.per_split = (P.nvec + P.nsplit - 1) / P.nsplit;
    if (static_cast<long long>(P.B) * P.J * P.nsplit > 0x7fffffffLL) return SPECKV_ERR_UNSUPPORTED;
    P.n_sweep = P.B * P.J * P.nsplit;
    P.v_begin = static_cast<int>(v_begin);
    P.export_state = 1;
    P.state = reinterpret_cast<float4*>(shard_state);
    P.tokl = reinterpret_cast<float2*>(shard_tokl);
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    {
        const DbgExtra ex[2] = {{shard_state, static_cast<size_t>(P.B) * P.J * sizeof(float4)},
                                {shard_tokl, static_cast<size_t>(P.B) * P.G * sizeof(float2)}};
        if (dbg_register(cs, local, true, workspace, workspace_bytes, ex, 2) != cudaSuccess) return SPECKV_ERR_CUDA;
    }
    if (cudaMemsetAsync(P.tick1, 0, (3 * static_cast<size_t>(P.B) + 4) * sizeof(int), cs) != cudaSuccess)
        return SPECKV_ERR_CUDA;
    if (cudaMemsetAsync(shard_tokl, 0, static_cast<size_t>(P.B) * P.G * sizeof(float2), cs) != cudaSuccess)
        return SPECKV_ERR_CUDA;
    const unsigned grid = static_cast<unsigned>(P.n_sweep);
    constexpr int Ub = kSweepLoads, Uf = (kSweepLoads + 1) / 2;
    const bool al = shard_aligned(local);
    // A slice row is short (V / n_shards columns).  One CTA per short row is mostly overhead and the
    // ring sweep pays per logit row as well (segment hand-over to its epilogue warp), so rows of up to
    // 64 KB are swept by one warp each, all of them resident at once; wider slices take the
    // CTA-per-slice sweep.
    const long long row_bytes = static_cast<long long>(P.V) * esize(local->dtype);
    if (row_bytes <= kShardWarpRowBytes) {
        const unsigned g2 = static_cast<unsigned>((static_cast<long long>(P.B) * P.J + kWarps - 1) / kWarps);
        if (local->dtype == SPECKV_BF16) {
            if (al) shard_rows_kernel<__nv_bfloat16, true, Ub><<<g2, kThreads, 0, cs>>>(P);
            else shard_rows_kernel<__nv_bfloat16, false, Ub><<<g2, kThreads, 0, cs>>>(P);
        } else {
            if (al) shard_rows_kernel<float, true, Uf><<<g2, kThreads, 0, cs>>>(P);
            else shard_rows_kernel<float, false, Uf><<<g2, kThreads, 0, cs>>>(P);
        }
        return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
    }
    if (local->dtype == SPECKV_BF16) {
        if (al) sweep_kernel<__nv_bfloat16, true, Ub><<<grid, kThreads, 0, cs>>>(P);
        else sweep_kernel<__nv_bfloat16, false, Ub><<<grid, kThreads, 0, cs>>>(P);
    } else {
        if (al) sweep_kernel<float, true, Uf><<<grid, kThreads, 0, cs>>>(P);
        else sweep_kernel<float, false, Uf><<<grid, kThreads, 0, cs>>>(P);
    }
    return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

speckv_status speckv_shard_finish(const speckv_batch* local, int32_t n_shards, int32_t shard_width, int32_t V_total,
                                  const float* all_state, const float* all_tokl, const float* comp,
                                  const speckv_mlp* mlp, float* H, float* C, float* feat, float* scores,
                                  int32_t* gamma_next, int32_t* n_accepted, int32_t* out_tokens, int32_t* row_status,
                                  void* row_info, void* cuda_stream) {
    speckv_status st = check_batch(local, true);
    if (st != SPECKV_OK) return st;
    if (n_shards < 1 || n_shards > 32 || shard_width < 1 || V_total < 1) return SPECKV_ERR_INVALID_ARG;
    if (static_cast<long long>(shard_width) * (n_shards - 1) >= V_total) return SPECKV_ERR_INVALID_ARG;
    if (local->B == 0) return SPECKV_OK;
    if (!all_state || !all_tokl || !n_accepted || !out_tokens || !row_info) return SPECKV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(row_info) % 16 != 0 || reinterpret_cast<uintptr_t>(all_state) % 16 != 0 ||
        reinterpret_cast<uintptr_t>(all_tokl) % 8 != 0)
        return SPECKV_ERR_INVALID_ARG;
    KParams P{};
    P.B = local->B; P.G = local->gamma_max; P.V = V_total; P.J = 2 * local->gamma_max + 1;
    P.mode = MODE_SIGNALS | MODE_VERIFY; P.bits = local->entropy_in_bits ? 1 : 0;
    if (mlp) {
        st = check_mlp(mlp);
        if (st != SPECKV_OK) return st;
        if (!gamma_next || !feat) return SPECKV_ERR_INVALID_ARG;
        P.mode |= MODE_MLP;
        fill_mlp(P, mlp, comp);
    }
    P.tok = local->draft_tokens; P.gamma = local->gamma; P.temp = local->temperature;
    P.temp_scalar = local->temperature_scalar; P.u = local->uniforms;
    P.H = H; P.C = C; P.feat = feat; P.scores = scores; P.gamma_next = gamma_next;
    P.n_acc = n_accepted; P.out_tok = out_tokens; P.status = row_status;
    P.part = const_cast<float4*>(reinterpret_cast<const float4*>(all_state));
    P.part_stride = P.B * P.J;
    P.n_shards = n_shards; P.shard_width = shard_width;
    P.tokl = const_cast<float2*>(reinterpret_cast<const float2*>(all_tokl));
    P.tokl_stride = static_cast<long long>(P.B) * P.G;
    P.info = static_cast<RowInfo*>(row_info);
    if (static_cast<long long>(P.B) * P.J > 0x7fffffffLL) return SPECKV_ERR_UNSUPPORTED;
    const unsigned grid = static_cast<unsigned>((P.B + kWarps - 1) / kWarps);
    {
        speckv_batch none{};  // this call reads no logits: only the gathered arrays and the row records
        const DbgExtra ex[3] = {{all_state, static_cast<size_t>(n_shards) * P.B * P.J * sizeof(float4)},
                                {all_tokl, static_cast<size_t>(n_shards) * P.B * P.G * sizeof(float2)},
                                {row_info, static_cast<size_t>(P.B) * sizeof(RowInfo)}};
        if (dbg_register(static_cast<cudaStream_t>(cuda_stream), &none, false, nullptr, 0, ex, 3) != cudaSuccess) return SPECKV_ERR_CUDA;
    }
    shard_finish_kernel<float><<<grid, kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(P);
    return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

speckv_status speckv_shard_draw_sums(const speckv_batch* local, const void* row_info, double* shard_weight,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
    KParams P{};
    ShardPlan pl;
    speckv_status st = shard_params(local, workspace, workspace_bytes, P, pl);
    if (st != SPECKV_OK || local->B == 0) return st;
    if (!row_info || !shard_weight) return SPECKV_ERR_INVALID_ARG;
    P.info = static_cast<RowInfo*>(const_cast<void*>(row_info));
    P.weight = shard_weight;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    {
        const DbgExtra ex[1] = {{row_info, static_cast<size_t>(P.B) * sizeof(RowInfo)}};
        if (dbg_register(cs, local, true, workspace, workspace_bytes, ex, 1) != cudaSuccess) return SPECKV_ERR_CUDA;
    }
    if (cudaMemsetAsync(P.tick2, 0, static_cast<size_t>(P.B) * sizeof(int), cs) != cudaSuccess) return SPECKV_ERR_CUDA;
    if (static_cast<long long>(P.B) * P.R > 0x7fffffffLL) return SPECKV_ERR_UNSUPPORTED;
    const unsigned grid = static_cast<unsigned>(P.B) * static_cast<unsigned>(P.R);
    const bool al = shard_aligned(local);
    if (local->dtype == SPECKV_BF16) {
        if (al) shard_sums_kernel<__nv_bfloat16, true><<<grid, kThreads, 0, cs>>>(P);
        else shard_sums_kernel<__nv_bfloat16, false><<<grid, kThreads, 0, cs>>>(P);
    } else {
        if (al) shard_sums_kernel<float, true><<<grid, kThreads, 0, cs>>>(P);
        else shard_sums_kernel<float, false><<<grid, kThreads, 0, cs>>>(P);
    }
    return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

speckv_status speckv_shard_draw_pick(const speckv_batch* local, int64_t v_begin, int32_t rank, int32_t n_shards,
                                     const void* row_info, const double* all_weight, int32_t* out_tokens,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
    KParams P{};
    ShardPlan pl;
    speckv_status st = shard_params(local, workspace, workspace_bytes, P, pl);
    if (st != SPECKV_OK || local->B == 0) return st;
    if (!row_info || !all_weight || !out_tokens) return SPECKV_ERR_INVALID_ARG;
    if (n_shards < 1 || n_shards > 32 || rank < 0 || rank >= n_shards || v_begin < 0 || v_begin > (1LL << 30))
        return SPECKV_ERR_INVALID_ARG;
    P.info = static_cast<RowInfo*>(const_cast<void*>(row_info));
    P.all_weight = all_weight;
    P.out_tok = out_tokens;
    P.rank = rank; P.n_shards = n_shards; P.v_begin = static_cast<int>(v_begin);
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    {
        const DbgExtra ex[1] = {{row_info, static_cast<size_t>(P.B) * sizeof(RowInfo)}};
        if (dbg_register(cs, local, true, workspace, workspace_bytes, ex, 1) != cudaSuccess) return SPECKV_ERR_CUDA;
    }
    const unsigned grid = static_cast<unsigned>(P.B);
    const bool al = shard_aligned(local);
    if (local->dtype == SPECKV_BF16) {
        if (al) shard_pick_kernel<__nv_bfloat16, true><<<grid, kThreads, 0, cs>>>(P);
        else shard_pick_kernel<__nv_bfloat16, false><<<grid, kThreads, 0, cs>>>(P);
    } else {
        if (al) shard_pick_kernel<float, true><<<grid, kThreads, 0, cs>>>(P);
        else shard_pick_kernel<float, false><<<grid, kThreads, 0, cs>>>(P);
    }
    return cudaGetLastError() == cudaSuccess ? SPECKV_OK : SPECKV_ERR_CUDA;
}

const char* speckv_status_string(speckv_status s) {
    switch (s) {
        case SPECKV_OK: return "ok";
        case SPECKV_ERR_INVALID_ARG: return "invalid argument";
        case SPECKV_ERR_UNSUPPORTED: return "unsupported size or type";
        case SPECKV_ERR_WORKSPACE: return "workspace too small";
        case SPECKV_ERR_CUDA: return "CUDA launch failed";
        case SPECKV_ERR_STATIC_LIMIT: return "batch needs more scratch than the built-in array holds";
    }
    return "unknown status";
}

int speckv_version(void) { return 100; }

}  // extern "C"
