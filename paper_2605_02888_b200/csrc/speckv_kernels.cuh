// Device code of libspeckv: the streaming sweep over vocabulary-sized logit rows, the
// per-row epilogue (signals, acceptance, controller) and the inverse-CDF resample.
//
// Scheme (sm_100a, CUDA cores only -- the work is a streaming reduction, not a contraction):
//   sweep kernel    one CTA per (row b, logit row j, vocabulary slice s).  Each thread keeps
//                   an online-softmax state over 16-byte vector loads, the CTA merges the
//                   256 states and stores one partial.  The last CTA of a batch row to finish
//                   (found with a ticket counter, nobody waits) merges that row's partials,
//                   decides the acceptances, raises the row's completion flag and then writes
//                   the signals and the controller outputs.
//   resample work   R CTAs per batch row rescan the stop position's draft/target rows, write
//                   per-256-element chunk sums of the residual weights, and the last of them
//                   locates the inverse-CDF threshold and writes the fresh token.  These CTAs
//                   sit behind the sweep CTAs in the sweep kernel's own grid and wait (bounded)
//                   for their row's flag, or run as a kernel of their own after the ring sweep
//                   of speckv_pipeline.cuh.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace speckv {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kVec = 8;                 // elements per lane per step
constexpr int kChunk = 32 * kVec;       // one warp step = one inverse-CDF chunk (256 elements)
constexpr int kMaxSplit = 32;
// Measured on b256 (same box, the two builds in turn, five times): 5 CTAs x 3 loads 156.7 us, 4 x 4 161.6 us,
// 5 x 4 163.6 us, 6 x 3 161.9 us; b256_g8 and b1024_loop the same within 0.1 %.
constexpr int kSweepLoads = 3;  // 16-byte loads in flight per thread (bf16); fp32 uses half as many vector steps
constexpr int kSweepCtasPerSm = 5;  // CTAs per SM the sweep kernel is compiled for (48 registers per thread)
constexpr float kFloor = -1.2676506002282294e30f;  // -2^100: logits below count as -inf
constexpr uint32_t kFloorBf16x2 = 0xF180F180u;     // -2^100 as two bf16
constexpr double kLn2 = 0.6931471805599453094;
constexpr double kLog2e = 1.4426950408889634074;

// ---- bounds-checked build (-DSPECKV_DEBUG) ---------------------------------------------------------
// Every global-memory access whose address comes out of index arithmetic (the logit loads of every
// kernel, the reads and writes of the workspace, the reads of the caller's state arrays in the sharded
// step) is first compared with the extents the host registered for the call.  An access outside them
// is counted, its address kept, and NOT performed: loads give a neutral value, stores are dropped.
// Nothing traps.  In the ordinary build the check is the constant true.
constexpr int kDbgRanges = 8;
struct DbgRanges { unsigned long long lo[kDbgRanges], hi[kDbgRanges]; };
#ifdef SPECKV_DEBUG
__device__ DbgRanges g_dbg_ranges;
__device__ unsigned long long g_dbg_report[4];  // violations, first offending address, its size, the kind of access
__device__ __forceinline__ bool dbg_ok(const void* p, unsigned bytes, int kind) {
    const unsigned long long a = reinterpret_cast<unsigned long long>(p);
#pragma unroll
    for (int k = 0; k < kDbgRanges; ++k)
        if (a >= g_dbg_ranges.lo[k] && a + bytes <= g_dbg_ranges.hi[k]) return true;
    if (atomicAdd(&g_dbg_report[0], 1ull) == 0ull) {
        g_dbg_report[1] = a;
        g_dbg_report[2] = bytes;
        g_dbg_report[3] = static_cast<unsigned long long>(kind);
    }
    return false;
}
#else
__device__ __forceinline__ bool dbg_ok(const void*, unsigned, int) { return true; }
#endif
enum : int { DBG_LOGIT16 = 1, DBG_LOGIT1 = 2, DBG_WS_LOAD = 3, DBG_WS_STORE = 4, DBG_COPY = 5 };

enum : int { MODE_SIGNALS = 1, MODE_VERIFY = 2, MODE_MLP = 4, MODE_SAMPLE = 8 };
enum : int { PATH_DRAFT = 0, PATH_TARGET = 1, PATH_ARGMAX = 2 };
enum : int { RS_NONE = 0, RS_RESIDUAL = 1, RS_BONUS = 2 };

struct RowInfo {  // written by the sweep kernel's row epilogue, read by the resample kernel
    int mode;     // RS_*
    int n;        // stop position
    float u2;     // uniform for the resample / bonus draw
    float scale;  // log2(e) / T as used by the sweep
    double lse2_p;  // log2-sum-exp2 of the target row at n
    double lse2_q;  // same for the draft row (residual only)
};

static_assert(sizeof(RowInfo) == 32, "the resample kernel reads a RowInfo as two 16-byte words");

struct KParams {
    int B, G, V, J, nsplit, nvec, per_split, nchunk, R, chunks_per_cta, mode, bits;
    int n_sweep;  // sweep kernel: CTAs that sweep; the rest of the grid (if any) does the resample work
    int sample;  // 1: draft-side sampling (every drafted position draws a token from its own row)
    int rs_tail, R2, chunks_per_cta2;  // resample: the last rs_tail draws in launch order use R2 CTAs each
    int wait_limit;  // polls a resample CTA spends on its row's completion flag before it gives the row up
    // Generation order of the sweep grid (verification, early != nullptr): first the draft and target rows of
    // positions 0..k_early of every batch row, then the remaining draft rows, last the remaining target rows,
    // which are left unread where the walk is already known to have stopped at a position <= k_early.
    int k_early, read_all;
    int* early;       // [B] 0 = not known yet, else stop position + 1, or G + 2 when the walk passes k_early
    int* tick_early;  // [B] arrivals of the first generation's CTAs
    int rs_reverse;  // resample kernel: 1 = last batch row first (after a sweep it cannot overlap: those rows are the freshest in L2)
    int Lg, Lp;  // staged sweep: 16-byte granules per logit row, and the same padded to whole ring stages
    const void* d; long long dsb, dsp;
    const void* t; long long tsb, tsp;
    const int* tok; const int* gamma; const float* temp; float temp_scalar; const float* u;
    // controller
    int n_in, n_hidden, n_out, layout, transform, n_comp;
    const float *W1, *b1, *W2, *b2, *comp;
    int gch[8];
    // outputs
    float *H, *C, *feat, *scores;
    int *gamma_next, *n_acc, *out_tok, *status;
    // workspace
    int *tick1, *tick2;
    int *qcount, *qhead, *qtail, *rowq;  // staged sweep: next quantum to hand out; queue of completed batch rows
    float2* tokl;  // [B, G] (draft logit, target logit) at the draft token, left by the register-staged sweep; may be NULL
    int* rdone;  // verification: rdone[b] = 1 once batch row b's epilogue has written everything the resample kernel reads
    RowInfo* info;
    float4* part;
    float* csum;
    // vocabulary-sharded verification (speckv_shard.cuh); all zero otherwise
    int part_stride;   // row epilogue: float4s between successive partials of one logit row (0 = adjacent)
    int n_shards;      // row epilogue: tokl holds one [B, G] table per shard, tokl_stride float2s apart
    int shard_width;   //   and the shard owning token x is min(x / shard_width, n_shards - 1)
    long long tokl_stride;
    int v_begin;       // sweep: first vocabulary index of this shard's slice (the batch's V is the slice width)
    int export_state;  // sweep: 1 = the row's last CTA writes the merged per-logit-row states instead of the row epilogue
    float4* state;     // [B, J] merged states of this shard (export)
    float* csum2;      // shard draw: chunk sums of p beside the residual's
    double* weight;    // shard draw: [B, 2] (residual mass, p mass) of this shard
    const double* all_weight;  // [n_shards, B, 2]
    int rank;
};

// ----------------------------------------------------------------------------------------
// small helpers
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Packed pairs of fp32 (sm_100 f32x2 arithmetic): one instruction works on two elements.
typedef unsigned long long f2;
__device__ __forceinline__ f2 pack2(float a, float b) {
    f2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(f2 v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ f2 add2(f2 a, f2 b) {
    f2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f2 sub2(f2 a, f2 b) {
    f2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f2 mul2(f2 a, f2 b) {
    f2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c) {
    f2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ f2 ex2_2(f2 a) {
    float x, y;
    unpack2(a, x, y);
    return pack2(ex2f(x), ex2f(y));
}
__device__ __forceinline__ float hsum2(f2 a) {
    float x, y;
    unpack2(a, x, y);
    return x + y;
}

__device__ __forceinline__ float max_nan(float a, float b) {  // NaN-propagating max
    float y;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b));
    return y;
}
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    if (!dbg_ok(p, 16, DBG_LOGIT16)) return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ __nv_bfloat162 as_bf2(uint32_t u) {
    return *reinterpret_cast<__nv_bfloat162*>(&u);
}
__device__ __forceinline__ uint32_t as_u32(__nv_bfloat162 h) {
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// Raw register image of kVec consecutive elements.
template <typename T> struct Raw;
template <> struct Raw<__nv_bfloat16> { uint4 a; };
template <> struct Raw<float> { uint4 a, b; };

template <typename T> __device__ __forceinline__ Raw<T> raw_fill(float v);
template <> __device__ __forceinline__ Raw<__nv_bfloat16> raw_fill<__nv_bfloat16>(float v) {
    uint32_t h = __float_as_uint(v) >> 16;  // callers pass bf16-representable values
    h |= h << 16;
    Raw<__nv_bfloat16> r; r.a = make_uint4(h, h, h, h); return r;
}
template <> __device__ __forceinline__ Raw<float> raw_fill<float>(float v) {
    uint32_t w = __float_as_uint(v);
    Raw<float> r; r.a = make_uint4(w, w, w, w); r.b = r.a; return r;
}

template <typename T> __device__ __forceinline__ void unpack(const Raw<T>& r, float (&x)[kVec]);
template <> __device__ __forceinline__ void unpack<__nv_bfloat16>(const Raw<__nv_bfloat16>& r, float (&x)[kVec]) {
    x[0] = bf_lo(r.a.x); x[1] = bf_hi(r.a.x); x[2] = bf_lo(r.a.y); x[3] = bf_hi(r.a.y);
    x[4] = bf_lo(r.a.z); x[5] = bf_hi(r.a.z); x[6] = bf_lo(r.a.w); x[7] = bf_hi(r.a.w);
}
template <> __device__ __forceinline__ void unpack<float>(const Raw<float>& r, float (&x)[kVec]) {
    x[0] = __uint_as_float(r.a.x); x[1] = __uint_as_float(r.a.y);
    x[2] = __uint_as_float(r.a.z); x[3] = __uint_as_float(r.a.w);
    x[4] = __uint_as_float(r.b.x); x[5] = __uint_as_float(r.b.y);
    x[6] = __uint_as_float(r.b.z); x[7] = __uint_as_float(r.b.w);
}

// the same kVec elements as four packed pairs
__device__ __forceinline__ void unpack_pairs(const Raw<__nv_bfloat16>& r, f2 (&x)[4]) {
    x[0] = pack2(bf_lo(r.a.x), bf_hi(r.a.x)); x[1] = pack2(bf_lo(r.a.y), bf_hi(r.a.y));
    x[2] = pack2(bf_lo(r.a.z), bf_hi(r.a.z)); x[3] = pack2(bf_lo(r.a.w), bf_hi(r.a.w));
}
__device__ __forceinline__ void unpack_pairs(const Raw<float>& r, f2 (&x)[4]) {
    x[0] = pack2(__uint_as_float(r.a.x), __uint_as_float(r.a.y));
    x[1] = pack2(__uint_as_float(r.a.z), __uint_as_float(r.a.w));
    x[2] = pack2(__uint_as_float(r.b.x), __uint_as_float(r.b.y));
    x[3] = pack2(__uint_as_float(r.b.z), __uint_as_float(r.b.w));
}

__device__ __forceinline__ float elem_to_float(const __nv_bfloat16* p, long long i) {
    if (!dbg_ok(p + i, 2, DBG_LOGIT1)) return 0.f;
    return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const unsigned short*>(p)[i]) << 16);
}
__device__ __forceinline__ float elem_to_float(const float* p, long long i) {
    if (!dbg_ok(p + i, 4, DBG_LOGIT1)) return 0.f;
    return p[i];
}

// kVec elements starting at element e0 of a row; elements at or beyond `hi` read as `pad`.
// ALIGNED: the row is 16-byte aligned, so a full vector is one (bf16) or two (fp32) 16-byte loads.
template <typename T, bool ALIGNED>
__device__ __forceinline__ Raw<T> load_raw(const T* row, int e0, int hi, float pad) {
    if (ALIGNED && e0 + kVec <= hi) {
        Raw<T> r;
        if constexpr (sizeof(T) == 2) {
            r.a = ldg_stream(row + e0);
        } else {
            r.a = ldg_stream(row + e0);
            r.b = ldg_stream(row + e0 + 4);
        }
        return r;
    }
    if (e0 >= hi) return raw_fill<T>(pad);
    float x[kVec];
#pragma unroll
    for (int j = 0; j < kVec; ++j) x[j] = (e0 + j < hi) ? elem_to_float(row, e0 + j) : pad;
    Raw<T> r;
    if constexpr (sizeof(T) == 2) {
        r.a.x = (__float_as_uint(x[0]) >> 16) | (__float_as_uint(x[1]) & 0xFFFF0000u);
        r.a.y = (__float_as_uint(x[2]) >> 16) | (__float_as_uint(x[3]) & 0xFFFF0000u);
        r.a.z = (__float_as_uint(x[4]) >> 16) | (__float_as_uint(x[5]) & 0xFFFF0000u);
        r.a.w = (__float_as_uint(x[6]) >> 16) | (__float_as_uint(x[7]) & 0xFFFF0000u);
    } else {
        r.a = make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
        r.b = make_uint4(__float_as_uint(x[4]), __float_as_uint(x[5]), __float_as_uint(x[6]), __float_as_uint(x[7]));
    }
    return r;
}

// NaN-propagating maximum of the kVec raw elements.
__device__ __forceinline__ float raw_max(const Raw<__nv_bfloat16>& r) {
    __nv_bfloat162 m = __hmax2_nan(__hmax2_nan(as_bf2(r.a.x), as_bf2(r.a.y)),
                                   __hmax2_nan(as_bf2(r.a.z), as_bf2(r.a.w)));
    uint32_t u = as_u32(m);
    return max_nan(bf_lo(u), bf_hi(u));
}
__device__ __forceinline__ float raw_max(const Raw<float>& r) {
    float a = max_nan(max_nan(__uint_as_float(r.a.x), __uint_as_float(r.a.y)),
                      max_nan(__uint_as_float(r.a.z), __uint_as_float(r.a.w)));
    float b = max_nan(max_nan(__uint_as_float(r.b.x), __uint_as_float(r.b.y)),
                      max_nan(__uint_as_float(r.b.z), __uint_as_float(r.b.w)));
    return max_nan(a, b);
}

// Does any raw element exceed `m` (or is any NaN)?  `STRICT`: exceed means >, else >=.
// For bf16 the test runs on packed pairs; `m` must be bf16-representable.
template <bool STRICT>
__device__ __forceinline__ bool raw_exceeds(const Raw<__nv_bfloat16>& r, float m) {
    __nv_bfloat162 mx = __hmax2_nan(__hmax2_nan(as_bf2(r.a.x), as_bf2(r.a.y)),
                                    __hmax2_nan(as_bf2(r.a.z), as_bf2(r.a.w)));
    uint32_t mb = __float_as_uint(m) >> 16;
    __nv_bfloat162 m2 = as_bf2(mb | (mb << 16));
    return STRICT ? !__hble2(mx, m2) : !__hblt2(mx, m2);
}
template <bool STRICT>
__device__ __forceinline__ bool raw_exceeds(const Raw<float>& r, float m) {
    float mx = raw_max(r);
    return STRICT ? !(mx <= m) : !(mx < m);
}

// Clamp the raw elements from below at kFloor (NaN becomes kFloor as well).
__device__ __forceinline__ void raw_floor(Raw<__nv_bfloat16>& r) {
    const __nv_bfloat162 f = as_bf2(kFloorBf16x2);
    r.a.x = as_u32(__hmax2(as_bf2(r.a.x), f));
    r.a.y = as_u32(__hmax2(as_bf2(r.a.y), f));
    r.a.z = as_u32(__hmax2(as_bf2(r.a.z), f));
    r.a.w = as_u32(__hmax2(as_bf2(r.a.w), f));
}
__device__ __forceinline__ void raw_floor(Raw<float>& r) {
    r.a.x = __float_as_uint(fmaxf(__uint_as_float(r.a.x), kFloor));
    r.a.y = __float_as_uint(fmaxf(__uint_as_float(r.a.y), kFloor));
    r.a.z = __float_as_uint(fmaxf(__uint_as_float(r.a.z), kFloor));
    r.a.w = __float_as_uint(fmaxf(__uint_as_float(r.a.w), kFloor));
    r.b.x = __float_as_uint(fmaxf(__uint_as_float(r.b.x), kFloor));
    r.b.y = __float_as_uint(fmaxf(__uint_as_float(r.b.y), kFloor));
    r.b.z = __float_as_uint(fmaxf(__uint_as_float(r.b.z), kFloor));
    r.b.w = __float_as_uint(fmaxf(__uint_as_float(r.b.w), kFloor));
}

// ----------------------------------------------------------------------------------------
// Per-thread sweep states.  All three share the shape (a, b, c, d) of a float4 partial.
//
// DRAFT   a = m (running max, logit units), b = cnt (elements equal to m that are kept out of
//         the sum so that a dominant token never absorbs the tail), c = Zx = sum over the other
//         elements of 2^((x-m)*scale), d = S = sum of 2^((x-m)*scale) * (x-m).
//         Z = cnt + Zx; entropy (nats) = ln Z - ln2*scale*S/Z; confidence = 1/Z  (Sec. 4.2).
//         cnt = NaN marks a NaN / +inf input.
// TARGET  a = r (reference, log2 units = m*scale), b = Z = sum 2^(x*scale - r); c,d unused.
//         NaN / +inf inputs surface as a non-finite Z.
// ARGMAX  a = best value, b = index (bit pattern), c = bad flag (non-zero: NaN / +inf seen).
// ----------------------------------------------------------------------------------------
struct DraftState {
    float m, cnt;
    f2 za, zb, sa, sb;  // four running sums each of Zx and S, as two packed pairs
    bool bad;
    __device__ __forceinline__ void init(float m0) {
        m = m0; cnt = 0.f; bad = false;
        za = zb = sa = sb = pack2(0.f, 0.f);
    }
    __device__ __forceinline__ float zsum() const { return hsum2(za) + hsum2(zb); }
    __device__ __forceinline__ float ssum() const { return hsum2(sa) + hsum2(sb); }

    template <typename T>
    __device__ __forceinline__ void slow(const Raw<T>& raw, float scale) {
        float x[kVec];
        unpack<T>(raw, x);
        float vmax = kFloor;
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            bad |= (x[j] != x[j]) || (x[j] == __int_as_float(0x7f800000));
            x[j] = fmaxf(x[j], kFloor);
            vmax = fmaxf(vmax, x[j]);
        }
        float z = zsum(), sv = ssum();
        if (vmax > m) {  // everything gathered so far moves below the new maximum
            float dm = m - vmax;
            float f = ex2f(dm * scale);
            float zall = cnt + z;
            z = zall * f;
            sv = fmaf(dm, zall, sv) * f;
            cnt = 0.f;
            m = vmax;
        }
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            if (x[j] == m) {
                cnt += 1.f;
            } else {
                float dx = x[j] - m;
                float e = ex2f(dx * scale);
                z += e;
                sv = fmaf(e, dx, sv);
            }
        }
        za = pack2(z, 0.f); zb = pack2(0.f, 0.f);
        sa = pack2(sv, 0.f); sb = pack2(0.f, 0.f);
    }

    template <typename T>
    __device__ __forceinline__ void step(Raw<T> raw, float scale) {
        if (raw_exceeds<false>(raw, m)) {  // an element >= m, or a NaN: rare after the warm start
            slow<T>(raw, scale);
            return;
        }
        raw_floor(raw);
        f2 x[4];
        unpack_pairs(raw, x);
        const f2 m2 = pack2(m, m), sc2 = pack2(scale, scale);
        const f2 d0 = sub2(x[0], m2), d1 = sub2(x[1], m2), d2 = sub2(x[2], m2), d3 = sub2(x[3], m2);
        const f2 e0 = ex2_2(mul2(d0, sc2)), e1 = ex2_2(mul2(d1, sc2));
        const f2 e2 = ex2_2(mul2(d2, sc2)), e3 = ex2_2(mul2(d3, sc2));
        za = add2(za, e0); zb = add2(zb, e1);
        sa = fma2(e0, d0, sa); sb = fma2(e1, d1, sb);
        za = add2(za, e2); zb = add2(zb, e3);
        sa = fma2(e2, d2, sa); sb = fma2(e3, d3, sb);
    }
    __device__ __forceinline__ float4 partial() const {
        return make_float4(m, bad ? __int_as_float(0x7fc00000) : cnt, zsum(), ssum());
    }
};

// (m, cnt, Zx, S) merge; `scale` converts logit units to log2 units.
__device__ __forceinline__ float4 merge_draft(float4 a, float4 b, float scale) {
    float m = fmaxf(a.x, b.x);
    float da = a.x - m, db = b.x - m;
    float fa = ex2f(da * scale), fb = ex2f(db * scale);
    float za = a.y + a.z, zb = b.y + b.z;
    float4 r;
    r.x = m;
    r.y = (a.x == m ? a.y : 0.f) + (b.x == m ? b.y : 0.f);
    r.z = (a.x == m ? a.z : za * fa) + (b.x == m ? b.z : zb * fb);
    r.w = (a.x == m ? a.w : fmaf(da, za, a.w) * fa) + (b.x == m ? b.w : fmaf(db, zb, b.w) * fb);
    // a NaN count must survive even when its side is scaled away
    if (a.y != a.y || b.y != b.y) r.y = __int_as_float(0x7fc00000);
    return r;
}

struct TargetState {
    float m, r;
    f2 za, zb;
    __device__ __forceinline__ void init(float m0, float scale) {
        m = m0; r = m0 * scale;
        za = zb = pack2(0.f, 0.f);
    }
    template <typename T>
    __device__ __forceinline__ void step(const Raw<T>& raw, float scale) {
        if (raw_exceeds<true>(raw, m)) {  // a new maximum (or NaN): move the reference
            float vmax = raw_max(raw);
            if (vmax == vmax) {  // NaN needs no rescale; it poisons Z below
                float rn = vmax * scale;
                float f = ex2f(r - rn);
                za = pack2((hsum2(za) + hsum2(zb)) * f, 0.f);
                zb = pack2(0.f, 0.f);
                r = rn; m = vmax;
            }
        }
        f2 x[4];
        unpack_pairs(raw, x);
        const f2 sc2 = pack2(scale, scale), nr2 = pack2(-r, -r);
        const f2 e0 = ex2_2(fma2(x[0], sc2, nr2)), e1 = ex2_2(fma2(x[1], sc2, nr2));
        const f2 e2 = ex2_2(fma2(x[2], sc2, nr2)), e3 = ex2_2(fma2(x[3], sc2, nr2));
        za = add2(za, e0); zb = add2(zb, e1);
        za = add2(za, e2); zb = add2(zb, e3);
    }
    __device__ __forceinline__ float4 partial() const {
        return make_float4(r, hsum2(za) + hsum2(zb), 0.f, 0.f);
    }
};

__device__ __forceinline__ float4 merge_target(float4 a, float4 b) {
    float r = fmaxf(a.x, b.x);
    float4 o;
    o.x = r;
    o.y = a.y * ex2f(a.x - r) + b.y * ex2f(b.x - r);
    if (a.y != a.y || b.y != b.y) o.y = __int_as_float(0x7fc00000);
    o.z = o.w = 0.f;
    return o;
}

struct ArgmaxState {
    float best; int idx; bool bad;
    __device__ __forceinline__ void init(float m0) { best = m0; idx = 0x7fffffff; bad = false; }
    template <typename T>
    __device__ __forceinline__ void step(const Raw<T>& raw, int e0) {
        if (!raw_exceeds<false>(raw, best)) return;
        float x[kVec];
        unpack<T>(raw, x);
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
            bad |= (x[j] != x[j]) || (x[j] == __int_as_float(0x7f800000));
            if (x[j] > best || (x[j] == best && e0 + j < idx)) { best = x[j]; idx = e0 + j; }
        }
    }
    __device__ __forceinline__ float4 partial() const {
        return make_float4(best, __int_as_float(idx), bad ? 1.f : 0.f, 0.f);
    }
};

__device__ __forceinline__ float4 merge_argmax(float4 a, float4 b) {
    int ia = __float_as_int(a.y), ib = __float_as_int(b.y);
    bool take_b = (b.x > a.x) || (b.x == a.x && ib < ia);
    float4 o = take_b ? b : a;
    o.z = a.z + b.z;
    return o;
}

template <int PATH>
__device__ __forceinline__ float4 merge_any(float4 a, float4 b, float scale) {
    if constexpr (PATH == PATH_DRAFT) return merge_draft(a, b, scale);
    else if constexpr (PATH == PATH_TARGET) return merge_target(a, b);
    else return merge_argmax(a, b);
}

__device__ __forceinline__ float4 shfl_xor4(float4 v, int mask) {
    v.x = __shfl_xor_sync(0xffffffffu, v.x, mask);
    v.y = __shfl_xor_sync(0xffffffffu, v.y, mask);
    v.z = __shfl_xor_sync(0xffffffffu, v.z, mask);
    v.w = __shfl_xor_sync(0xffffffffu, v.w, mask);
    return v;
}

// ----------------------------------------------------------------------------------------
// Warp-level merge of the 32 per-thread partials (result valid in every lane).
// DRAFT / TARGET: bring every lane to the warp-wide reference, then plain sums.
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sumf(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_maxf(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <int PATH>
__device__ __forceinline__ float4 warp_merge(float4 p, float scale) {
    if constexpr (PATH == PATH_DRAFT) {
        const float M = warp_maxf(p.x);
        if (p.x != M) {  // this lane's maximum is not the warp's: its count joins the scaled sum
            const float dm = p.x - M, f = ex2f(dm * scale), za = p.y + p.z;
            p.w = fmaf(dm, za, p.w) * f;
            p.z = za * f;
            p.y = 0.f;
        }
        return make_float4(M, warp_sumf(p.y), warp_sumf(p.z), warp_sumf(p.w));
    } else if constexpr (PATH == PATH_TARGET) {
        const float R = warp_maxf(p.x);
        return make_float4(R, warp_sumf(p.y * ex2f(p.x - R)), 0.f, 0.f);
    } else {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) p = merge_argmax(p, shfl_xor4(p, o));
        return p;
    }
}

template <typename T>
__device__ __forceinline__ Raw<T> ld_vec(const T* p) {
    Raw<T> r;
    if constexpr (sizeof(T) == 2) {
        r.a = ldg_stream(p);
    } else {
        r.a = ldg_stream(p);
        r.b = ldg_stream(p + 4);
    }
    return r;
}

// ----------------------------------------------------------------------------------------
// One WARP sweeps elements [lo, hi) of one logit row and returns the merged partial in every
// lane.  Lane l owns vectors l, l+32, ... of the range; U of them are in flight.  Warps of a
// CTA never wait for one another.
// ----------------------------------------------------------------------------------------
// CTA_WARM: the warps of the CTA sweep slices of the same row and share their warm starts (one
// barrier, every warp of the CTA must call); false: the warp is on its own row.
template <typename T, bool ALIGNED, int PATH, int U, int STEP, bool CTA_WARM = true>
__device__ __forceinline__ float4 sweep_warp(const T* __restrict__ row, int lo, int hi, int first, float scale,
                                             volatile float* sh_m0) {
    // this thread owns vectors first, first+STEP, ... of the range [lo, hi)
    const float pad = (PATH == PATH_DRAFT) ? kFloor : __int_as_float(0xff800000);
    constexpr int kStride = STEP * kVec;                    // elements between a thread's vectors
    const int nv = (hi > lo) ? (hi - lo + kVec - 1) / kVec : 0;  // vectors in the range (last may be ragged)
    const int my_n = (nv > first) ? (nv - first + STEP - 1) / STEP : 0;
    // vectors this thread takes through the unguarded 16-byte path
    int n_main = my_n;
    if (!ALIGNED) n_main = 0;
    else if (my_n > 0 && lo + (first + (my_n - 1) * STEP) * kVec + kVec > hi) n_main = my_n - 1;
    const T* p = row + lo + first * kVec;

    Raw<T> buf[U];
#pragma unroll
    for (int k = 0; k < U; ++k) buf[k] = (k < n_main) ? ld_vec<T>(p + k * kStride) : raw_fill<T>(pad);

    // warm start: the warp-wide maximum of the first U vectors of every lane.  A vector holding
    // NaN / +inf / only -inf contributes the floor; its owner meets the offending element again
    // in its own state and flags it there.
    float m0 = kFloor;
#pragma unroll
    for (int k = 0; k < U; ++k) {
        float v = raw_max(buf[k]);
        if (v >= kFloor && v < __int_as_float(0x7f800000)) m0 = fmaxf(m0, v);
    }
    if (n_main == 0 && my_n > 0) {
        float v = raw_max(load_raw<T, false>(row, lo + first * kVec, hi, pad));
        if (v >= kFloor && v < __int_as_float(0x7f800000)) m0 = fmaxf(m0, v);
    }
    m0 = warp_maxf(m0);
    // share the warm start across the CTA's warps (one barrier per CTA, before the streaming loop)
    if (CTA_WARM) {
        if ((threadIdx.x & 31) == 0) sh_m0[threadIdx.x >> 5] = m0;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kWarps; ++w) m0 = fmaxf(m0, sh_m0[w]);
    }

    DraftState ds; TargetState ts; ArgmaxState as;
    if constexpr (PATH == PATH_DRAFT) ds.init(m0);
    else if constexpr (PATH == PATH_TARGET) ts.init(m0, scale);
    else as.init(m0);

    auto process = [&](const Raw<T>& v, int idx) {
        if constexpr (PATH == PATH_DRAFT) ds.template step<T>(v, scale);
        else if constexpr (PATH == PATH_TARGET) ts.template step<T>(v, scale);
        else as.template step<T>(v, lo + (first + idx * STEP) * kVec);
    };

    int i = 0;
    for (; i + U <= n_main; i += U) {
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const Raw<T> cur = buf[k];
            const int nx = i + U + k;
            if (nx < n_main) buf[k] = ld_vec<T>(p + nx * kStride);
            process(cur, i + k);
        }
    }
#pragma unroll
    for (int k = 0; k < U; ++k)
        if (i + k < n_main) process(buf[k], i + k);
    // vectors that need the guarded element-wise load: a ragged last vector, or every vector
    // of a row that is not 16-byte aligned
    for (int j = n_main; j < my_n; ++j)
        process(load_raw<T, false>(row, lo + (first + j * STEP) * kVec, hi, pad), j);

    float4 part;
    if constexpr (PATH == PATH_DRAFT) part = ds.partial();
    else if constexpr (PATH == PATH_TARGET) part = ts.partial();
    else part = as.partial();
    return warp_merge<PATH>(part, scale);
}

// ----------------------------------------------------------------------------------------
// Row epilogue helpers (one warp, double precision; a few dozen values per row)
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float4 ldcg4(const float4* p) {
    if (!dbg_ok(p, 16, DBG_WS_LOAD)) return make_float4(0.f, 0.f, 0.f, 0.f);
    return __ldcg(p);
}
// a store into the workspace (or a caller's state array) at an index that was computed
#define SPECKV_ST(lvalue, value) do { if (dbg_ok(&(lvalue), sizeof(lvalue), DBG_WS_STORE)) (lvalue) = (value); } while (0)

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_min(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmin(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Controller (Sec. 4.3, Eq. 1) for one row, executed by a full warp.  The parameters are fetched
// first, all at once (ctl_load), so that their memory latency overlaps whatever comes between
// the load and the evaluation.  Lane k holds hidden unit k's weights, b2[k] and comp[k].
struct CtlRegs {
    float w1[8], w2[8];
    float b1, b2k, compk;
};
__device__ __forceinline__ CtlRegs ctl_load(const KParams& P, int b, int lane) {
    CtlRegs c;
    const bool hid = lane < P.n_hidden;
#pragma unroll
    for (int f = 0; f < 8; ++f) c.w1[f] = (hid && f < P.n_in) ? __ldg(P.W1 + lane * P.n_in + f) : 0.f;
    if (P.layout == 2) {
        // the paper's f(x, gamma): one output head; without hidden units W2 weighs the inputs directly
#pragma unroll
        for (int j = 1; j < 8; ++j) c.w2[j] = 0.f;
        c.w2[0] = (P.n_hidden > 0 ? hid : lane < P.n_in) ? __ldg(P.W2 + lane) : 0.f;
        c.b2k = lane == 0 ? __ldg(P.b2) : 0.f;
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) c.w2[j] = (hid && j < P.n_out) ? __ldg(P.W2 + j * P.n_hidden + lane) : 0.f;
        c.b2k = lane < P.n_out ? __ldg(P.b2 + lane) : 0.f;
    }
    c.b1 = hid ? __ldg(P.b1 + lane) : 0.f;
    c.compk = (P.comp && lane < P.n_comp) ? __ldg(P.comp + static_cast<long long>(b) * P.n_comp + lane) : 0.f;
    return c;
}
// f4 = Hbar, cbar, Hmax, cmin.  fp32 throughout: 164 multiply-adds on values of order one.
__device__ __forceinline__ void ctl_eval(const KParams& P, const CtlRegs& c, const float (&f4)[4],
                                         float* scores_row, int* gamma_next) {
    const int lane = threadIdx.x & 31;
    if (P.layout == 2) {
        // Sec. 4.3 as printed: a_hat = f([Hbar, cbar, Hmax, cmin, comp.., gamma_j]) for every candidate
        float x[8];
        x[0] = f4[0]; x[1] = f4[1]; x[2] = f4[2]; x[3] = f4[3];
#pragma unroll
        for (int k = 4; k < 8; ++k) {
            const float cv = __shfl_sync(0xffffffffu, c.compk, k - 4);
            x[k] = (k < P.n_in - 1) ? cv : 0.f;
        }
        float base = c.b1, wg = 0.f, xl = 0.f;  // hidden pre-activation without gamma; gamma's weight; x[lane]
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            if (f < P.n_in - 1) base = fmaf(c.w1[f], x[f], base);
            if (f == P.n_in - 1) wg = c.w1[f];
            if (f == lane) xl = x[f];
        }
        const float b2 = __shfl_sync(0xffffffffu, c.b2k, 0);
        float best = 0.f;
        int best_j = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (j < P.n_out) {  // uniform across the warp
                const float g = static_cast<float>(P.gch[j]);
                float term;
                if (P.n_hidden > 0) {
                    const float h = fmaf(wg, g, base);
                    term = (lane < P.n_hidden && h > 0.f) ? c.w2[0] * h : 0.f;
                } else {
                    term = lane < P.n_in - 1 ? c.w2[0] * xl : (lane == P.n_in - 1 ? c.w2[0] * g : 0.f);
                }
                const float a_hat = warp_sumf(term) + b2;
                const float e = (P.transform == 0) ? fmaf(a_hat, g, 1.f) : a_hat;
                if (scores_row && lane == 0) scores_row[j] = e;
                if (j == 0 || e > best) { best = e; best_j = j; }
            }
        }
        if (gamma_next && lane == 0) *gamma_next = P.gch[best_j];
        return;
    }
    float x[8];
    const int first_comp = (P.layout == 0) ? 3 : 4;
    if (P.layout == 0) { x[0] = f4[0]; x[1] = f4[1]; x[2] = f4[3]; x[3] = 0.f; }
    else { x[0] = f4[0]; x[1] = f4[1]; x[2] = f4[2]; x[3] = f4[3]; }
#pragma unroll
    for (int k = 3; k < 8; ++k) {
        const float cv = __shfl_sync(0xffffffffu, c.compk, (k - first_comp) & 31);
        if (k >= first_comp) x[k] = (k < P.n_in) ? cv : 0.f;
    }
    float h = c.b1;
#pragma unroll
    for (int f = 0; f < 8; ++f)
        if (f < P.n_in) h = fmaf(c.w1[f], x[f], h);
    h = (lane < P.n_hidden && h > 0.f) ? h : 0.f;
    float best = 0.f;
    int best_j = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float b2 = __shfl_sync(0xffffffffu, c.b2k, j);
        if (j < P.n_out) {  // uniform across the warp
            const float o = warp_sumf(c.w2[j] * h) + b2;
            const float e = (P.transform == 0) ? fmaf(o, static_cast<float>(P.gch[j]), 1.f) : o;
            if (scores_row && lane == 0) scores_row[j] = e;
            if (j == 0 || e > best) { best = e; best_j = j; }
        }
    }
    if (gamma_next && lane == 0) *gamma_next = P.gch[best_j];
}

// log2 of a positive finite number in double: it enters the normalisers of p and q, and the residual
// max(0, p - q) sees the difference of their errors magnified by 1 / (its own mass); a few dozen calls
// per batch row, so the cost does not show
__device__ __forceinline__ double log2_split(double z) { return log2(z); }

// End of a row epilogue (whole warp): everything the warp wrote for batch row b becomes visible
// before the row's completion flag does.  The resample kernel polls the flag instead of waiting for
// the whole sweep grid, so it can work on finished rows while the sweep's last CTAs drain.
constexpr int kRowDoneTimeout = 1 << 30;  // a resample CTA gave up waiting for this row
__device__ __forceinline__ void row_done_signal(const KParams& P, int b, int mode, int n) {
    if (!P.rdone) return;
    __threadfence();
    __syncwarp();
    // the flag carries what a resample CTA needs to start fetching logits: draw mode and stop position
    const int v = 1 | (mode << 8) | (n << 16);
    if ((threadIdx.x & 31) == 0) {
        const int old = atomicOr(P.rdone + b, v);
        // a resample CTA whose bounded wait ran out before this point left its mark here: the row's fresh
        // token will never be drawn, and the status written above must say so
        if ((old & kRowDoneTimeout) && P.status) atomicOr(P.status + b, 16);
    }
}

// Bounded wait for a row's completion flag (one thread polls).  The flag's value, 0 when the bound ran out.
__device__ __forceinline__ int row_done_wait(const int* flag, int limit) {
    for (int it = 0; it < limit; ++it) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
        if (v & 1) return v;
        __nanosleep(it < 64 ? 100 : 1000);
    }
    return 0;
}

// What one lane of a row's epilogue learns about its position (lane i: draft position i, target position i).
struct RowDecide {
    int x;            // draft token (-1 where the lane has none)
    float u_res;      // second uniform of the position
    float Hi, ci;     // entropy (nats) and confidence of the draft distribution
    double lse2_q, lse2_p;  // log2-normalisers of draft and target
    int amax;         // greedy rows: argmax of the target row
    bool dbad, tbad;  // non-finite draft row / target row at this position
    bool badtok, accept, any_dbad;
};

// The per-position part of the row epilogue: lane i < n_lanes merges the nd partials at pd (draft position
// i) and the nt partials at pt (target position i) and takes the acceptance test of its position.  One
// compiled body serves the row epilogue and the prefix epilogue below, so that both reach the same bits.
template <typename T>
__device__ __noinline__ void row_decide(const KParams& P, int b, int gam, float Tf, int status, int n_lanes,
                                        const float4* pd, int nd, const float4* pt, int nt, RowDecide& o) {
    const int lane = threadIdx.x & 31;
    const int G = P.G;
    const bool verify = (P.mode & MODE_VERIFY) != 0;
    constexpr int kPre = 4;  // partials fetched ahead per lane; more are rare
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    const double sd = static_cast<double>(scale);
    const bool in = lane < n_lanes;
    const bool dr_on = in && !status && lane < gam;
    const bool tg_on = in && !status && verify && lane <= gam;
    const bool tok_on = in && !status && verify && lane < gam;

    // ---- first round trip ----
    const long long ps = P.part_stride > 0 ? P.part_stride : 1;  // partials of a logit row: adjacent, or one per shard
    float4 qd[kPre], qt[kPre];
#pragma unroll
    for (int k = 0; k < kPre; ++k) {
        qd[k] = (dr_on && k < nd) ? ldcg4(pd + k * ps) : make_float4(0.f, 0.f, 0.f, 0.f);
        qt[k] = (tg_on && k < nt) ? ldcg4(pt + k * ps) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const long long urow = (static_cast<long long>(b) * (G + 1) + lane) * 2;
    const int x = tok_on ? __ldg(P.tok + static_cast<long long>(b) * G + lane) : -1;
    const float u_acc = tok_on ? __ldg(P.u + urow) : 0.f;
    const float u_res = tg_on ? __ldg(P.u + urow + 1) : 0.f;
    // the two logits at the draft token: left by the sweep CTA of the draft position when the sweep
    // does that (same round trip), else fetched below (a second one)
    float2 tl = make_float2(0.f, 0.f);
    if (P.tokl && tok_on && !greedy) {
        long long at = static_cast<long long>(b) * G + lane;
        if (P.shard_width > 0)  // the table of the shard whose slice holds the token (one more dependent load)
            at += (x > 0 ? min(x / P.shard_width, P.n_shards - 1) : 0) * P.tokl_stride;
        tl = __ldcg(P.tokl + at);
    }

    const bool badtok = tok_on && (x < 0 || x >= P.V);
    float dxf = tl.x, txf = tl.y;
    if (!P.tokl && tok_on && !badtok && !greedy) {
        const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb;
        const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb;
        dxf = elem_to_float(drow + static_cast<long long>(lane) * P.dsp, x);
        txf = elem_to_float(trow + static_cast<long long>(lane) * P.tsp, x);
    }

    float Hi = 0.f, ci = 0.f;
    double lse2_q = 0.0, lse2_p = 0.0;
    int amax = -1;
    bool dbad = false, tbad = false, accept = true;  // non-finite draft row / target row at this lane's position
    bool any_dbad = false;

    if (!status) {
        // Partials are merged in fp32 with the same branch-free rules the sweep uses; the draft and
        // the target chain are independent, so their instructions interleave.  Only what decides an
        // acceptance (the log2-normalisers and the test itself) is carried in double.
        float4 ad = qd[0], at = qt[0];
#pragma unroll
        for (int k = 1; k < kPre; ++k) {
            if (k < nd) ad = merge_draft(ad, qd[k], scale);
            if (k < nt) at = greedy ? merge_argmax(at, qt[k]) : merge_target(at, qt[k]);
        }
        // (only lanes that have a position: the partials of the others would lie outside the array)
        if (dr_on)
            for (int k = kPre; k < nd; ++k) ad = merge_draft(ad, ldcg4(pd + k * ps), scale);
        if (tg_on)
            for (int k = kPre; k < nt; ++k) at = greedy ? merge_argmax(at, ldcg4(pt + k * ps)) : merge_target(at, ldcg4(pt + k * ps));
        if (dr_on) {
            const float m = ad.x, cnt = ad.y, Zx = ad.z, S = ad.w;
            const float Z = cnt + Zx;
            if (!(cnt >= 1.f) || !(Z < 3e38f) || !(m > kFloor)) {
                dbad = true;
            } else {
                const float lnZ = (cnt == 1.f) ? log1pf(Zx) : logf(cnt) + log1pf(Zx / cnt);
                const float rZ = 1.f / Z;
                Hi = fmaxf(lnZ - static_cast<float>(kLn2) * scale * S * rZ, 0.f);
                ci = rZ;
                lse2_q = static_cast<double>(m) * sd + log2_split(static_cast<double>(cnt) + static_cast<double>(Zx));
            }
        }
        if (tg_on) {
            if (greedy) {
                const int bi = __float_as_int(at.y);
                if (at.z != 0.f || bi == 0x7fffffff || !(at.x > kFloor)) tbad = true;
                amax = bi;
            } else {
                if (!(at.y > 0.f) || !(at.y < 3e38f)) tbad = true;
                else lse2_p = static_cast<double>(at.x) + log2_split(static_cast<double>(at.y));
            }
        }
        any_dbad = __any_sync(0xffffffffu, dbad);
    }

    if (status == 0 && !any_dbad && tok_on && !badtok && !tbad) {
        if (greedy) {
            accept = (x == amax);
        } else {
            const double lq = static_cast<double>(dxf) * sd - lse2_q;
            const double lp = static_cast<double>(txf) * sd - lse2_p;
            // u * q(x) < p(x); u = 0 gives -inf on the left
            const double l2u = (u_acc > 0.f) ? log2_split(static_cast<double>(u_acc)) : -__longlong_as_double(0x7ff0000000000000LL);
            accept = (l2u + lq) < lp;
        }
    }
    o.x = x; o.u_res = u_res; o.Hi = Hi; o.ci = ci; o.lse2_q = lse2_q; o.lse2_p = lse2_p; o.amax = amax;
    o.dbad = dbad; o.tbad = tbad; o.badtok = badtok; o.accept = accept; o.any_dbad = any_dbad;
}

// Prefix epilogue (one warp): run when the partials of a batch row's first positions 0..k are in, while
// the rest of the row is still being swept.  It takes the acceptance tests of those positions and
// publishes where the walk stops if it stops there, so that CTAs which have not started yet can leave
// target rows behind that position unread.  early[b] = stop position + 1, or G + 2 when the walk passes k.
template <typename T>
__device__ __noinline__ void prefix_epilogue(const KParams& P, int b, int gam, float Tf) {
    const int lane = threadIdx.x & 31;
    const long long row0 = static_cast<long long>(b) * P.J;
    RowDecide d;
    row_decide<T>(P, b, gam, Tf, 0, P.k_early + 1, P.part + (row0 + P.G + 1 + lane) * P.nsplit, P.nsplit,
                  P.part + (row0 + lane) * P.nsplit, P.nsplit, d);
    const bool in = lane <= P.k_early && lane <= gam;
    const unsigned stop = __ballot_sync(0xffffffffu, in && (d.tbad || d.dbad || (lane < gam && (d.badtok || !d.accept))));
    if (lane == 0) {
        const int e = stop ? __ffs(stop) : P.G + 2;
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(P.early + b), "r"(e) : "memory");
    }
}

// Row epilogue: one warp, run by whoever learns that all partials of batch row b are in.  Lane i
// merges the nd partials at pd (draft position i) and the nt partials at pt (target position i).
// gam and Tf are the row's gamma and temperature as the sweep read them.  Everything the row
// needs from memory that does not depend on other loads is requested first, so the epilogue
// costs one memory round trip (two when the sweep did not leave the logits at the draft tokens).
// Order: what the resample kernel needs (acceptance, stop position, normalisers), the row's
// completion flag, then the signals and the controller.
template <typename T>
__device__ __noinline__ void row_epilogue(const KParams& P, int b, int gam, float Tf, const float4* pd, int nd,
                                          const float4* pt, int nt) {
    const int lane = threadIdx.x & 31;
    const int G = P.G;
    const bool verify = (P.mode & MODE_VERIFY) != 0;

    int status = 0;
    if (gam < 1 || gam > G) status |= 1;
    if (!(Tf >= 0.f) || Tf == __int_as_float(0x7f800000)) status |= 8;
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    const bool tg_on = !status && verify && lane <= gam;

    CtlRegs ctl;
    if ((P.mode & MODE_MLP) && !status) ctl = ctl_load(P, b, lane);
    RowDecide dec;
    row_decide<T>(P, b, gam, Tf, status, 32, pd, nd, pt, nt, dec);
    const int x = dec.x;
    const float u_res = dec.u_res, Hi = dec.Hi, ci = dec.ci;
    const double lse2_q = dec.lse2_q, lse2_p = dec.lse2_p;
    const int amax = dec.amax;
    const bool tbad = dec.tbad, badtok = dec.badtok, accept = dec.accept, any_dbad = dec.any_dbad;

    // The positions are walked in order; the walk ends at the first one whose target row is non-finite
    // (which flags the row), whose draft token is out of range, or whose token is rejected.  Target rows
    // behind that position are not part of the step (Sec. 3.1 discards what follows the first mismatch):
    // whatever they hold flags nothing.  A non-finite draft row flags the row wherever it is.
    const unsigned stop = __ballot_sync(0xffffffffu, tg_on && (tbad || (lane < gam && (badtok || !accept))));
    const int first = stop ? (__ffs(stop) - 1) : gam;
    const bool tbad_first = __shfl_sync(0xffffffffu, tbad ? 1 : 0, first & 31) != 0;
    if (status == 0) {
        if (any_dbad || (verify && tbad_first)) status |= 4;
        if (__any_sync(0xffffffffu, badtok)) status |= 2;
    }
    const int n = (status == 0 && verify) ? first : 0;

    const int rs_mode = (verify && status == 0 && !greedy) ? (n < gam ? RS_RESIDUAL : RS_BONUS) : RS_NONE;
    if (verify) {
        // fresh token: known here for greedy rows, drawn by the resample step otherwise
        const int amax_n = __shfl_sync(0xffffffffu, amax, n);
        const double lp_n = __shfl_sync(0xffffffffu, lse2_p, n);
        const double lq_n = __shfl_sync(0xffffffffu, lse2_q, n < gam ? n : 0);
        const float u2_n = __shfl_sync(0xffffffffu, u_res, n);
        if (lane <= G) {
            int v = -1;
            if (status == 0) {
                if (lane < n) v = x;
                else if (lane == n && greedy) v = amax_n;
            }
            P.out_tok[static_cast<long long>(b) * (G + 1) + lane] = v;
        }
        if (lane == 0) {
            P.n_acc[b] = n;
            RowInfo ri;
            ri.mode = rs_mode;
            ri.n = n;
            ri.u2 = (status == 0 && !greedy) ? u2_n : 0.f;
            ri.scale = scale;
            ri.lse2_p = lp_n;
            ri.lse2_q = lq_n;
            SPECKV_ST(P.info[b], ri);
        }
    }
    if (P.status && lane == 0) P.status[b] = status;
    row_done_signal(P, b, rs_mode, n);

    // signals
    const float in_bits = P.bits ? static_cast<float>(kLog2e) : 1.f;
    const float Hout = (status == 0 && lane < gam) ? Hi * in_bits : 0.f;
    const float Cout = (status == 0 && lane < gam) ? ci : 0.f;
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
            ctl_eval(P, ctl, f4, P.scores ? P.scores + static_cast<long long>(b) * P.n_out : nullptr,
                     P.gamma_next + b);
        } else {
            if (P.scores && lane < P.n_out) P.scores[static_cast<long long>(b) * P.n_out + lane] = 0.f;
            if (lane == 0) P.gamma_next[b] = 0;
        }
    }
}

// Epilogue of the draft-side sampling sweep (one warp per batch row): lane i merges the partials
// of drafted position i into the row's log2-normaliser (or its argmax for a greedy row) and leaves
// one RowInfo per position for the resample kernel, which then draws from softmax(d_i / T).
__device__ __noinline__ void sample_epilogue(const KParams& P, int b, int gam, float Tf, const float4* pt, int nt) {
    const int lane = threadIdx.x & 31;
    const int G = P.G;
    int status = 0;
    if (gam < 1 || gam > G) status |= 1;
    if (!(Tf >= 0.f) || Tf == __int_as_float(0x7f800000)) status |= 8;
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    const bool on = !status && lane < gam;
    double lse2 = 0.0;
    int amax = -1;
    bool nonfinite = false;
    if (on) {
        float4 at = ldcg4(pt);
        for (int k = 1; k < nt; ++k) at = greedy ? merge_argmax(at, ldcg4(pt + k)) : merge_target(at, ldcg4(pt + k));
        if (greedy) {
            amax = __float_as_int(at.y);
            if (at.z != 0.f || amax == 0x7fffffff || !(at.x > kFloor)) nonfinite = true;
        } else {
            if (!(at.y > 0.f) || !(at.y < 3e38f)) nonfinite = true;
            else lse2 = static_cast<double>(at.x) + log2_split(static_cast<double>(at.y));
        }
    }
    if (__any_sync(0xffffffffu, nonfinite)) status |= 4;
    if (lane < G) {
        const long long r = static_cast<long long>(b) * G + lane;
        const bool ok = (status == 0 && lane < gam);
        RowInfo ri;
        ri.mode = (ok && !greedy) ? RS_BONUS : RS_NONE;
        ri.n = lane;
        ri.u2 = (ok && !greedy) ? __ldg(P.u + r) : 0.f;
        ri.scale = scale;
        ri.lse2_p = lse2;
        ri.lse2_q = 0.0;
        SPECKV_ST(P.info[r], ri);
        P.out_tok[r] = (ok && greedy) ? amax : -1;
    }
    if (P.status && lane == 0) P.status[b] = status;
    row_done_signal(P, b, RS_NONE, 0);  // every position of the row has its own record: the flag only says they are written
}

// Epilogue of a vocabulary shard's sweep (one warp per batch row): lane i merges this shard's nd
// partials of draft position i and nt partials of target position i (the counts may differ from lane
// to lane) and writes the two merged states; the row epilogue proper runs later on the states of all
// shards.  An argmax index becomes a global vocabulary index.
__device__ __noinline__ void export_epilogue(const KParams& P, int b, int gam, float Tf, const float4* pd, int nd,
                                             const float4* pt, int nt) {
    const int lane = threadIdx.x & 31;
    const int G = P.G;
    const bool ok = (gam >= 1 && gam <= G) && (Tf >= 0.f) && (Tf != __int_as_float(0x7f800000));
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    float4* out = P.state + static_cast<long long>(b) * P.J;
    if (lane < G) {
        float4 ad = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ok && lane < gam && nd > 0) {
            ad = ldcg4(pd);
            for (int k = 1; k < nd; ++k) ad = merge_draft(ad, ldcg4(pd + k), scale);
        }
        SPECKV_ST(out[G + 1 + lane], ad);
    }
    if (lane <= G) {
        float4 at = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ok && lane <= gam && nt > 0) {
            at = ldcg4(pt);
            for (int k = 1; k < nt; ++k) at = greedy ? merge_argmax(at, ldcg4(pt + k)) : merge_target(at, ldcg4(pt + k));
            if (greedy) {
                const int idx = __float_as_int(at.y);
                if (idx != 0x7fffffff) at.y = __int_as_float(idx + P.v_begin);
            }
        }
        SPECKV_ST(out[lane], at);
    }
}

// One CTA's share of a batch row's fresh-token draw (defined with the resample kernel below).
template <typename T, bool ALIGNED>
__device__ __forceinline__ void resample_body(const KParams& P, const int bid);
template <typename T, bool ALIGNED>
__device__ __forceinline__ void resample_row(const KParams& P, const int b, const int r, const int mode, const int n,
                                             const int4 lo4, const int4 hi4, const int share, const int Rr, const int cpc);

// ----------------------------------------------------------------------------------------
// Sweep kernel.  CTAs 0 .. n_sweep-1 sweep one slice of one logit row each.  With verification the
// grid may carry B*R more CTAs behind them that do the resample kernel's work in the same launch:
// CTAs start in index order, so these start exactly when the sweep runs out of slices, wait (with
// a bound) for their batch row's completion flag and fill the SMs that the sweep's last CTAs
// leave one by one.  A second launch, even a programmatic dependent one, starts microseconds
// after the last sweep CTA has started and leaves most of the drain unused.
// ----------------------------------------------------------------------------------------
template <typename T, bool ALIGNED, int U>
__global__ void __launch_bounds__(kThreads, kSweepCtasPerSm) sweep_kernel(const __grid_constant__ KParams P) {
    if (static_cast<int>(blockIdx.x) >= P.n_sweep) {
        resample_body<T, ALIGNED>(P, static_cast<int>(blockIdx.x) - P.n_sweep);
        return;
    }
    __shared__ float4 sh_part[kWarps];
    __shared__ int sh_count;
    __shared__ int sh_early;
    __shared__ float sh_m0[kWarps];
    asm volatile("griddepcontrol.launch_dependents;");  // a dependent resample kernel may be scheduled as SMs free up
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool verify = (P.mode & MODE_VERIFY) != 0;
    int b, j, s, gen = 0;
    if (P.early) {
        // generation order: CTAs start in index order, so a later generation starts when the earlier ones
        // are all under way and, for all but the smallest batches, long after the first one has finished
        const int ns = P.nsplit, k1 = P.k_early + 1;
        const int nA = k1 * P.B * 2 * ns, nB = (P.G - k1) * P.B * ns;
        int i = blockIdx.x, p, is_draft;
        if (i < nA) {
            p = i / (2 * P.B * ns); i -= p * (2 * P.B * ns);
            b = i / (2 * ns); i -= b * (2 * ns);
            is_draft = i / ns; s = i - is_draft * ns;
        } else {
            // the later generations go batch row by batch row, so that the rows complete one after another
            gen = (i < nA + nB) ? 1 : 2;
            i -= (gen == 1) ? nA : nA + nB;
            const int per_b = (gen == 1 ? P.G - k1 : P.G + 1 - k1) * ns;
            b = i / per_b; i -= b * per_b;
            p = i / ns; s = i - p * ns;
            p += k1;
            is_draft = (gen == 1);
        }
        j = is_draft ? P.G + 1 + p : p;
    } else {
        const int per_row = P.J * P.nsplit;
        b = blockIdx.x / per_row;
        const int r = blockIdx.x - b * per_row;
        j = r / P.nsplit;
        s = r - j * P.nsplit;
    }
    // the row's gamma and temperature travel together with the one thing a CTA of the last generation has
    // to learn first: one memory round trip before the CTA knows whether it has work
    int gam = P.gamma ? P.gamma[b] : P.G;
    float Tf = P.temp ? P.temp[b] : P.temp_scalar;
    if (threadIdx.x == 0) {
        sh_count = 0;
        // one thread reads what is known of the row's stop position, so that the whole CTA takes one decision
        int e = 0;
        if (gen == 2 && !P.read_all)
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(e) : "l"(P.early + b) : "memory");
        sh_early = e;
    }
    if (threadIdx.x < kWarps) sh_m0[threadIdx.x] = kFloor;
    __syncthreads();  // before any load is issued
    const int rem = j * P.nsplit + s;

    const bool row_ok = (gam >= 1 && gam <= P.G) && (Tf >= 0.f) && (Tf != __int_as_float(0x7f800000));
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));

    // logit row handled by this CTA: with verification, j <= G are target positions and the
    // rest draft positions; signals alone sweep draft positions only
    // (draft-side sampling sweeps the drafted positions with the target statistics: only the
    // normaliser, or the argmax, of each row is needed; P.t then points at the draft logits)
    const bool is_target = P.sample || (verify && j <= P.G);
    const int pos = is_target ? j : (verify ? j - (P.G + 1) : j);
    const bool active = row_ok && ((is_target && !P.sample) ? pos <= gam : pos < gam);
    const long long pidx = (static_cast<long long>(b) * P.J + j) * P.nsplit + s;  // this CTA's partial

    // the walk stopped at a position before this one
    const bool skipped = active && gen == 2 && sh_early != 0 && sh_early <= P.k_early + 1;
    if (skipped) {
        // the row epilogue never looks behind the stop position; the partial only has to be finite
        if (warp != 0) return;
        if (lane == 0)
            SPECKV_ST(P.part[pidx], greedy ? make_float4(kFloor, __int_as_float(0x7fffffff), 0.f, 0.f)
                                           : make_float4(kFloor, 0.f, 0.f, 0.f));
    } else if (active) {
        // the CTA's slice of the row
        const int v0 = s * P.per_split;
        const int v1 = min(P.nvec, v0 + P.per_split);
        // the CTA's threads interleave over the slice: consecutive warps read consecutive 512 bytes
        constexpr int STEP = kThreads;
        const int first = threadIdx.x;
        const int lo = v0 * kVec;
        const int hi = min(P.V, v1 * kVec);
        float4 part;
        int path;
        if (is_target) {
            const T* row = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb +
                           static_cast<long long>(pos) * P.tsp;
            if (greedy) { part = sweep_warp<T, ALIGNED, PATH_ARGMAX, U, STEP>(row, lo, hi, first, scale, sh_m0); path = PATH_ARGMAX; }
            else { part = sweep_warp<T, ALIGNED, PATH_TARGET, U, STEP>(row, lo, hi, first, scale, sh_m0); path = PATH_TARGET; }
        } else {
            const T* row = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb +
                           static_cast<long long>(pos) * P.dsp;
            if (verify && P.tokl && s == 0 && threadIdx.x == 0 && !greedy) {
                // the acceptance test of this position needs both logits at the draft token: fetch them
                // now, while the sweep hides the latency, and leave them for the row epilogue
                const int x = __ldg(P.tok + static_cast<long long>(b) * P.G + pos) - P.v_begin;  // index in this slice
                if (x >= 0 && x < P.V) {
                    const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb +
                                    static_cast<long long>(pos) * P.tsp;
                    SPECKV_ST(P.tokl[static_cast<long long>(b) * P.G + pos], make_float2(elem_to_float(row, x), elem_to_float(trow, x)));
                }
            }
            part = sweep_warp<T, ALIGNED, PATH_DRAFT, U, STEP>(row, lo, hi, first, scale, sh_m0);
            path = PATH_DRAFT;
        }
        // the last warp of the CTA to finish merges the eight warp partials; nobody waits
        int last = 0;
        if (lane == 0) {
            sh_part[warp] = part;
            __threadfence_block();
            last = (atomicAdd(&sh_count, 1) == kWarps - 1);
        }
        if (!__shfl_sync(0xffffffffu, last, 0)) return;
        if (lane == 0) {
            __threadfence_block();
            const volatile float4* vp = sh_part;
            float4 acc = make_float4(vp[0].x, vp[0].y, vp[0].z, vp[0].w);
            for (int w = 1; w < kWarps; ++w) {
                float4 o = make_float4(vp[w].x, vp[w].y, vp[w].z, vp[w].w);
                acc = (path == PATH_DRAFT) ? merge_draft(acc, o, scale)
                    : (path == PATH_TARGET) ? merge_target(acc, o) : merge_argmax(acc, o);
            }
            SPECKV_ST(P.part[pidx], acc);
        }
        if (P.early && gen == 0) {
            // first generation: the last of the row's CTAs of positions 0..k_early takes their acceptance tests
            const int n_pre = (min(P.k_early, gam) + 1 + min(P.k_early + 1, gam)) * P.nsplit;
            int last_pre = 0;
            if (lane == 0) {
                __threadfence();
                last_pre = (atomicAdd(P.tick_early + b, 1) == n_pre - 1);
            }
            if (__shfl_sync(0xffffffffu, last_pre, 0)) {
                __threadfence();
                prefix_epilogue<T>(P, b, gam, Tf);
            }
        }
    } else if (row_ok || rem != 0 || warp != 0) {
        return;  // unused position: nothing to count; a flagged row keeps its first CTA for the epilogue
    }

    // ticket: the last of the row's active CTAs runs the row epilogue; nobody waits
    const int n_rows = P.sample ? gam : (verify ? 2 * gam + 1 : gam);
    const int n_tickets = row_ok ? n_rows * P.nsplit : 1;
    const long long row0 = static_cast<long long>(b) * P.J;
    int last_row = 0;
    if (lane == 0) {
        __threadfence();
        last_row = (atomicAdd(P.tick1 + b, 1) == n_tickets - 1);
    }
    if (!__shfl_sync(0xffffffffu, last_row, 0)) return;
    __threadfence();
    if (P.sample) {
        sample_epilogue(P, b, gam, Tf, P.part + (row0 + lane) * P.nsplit, P.nsplit);
        return;
    }
    if (P.export_state) {
        export_epilogue(P, b, gam, Tf, P.part + (row0 + P.G + 1 + lane) * P.nsplit, P.nsplit,
                           P.part + (row0 + lane) * P.nsplit, P.nsplit);
        return;
    }
    row_epilogue<T>(P, b, gam, Tf, P.part + (row0 + (verify ? P.G + 1 + lane : lane)) * P.nsplit, P.nsplit,
                    P.part + (row0 + lane) * P.nsplit, P.nsplit);
}

// ----------------------------------------------------------------------------------------
// Resample kernel: inverse CDF over the stop position's weights, vocabulary order.
//   residual: w_v = max(0, p_v - q_v);   bonus: w_v = p_v
// p_v and q_v are evaluated with fp32 exp2 against normalisers carried as two floats; the chunk
// sums are fp32, everything above a chunk is summed in double.  A residual whose total mass is
// below 1e-6 cannot be told from rounding noise and is treated as empty (p == q at the stop
// position): the token is then drawn from p.
// ----------------------------------------------------------------------------------------
struct RsConst {
    int mode;
    float scale, lp_hi, lp_lo, lq_hi, lq_lo;
};

__device__ __forceinline__ RsConst rs_const(const RowInfo& ri, int mode) {
    RsConst c;
    c.mode = mode;
    c.scale = ri.scale;
    // log2-normalisers split into two floats so that the exponent argument keeps the bits a
    // single float would drop
    c.lp_hi = static_cast<float>(ri.lse2_p);
    c.lp_lo = static_cast<float>(ri.lse2_p - static_cast<double>(c.lp_hi));
    c.lq_hi = static_cast<float>(ri.lse2_q);
    c.lq_lo = static_cast<float>(ri.lse2_q - static_cast<double>(c.lq_hi));
    return c;
}

// w = p (bonus) or max(0, p - q) (residual); explicit roundings so that the first pass and the
// rescan of the located chunk produce the same bits
__device__ __forceinline__ float rs_weight(const RsConst& c, float xt, float xd) {
    const float p = ex2f(__fsub_rn(__fmaf_rn(xt, c.scale, -c.lp_hi), c.lp_lo));
    if (c.mode == RS_BONUS) return p;
    const float q = ex2f(__fsub_rn(__fmaf_rn(xd, c.scale, -c.lq_hi), c.lq_lo));
    return fmaxf(__fsub_rn(p, q), 0.f);
}

// A lane's kVec elements of a 256-element chunk.  bf16: eight adjacent elements (one 16-byte load, the warp
// reads 512 contiguous bytes).  fp32: four adjacent elements of the chunk's first half and four of its
// second half, so that each of the two loads of the warp covers 512 contiguous bytes (with eight
// adjacent floats per lane every 32-byte sector would be requested twice).  rs_elem gives the vocabulary
// index of element j.
template <typename T>
__device__ __forceinline__ int rs_elem(int chunk, int lane, int j) {
    if constexpr (sizeof(T) == 2) return chunk * kChunk + lane * kVec + j;
    else return chunk * kChunk + (j < kVec / 2 ? lane * (kVec / 2) + j : kChunk / 2 + lane * (kVec / 2) + j - kVec / 2);
}
template <bool ALIGNED>
__device__ __forceinline__ uint4 rs_load4(const float* row, int e, int hi, float pad) {
    if (ALIGNED && e + 4 <= hi) return ldg_stream(row + e);
    float x[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) x[j] = (e + j < hi) ? elem_to_float(row, e + j) : pad;
    return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
}
template <typename T, bool ALIGNED>
__device__ __forceinline__ Raw<T> rs_load_lane(const T* row, int chunk, int V, float pad) {
    const int lane = threadIdx.x & 31;
    if constexpr (sizeof(T) == 2) {
        return load_raw<T, ALIGNED>(row, chunk * kChunk + lane * kVec, V, pad);
    } else {
        Raw<T> r;
        r.a = rs_load4<ALIGNED>(row, chunk * kChunk + lane * 4, V, pad);
        r.b = rs_load4<ALIGNED>(row, chunk * kChunk + kChunk / 2 + lane * 4, V, pad);
        return r;
    }
}

template <typename T, bool ALIGNED>
__device__ __forceinline__ void rs_load(const RsConst& c, const T* trow, const T* drow, int chunk, int V,
                                        Raw<T>& rt, Raw<T>& rd) {
    const float ninf = __int_as_float(0xff800000);
    rt = rs_load_lane<T, ALIGNED>(trow, chunk, V, ninf);
    if (c.mode == RS_RESIDUAL) rd = rs_load_lane<T, ALIGNED>(drow, chunk, V, ninf);
    else rd = raw_fill<T>(ninf);
}

// the kVec weights of one lane, two elements per instruction; per element the same operations and
// roundings as rs_weight, so both give the same bits
template <typename T>
__device__ __forceinline__ void rs_weights(const RsConst& c, const Raw<T>& rt, const Raw<T>& rd, float (&w)[kVec]) {
    const f2 sc2 = pack2(c.scale, c.scale);
    const f2 ph2 = pack2(-c.lp_hi, -c.lp_hi), pl2 = pack2(c.lp_lo, c.lp_lo);
    f2 xt[4];
    unpack_pairs(rt, xt);
    if (c.mode == RS_BONUS) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const f2 p = ex2_2(sub2(fma2(xt[i], sc2, ph2), pl2));
            unpack2(p, w[2 * i], w[2 * i + 1]);
        }
        return;
    }
    const f2 qh2 = pack2(-c.lq_hi, -c.lq_hi), ql2 = pack2(c.lq_lo, c.lq_lo);
    f2 xd[4];
    unpack_pairs(rd, xd);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const f2 p = ex2_2(sub2(fma2(xt[i], sc2, ph2), pl2));
        const f2 q = ex2_2(sub2(fma2(xd[i], sc2, qh2), ql2));
        float lo, hi;
        unpack2(sub2(p, q), lo, hi);
        w[2 * i] = fmaxf(lo, 0.f);
        w[2 * i + 1] = fmaxf(hi, 0.f);
    }
}

template <typename T, bool ALIGNED>
__device__ __forceinline__ void rs_chunk_weights(const RsConst& c, const T* trow, const T* drow, int chunk,
                                                 int V, float (&w)[kVec]) {
    Raw<T> rt, rd;
    rs_load<T, ALIGNED>(c, trow, drow, chunk, V, rt, rd);
    rs_weights<T>(c, rt, rd, w);
}

// Each warp takes KU chunks at a time (c0+warp, +8, ...) and requests the next KU before it evaluates
// the current ones, so the memory latency is paid once per CTA, not once per batch.  MODE is the
// row's mode as a constant: a bonus draw never touches the draft row, so its registers go into a
// deeper batch instead.  The buffers of both batches stay within 32 registers per thread for
// either element type; more than that spills and the kernel falls to a fraction of its rate.
template <typename T, bool ALIGNED, int MODE, int KU>
__device__ __forceinline__ void rs_load_batch(const T* trow, const T* drow, int base, int c1, int V,
                                              Raw<T> (&rt)[KU], Raw<T> (&rd)[KU]) {
    const float ninf = __int_as_float(0xff800000);
#pragma unroll
    for (int u = 0; u < KU; ++u) {
        const int ch = base + u * kWarps;
        if (ch < c1) {
            rt[u] = rs_load_lane<T, ALIGNED>(trow, ch, V, ninf);
            if (MODE == RS_RESIDUAL) rd[u] = rs_load_lane<T, ALIGNED>(drow, ch, V, ninf);
        } else {
            rt[u] = raw_fill<T>(ninf);
            if (MODE == RS_RESIDUAL) rd[u] = rt[u];
        }
    }
}

// make_const() yields the row's constants; it is called after the first batch of loads has been issued,
// so constants that are themselves still on their way from memory do not hold the loads up.
template <typename T, bool ALIGNED, int MODE, int KU, class F>
__device__ __forceinline__ void rs_chunk_sums_mode(F make_const, const T* trow, const T* drow, int c0, int c1,
                                                   int V, float* csum) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int base = c0 + warp;
    if (base >= c1) return;
    Raw<T> rt[KU], rd[KU];
    rs_load_batch<T, ALIGNED, MODE, KU>(trow, drow, base, c1, V, rt, rd);
    RsConst c = make_const();
    c.mode = MODE;
    while (base < c1) {
        const int next = base + kWarps * KU;
        Raw<T> nt[KU], nd[KU];
        if (next < c1) rs_load_batch<T, ALIGNED, MODE, KU>(trow, drow, next, c1, V, nt, nd);
        float s[KU];
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            float w[kVec];
            rs_weights<T>(c, rt[u], rd[u], w);
            s[u] = 0.f;
#pragma unroll
            for (int j = 0; j < kVec; ++j) s[u] = __fadd_rn(s[u], w[j]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int u = 0; u < KU; ++u) s[u] = __fadd_rn(s[u], __shfl_xor_sync(0xffffffffu, s[u], o));
        }
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            const int ch = base + u * kWarps;
            if (lane == 0 && ch < c1) SPECKV_ST(csum[ch], s[u]);
        }
        if (next < c1) {
#pragma unroll
            for (int u = 0; u < KU; ++u) {
                rt[u] = nt[u];
                if (MODE == RS_RESIDUAL) rd[u] = nd[u];
            }
        }
        base = next;
    }
}

template <typename T, bool ALIGNED>
__device__ __forceinline__ void rs_chunk_sums(const RsConst& c, const T* trow, const T* drow, int c0, int c1,
                                              int V, float* csum) {
    constexpr int kResidual = sizeof(T) == 2 ? 2 : 1;  // chunks per batch: two rows to buffer
    constexpr int kBonus = 2;  // one row to buffer; measured: deeper bf16 batches leave a warp too few iterations
    auto mk = [&]() { return c; };
    if (c.mode == RS_BONUS) rs_chunk_sums_mode<T, ALIGNED, RS_BONUS, kBonus>(mk, trow, drow, c0, c1, V, csum);
    else rs_chunk_sums_mode<T, ALIGNED, RS_RESIDUAL, kResidual>(mk, trow, drow, c0, c1, V, csum);
}

// RowInfo as the two 16-byte words it is loaded as
__device__ __forceinline__ RowInfo row_info_from(const int4& lo4, const int4& hi4) {
    RowInfo ri;
    ri.mode = lo4.x; ri.n = lo4.y; ri.u2 = __int_as_float(lo4.z); ri.scale = __int_as_float(lo4.w);
    ri.lse2_p = __hiloint2double(hi4.y, hi4.x);
    ri.lse2_q = __hiloint2double(hi4.w, hi4.z);
    return ri;
}
// The same sums for a row whose mode is known but whose RowInfo words may still be in flight
template <typename T, bool ALIGNED>
__device__ __forceinline__ void rs_chunk_sums_info(int mode, const int4& lo4, const int4& hi4, const T* trow, const T* drow,
                                                   int c0, int c1, int V, float* csum) {
    constexpr int kResidual = sizeof(T) == 2 ? 2 : 1;
    constexpr int kBonus = 2;
    auto mk = [&]() { return rs_const(row_info_from(lo4, hi4), mode); };
    if (mode == RS_BONUS) rs_chunk_sums_mode<T, ALIGNED, RS_BONUS, kBonus>(mk, trow, drow, c0, c1, V, csum);
    else rs_chunk_sums_mode<T, ALIGNED, RS_RESIDUAL, kResidual>(mk, trow, drow, c0, c1, V, csum);
}

// The last CTA of a row copies the row's chunk sums into shared memory (one memory round trip for
// all of them) before it searches them; rows with more chunks than fit are searched in place.
constexpr int kRsStage = 2048;
struct RsSums {
    const float* sh;    // staged copy, or nullptr
    const float* glob;
    __device__ __forceinline__ float operator[](int ch) const {
        if (sh) return sh[ch];
        return dbg_ok(glob + ch, 4, DBG_WS_LOAD) ? __ldcg(glob + ch) : 0.f;
    }
};
__device__ __forceinline__ RsSums rs_stage_sums(float* sh_cs, const float* csum, int nchunk) {
    RsSums r;
    r.glob = csum;
    r.sh = nullptr;
    if (nchunk <= kRsStage) {
        for (int ch = threadIdx.x; ch < nchunk; ch += kThreads) sh_cs[ch] = dbg_ok(csum + ch, 4, DBG_WS_LOAD) ? __ldcg(csum + ch) : 0.f;
        r.sh = sh_cs;
    }
    __syncthreads();
    return r;
}

// warp 0: total weight W of the row from its chunk sums
__device__ __forceinline__ double rs_total(const RsSums& cs, int nchunk, int per_lane, double* own_out) {
    const int lane = threadIdx.x & 31;
    double own = 0.0;
    const int a = lane * per_lane, e = min(nchunk, a + per_lane);
    for (int ch = a; ch < e; ++ch) own += static_cast<double>(cs[ch]);
    *own_out = own;
    return warp_sum(own);
}

// Warp 0 of the CTA that holds a row's chunk sums: the vocabulary index at which the running sum of the
// weights first exceeds tau (the last index with weight if rounding leaves tau at or above the total).
// own = this lane's share of the chunk sums as rs_total left it.  The located chunk's weights are
// recomputed, bit-identical to the first pass.  Every lane returns the index.
template <typename T, bool ALIGNED>
__device__ __forceinline__ int rs_search(const RsConst& c, const T* trow, const T* drow, const RsSums& cs, int nchunk,
                                         int V, double tau, double own, int per_lane) {
    const int lane = threadIdx.x & 31;
    // inclusive scan of the per-lane group sums
    double incl = own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    unsigned hit = __ballot_sync(0xffffffffu, incl > tau && own > 0.0);
    unsigned pos = __ballot_sync(0xffffffffu, own > 0.0);
    int src = hit ? (__ffs(hit) - 1) : (31 - __clz(pos));  // fallback: last group with weight
    // the chosen lane walks its chunks
    int chunk = -1;
    double before = 0.0;
    if (lane == src) {
        double run = incl - own;
        const int a = lane * per_lane, e = min(nchunk, a + per_lane);
        int last_pos = -1;
        double last_before = 0.0;
        for (int ch = a; ch < e; ++ch) {
            double sv = static_cast<double>(cs[ch]);
            if (sv > 0.0) { last_pos = ch; last_before = run; }
            if (run + sv > tau && sv > 0.0) { chunk = ch; before = run; break; }
            run += sv;
        }
        if (chunk < 0) { chunk = last_pos; before = last_before; }
    }
    chunk = __shfl_sync(0xffffffffu, chunk, src);
    before = __shfl_sync(0xffffffffu, before, src);

    // recompute the chunk's weights (bit-identical to the first pass) and scan them
    float w[kVec];
    rs_chunk_weights<T, ALIGNED>(c, trow, drow, chunk, V, w);
    // a lane's elements form one run of the chunk (bf16) or two (fp32, see rs_elem): scan run by run
    constexpr int kSeg = sizeof(T) == 2 ? 1 : 2, kSegLen = kVec / kSeg;
    int found = 0x7fffffff, lastw = -1;
    double seg_base = before;
#pragma unroll
    for (int sg = 0; sg < kSeg; ++sg) {
        double lane_tot = 0.0;
#pragma unroll
        for (int j = 0; j < kSegLen; ++j) lane_tot += static_cast<double>(w[sg * kSegLen + j]);
        double lincl = lane_tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            double v = __shfl_up_sync(0xffffffffu, lincl, o);
            if (lane >= o) lincl += v;
        }
        double run = seg_base + (lincl - lane_tot);
#pragma unroll
        for (int j = 0; j < kSegLen; ++j) {
            run += static_cast<double>(w[sg * kSegLen + j]);
            const int idx = rs_elem<T>(chunk, lane, sg * kSegLen + j);
            if (w[sg * kSegLen + j] > 0.f) {
                lastw = max(lastw, idx);
                if (run > tau && found == 0x7fffffff) found = idx;
            }
        }
        seg_base += __shfl_sync(0xffffffffu, lincl, 31);  // the whole run
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
        lastw = max(lastw, __shfl_xor_sync(0xffffffffu, lastw, o));
    }
    return (found != 0x7fffffff) ? found : lastw;
}

template <typename T, bool ALIGNED>
__device__ __forceinline__ void resample_body(const KParams& P, const int bid) {
    __shared__ int sh_flag;
    // one-dimensional grid, R consecutive CTAs per batch row: the CTAs of a row are neighbours in
    // launch order, so rows finish one after the other and their searches overlap the other rows' sums
    // (draft-side sampling: one draw per drafted position; r counts positions, b = r / gamma_max)
    // the last rs_tail draws (in launch order) are cut into R2 >= R shares: their rows are the last to
    // be swept, nothing is left to overlap their draw with, and more CTAs per row shorten it
    const int n_all = P.sample ? P.B * P.G : P.B;
    const int n_head = (n_all - P.rs_tail) * P.R;
    const bool tail = bid >= n_head;
    const int Rr = tail ? P.R2 : P.R;
    const int cpc = tail ? P.chunks_per_cta2 : P.chunks_per_cta;
    const int bq = tail ? (n_all - P.rs_tail) + (bid - n_head) / Rr : bid / Rr;
    const int share = tail ? (bid - n_head) % Rr : bid % Rr;
    const int r = P.rs_reverse ? (P.sample ? P.B * P.G : P.B) - 1 - bq : bq;
    const int b = P.sample ? r / P.G : r;
    // Launched as a programmatic dependent of the sweep kernel, so its CTAs become resident as the
    // sweep's last CTAs leave.  With completion flags a CTA waits only for its own batch row (rows
    // are taken in the order the sweep finishes them unless rs_reverse is set) and the stop positions of finished rows are
    // summed while the sweep drains; every sweep CTA is resident or done before the first CTA of
    // this kernel starts, so the wait ends, and it is bounded all the same.  Without flags the CTA
    // waits for the whole sweep grid.
    const int4* ip = reinterpret_cast<const int4*>(P.info + r);
    int mode, n;
    int4 lo4, hi4;
    if (P.rdone) {
        if (threadIdx.x == 0) sh_flag = row_done_wait(P.rdone + b, P.wait_limit);
        __syncthreads();
        const int v = sh_flag;
        if (!v) {
            // Gave up.  The mark goes on the row's flag: if the row epilogue has already written the
            // status (the flag went up just after the last poll) the bit is added here, otherwise the
            // epilogue finds the mark when it raises the flag and adds the bit itself.
            if (threadIdx.x == 0 && share == 0) {
                const int old = atomicOr(P.rdone + b, kRowDoneTimeout);
                if ((old & 1) && P.status) atomicOr(P.status + b, 16);
            }
            return;
        }
        __syncthreads();  // sh_flag is reused below
        // mode and stop position came with the flag: the logit loads below can go out at once, the
        // rest of the row's record (normalisers, second uniform) travels beside them
        lo4 = __ldcg(ip); hi4 = __ldcg(ip + 1);
        if (P.sample) {  // one record per drafted position behind one flag per batch row
            mode = lo4.x;
            n = lo4.y;
        } else {
            mode = (v >> 8) & 3;
            n = (v >> 16) & 0xff;
        }
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        lo4 = __ldcg(ip); hi4 = __ldcg(ip + 1);
        mode = lo4.x;
        n = lo4.y;
    }
    resample_row<T, ALIGNED>(P, b, r, mode, n, lo4, hi4, share, Rr, cpc);
}

// One CTA's share (chunks share*cpc ...) of draw r of batch row b; the last of the draw's Rr CTAs to arrive
// locates the token.  lo4 / hi4: the row's record as loaded from P.info[r].
template <typename T, bool ALIGNED>
__device__ __forceinline__ void resample_row(const KParams& P, const int b, const int r, const int mode, const int n,
                                             const int4 lo4, const int4 hi4, const int share, const int Rr, const int cpc) {
    __shared__ int sh_flag;
    __shared__ int sh_empty;
    __shared__ float sh_cs[kRsStage];
    const int4* ip = reinterpret_cast<const int4*>(P.info + r);
    if (mode == RS_NONE) return;  // greedy or flagged row: nothing to draw
    const long long out_at = P.sample ? static_cast<long long>(r) : static_cast<long long>(b) * (P.G + 1) + n;

    const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb +
                    static_cast<long long>(n) * P.tsp;
    const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb +
                    static_cast<long long>(n) * P.dsp;
    float* csum = P.csum + static_cast<long long>(r) * P.nchunk;

    const int c0 = share * cpc;
    const int c1 = min(P.nchunk, c0 + cpc);
    rs_chunk_sums_info<T, ALIGNED>(mode, lo4, hi4, trow, drow, c0, c1, P.V, csum);

    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        int old = atomicAdd(P.tick2 + r, 1);
        sh_flag = (old == Rr - 1);
    }
    __syncthreads();
    if (!sh_flag) return;
    __threadfence();

    // ---- last CTA of the row: locate the threshold ----
    const RowInfo ri = row_info_from(__ldcg(ip), __ldcg(ip + 1));  // fetched again rather than kept in registers
    RsConst c = rs_const(ri, mode);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int per_lane = (P.nchunk + 31) / 32;
    double own = 0.0, W = 0.0;
    RsSums cs = rs_stage_sums(sh_cs, csum, P.nchunk);
    if (warp == 0) {
        W = rs_total(cs, P.nchunk, per_lane, &own);
        if (lane == 0) sh_empty = (W > (c.mode == RS_RESIDUAL ? 1e-6 : 0.0)) ? 0 : 1;
    }
    __syncthreads();
    if (sh_empty) {
        // numerically empty residual (p == q at the stop position): draw from p instead
        if (c.mode != RS_RESIDUAL) {  // p itself has no mass: cannot happen for a finite row
            if (threadIdx.x == 0) P.out_tok[out_at] = 0;
            return;
        }
        c.mode = RS_BONUS;
        rs_chunk_sums<T, ALIGNED>(c, trow, drow, 0, P.nchunk, P.V, csum);
        __syncthreads();
        cs = rs_stage_sums(sh_cs, csum, P.nchunk);
        if (warp == 0) W = rs_total(cs, P.nchunk, per_lane, &own);
    }
    if (warp != 0) return;

    const double tau = static_cast<double>(ri.u2) * W;
    const int tok = rs_search<T, ALIGNED>(c, trow, drow, cs, P.nchunk, P.V, tau, own, per_lane);
    if (lane == 0) P.out_tok[out_at] = tok;
}

template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(kThreads, 4) resample_kernel(const __grid_constant__ KParams P) {
    resample_body<T, ALIGNED>(P, static_cast<int>(blockIdx.x));
}

// ----------------------------------------------------------------------------------------
// Stand-alone controller: one warp per row.
// ----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) select_gamma_kernel(const __grid_constant__ KParams P, const float* feat_in) {
    const int b = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b >= P.B) return;
    float f4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) f4[k] = feat_in[static_cast<long long>(b) * 4 + k];
    const CtlRegs ctl = ctl_load(P, b, threadIdx.x & 31);
    ctl_eval(P, ctl, f4, P.scores ? P.scores + static_cast<long long>(b) * P.n_out : nullptr, P.gamma_next + b);
}

}  // namespace speckv
