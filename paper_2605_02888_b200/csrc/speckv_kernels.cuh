// Device code of libspeckv: the streaming sweep over vocabulary-sized logit rows, the
// per-row epilogue (signals, acceptance, controller) and the inverse-CDF resample.
//
// Scheme (sm_100a, CUDA cores only -- the work is a streaming reduction, not a contraction):
//   sweep kernel    one CTA per (row b, logit row j, vocabulary slice s).  Each thread keeps
//                   an online-softmax state over 16-byte vector loads, the CTA merges the
//                   256 states and stores one partial.  The last CTA of a batch row to finish
//                   (found with a ticket counter, nobody waits) merges that row's partials in
//                   double precision and writes signals, acceptance, controller outputs.
//   resample kernel R CTAs per batch row rescan the stop position's draft/target rows, write
//                   per-256-element chunk sums of the residual weights, and the last of them
//                   locates the inverse-CDF threshold and writes the fresh token.
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
constexpr float kFloor = -1.2676506002282294e30f;  // -2^100: logits below count as -inf
constexpr uint32_t kFloorBf16x2 = 0xF180F180u;     // -2^100 as two bf16
constexpr double kLn2 = 0.6931471805599453094;
constexpr double kLog2e = 1.4426950408889634074;

enum : int { MODE_SIGNALS = 1, MODE_VERIFY = 2, MODE_MLP = 4 };
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

struct KParams {
    int B, G, V, J, nsplit, nvec, per_split, nchunk, R, chunks_per_cta, mode, bits;
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
    RowInfo* info;
    float4* part;
    float* csum;
};

// ----------------------------------------------------------------------------------------
// small helpers
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max_nan(float a, float b) {  // NaN-propagating max
    float y;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b));
    return y;
}
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
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

__device__ __forceinline__ float elem_to_float(const __nv_bfloat16* p, long long i) {
    return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const unsigned short*>(p)[i]) << 16);
}
__device__ __forceinline__ float elem_to_float(const float* p, long long i) { return p[i]; }

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
    float m, cnt, z0, z1, s0, s1;
    bool bad;
    __device__ __forceinline__ void init(float m0) { m = m0; cnt = 0.f; z0 = z1 = s0 = s1 = 0.f; bad = false; }

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
        if (vmax > m) {  // everything gathered so far moves below the new maximum
            float dm = m - vmax;
            float f = ex2f(dm * scale);
            float zall = cnt + (z0 + z1);
            float sall = s0 + s1;
            z0 = zall * f; z1 = 0.f;
            s0 = fmaf(dm, zall, sall) * f; s1 = 0.f;
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
                z0 += e;
                s0 = fmaf(e, dx, s0);
            }
        }
    }

    template <typename T>
    __device__ __forceinline__ void step(Raw<T> raw, float scale) {
        if (raw_exceeds<false>(raw, m)) {  // an element >= m, or a NaN: rare after the warm start
            slow<T>(raw, scale);
            return;
        }
        raw_floor(raw);
        float x[kVec];
        unpack<T>(raw, x);
#pragma unroll
        for (int j = 0; j < kVec; j += 2) {
            float d0 = x[j] - m, d1 = x[j + 1] - m;
            float e0 = ex2f(d0 * scale), e1 = ex2f(d1 * scale);
            z0 += e0; z1 += e1;
            s0 = fmaf(e0, d0, s0); s1 = fmaf(e1, d1, s1);
        }
    }
    __device__ __forceinline__ float4 partial() const {
        return make_float4(m, bad ? __int_as_float(0x7fc00000) : cnt, z0 + z1, s0 + s1);
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
    float m, r, z0, z1;
    __device__ __forceinline__ void init(float m0, float scale) { m = m0; r = m0 * scale; z0 = z1 = 0.f; }
    template <typename T>
    __device__ __forceinline__ void step(const Raw<T>& raw, float scale) {
        if (raw_exceeds<true>(raw, m)) {  // a new maximum (or NaN): move the reference
            float vmax = raw_max(raw);
            if (vmax == vmax) {  // NaN needs no rescale; it poisons Z below
                float rn = vmax * scale;
                float f = ex2f(r - rn);
                z0 = (z0 + z1) * f; z1 = 0.f;
                r = rn; m = vmax;
            }
        }
        float x[kVec];
        unpack<T>(raw, x);
#pragma unroll
        for (int j = 0; j < kVec; j += 2) {
            z0 += ex2f(fmaf(x[j], scale, -r));
            z1 += ex2f(fmaf(x[j + 1], scale, -r));
        }
    }
    __device__ __forceinline__ float4 partial() const { return make_float4(r, z0 + z1, 0.f, 0.f); }
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
// One CTA sweeps elements [lo, hi) of one logit row and returns the merged partial in
// thread 0.  Thread t owns vectors t, t+256, ... of the slice; U of them are in flight.
// ----------------------------------------------------------------------------------------
template <typename T, bool ALIGNED, int PATH, int U>
__device__ __forceinline__ float4 sweep_slice(const T* __restrict__ row, int lo, int hi, float scale,
                                              float4* sh_part) {
    const int tid = threadIdx.x;
    const float pad = (PATH == PATH_DRAFT) ? kFloor : __int_as_float(0xff800000);
    constexpr int kStride = kThreads * kVec;               // elements between a thread's vectors
    const int nv = (hi - lo + kVec - 1) / kVec;             // vectors in the slice (last may be ragged)
    const int my_n = (nv > tid) ? (nv - tid + kThreads - 1) / kThreads : 0;
    // vectors this thread takes through the unguarded 16-byte path
    int n_main = my_n;
    if (!ALIGNED) n_main = 0;
    else if (my_n > 0 && lo + (tid + (my_n - 1) * kThreads) * kVec + kVec > hi) n_main = my_n - 1;
    const T* p = row + lo + tid * kVec;

    Raw<T> buf[U];
#pragma unroll
    for (int k = 0; k < U; ++k) buf[k] = (k < n_main) ? ld_vec<T>(p + k * kStride) : raw_fill<T>(pad);
    Raw<T> first = buf[0];
    if (n_main == 0 && my_n > 0) first = load_raw<T, false>(row, lo + tid * kVec, hi, pad);

    // warm start: the CTA-wide maximum of every thread's first vector.  A first vector holding
    // NaN / +inf / only -inf contributes the floor; its owner meets the offending element again
    // in its own state and flags it there.
    float m0 = raw_max(first);
    if (!(m0 >= kFloor && m0 < __int_as_float(0x7f800000))) m0 = kFloor;
    m0 = warp_maxf(m0);
    __shared__ float sh_m0[kWarps];
    if ((tid & 31) == 0) sh_m0[tid >> 5] = m0;
    __syncthreads();
    m0 = sh_m0[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) m0 = fmaxf(m0, sh_m0[w]);

    DraftState ds; TargetState ts; ArgmaxState as;
    if constexpr (PATH == PATH_DRAFT) ds.init(m0);
    else if constexpr (PATH == PATH_TARGET) ts.init(m0, scale);
    else as.init(m0);

    auto process = [&](const Raw<T>& v, int idx) {
        if constexpr (PATH == PATH_DRAFT) ds.template step<T>(v, scale);
        else if constexpr (PATH == PATH_TARGET) ts.template step<T>(v, scale);
        else as.template step<T>(v, lo + (tid + idx * kThreads) * kVec);
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
        process(load_raw<T, false>(row, lo + (tid + j * kThreads) * kVec, hi, pad), j);

    float4 part;
    if constexpr (PATH == PATH_DRAFT) part = ds.partial();
    else if constexpr (PATH == PATH_TARGET) part = ts.partial();
    else part = as.partial();
    part = warp_merge<PATH>(part, scale);
    if ((tid & 31) == 0) sh_part[tid >> 5] = part;
    __syncthreads();
    if (tid == 0) {
#pragma unroll
        for (int w = 1; w < kWarps; ++w) part = merge_any<PATH>(part, sh_part[w], scale);
    }
    return part;
}

// ----------------------------------------------------------------------------------------
// Row epilogue helpers (one warp, double precision; a few dozen values per row)
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float4 ldcg4(const float4* p) { return __ldcg(p); }

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

// Controller (Sec. 4.3, Eq. 1) for one row, executed by a full warp.  f4 = Hbar, cbar, Hmax, cmin.
__device__ __forceinline__ void controller_row(const KParams& P, int b, const double (&f4)[4],
                                               float* scores_row, int* gamma_next) {
    const int lane = threadIdx.x & 31;
    double x[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) x[k] = 0.0;
    const float* comp = P.comp ? P.comp + static_cast<long long>(b) * P.n_comp : nullptr;
    if (P.layout == 0) {
        x[0] = f4[0]; x[1] = f4[1]; x[2] = f4[3];
        for (int k = 3; k < P.n_in; ++k) x[k] = comp ? static_cast<double>(comp[k - 3]) : 0.0;
    } else {
        x[0] = f4[0]; x[1] = f4[1]; x[2] = f4[2]; x[3] = f4[3];
        for (int k = 4; k < P.n_in; ++k) x[k] = comp ? static_cast<double>(comp[k - 4]) : 0.0;
    }
    double h = 0.0;
    if (lane < P.n_hidden) {
        h = static_cast<double>(P.b1[lane]);
        for (int f = 0; f < P.n_in; ++f) h += static_cast<double>(P.W1[lane * P.n_in + f]) * x[f];
        h = h > 0.0 ? h : 0.0;
    }
    double best = 0.0;
    int best_j = 0;
    for (int j = 0; j < P.n_out; ++j) {
        double part = (lane < P.n_hidden) ? static_cast<double>(P.W2[j * P.n_hidden + lane]) * h : 0.0;
        double o = warp_sum(part) + static_cast<double>(P.b2[j]);
        double e = (P.transform == 0) ? o * P.gch[j] + 1.0 : o;
        if (scores_row && lane == 0) scores_row[j] = static_cast<float>(e);
        if (j == 0 || e > best) { best = e; best_j = j; }
    }
    if (gamma_next && lane == 0) *gamma_next = P.gch[best_j];
}

// Row epilogue: runs in warp 0 of the last CTA of batch row b.
template <typename T>
__device__ __noinline__ void row_epilogue(const KParams& P, int b) {
    const int lane = threadIdx.x & 31;
    const int G = P.G;
    const bool verify = (P.mode & MODE_VERIFY) != 0;

    int gam = P.gamma ? P.gamma[b] : G;
    float Tf = P.temp ? P.temp[b] : P.temp_scalar;
    int status = 0;
    if (gam < 1 || gam > G) status |= 1;
    if (!(Tf >= 0.f) || Tf == __int_as_float(0x7f800000)) status |= 8;
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));
    const double sd = static_cast<double>(scale);

    const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb;
    const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb;

    double Hi = 0.0, ci = 0.0, lse2_q = 0.0, lse2_p = 0.0;
    int amax = -1;
    bool nonfinite = false, badtok = false, accept = true;

    if (!status) {
        const bool dr_on = lane < gam;
        const bool tg_on = verify && lane <= gam;
        if (dr_on) {
            const int j = verify ? (G + 1 + lane) : lane;
            const float4* pp = P.part + (static_cast<long long>(b) * P.J + j) * P.nsplit;
            double m = 0, cnt = 0, Zx = 0, S = 0;
            for (int k = 0; k < P.nsplit; ++k) {
                float4 q = ldcg4(pp + k);
                double qm = q.x, qc = q.y, qz = q.z, qs = q.w;
                if (k == 0) { m = qm; cnt = qc; Zx = qz; S = qs; continue; }
                if (qm > m) {
                    double dm = m - qm, f = exp2(dm * sd), za = cnt + Zx;
                    Zx = za * f + qz; S = (S + dm * za) * f + qs; cnt = qc; m = qm;
                } else if (qm == m) {
                    cnt += qc; Zx += qz; S += qs;
                } else {
                    double dm = qm - m, f = exp2(dm * sd), za = qc + qz;
                    Zx += za * f; S += (qs + dm * za) * f;
                    if (qc != qc) cnt = qc;
                }
            }
            double Z = cnt + Zx;
            if (!(cnt >= 1.0) || !(Z < 1e300) || !(m > static_cast<double>(kFloor))) {
                nonfinite = true;
            } else {
                double lnZ = log(cnt) + log1p(Zx / cnt);
                Hi = lnZ - kLn2 * sd * S / Z;
                if (Hi < 0.0) Hi = 0.0;
                ci = 1.0 / Z;
                lse2_q = m * sd + lnZ * kLog2e;
            }
        }
        if (tg_on) {
            const float4* pp = P.part + (static_cast<long long>(b) * P.J + lane) * P.nsplit;
            if (greedy) {
                float bv = 0.f; int bi = 0x7fffffff; float bad = 0.f;
                for (int k = 0; k < P.nsplit; ++k) {
                    float4 q = ldcg4(pp + k);
                    int qi = __float_as_int(q.y);
                    if (k == 0 || q.x > bv || (q.x == bv && qi < bi)) { bv = q.x; bi = qi; }
                    bad += q.z;
                }
                if (bad != 0.f || bi == 0x7fffffff || !(bv > kFloor)) nonfinite = true;
                amax = bi;
            } else {
                double R = 0, Z = 0;
                for (int k = 0; k < P.nsplit; ++k) {
                    float4 q = ldcg4(pp + k);
                    double qr = q.x, qz = q.y;
                    if (k == 0) { R = qr; Z = qz; continue; }
                    if (qr > R) { Z = Z * exp2(R - qr) + qz; R = qr; }
                    else { Z += qz * exp2(qr - R); }
                }
                if (!(Z > 0.0) || !(Z < 1e300)) nonfinite = true;
                else lse2_p = R + log2(Z);
            }
        }
        if (verify && lane < gam) {
            int x = P.tok[static_cast<long long>(b) * G + lane];
            if (x < 0 || x >= P.V) {
                badtok = true;
            } else if (greedy) {
                accept = (x == amax);
            } else if (!nonfinite) {
                double dx = static_cast<double>(elem_to_float(drow + static_cast<long long>(lane) * P.dsp, x));
                double tx = static_cast<double>(elem_to_float(trow + static_cast<long long>(lane) * P.tsp, x));
                double lq = dx * sd - lse2_q;
                double lp = tx * sd - lse2_p;
                double u = static_cast<double>(P.u[(static_cast<long long>(b) * (G + 1) + lane) * 2]);
                accept = (log2(u) + lq) < lp;  // u * q(x) < p(x)
            }
        }
        if (__any_sync(0xffffffffu, nonfinite)) status |= 4;
        if (__any_sync(0xffffffffu, badtok)) status |= 2;
    }

    // first rejected position
    unsigned rej = __ballot_sync(0xffffffffu, !accept && lane < gam);
    int n = (status == 0 && verify) ? (rej ? (__ffs(rej) - 1) : gam) : 0;

    // signals
    const double in_bits = P.bits ? kLog2e : 1.0;
    double Hout = (status == 0 && lane < gam) ? Hi * in_bits : 0.0;
    double Cout = (status == 0 && lane < gam) ? ci : 0.0;
    double f4[4] = {0, 0, 0, 0};
    if (status == 0) {
        f4[0] = warp_sum(Hout) / gam;
        f4[1] = warp_sum(Cout) / gam;
        f4[2] = warp_max(Hout);
        f4[3] = warp_min(lane < gam ? Cout : 2.0);
    }
    if (lane < G) {
        if (P.H) P.H[static_cast<long long>(b) * G + lane] = static_cast<float>(Hout);
        if (P.C) P.C[static_cast<long long>(b) * G + lane] = static_cast<float>(Cout);
    }
    if (P.feat && lane < 4) P.feat[static_cast<long long>(b) * 4 + lane] = static_cast<float>(f4[lane]);

    if (P.mode & MODE_MLP) {
        if (status == 0) {
            controller_row(P, b, f4, P.scores ? P.scores + static_cast<long long>(b) * P.n_out : nullptr,
                           P.gamma_next + b);
        } else {
            if (P.scores && lane < P.n_out) P.scores[static_cast<long long>(b) * P.n_out + lane] = 0.f;
            if (lane == 0) P.gamma_next[b] = 0;
        }
    }

    if (verify) {
        // fresh token: known here for greedy rows, drawn by the resample kernel otherwise
        int amax_n = __shfl_sync(0xffffffffu, amax, n);
        double lp_n = __shfl_sync(0xffffffffu, lse2_p, n);
        double lq_n = __shfl_sync(0xffffffffu, lse2_q, n < gam ? n : 0);
        if (lane <= G) {
            int v = -1;
            if (status == 0) {
                if (lane < n) v = P.tok[static_cast<long long>(b) * G + lane];
                else if (lane == n && greedy) v = amax_n;
            }
            P.out_tok[static_cast<long long>(b) * (G + 1) + lane] = v;
        }
        if (lane == 0) {
            P.n_acc[b] = n;
            RowInfo ri;
            ri.mode = (status == 0 && !greedy) ? (n < gam ? RS_RESIDUAL : RS_BONUS) : RS_NONE;
            ri.n = n;
            ri.u2 = (status == 0 && !greedy) ? P.u[(static_cast<long long>(b) * (G + 1) + n) * 2 + 1] : 0.f;
            ri.scale = scale;
            ri.lse2_p = lp_n;
            ri.lse2_q = lq_n;
            P.info[b] = ri;
        }
    }
    if (P.status && lane == 0) P.status[b] = status;
}

// ----------------------------------------------------------------------------------------
// Sweep kernel
// ----------------------------------------------------------------------------------------
template <typename T, bool ALIGNED, int U>
__global__ void __launch_bounds__(kThreads, 4) sweep_kernel(const __grid_constant__ KParams P) {
    __shared__ float4 sh_part[kWarps];
    __shared__ int sh_last;

    const int per_row = P.J * P.nsplit;
    const int b = blockIdx.x / per_row;
    const int rem = blockIdx.x - b * per_row;
    const int j = rem / P.nsplit;
    const int s = rem - j * P.nsplit;
    const bool verify = (P.mode & MODE_VERIFY) != 0;

    int gam = P.gamma ? P.gamma[b] : P.G;
    float Tf = P.temp ? P.temp[b] : P.temp_scalar;
    const bool row_ok = (gam >= 1 && gam <= P.G) && (Tf >= 0.f) && (Tf != __int_as_float(0x7f800000));
    const bool greedy = (Tf == 0.f);
    const float scale = static_cast<float>(kLog2e / static_cast<double>(greedy ? 1.f : Tf));

    // logit row handled by this CTA: with verification, j <= G are target positions and the
    // rest draft positions; signals alone sweep draft positions only
    const bool is_target = verify && j <= P.G;
    const int pos = is_target ? j : (verify ? j - (P.G + 1) : j);
    const bool active = row_ok && (is_target ? pos <= gam : pos < gam);

    if (active) {
        const int v0 = s * P.per_split;
        const int v1 = min(P.nvec, v0 + P.per_split);
        const int lo = v0 * kVec;
        const int hi = min(P.V, v1 * kVec);
        float4 part = make_float4(0.f, 0.f, 0.f, 0.f);
        if (is_target) {
            const T* row = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb +
                           static_cast<long long>(pos) * P.tsp;
            if (greedy) part = sweep_slice<T, ALIGNED, PATH_ARGMAX, U>(row, lo, hi, scale, sh_part);
            else part = sweep_slice<T, ALIGNED, PATH_TARGET, U>(row, lo, hi, scale, sh_part);
        } else {
            const T* row = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb +
                           static_cast<long long>(pos) * P.dsp;
            part = sweep_slice<T, ALIGNED, PATH_DRAFT, U>(row, lo, hi, scale, sh_part);
        }
        if (threadIdx.x == 0) P.part[static_cast<long long>(blockIdx.x)] = part;
    }

    // ticket: the last CTA of this batch row runs the row epilogue; nobody waits
    if (threadIdx.x == 0) {
        __threadfence();
        int old = atomicAdd(P.tick1 + b, 1);
        sh_last = (old == per_row - 1);
    }
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    if (threadIdx.x < 32) row_epilogue<T>(P, b);
}

// ----------------------------------------------------------------------------------------
// Resample kernel: inverse CDF over the stop position's weights, vocabulary order.
//   residual: w_v = max(0, p_v - q_v);   bonus: w_v = p_v
// The weights are evaluated without cancellation: for p_v < 2 q_v they are formed as
// q_v * expm1(ln p_v - ln q_v), the log-ratio coming from the exact difference of the two
// logits, so a draft that is close to the target still gives accurate small weights.
// ----------------------------------------------------------------------------------------
struct RsConst {
    int mode;
    float scale, lp_hi, lp_lo, lq_hi, lq_lo, dl_hi, dl_lo;
};

__device__ __forceinline__ RsConst rs_const(const RowInfo& ri, int mode) {
    RsConst c;
    c.mode = mode;
    c.scale = ri.scale;
    c.lp_hi = static_cast<float>(ri.lse2_p);
    c.lp_lo = static_cast<float>(ri.lse2_p - static_cast<double>(c.lp_hi));
    c.lq_hi = static_cast<float>(ri.lse2_q);
    c.lq_lo = static_cast<float>(ri.lse2_q - static_cast<double>(c.lq_hi));
    double dl = ri.lse2_p - ri.lse2_q;
    c.dl_hi = static_cast<float>(dl);
    c.dl_lo = static_cast<float>(dl - static_cast<double>(c.dl_hi));
    return c;
}

// expm1(z) for 0 < z < ln 2, Taylor to z^10 (truncation below 2e-9 relative)
__device__ __forceinline__ float expm1_small(float z) {
    float p = 2.755731922e-7f;                 // 1/10!
    p = __fmaf_rn(p, z, 2.755731922e-6f);      // 1/9!
    p = __fmaf_rn(p, z, 2.480158730e-5f);      // 1/8!
    p = __fmaf_rn(p, z, 1.984126984e-4f);      // 1/7!
    p = __fmaf_rn(p, z, 1.388888889e-3f);      // 1/6!
    p = __fmaf_rn(p, z, 8.333333333e-3f);      // 1/5!
    p = __fmaf_rn(p, z, 4.166666667e-2f);      // 1/4!
    p = __fmaf_rn(p, z, 1.666666667e-1f);      // 1/3!
    p = __fmaf_rn(p, z, 0.5f);
    p = __fmaf_rn(p, z, 1.0f);
    return __fmul_rn(p, z);
}

__device__ __forceinline__ float rs_weight(const RsConst& c, float xt, float xd) {
    float p = ex2f(__fsub_rn(__fmaf_rn(xt, c.scale, -c.lp_hi), c.lp_lo));
    if (c.mode == RS_BONUS) return p;
    float q = ex2f(__fsub_rn(__fmaf_rn(xd, c.scale, -c.lq_hi), c.lq_lo));
    float dl = __fsub_rn(__fmaf_rn(__fsub_rn(xt, xd), c.scale, -c.dl_hi), c.dl_lo);  // log2(p/q)
    float w = 0.f;
    if (dl >= 1.0f) w = __fsub_rn(p, q);
    else if (dl > 0.0f) w = __fmul_rn(q, expm1_small(__fmul_rn(dl, 0.693147180559945f)));
    return w;
}

template <typename T, bool ALIGNED>
__device__ __forceinline__ void rs_chunk_weights(const RsConst& c, const T* trow, const T* drow, int chunk,
                                                 int V, float (&w)[kVec]) {
    const int lane = threadIdx.x & 31;
    const int e0 = chunk * kChunk + lane * kVec;
    const float ninf = __int_as_float(0xff800000);
    Raw<T> rt = load_raw<T, ALIGNED>(trow, e0, V, ninf);
    float xt[kVec], xd[kVec];
    unpack<T>(rt, xt);
    if (c.mode == RS_RESIDUAL) {
        Raw<T> rd = load_raw<T, ALIGNED>(drow, e0, V, ninf);
        unpack<T>(rd, xd);
    } else {
#pragma unroll
        for (int j = 0; j < kVec; ++j) xd[j] = ninf;
    }
#pragma unroll
    for (int j = 0; j < kVec; ++j) w[j] = rs_weight(c, xt[j], xd[j]);
}

template <typename T, bool ALIGNED>
__device__ __forceinline__ void rs_chunk_sums(const RsConst& c, const T* trow, const T* drow, int c0, int c1,
                                              int V, float* csum) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int ch = c0 + warp; ch < c1; ch += kWarps) {
        float w[kVec];
        rs_chunk_weights<T, ALIGNED>(c, trow, drow, ch, V, w);
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < kVec; ++j) s = __fadd_rn(s, w[j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, o));
        if (lane == 0) csum[ch] = s;
    }
}

// warp 0: total weight W of the row from its chunk sums
__device__ __forceinline__ double rs_total(const float* csum, int nchunk, int per_lane, double* own_out) {
    const int lane = threadIdx.x & 31;
    double own = 0.0;
    const int a = lane * per_lane, e = min(nchunk, a + per_lane);
    for (int ch = a; ch < e; ++ch) own += static_cast<double>(__ldcg(csum + ch));
    *own_out = own;
    return warp_sum(own);
}

template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(kThreads, 4) resample_kernel(const __grid_constant__ KParams P) {
    __shared__ int sh_flag;
    __shared__ int sh_empty;
    const int b = blockIdx.x;  // batch row; blockIdx.y = which share of the row's chunks
    const RowInfo ri = P.info[b];
    if (ri.mode == RS_NONE) return;  // greedy or flagged row: nothing to draw

    const T* trow = static_cast<const T*>(P.t) + static_cast<long long>(b) * P.tsb +
                    static_cast<long long>(ri.n) * P.tsp;
    const T* drow = static_cast<const T*>(P.d) + static_cast<long long>(b) * P.dsb +
                    static_cast<long long>(ri.n) * P.dsp;
    float* csum = P.csum + static_cast<long long>(b) * P.nchunk;
    RsConst c = rs_const(ri, ri.mode);

    const int c0 = blockIdx.y * P.chunks_per_cta;
    const int c1 = min(P.nchunk, c0 + P.chunks_per_cta);
    rs_chunk_sums<T, ALIGNED>(c, trow, drow, c0, c1, P.V, csum);

    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        int old = atomicAdd(P.tick2 + b, 1);
        sh_flag = (old == static_cast<int>(gridDim.y) - 1);
    }
    __syncthreads();
    if (!sh_flag) return;
    __threadfence();

    // ---- last CTA of the row: locate the threshold ----
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int per_lane = (P.nchunk + 31) / 32;
    double own = 0.0, W = 0.0;
    if (warp == 0) {
        W = rs_total(csum, P.nchunk, per_lane, &own);
        if (lane == 0) sh_empty = (W > 0.0) ? 0 : 1;
    }
    __syncthreads();
    if (sh_empty) {
        // numerically empty residual (p == q at the stop position): draw from p instead
        if (c.mode != RS_RESIDUAL) {  // p itself has no mass: cannot happen for a finite row
            if (threadIdx.x == 0) P.out_tok[static_cast<long long>(b) * (P.G + 1) + ri.n] = 0;
            return;
        }
        c.mode = RS_BONUS;
        rs_chunk_sums<T, ALIGNED>(c, trow, drow, 0, P.nchunk, P.V, csum);
        __syncthreads();
        if (warp == 0) W = rs_total(csum, P.nchunk, per_lane, &own);
    }
    if (warp != 0) return;

    const double tau = static_cast<double>(ri.u2) * W;
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
        const int a = lane * per_lane, e = min(P.nchunk, a + per_lane);
        int last_pos = -1;
        double last_before = 0.0;
        for (int ch = a; ch < e; ++ch) {
            double sv = static_cast<double>(__ldcg(csum + ch));
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
    rs_chunk_weights<T, ALIGNED>(c, trow, drow, chunk, P.V, w);
    double lane_tot = 0.0;
#pragma unroll
    for (int j = 0; j < kVec; ++j) lane_tot += static_cast<double>(w[j]);
    double lincl = lane_tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double v = __shfl_up_sync(0xffffffffu, lincl, o);
        if (lane >= o) lincl += v;
    }
    double run = before + (lincl - lane_tot);
    int found = 0x7fffffff, lastw = -1;
#pragma unroll
    for (int j = 0; j < kVec; ++j) {
        run += static_cast<double>(w[j]);
        const int idx = chunk * kChunk + lane * kVec + j;
        if (w[j] > 0.f) {
            lastw = idx;
            if (run > tau && found == 0x7fffffff) found = idx;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
        lastw = max(lastw, __shfl_xor_sync(0xffffffffu, lastw, o));
    }
    if (lane == 0) {
        int tok = (found != 0x7fffffff) ? found : lastw;
        P.out_tok[static_cast<long long>(b) * (P.G + 1) + ri.n] = tok;
    }
}

// ----------------------------------------------------------------------------------------
// Stand-alone controller: one warp per row.
// ----------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) select_gamma_kernel(const __grid_constant__ KParams P, const float* feat_in) {
    const int b = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b >= P.B) return;
    double f4[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) f4[k] = static_cast<double>(feat_in[static_cast<long long>(b) * 4 + k]);
    controller_row(P, b, f4, P.scores ? P.scores + static_cast<long long>(b) * P.n_out : nullptr,
                   P.gamma_next + b);
}

}  // namespace speckv
