// gv_device.cuh -- device-side building blocks of the output verifier (sm_100a).
//
// Everything here follows the per-element rule and the content hash stated in include/gv.h
// (the tolerance-based comparison of Section 3.1 of the GEAK paper). Float arithmetic on the
// compare path uses the explicitly rounded intrinsics so that no compiler flag can contract it
// into a fused multiply-add or flush subnormals.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "gv.h"

namespace gv {

constexpr int kThreads = 256;          // threads per CTA in every verify kernel
constexpr int kChunk = 16;             // candidates whose accumulators a CTA keeps alive at once
constexpr int kMaxPtrs = 256;          // candidate pointers per dense launch (kernel parameters)
constexpr uint32_t kWaitLimit = 1u << 16;   // polls of a bounded mbarrier wait before giving up
constexpr uint32_t kWaitHintNs = 20000;     // each poll may suspend the thread for up to this long

// status word bits (workspace[0])
constexpr uint32_t kStatusTimeout = 1u;
constexpr uint32_t kStatusBadTable = 2u;

template <int DT> struct Traits;
template <> struct Traits<GV_F32>  { static constexpr int ESZ = 4; static constexpr bool IS_FLOAT = true;  };
template <> struct Traits<GV_BF16> { static constexpr int ESZ = 2; static constexpr bool IS_FLOAT = true;  };
template <> struct Traits<GV_F16>  { static constexpr int ESZ = 2; static constexpr bool IS_FLOAT = true;  };
template <> struct Traits<GV_I32>  { static constexpr int ESZ = 4; static constexpr bool IS_FLOAT = false; };
template <> struct Traits<GV_I64>  { static constexpr int ESZ = 8; static constexpr bool IS_FLOAT = false; };

__host__ __device__ inline int elem_size(int dt) {
    return dt == GV_F32 ? 4 : dt == GV_BF16 ? 2 : dt == GV_F16 ? 2 : dt == GV_I32 ? 4 : dt == GV_I64 ? 8 : 0;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ------------------------------------------------------------------------------------------
// content hash
// ------------------------------------------------------------------------------------------
// The mixing function of the content hash (the SplitMix64 finaliser), written the plain way. Moving part of
// its shifts and additions to the multiplier pipe was measured (a dozen formulations) and brought nothing:
// the plain form is what ships.
__device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ __forceinline__ uint64_t pack64(uint32_t lo, uint32_t hi) {
    return (static_cast<uint64_t>(hi) << 32) | lo;
}

// Hash contribution of one 16-byte vector whose first word has index k0 (k0 even when the vector
// is 16-byte aligned relative to the tensor start). nwords = how many of its two words exist.
__device__ __forceinline__ uint64_t hash_vec(const uint4& v, uint64_t k0, int nwords) {
    uint64_t h = 0;
    if (nwords > 0) h += splitmix64(k0 ^ pack64(v.x, v.y));
    if (nwords > 1) h += splitmix64((k0 + 1) ^ pack64(v.z, v.w));
    return h;
}
__device__ __forceinline__ uint64_t hash_vec_full(const uint4& v, uint64_t k0) {
    return splitmix64(k0 ^ pack64(v.x, v.y)) + splitmix64((k0 + 1) ^ pack64(v.z, v.w));
}

// Full vector whose word indices fit 32 bits (tensors below 32 GiB): the high half of the index is
// zero, so only the low halves are xored.
__device__ __forceinline__ uint64_t hash_vec_full_k32(const uint4& v, uint32_t k0) {
    return splitmix64(pack64(v.x ^ k0, v.y)) + splitmix64(pack64(v.z ^ (k0 + 1u), v.w));
}

// ------------------------------------------------------------------------------------------
// loads
// ------------------------------------------------------------------------------------------
// Streaming 128-bit load: candidates are read exactly once, keep them out of L1.
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Per-thread asynchronous 16-byte copy global -> shared (L2 only, bypasses L1) and its group
// bookkeeping: each thread later reads back only the bytes it copied itself, so completion needs no
// barrier, only the thread's own wait.
__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}
// the same with an L2 eviction hint (policy from l2_evict_first_policy()): streaming candidate bytes are
// read exactly once and should not push the reference out of L2
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void cp_async16_hint(uint32_t smem_dst, const void* gsrc, uint64_t policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gsrc), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t smem_addr, const uint4& v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(smem_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
// the same store under a predicate (no branch: the lanes of a warp that store and those that do not stay together)
__device__ __forceinline__ void sts128_if(uint32_t smem_addr, const uint4& v, bool on) {
    asm volatile("{ .reg .pred p; setp.ne.u32 p, %5, 0; @p st.shared.v4.u32 [%0], {%1,%2,%3,%4}; }"
                 ::"r"(smem_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(static_cast<uint32_t>(on))
                 : "memory");
}
// three such stores, `plane` bytes apart, under one predicate (one queue entry)
__device__ __forceinline__ void sts128x3_if(uint32_t smem_addr, uint32_t plane, const uint4& a, const uint4& b, const uint4& c,
                                            bool on) {
    asm volatile(
        "{ .reg .pred p; .reg .u32 a1, a2;\n\t"
        "setp.ne.u32 p, %14, 0;\n\t"
        "add.u32 a1, %0, %13;\n\t"
        "add.u32 a2, a1, %13;\n\t"
        "@p st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n\t"
        "@p st.shared.v4.u32 [a1], {%5,%6,%7,%8};\n\t"
        "@p st.shared.v4.u32 [a2], {%9,%10,%11,%12}; }"
        ::"r"(smem_addr), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w), "r"(c.x), "r"(c.y),
          "r"(c.z), "r"(c.w), "r"(plane), "r"(static_cast<uint32_t>(on))
        : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t smem_addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(smem_addr)
                 : "memory");
    return v;
}

// Generic vector fetch for ragged edges and bases that are not 16-byte aligned: element-sized
// loads of the elements that exist, zero fill for the rest. `base` points at the tensor start,
// `byte_off` is the vector's offset in it, `nbytes` the tensor's size in bytes.
template <int ESZ>
__device__ __forceinline__ uint4 load_vec_generic(const unsigned char* base, uint64_t byte_off, uint64_t nbytes) {
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (ESZ == 2) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint64_t o = byte_off + 2u * e;
            if (o < nbytes) {
                const uint32_t x = *reinterpret_cast<const unsigned short*>(base + o);
                w[e >> 1] |= x << (16 * (e & 1));
            }
        }
    } else if (ESZ == 4) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint64_t o = byte_off + 4u * e;
            if (o < nbytes) w[e] = *reinterpret_cast<const uint32_t*>(base + o);
        }
    } else {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const uint64_t o = byte_off + 8u * e;
            if (o < nbytes) {
                const uint64_t x = *reinterpret_cast<const unsigned long long*>(base + o);
                w[2 * e] = static_cast<uint32_t>(x);
                w[2 * e + 1] = static_cast<uint32_t>(x >> 32);
            }
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// ------------------------------------------------------------------------------------------
// widening of 16-byte vectors to binary32 (exact)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float f16_to_f32(uint32_t h16) {
    float f;
    asm("{ .reg .b16 t; cvt.u16.u32 t, %1; cvt.f32.f16 %0, t; }" : "=f"(f) : "r"(h16));
    return f;
}

template <int DT> struct Widen;
template <> struct Widen<GV_F32> {
    static constexpr int EPV = 4;
    static __device__ __forceinline__ void run(const uint4& v, float (&o)[4]) {
        o[0] = __uint_as_float(v.x); o[1] = __uint_as_float(v.y);
        o[2] = __uint_as_float(v.z); o[3] = __uint_as_float(v.w);
    }
};
template <> struct Widen<GV_BF16> {
    static constexpr int EPV = 8;
    static __device__ __forceinline__ void run(const uint4& v, float (&o)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            o[2 * i] = __uint_as_float(w[i] << 16);
            o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};
template <> struct Widen<GV_F16> {
    static constexpr int EPV = 8;
    static __device__ __forceinline__ void run(const uint4& v, float (&o)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            o[2 * i] = f16_to_f32(w[i] & 0xFFFFu);
            o[2 * i + 1] = f16_to_f32(w[i] >> 16);
        }
    }
};

// |fl32(c_e - r_e)| for the elements of a candidate vector against an already widened reference vector.
// For the 16-bit types the subtraction takes the candidate element as it is: sm_100's mixed-precision
// subtract (sub.rn.f32.f16 / .bf16: the 16-bit operand is converted exactly, then one correctly rounded
// binary32 subtraction, subnormals kept) does in one instruction what "widen, then subtract" does in two
// or three -- the same value, bit for bit.
template <int DT> struct AbsDiff;
template <> struct AbsDiff<GV_F32> {
    static __device__ __forceinline__ void run(const uint4& c, const float (&rf)[4], float (&ad)[4]) {
        ad[0] = fabsf(__fsub_rn(__uint_as_float(c.x), rf[0])); ad[1] = fabsf(__fsub_rn(__uint_as_float(c.y), rf[1]));
        ad[2] = fabsf(__fsub_rn(__uint_as_float(c.z), rf[2])); ad[3] = fabsf(__fsub_rn(__uint_as_float(c.w), rf[3]));
    }
};
template <> struct AbsDiff<GV_BF16> {
    static __device__ __forceinline__ void run(const uint4& c, const float (&rf)[8], float (&ad)[8]) {
        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float d0, d1;
            asm("{ .reg .b16 lo, hi;\n\t mov.b32 {lo, hi}, %2;\n\t sub.rn.f32.bf16 %0, lo, %3;\n\t sub.rn.f32.bf16 %1, hi, %4; }"
                : "=f"(d0), "=f"(d1) : "r"(w[i]), "f"(rf[2 * i]), "f"(rf[2 * i + 1]));
            ad[2 * i] = fabsf(d0);
            ad[2 * i + 1] = fabsf(d1);
        }
    }
};
template <> struct AbsDiff<GV_F16> {
    static __device__ __forceinline__ void run(const uint4& c, const float (&rf)[8], float (&ad)[8]) {
        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float d0, d1;
            asm("{ .reg .b16 lo, hi;\n\t mov.b32 {lo, hi}, %2;\n\t sub.rn.f32.f16 %0, lo, %3;\n\t sub.rn.f32.f16 %1, hi, %4; }"
                : "=f"(d0), "=f"(d1) : "r"(w[i]), "f"(rf[2 * i]), "f"(rf[2 * i + 1]));
            ad[2 * i] = fabsf(d0);
            ad[2 * i + 1] = fabsf(d1);
        }
    }
};

// ------------------------------------------------------------------------------------------
// per-thread partial statistics of one candidate visit
// ------------------------------------------------------------------------------------------
struct Acc {
    uint64_t hash;
    uint64_t first;      // smallest mismatching element index seen (tensor-relative)
    uint64_t maxint;     // integer dtypes
    uint32_t cnt;        // mismatches
    uint32_t nan;        // NaN disagreements
    uint32_t inf;        // Inf disagreements
    uint32_t maxabs;     // bit pattern of a non-negative float
    uint32_t maxrel;     // bit pattern of a non-negative float
    __device__ __forceinline__ void clear() {
        hash = 0; first = ~0ull; maxint = 0; cnt = 0; nan = 0; inf = 0; maxabs = 0; maxrel = 0;
    }
};

// Per-candidate accumulators of one CTA (shared memory). Rare quantities are updated with
// shared-memory atomics from the compare path; the common ones once per flush.
// (16-byte aligned: {maxabs, maxrel, thr, pad} is read with one 128-bit shared load)
struct __align__(16) CtaAcc {
    unsigned long long hash, cnt, first, nan, inf, maxint;
    unsigned int maxabs, maxrel;
    unsigned int thr;      // relative-error filter threshold derived from maxrel (see rel_threshold_bits)
    unsigned int pad;
    unsigned int pad2[2];
    __device__ __forceinline__ void clear() {
        hash = 0; cnt = 0; first = ~0ull; nan = 0; inf = 0; maxint = 0; maxabs = 0; maxrel = 0; thr = 0; pad = 0;
        pad2[0] = 0; pad2[1] = 0;
    }
};

struct TolF {
    float atol, rtol;
    int equal_nan;
};

__device__ __forceinline__ bool is_nan_bits(uint32_t b) { return (b & 0x7FFFFFFFu) > 0x7F800000u; }
__device__ __forceinline__ bool is_inf_bits(uint32_t b) { return (b & 0x7FFFFFFFu) == 0x7F800000u; }
__device__ __forceinline__ bool is_finite_bits(uint32_t b) { return (b & 0x7F800000u) != 0x7F800000u; }

// The per-element rule, written out once, exactly as the header states it. Used for every
// element on the general path and for the elements of vectors the fast path cannot settle.
// 2^-50 as binary32 bits: below this magnitude a reference element (or a running maximum) is "tiny"
// and the cheap relative-error filter is not trusted (see rel_threshold_bits).
constexpr uint32_t kTinyBits = 0x26800000u;

// GUARDED: the exact quotient is only needed when it can exceed the running maximum M. Callers that
// hold a threshold from rel_threshold_bits (T = M, or 0 while M is tiny) pass it, and the
// division is skipped for elements with |d| <= T |r| (sign of one fused multiply-add).
template <bool GUARDED>
__device__ __forceinline__ void element_rule(float c, float r, const TolF& t, uint64_t idx, Acc& a,
                                             uint32_t thr_bits = 0u) {
    const uint32_t cb = __float_as_uint(c), rb = __float_as_uint(r);
    const float d = __fsub_rn(c, r);
    const float ad = fabsf(d);
    const float tol = __fadd_rn(t.atol, __fmul_rn(t.rtol, fabsf(r)));
    const bool cn = is_nan_bits(cb), rn = is_nan_bits(rb);
    bool close = (c == r);
    close = close || (t.equal_nan && cn && rn);
    close = close || (ad < __uint_as_float(0x7F800000u) && ad <= tol);
    if (!close) {
        a.cnt += 1;
        a.first = idx < a.first ? idx : a.first;
    }
    a.nan += (cn != rn) ? 1u : 0u;
    const bool ci = is_inf_bits(cb), ri = is_inf_bits(rb);
    // classes differ unless both are non-infinite or both are the same infinity
    a.inf += ((ci != ri) || (ci && ri && cb != rb)) ? 1u : 0u;
    if (is_finite_bits(cb) && is_finite_bits(rb)) {
        const uint32_t adb = __float_as_uint(ad);          // ad >= +0, possibly +Inf by overflow
        a.maxabs = adb > a.maxabs ? adb : a.maxabs;
        const uint32_t rab = rb & 0x7FFFFFFFu;
        if (rab != 0u) {
            bool need = true;
            if (GUARDED && thr_bits != 0u && rab >= kTinyBits)
                need = __fmaf_rn(-__uint_as_float(thr_bits), fabsf(r), ad) > 0.0f;
            if (need) {
                const uint32_t qe = __float_as_uint(__fdiv_rn(ad, fabsf(r)));
                a.maxrel = qe > a.maxrel ? qe : a.maxrel;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// fast path for full, aligned vectors of float dtypes
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float max3_nan(float a, float b, float c) {     // NaN if any input is NaN
    float d;
    asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float max2_nan(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// Values derived from one reference vector, computed once per tile and reused for every
// candidate of the chunk.
//   rf      reference widened to binary32
//   tolmin  the smallest tolc = min(tol, FLT_MAX) of the vector, tol = fl(atol + fl(rtol*|r|)):
//           max |d| <= tolmin settles "every element is close" with one comparison
template <int EPV>
struct RefVec {
    float rf[EPV];
    float tolmin;
};

// tolc of one element, as the rule defines it (two roundings, then the clamp that encodes |d| < Inf)
__device__ __forceinline__ float tolc_of(float abs_r, const TolF& t) {
    return fminf(__fadd_rn(t.atol, __fmul_rn(t.rtol, abs_r)), __uint_as_float(0x7F7FFFFFu));
}

// flags: bit 1 = the vector holds a nonzero element below 2^-50 (relative filter not trusted)
template <int DT>
__device__ __forceinline__ void hoist_ref(const uint4& raw, const TolF& t, RefVec<16 / Traits<DT>::ESZ>& o,
                                          uint32_t& flags) {
    constexpr int EPV = 16 / Traits<DT>::ESZ;
    Widen<DT>::run(raw, o.rf);
    // tol is a monotone function of |r| (two correctly rounded monotone steps), so the smallest tol of
    // the vector is the tol of its smallest |r|. fminf skips NaNs: a NaN element makes d NaN anyway.
    float amin = __uint_as_float(0x7F800000u);
#pragma unroll
    for (int e = 0; e < EPV; ++e) amin = fminf(amin, fabsf(o.rf[e]));
    o.tolmin = tolc_of(amin, t);
    // A nonzero element below 2^-50 can only exist when the smallest |r| is below 2^-50 (it may be a
    // zero, so look at the elements then; f16 has no nonzero value that small).
    flags = 0u;
    if (DT != GV_F16 && __float_as_uint(amin) < kTinyBits) {
        uint32_t umin1 = 0xFFFFFFFFu;
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            const uint32_t u1 = (__float_as_uint(o.rf[e]) & 0x7FFFFFFFu) - 1u;   // zero wraps to the top: ignored
            umin1 = u1 < umin1 ? u1 : umin1;
        }
        flags = (umin1 < kTinyBits - 1u) ? 2u : 0u;
    }
}

// Relative-error filter of one (CTA, candidate). M = largest quotient fl(|d| / |r|) recorded so far; the
// threshold T is M itself, or 0 while M < 2^-50. Rounding is monotone and M is a binary32 value, so an
// element can raise M only if the real quotient exceeds M, i.e. x = |d| - M |r| > 0. The fused
// multiply-add w = fma(-T, |r|, |d|) rounds that exact x once, which keeps its sign unless a nonzero x
// rounds to zero; with M >= 2^-50 and |r| >= 2^-50 the product M |r| is a multiple of 2^-146 and |d| one
// of 2^-149, so a positive x is at least 2^-149 and stays positive: w > 0 exactly when the quotient
// exceeds M. Elements whose quotient only ties with M -- every element of a candidate of zeros, of a
// negated or a scaled one, and the usual case in quantised noise -- therefore stop at the filter.
// Vectors holding a nonzero |r| < 2^-50 skip the filter (flag from hoist_ref), and while T == 0 every
// nonzero |d| passes (w = |d|). When M |r| overflows the quotient is below M and w is -Inf. Elements
// with r == 0 pass whenever |d| != 0 and are dropped afterwards (no relative error).
__device__ __forceinline__ uint32_t rel_threshold_bits(uint32_t m_bits) {
    return m_bits < kTinyBits ? 0u : m_bits;
}

// Add a 32-bit count to a 64-bit counter in shared memory. A 64-bit atomic add on shared memory behaves
// like a compare-and-swap loop: when the lanes of a warp add to the same counter (a batch of entries of
// one candidate that mismatch everywhere) its cost grows with the number of lanes that collide (measured:
// shared-memory stalls dominated such launches); the 32-bit add resolves the conflict in hardware. The carry into the upper word is added separately (exact:
// the sum wraps mod 2^64, and nothing reads the counter before the CTA's final barrier).
__device__ __forceinline__ void add_count(unsigned long long* counter, uint32_t v) {
    uint32_t* w = reinterpret_cast<uint32_t*>(counter);
    const uint32_t old = atomicAdd(w, v);
    if (old + v < old) atomicAdd(w + 1, 1u);
}

// Raise the CTA's running maxima (bit patterns of non-negative floats).
__device__ __forceinline__ void raise_maxabs(CtaAcc* s, uint32_t bits) {
    if (bits > *reinterpret_cast<volatile unsigned int*>(&s->maxabs)) {
        atomicMax(&s->maxabs, bits);
    }
}
__device__ __forceinline__ void raise_maxrel(CtaAcc* s, uint32_t bits) {
    if (bits > *reinterpret_cast<volatile unsigned int*>(&s->maxrel)) {
        atomicMax(&s->maxrel, bits);
        atomicMax(&s->thr, rel_threshold_bits(bits));
    }
}

// One element that passed the relative-error filter (out of line: the hot loop only tests and calls).
// First decides exactly, without dividing, whether the real quotient |d| / |r| exceeds M:
// |d| > M |r|  <=>  |d| - p > e  with p = fl(M |r|) and e = M |r| - p, the exact rounding error of the
// product, delivered by one fused multiply-add. Elements that only tie with M -- the norm in
// quantised data -- stop there: rounding is monotone, so a real quotient <= M cannot round above M.
// Returns the bits of the IEEE quotient, or 0 when it cannot raise M. thr_bits == 0: M unknown/tiny.
__device__ __noinline__ uint32_t rel_candidate_bits(float ad, float ar, float M, uint32_t thr_bits) {
    if (ar == 0.0f) return 0u;                              // r == 0: no relative error
    if (thr_bits != 0u) {
        const float pm = __fmul_rn(M, ar);
        if (__float_as_uint(pm) >= 0x0D800000u && __float_as_uint(pm) < 0x7F800000u) {   // 2^-100 <= p < Inf: e is exact
            const float err = __fmaf_rn(M, ar, -pm);
            if (!(__fsub_rn(ad, pm) > err)) return 0u;
        }
    }
    return __float_as_uint(__fdiv_rn(ad, ar));
}

// Compare one full vector on the fast path. Returns true when the vector is settled here: every pair
// is a finite pair (both values finite, |d| finite). Close elements only feed the maxima; elements
// that are not close are counted (a finite pair is close exactly when |d| <= tolc) and the first
// index is merged. Max |d| and, for the elements whose estimate passes the filter, the exact relative
// error go to the CTA accumulators. Returns false when a NaN or an infinity is involved: the caller
// then runs the exact per-element rule on this vector (nothing has been recorded in that case).
// n_not_close: the number of elements found not close is ADDED to this per-lane counter; the caller
// merges it into the accumulator at a point where the whole warp is converged (one reduction and one
// atomic per warp) -- inside this function the set of lanes present is not known reliably.
// ADD_NOW: add the count to the accumulator at once (callers whose lanes each work for their own
// candidate) instead of returning it in n_not_close.
template <int DT, bool ADD_NOW = false, bool REL_OK = ADD_NOW>
__device__ __forceinline__ bool vec_fast_float(const uint4& c, const RefVec<16 / Traits<DT>::ESZ>& r, uint32_t flags,
                                               const TolF& t, CtaAcc* s, uint64_t elem0, uint32_t& n_not_close) {
    constexpr int EPV = 16 / Traits<DT>::ESZ;
    // running maxima of this (CTA, candidate): max|d| bits, max relative error bits, filter threshold
    const uint4 run = lds128(smem_u32(&s->maxabs));
    const float nT = -__uint_as_float(run.z);
    float ad[EPV], w[EPV];
    AbsDiff<DT>::run(c, r.rf, ad);
#pragma unroll
    for (int e = 0; e < EPV; ++e) w[e] = __fmaf_rn(nT, fabsf(r.rf[e]), ad[e]);         // > 0  <=  the quotient could exceed M
    float va, vw;       // va propagates NaN: a NaN anywhere (candidate or reference) must not be skipped
    if (EPV == 8) {
        va = max2_nan(max3_nan(ad[0], ad[1], ad[2]), max3_nan(max3_nan(ad[3], ad[4], ad[5]), ad[6], ad[7]));
        vw = fmaxf(max3(w[0], w[1], w[2]), max3(max3(w[3], w[4], w[5]), w[6], w[7]));
    } else {
        va = max2_nan(max3_nan(ad[0], ad[1], ad[2]), ad[3]);
        vw = fmaxf(max3(w[0], w[1], w[2]), w[3]);
    }
    const uint32_t vab = __float_as_uint(va);
    // Common case: every element within the smallest tolerance, no running maximum raised -> one test.
    // Second way to "all close": while the running maximum M of |d| / |r| (the filter's T) is at most rtol,
    // an element with |d| <= T |r| (w <= 0; the sign is exact for the magnitudes the filter trusts) has
    // |d| <= rtol |r|, hence |d| <= fl(rtol |r|) <= fl(atol + fl(rtol |r|)) = tol, rounding being monotone
    // and |d| a binary32 value. So when no element of the vector exceeds M (vw <= 0) and all |d| are
    // finite, every element is close whatever the smallest tolerance of the vector says: with an
    // essentially relative tolerance (atol << rtol |r|) the vector's largest |d| sits on a large element
    // and exceeds the tolerance of its smallest one all the time. (REL_OK: the callers with one lane per
    // entry always; the in-place loop of the dense kernel, where the two extra instructions cost 3-4 % on
    // data that does not need them, in the instance the host picks when atol is far below rtol.)
    const float lim = (REL_OK && run.z <= __float_as_uint(t.rtol)) ? __uint_as_float(0x7F7FFFFFu) : r.tolmin;
    const bool raise_abs = vab > run.x;
    const bool maybe_rel = vw > 0.0f || ((flags & 2u) && vab != 0u);
    if (va <= lim && !(raise_abs || maybe_rel)) return true;
    const bool over_tol = !(va <= ((maybe_rel || (flags & 2u)) ? r.tolmin : lim));
    if (over_tol) {
        // Some |d| exceeds the smallest tolerance of the vector, or a NaN is present. NaN or Inf:
        // the caller runs the exact rule. Otherwise every pair is finite and an element is close
        // exactly when |d| <= its own tolc.
        if (va != va || vab >= 0x7F800000u) return false;
        // (every |d| is finite here, so the clamp of tolc_of is not needed: |d| > tol is false for tol = +Inf)
        uint32_t bad = 0u;
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            if (ad[e] > __fadd_rn(t.atol, __fmul_rn(t.rtol, fabsf(r.rf[e])))) bad |= 1u << e;
        }
        if (bad) {
            const uint32_t cnt = static_cast<uint32_t>(__popc(bad));
            if (ADD_NOW) add_count(&s->cnt, cnt);
            else n_not_close += cnt;
            const unsigned long long idx = elem0 + static_cast<uint32_t>(__ffs(bad) - 1);
            if (idx < *reinterpret_cast<volatile unsigned long long*>(&s->first)) atomicMin(&s->first, idx);
        }
    }
    if (raise_abs) raise_maxabs(s, vab);
    if (maybe_rel) {
        // some element may raise the relative maximum M: each one that passes the filter is examined
        const float M = __uint_as_float(run.y);
        uint32_t best = 0u;
        // A quotient above M still rounds to M unless it reaches M + half an ulp, i.e. |d| - M |r| >= half |r|
        // (w is monotone in that difference and half |r| is exact). Without this test the elements of a
        // quantised candidate whose quotient lies just above the maximum it rounds to would divide every time.
        const float half = (run.z != 0u && run.z < 0x7F800000u) ? __uint_as_float(((run.z >> 23) - 24u) << 23) : 0.0f;
        if constexpr (ADD_NOW) {
        // (callers with one lane per entry: one call site for all elements keeps the batch function short)
        uint32_t pass = 0u;
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            if ((w[e] > 0.0f && w[e] >= __fmul_rn(half, fabsf(r.rf[e]))) || ((flags & 2u) && ad[e] != 0.0f)) pass |= 1u << e;
        }
        while (pass) {                                  // one call site for all elements
            const int e = __ffs(pass) - 1;
            pass &= pass - 1u;
            float ade = ad[0], are = r.rf[0];
#pragma unroll
            for (int k = 1; k < EPV; ++k) {
                if (e == k) { ade = ad[k]; are = r.rf[k]; }
            }
            const uint32_t qe = rel_candidate_bits(ade, fabsf(are), M, run.z);
            best = qe > best ? qe : best;
        }
        } else {
#pragma unroll
        for (int e = 0; e < EPV; ++e) {
            if ((w[e] > 0.0f && w[e] >= __fmul_rn(half, fabsf(r.rf[e]))) || ((flags & 2u) && ad[e] != 0.0f)) {
                const uint32_t qe = rel_candidate_bits(ad[e], fabsf(r.rf[e]), M, run.z);
                best = qe > best ? qe : best;
            }
        }
        }
        if (best > run.y) raise_maxrel(s, best);
    }
    return true;
}

// Exact per-element rule over a full vector, using the hoisted reference values (the path taken
// by vectors the fast path could not settle).
template <int DT>
__device__ __forceinline__ void vec_exact_float(const uint4& c, const RefVec<16 / Traits<DT>::ESZ>& r,
                                                uint64_t elem0, const TolF& t, uint32_t thr_bits, Acc& a) {
    constexpr int EPV = 16 / Traits<DT>::ESZ;
    float cf[EPV];
    Widen<DT>::run(c, cf);
#pragma unroll
    for (int e = 0; e < EPV; ++e) element_rule<true>(cf[e], r.rf[e], t, elem0 + e, a, thr_bits);
}

// One 16-byte vector of a float dtype, general path: every element through the rule.
// nvalid = number of elements of the vector that exist (EPV for a full vector).
template <int DT>
__device__ __forceinline__ void vec_general_float(const uint4& c, const uint4& r, uint64_t elem0, int nvalid,
                                                  const TolF& t, Acc& a) {
    constexpr int EPV = Widen<DT>::EPV;
    float cf[EPV], rf[EPV];
    Widen<DT>::run(c, cf);
    Widen<DT>::run(r, rf);
#pragma unroll
    for (int e = 0; e < EPV; ++e) {
        if (e < nvalid) element_rule<false>(cf[e], rf[e], t, elem0 + e, a);
    }
}

// One 16-byte vector of an integer dtype: exact equality, exact |c - r|.
template <int DT>
__device__ __forceinline__ void vec_int(const uint4& c, const uint4& r, uint64_t elem0, int nvalid, Acc& a) {
    if (((c.x ^ r.x) | (c.y ^ r.y) | (c.z ^ r.z) | (c.w ^ r.w)) == 0u) return;   // identical vector
    if (DT == GV_I32) {
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (e < nvalid && cw[e] != rw[e]) {
                const int64_t cv = static_cast<int32_t>(cw[e]), rv = static_cast<int32_t>(rw[e]);
                const uint64_t diff = cv > rv ? static_cast<uint64_t>(cv - rv) : static_cast<uint64_t>(rv - cv);
                a.cnt += 1;
                a.first = (elem0 + e) < a.first ? (elem0 + e) : a.first;
                a.maxint = diff > a.maxint ? diff : a.maxint;
            }
        }
    } else {
        const uint64_t cw[2] = {pack64(c.x, c.y), pack64(c.z, c.w)}, rw[2] = {pack64(r.x, r.y), pack64(r.z, r.w)};
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            if (e < nvalid && cw[e] != rw[e]) {
                const int64_t cv = static_cast<int64_t>(cw[e]), rv = static_cast<int64_t>(rw[e]);
                const uint64_t diff = cv > rv ? cw[e] - rw[e] : rw[e] - cw[e];      // exact mod 2^64
                a.cnt += 1;
                a.first = (elem0 + e) < a.first ? (elem0 + e) : a.first;
                a.maxint = diff > a.maxint ? diff : a.maxint;
            }
        }
    }
}

template <int DT>
__device__ __forceinline__ void vec_compare(const uint4& c, const uint4& r, uint64_t elem0, int nvalid,
                                            const TolF& t, Acc& a) {
    if constexpr (Traits<DT>::IS_FLOAT) vec_general_float<DT>(c, r, elem0, nvalid, t, a);
    else vec_int<DT>(c, r, elem0, nvalid, a);
}

// ------------------------------------------------------------------------------------------
// mbarrier + bulk async copy (TMA, 1-D, this CTA's shared memory only)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// orders this thread's earlier ordinary shared-memory accesses before later async-proxy ones
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// global -> this CTA's shared memory; bytes and both addresses multiples of 16
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kWaitHintNs)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false when the limit is reached (the caller flags a timeout and leaves).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit = kWaitLimit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}

// ------------------------------------------------------------------------------------------
// warp / block combines (all on integers, so any order gives the same bytes)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t warp_sum_u64(uint64_t v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ uint64_t warp_min_u64(uint64_t v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t x = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = x < v ? x : v;
    }
    return v;
}
__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t x = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = x > v ? x : v;
    }
    return v;
}

// Merge per-lane mismatch counts at a point where all 32 lanes of the warp are converged.
__device__ __forceinline__ void merge_counts_converged(CtaAcc* s, uint32_t lane_cnt) {
    const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, lane_cnt);
    if (total && (threadIdx.x & 31) == 0) add_count(&s->cnt, total);
}

// Rare-path partials of one thread's visit -> CTA accumulators.
// (Reads before the atomics keep hot addresses quiet: a value that cannot change the
// accumulator is dropped without an atomic.)
__device__ __forceinline__ void push_rare(CtaAcc* s, const Acc& a) {
    if (a.cnt && a.first < *reinterpret_cast<volatile unsigned long long*>(&s->first))
        atomicMin(&s->first, static_cast<unsigned long long>(a.first));
    if (a.nan) add_count(&s->nan, a.nan);
    if (a.inf) add_count(&s->inf, a.inf);
    if (a.maxint > *reinterpret_cast<volatile unsigned long long*>(&s->maxint))
        atomicMax(&s->maxint, static_cast<unsigned long long>(a.maxint));
    raise_maxrel(s, a.maxrel);
}

// CTA accumulators -> result record in global memory (skips identities).
__device__ __forceinline__ void push_global(gv_result* res, const CtaAcc& s) {
    if (s.cnt) atomicAdd(reinterpret_cast<unsigned long long*>(&res->n_mismatch), s.cnt);
    if (s.first != ~0ull) atomicMin(reinterpret_cast<unsigned long long*>(&res->first_mismatch), s.first);
    if (s.nan) atomicAdd(reinterpret_cast<unsigned long long*>(&res->n_nan_disagree), s.nan);
    if (s.inf) atomicAdd(reinterpret_cast<unsigned long long*>(&res->n_inf_disagree), s.inf);
    if (s.hash) atomicAdd(reinterpret_cast<unsigned long long*>(&res->hash), s.hash);
    if (s.maxint) atomicMax(reinterpret_cast<unsigned long long*>(&res->max_abs_diff_int), s.maxint);
    if (s.maxabs) atomicMax(reinterpret_cast<unsigned int*>(&res->max_abs_err), s.maxabs);
    if (s.maxrel) atomicMax(reinterpret_cast<unsigned int*>(&res->max_rel_err), s.maxrel);
}

static_assert(sizeof(CtaAcc) % 16 == 0 && offsetof(CtaAcc, maxabs) % 16 == 0, "CtaAcc layout");

}  // namespace gv
