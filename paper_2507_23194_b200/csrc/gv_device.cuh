// gv_device.cuh -- device-side building blocks of the output verifier (sm_100a).
//
// Everything here follows the per-element rule and the content hash stated in include/gv.h
// (the tolerance-based comparison of Section 3.1 of the GEAK paper). Float arithmetic on the
// compare path uses the explicitly rounded intrinsics so that no compiler flag can contract it
// into a fused multiply-add or flush subnormals.
#pragma once

#include <cuda_runtime.h>
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

// ------------------------------------------------------------------------------------------
// content hash
// ------------------------------------------------------------------------------------------
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

struct TolF {
    float atol, rtol;
    int equal_nan;
};

__device__ __forceinline__ bool is_nan_bits(uint32_t b) { return (b & 0x7FFFFFFFu) > 0x7F800000u; }
__device__ __forceinline__ bool is_inf_bits(uint32_t b) { return (b & 0x7FFFFFFFu) == 0x7F800000u; }
__device__ __forceinline__ bool is_finite_bits(uint32_t b) { return (b & 0x7F800000u) != 0x7F800000u; }

// The per-element rule, written out once, exactly as the header states it. Used for every
// element on the general path and for the elements of vectors the fast path cannot settle.
__device__ __forceinline__ void element_rule(float c, float r, const TolF& t, uint64_t idx, Acc& a) {
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
        if ((rb & 0x7FFFFFFFu) != 0u) {
            const uint32_t q = __float_as_uint(__fdiv_rn(ad, fabsf(r)));
            a.maxrel = q > a.maxrel ? q : a.maxrel;
        }
    }
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
        if (e < nvalid) element_rule(cf[e], rf[e], t, elem0 + e, a);
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
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
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
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
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

// Per-candidate accumulators of one CTA (shared memory). Rare quantities are updated with
// shared-memory atomics from the compare path; the common ones once per flush.
struct CtaAcc {
    unsigned long long hash, cnt, first, nan, inf, maxint;
    unsigned int maxabs, maxrel;
    __device__ __forceinline__ void clear() {
        hash = 0; cnt = 0; first = ~0ull; nan = 0; inf = 0; maxint = 0; maxabs = 0; maxrel = 0;
    }
};

// Rare-path partials of one thread's visit -> CTA accumulators.
__device__ __forceinline__ void push_rare(CtaAcc* s, const Acc& a) {
    if (a.cnt) atomicMin(&s->first, static_cast<unsigned long long>(a.first));
    if (a.nan) atomicAdd(&s->nan, static_cast<unsigned long long>(a.nan));
    if (a.inf) atomicAdd(&s->inf, static_cast<unsigned long long>(a.inf));
    if (a.maxint) atomicMax(&s->maxint, static_cast<unsigned long long>(a.maxint));
    if (a.maxrel) atomicMax(&s->maxrel, a.maxrel);
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

}  // namespace gv
