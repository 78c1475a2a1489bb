// Error profile of one candidate against the reference: device code.
//
// What an Evaluator can hand to the Reflector when the functionality test fails (paper Sections
// 4.1 and 4.2: the error trace of a failing run is fed back): a histogram of the distance between
// candidate and reference in units of the dtype's own spacing, the mismatching element with the
// largest error, the first eight mismatching elements and, optionally, mismatch counts per row.
// It runs on demand over the few candidates that failed, as a pass of its own, so the verifier's
// hot loop carries none of it. One cooperative launch: the grid clears the outputs, synchronises,
// streams both tensors once (every byte read once, 128-bit loads) into per-warp / per-CTA partials,
// synchronises again, and its first CTA finalises; all results are exact integers or bit patterns
// and do not depend on scheduling.
#pragma once
#include <cooperative_groups.h>
#include <stdint.h>

#include "gv.h"
#include "gv_device.cuh"

namespace gv {

constexpr int kProfileThreads = 256;
constexpr int kProfileWarps = kProfileThreads / 32;
constexpr int kProfileMaxCtas = 2048;

struct ProfileWorst {              // per-CTA partial: the worst mismatching element it met
    unsigned long long key;        // error used for ranking (see profile_element)
    unsigned long long index;      // all ones: none
    unsigned long long c_raw, r_raw;
};

struct ProfileParams {
    const unsigned char* ref;
    const unsigned char* cand;
    uint64_t n;
    float atol, rtol;
    int equal_nan;
    int aligned;                   // both bases 16-byte aligned
    uint64_t row_len;              // 0: no per-row counts
    gv_profile* out;
    uint32_t* rows;
    ProfileWorst* cta_worst;       // [gridDim.x]
    unsigned long long* cta_first;   // [gridDim.x][GV_PROFILE_LIST]: the CTA's smallest mismatching indices, all ones = unused
};

// bucket of a distance: 0 for 0, else 1 + floor(log2 distance)
__device__ __forceinline__ int profile_bucket(uint64_t dist) { return dist ? 64 - __clzll(static_cast<long long>(dist)) : 0; }

// One element: raw bits (zero-extended) of candidate and reference -> close?, ranking key, bucket.
template <int DT>
__device__ __forceinline__ void profile_element(uint64_t c_raw, uint64_t r_raw, const TolF& t, bool& close, uint64_t& key,
                                                int& bucket) {
    if constexpr (!Traits<DT>::IS_FLOAT) {
        const int64_t c = DT == GV_I32 ? static_cast<int64_t>(static_cast<int32_t>(c_raw)) : static_cast<int64_t>(c_raw);
        const int64_t r = DT == GV_I32 ? static_cast<int64_t>(static_cast<int32_t>(r_raw)) : static_cast<int64_t>(r_raw);
        const uint64_t diff = c > r ? static_cast<uint64_t>(c) - static_cast<uint64_t>(r)
                                    : static_cast<uint64_t>(r) - static_cast<uint64_t>(c);
        close = c == r;
        key = diff;
        bucket = profile_bucket(diff);
    } else {
        constexpr int W = Traits<DT>::ESZ * 8;
        float c, r;
        if constexpr (DT == GV_F32) {
            c = __uint_as_float(static_cast<uint32_t>(c_raw));
            r = __uint_as_float(static_cast<uint32_t>(r_raw));
        } else if constexpr (DT == GV_BF16) {
            c = __uint_as_float(static_cast<uint32_t>(c_raw) << 16);
            r = __uint_as_float(static_cast<uint32_t>(r_raw) << 16);
        } else {
            c = f16_to_f32(static_cast<uint32_t>(c_raw));
            r = f16_to_f32(static_cast<uint32_t>(r_raw));
        }
        const float ad = fabsf(__fsub_rn(c, r));
        const float tol = __fadd_rn(t.atol, __fmul_rn(t.rtol, fabsf(r)));
        const bool cn = is_nan_bits(__float_as_uint(c)), rn = is_nan_bits(__float_as_uint(r));
        close = (c == r) || (t.equal_nan && cn && rn) || (ad < __uint_as_float(0x7F800000u) && ad <= tol);
        const uint32_t adb = __float_as_uint(ad);
        key = is_nan_bits(adb) ? 0xFFFFFFFFull : static_cast<uint64_t>(adb);
        if (cn || rn) {
            bucket = GV_PROFILE_BUCKETS - 1;
        } else {
            constexpr uint64_t kSign = 1ull << (W - 1);
            const int64_t oc = (c_raw & kSign) ? -static_cast<int64_t>(c_raw & (kSign - 1)) : static_cast<int64_t>(c_raw);
            const int64_t orf = (r_raw & kSign) ? -static_cast<int64_t>(r_raw & (kSign - 1)) : static_cast<int64_t>(r_raw);
            bucket = profile_bucket(static_cast<uint64_t>(oc > orf ? oc - orf : orf - oc));
        }
    }
}

template <int ESZ>
__device__ __forceinline__ uint64_t profile_raw(const uint4& v, int e) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (ESZ == 2) return (w[e >> 1] >> (16 * (e & 1))) & 0xFFFFu;
    if (ESZ == 4) return w[e];
    return static_cast<uint64_t>(w[2 * e + 1]) << 32 | w[2 * e];
}

// "a ranks before b": larger key, then smaller index
__device__ __forceinline__ bool profile_better(uint64_t ka, uint64_t ia, uint64_t kb, uint64_t ib) {
    return ib == ~0ull ? ia != ~0ull : (ia != ~0ull && (ka > kb || (ka == kb && ia < ib)));
}

template <int DT>
__device__ __forceinline__ void profile_finalize(const ProfileParams& p, unsigned int n_ctas);

// Launched cooperatively (all CTAs resident), because the outputs the grid accumulates into with atomics
// are cleared by the grid itself first, and the finalisation needs every CTA's partials.
template <int DT>
__global__ void __launch_bounds__(kProfileThreads) profile_kernel(ProfileParams p) {
    constexpr int ESZ = Traits<DT>::ESZ;
    constexpr int EPV = 16 / ESZ;
    cooperative_groups::grid_group grid = cooperative_groups::this_grid();
    {
        // clear what the atomics below add to: the whole output record and, if asked for, the row counts
        const uint64_t gtid = blockIdx.x * static_cast<uint64_t>(kProfileThreads) + threadIdx.x;
        const uint64_t gsize = static_cast<uint64_t>(gridDim.x) * kProfileThreads;
        unsigned long long* o = reinterpret_cast<unsigned long long*>(p.out);
        for (uint64_t i = gtid; i < sizeof(gv_profile) / 8; i += gsize) o[i] = 0ull;
        if (p.row_len) {
            const uint64_t n_rows = (p.n + p.row_len - 1) / p.row_len;
            for (uint64_t i = gtid; i < n_rows; i += gsize) p.rows[i] = 0u;
        }
    }
    grid.sync();
    __shared__ unsigned int s_hist[kProfileWarps][GV_PROFILE_BUCKETS];     // one per warp: fewer same-address collisions
    __shared__ unsigned long long s_first[kProfileWarps][GV_PROFILE_LIST];
    __shared__ ProfileWorst s_worst[kProfileWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int b = tid; b < kProfileWarps * GV_PROFILE_BUCKETS; b += kProfileThreads) (&s_hist[0][0])[b] = 0u;
    if (lane < GV_PROFILE_LIST) s_first[warp][lane] = ~0ull;
    __syncthreads();

    const TolF tol = {p.atol, p.rtol, p.equal_nan};
    const uint64_t nbytes = p.n * ESZ;
    const uint64_t tiles = (nbytes + 511) / 512;
    const uint64_t gw = static_cast<uint64_t>(blockIdx.x) * kProfileWarps + warp;
    const uint64_t GW = static_cast<uint64_t>(gridDim.x) * kProfileWarps;
    unsigned long long zero_cnt = 0, mism_cnt = 0;
    uint64_t best_key = 0, best_idx = ~0ull, best_c = 0, best_r = 0;
    uint32_t wn = 0;                                   // entries in this warp's list of first mismatches (warp-uniform)

    for (uint64_t t = gw; t < tiles; t += GW) {        // a warp meets its tiles in increasing order
        const uint64_t voff = t * 512 + lane * 16;
        const uint64_t rem = voff < nbytes ? nbytes - voff : 0;
        const int nvalid = rem >= 16 ? EPV : static_cast<int>(rem / ESZ);
        uint4 c = make_uint4(0u, 0u, 0u, 0u), r = c;
        if (nvalid == EPV && p.aligned) {
            c = ldg_stream(p.cand + voff);
            r = ldg_stream(p.ref + voff);
        } else if (nvalid > 0) {
            c = load_vec_generic<ESZ>(p.cand, voff, nbytes);
            r = load_vec_generic<ESZ>(p.ref, voff, nbytes);
        }
        const uint64_t elem0 = voff / ESZ;
        uint32_t bad = 0u;                             // bit e: element e of this lane's vector is not close
        const bool same = c.x == r.x && c.y == r.y && c.z == r.z && c.w == r.w;
        bool plain_same = same && nvalid > 0;
        if constexpr (Traits<DT>::IS_FLOAT) {
            // identical bits are distance 0 and close unless a NaN is involved (NaN == NaN only with equal_nan)
            if (plain_same) {
                bool any_nan = false;
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    const uint64_t x = profile_raw<ESZ>(r, e);
                    constexpr uint64_t kAbs = (1ull << (ESZ * 8 - 1)) - 1;
                    constexpr uint64_t kInf = DT == GV_F32 ? 0x7F800000ull : DT == GV_BF16 ? 0x7F80ull : 0x7C00ull;
                    any_nan = any_nan || (x & kAbs) > kInf;
                }
                plain_same = !any_nan;
            }
        }
        if (plain_same) {
            zero_cnt += static_cast<unsigned>(nvalid);
        } else {
#pragma unroll
            for (int e = 0; e < EPV; ++e) {
                if (e < nvalid) {
                    const uint64_t c_raw = profile_raw<ESZ>(c, e), r_raw = profile_raw<ESZ>(r, e);
                    bool close;
                    uint64_t key;
                    int bucket;
                    profile_element<DT>(c_raw, r_raw, tol, close, key, bucket);
                    if (bucket == 0) zero_cnt += 1;
                    else atomicAdd(&s_hist[warp][bucket], 1u);
                    if (!close) {
                        bad |= 1u << e;
                        mism_cnt += 1;
                        if (best_idx == ~0ull || key > best_key) {      // indices only grow: strict > keeps the first
                            best_key = key; best_idx = elem0 + e; best_c = c_raw; best_r = r_raw;
                        }
                    }
                }
            }
        }
        const uint32_t any_bad = __ballot_sync(0xFFFFFFFFu, bad != 0u);
        if (any_bad) {
            if (p.row_len) {
                const uint64_t row_a = elem0 / p.row_len;
                if (bad) {
                    if ((elem0 + EPV - 1) / p.row_len == row_a) {
                        atomicAdd(&p.rows[row_a], static_cast<unsigned>(__popc(bad)));
                    } else {
#pragma unroll
                        for (int e = 0; e < EPV; ++e)
                            if (bad & (1u << e)) atomicAdd(&p.rows[(elem0 + e) / p.row_len], 1u);
                    }
                }
            }
            if (wn < GV_PROFILE_LIST) {
                // position of this lane's mismatches in index order: exclusive prefix of the counts over the lanes
                const uint32_t mine = __popc(bad);
                uint32_t incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += y;
                }
                uint32_t pos = wn + incl - mine;
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    if (bad & (1u << e)) {
                        if (pos < GV_PROFILE_LIST) s_first[warp][pos] = elem0 + e;
                        ++pos;
                    }
                }
                const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
                wn = min(wn + total, static_cast<uint32_t>(GV_PROFILE_LIST));
                __syncwarp();
            }
        }
    }

    // ---- per-CTA combine ----
    zero_cnt = warp_sum_u64(zero_cnt);
    mism_cnt = warp_sum_u64(mism_cnt);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const uint64_t k2 = __shfl_xor_sync(0xFFFFFFFFu, best_key, o), i2 = __shfl_xor_sync(0xFFFFFFFFu, best_idx, o);
        const uint64_t c2 = __shfl_xor_sync(0xFFFFFFFFu, best_c, o), r2 = __shfl_xor_sync(0xFFFFFFFFu, best_r, o);
        if (profile_better(k2, i2, best_key, best_idx)) { best_key = k2; best_idx = i2; best_c = c2; best_r = r2; }
    }
    if (lane == 0) {
        if (zero_cnt) atomicAdd(reinterpret_cast<unsigned long long*>(&p.out->ulp_hist[0]), zero_cnt);
        if (mism_cnt) atomicAdd(reinterpret_cast<unsigned long long*>(&p.out->n_mismatch), mism_cnt);
        s_worst[warp] = {best_key, best_idx, best_c, best_r};
    }
    __syncthreads();
    for (int b = tid; b < GV_PROFILE_BUCKETS; b += kProfileThreads) {
        unsigned long long h = 0;
        for (int i = 0; i < kProfileWarps; ++i) h += s_hist[i][b];
        if (h) atomicAdd(reinterpret_cast<unsigned long long*>(&p.out->ulp_hist[b]), h);
    }
    if (tid == 0) {
        ProfileWorst w = s_worst[0];
        for (int i = 1; i < kProfileWarps; ++i)
            if (profile_better(s_worst[i].key, s_worst[i].index, w.key, w.index)) w = s_worst[i];
        p.cta_worst[blockIdx.x] = w;
    }
    // the CTA's eight smallest mismatching indices out of its warps' lists: warp 0, two entries per lane,
    // eight rounds of a warp-wide minimum above the previous pick
    if (warp == 0) {
        __syncwarp();
        static_assert(kProfileWarps * GV_PROFILE_LIST == 64, "two entries per lane");
        const unsigned long long e0 = s_first[lane >> 3][lane & 7], e1 = s_first[4 + (lane >> 3)][lane & 7];
        unsigned long long last = 0;
        bool have_last = false;
        for (int round = 0; round < GV_PROFILE_LIST; ++round) {
            unsigned long long m = ~0ull;
            if (e0 < m && (!have_last || e0 > last)) m = e0;
            if (e1 < m && (!have_last || e1 > last)) m = e1;
            m = warp_min_u64(m);
            if (lane == 0) p.cta_first[static_cast<size_t>(blockIdx.x) * GV_PROFILE_LIST + round] = m;
            last = m;
            have_last = true;
        }
    }
    grid.sync();
    if (blockIdx.x == 0) profile_finalize<DT>(p, gridDim.x);
}

// One CTA: the worst element over the per-CTA partials, the eight smallest indices over the
// per-CTA lists (eight rounds of a block-wide minimum above the previous pick), and their raw values.
template <int DT>
__device__ __forceinline__ void profile_finalize(const ProfileParams& p, unsigned int n_ctas) {
    constexpr int ESZ = Traits<DT>::ESZ;
    __shared__ ProfileWorst s_w[kProfileWarps];
    __shared__ unsigned long long s_min[kProfileWarps];
    __shared__ unsigned long long s_pick[GV_PROFILE_LIST];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    ProfileWorst w = {0ull, ~0ull, 0ull, 0ull};
    for (unsigned int i = tid; i < n_ctas; i += kProfileThreads) {
        const ProfileWorst x = p.cta_worst[i];
        if (profile_better(x.key, x.index, w.key, w.index)) w = x;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ProfileWorst x;
        x.key = __shfl_xor_sync(0xFFFFFFFFu, w.key, o);
        x.index = __shfl_xor_sync(0xFFFFFFFFu, w.index, o);
        x.c_raw = __shfl_xor_sync(0xFFFFFFFFu, w.c_raw, o);
        x.r_raw = __shfl_xor_sync(0xFFFFFFFFu, w.r_raw, o);
        if (profile_better(x.key, x.index, w.key, w.index)) w = x;
    }
    if (lane == 0) s_w[warp] = w;
    __syncthreads();
    if (tid == 0) {
        for (int i = 1; i < kProfileWarps; ++i)
            if (profile_better(s_w[i].key, s_w[i].index, w.key, w.index)) w = s_w[i];
        p.out->worst_index = w.index;
        p.out->worst_c_raw = w.index == ~0ull ? 0ull : w.c_raw;
        p.out->worst_r_raw = w.index == ~0ull ? 0ull : w.r_raw;
    }
    // each thread keeps the eight smallest of the entries it reads (one pass, independent loads) ...
    const uint64_t entries = static_cast<uint64_t>(n_ctas) * GV_PROFILE_LIST;
    unsigned long long t8[GV_PROFILE_LIST];
#pragma unroll
    for (int j = 0; j < GV_PROFILE_LIST; ++j) t8[j] = ~0ull;
    for (uint64_t i = tid; i < entries; i += kProfileThreads) {
        unsigned long long x = p.cta_first[i];
        if (x < t8[GV_PROFILE_LIST - 1]) {
#pragma unroll
            for (int j = 0; j < GV_PROFILE_LIST; ++j) {        // insertion into the ascending list
                const unsigned long long y = t8[j];
                if (x < y) { t8[j] = x; x = y; }
            }
        }
    }
    // ... then eight rounds of a block-wide minimum over the threads' current heads (indices are unique)
    for (int round = 0; round < GV_PROFILE_LIST; ++round) {
        unsigned long long m = warp_min_u64(t8[0]);
        if (lane == 0) s_min[warp] = m;
        __syncthreads();
        m = s_min[0];
        for (int i = 1; i < kProfileWarps; ++i) m = s_min[i] < m ? s_min[i] : m;
        if (tid == 0) s_pick[round] = m;
        if (m != ~0ull && t8[0] == m) {                        // the owner drops its head
#pragma unroll
            for (int j = 0; j + 1 < GV_PROFILE_LIST; ++j) t8[j] = t8[j + 1];
            t8[GV_PROFILE_LIST - 1] = ~0ull;
        }
        __syncthreads();
    }
    __syncthreads();
    if (tid < GV_PROFILE_LIST) {
        const unsigned long long idx = s_pick[tid];
        p.out->first_index[tid] = idx;
        unsigned long long c_raw = 0, r_raw = 0;
        if (idx != ~0ull) {
            for (int b = ESZ - 1; b >= 0; --b) {
                c_raw = c_raw << 8 | p.cand[idx * ESZ + b];
                r_raw = r_raw << 8 | p.ref[idx * ESZ + b];
            }
        }
        p.out->first_c_raw[tid] = c_raw;
        p.out->first_r_raw[tid] = r_raw;
    }
    if (tid == 0) {
        unsigned long long cnt = 0;
        for (int i = 0; i < GV_PROFILE_LIST; ++i) cnt += s_pick[i] != ~0ull;
        p.out->n_first = cnt;
    }
}

}  // namespace gv
