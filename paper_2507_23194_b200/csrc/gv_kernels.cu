// gv_kernels.cu -- kernels and C ABI of the batched output verifier (sm_100a).
//
// Hot path (one call of gv_verify_batch): record initialisation, a sampling pass that classifies the
// candidates, then one persistent kernel in which every WARP works alone on 512-byte warp-tiles of the
// reference (one 16-byte vector per lane) for one chunk of up to 16 candidates at a time. The warp's
// reference tile arrives by a 1-D bulk async copy (TMA) on the warp's own mbarrier, double buffered;
// each lane keeps its reference vector in registers for the whole chunk and streams its own 16 bytes
// of every candidate through a private ring of asynchronous 16-byte copies in shared memory. A
// candidate vector identical to the reference vector costs an identity test only (it shares the
// reference's hash terms); vectors that differ are hashed and compared, either in place or through a
// per-warp queue, depending on the candidate's class. Hash partials live in per-(candidate, lane)
// shared-memory slots, the other statistics in per-CTA accumulators; one block combine and one set
// of global integer atomics per (CTA, candidate). The comment above dense_kernel has the details; the
// ragged path and the follow-on calls are described where they are defined.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <type_traits>

#include "gv.h"
#include "gv_device.cuh"
#include "gv_group.cuh"
#include "gv_profile.cuh"
#include "gv_stats.cuh"

namespace gv {

// =============================================================================================
// result initialisation
// =============================================================================================
__global__ void init_results_kernel(gv_result* res, uint64_t count, uint32_t* status, uint64_t* ref_hash) {
    const uint64_t i = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x;
    if (i < count) {
        gv_result z;
        z.n_mismatch = 0; z.first_mismatch = GV_NO_INDEX; z.n_nan_disagree = 0; z.n_inf_disagree = 0;
        z.hash = 0; z.max_abs_diff_int = 0; z.max_abs_err = 0.0f; z.max_rel_err = 0.0f; z.reserved = 0;
        res[i] = z;
    }
    if (i == 0) {
        if (status) { status[0] = 0; status[1] = 0; status[2] = 0; status[3] = 0; }
        if (ref_hash) *ref_hash = 0;
    }
}

// A bounded wait that is certain to expire: the barrier expects 16 bytes of a bulk copy nobody issues.
// The expiry is reported the way the verify kernels report theirs (status bit), and the kernel returns.
__global__ void wait_expiry_kernel(uint32_t* status) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        status[0] = 0;
        mbar_init(&bar, 1);
        mbar_fence_init();
        mbar_expect_tx(&bar, 16);
    }
    __syncwarp();
    const bool ok = mbar_wait_bounded(&bar, 0u, 256u);
    if (!__all_sync(0xFFFFFFFFu, ok) && threadIdx.x == 0) atomicOr(status, kStatusTimeout);
}

// Read-only bandwidth probe: the wrapping sum of all 32-bit words of a buffer. Eight independent 128-bit
// streaming loads per thread and iteration, three integer additions per load: nothing but the memory
// system limits it, so its rate is the read bandwidth a verify kernel could at best reach.
__global__ void __launch_bounds__(kThreads) read_sum_kernel(const uint4* buf, uint64_t nvec, unsigned long long* out) {
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t v = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x;
    unsigned long long acc = 0;
    for (; v + 7 * stride < nvec; v += 8 * stride) {
        uint4 x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = ldg_stream(buf + v + j * stride);
        // (the additions start only when all eight loads have been issued)
        asm volatile("" ::: "memory");
#pragma unroll
        for (int j = 0; j < 8; ++j) acc += static_cast<unsigned long long>(x[j].x) + x[j].y + static_cast<unsigned long long>(x[j].z) + x[j].w;
    }
    for (; v < nvec; v += stride) {
        const uint4 x = ldg_stream(buf + v);
        acc += static_cast<unsigned long long>(x.x) + x.y + static_cast<unsigned long long>(x.z) + x.w;
    }
    acc = warp_sum_u64(acc);
    if ((threadIdx.x & 31) == 0 && acc) atomicAdd(out, acc);
}

// =============================================================================================
// gv_hash
// =============================================================================================
// LANE2: the second hash lane -- the word index is multiplied by the odd constant kGamma before the xor.
constexpr uint64_t kGamma = 0x9E3779B97F4A7C15ull;
template <bool LANE2>
__global__ void __launch_bounds__(kThreads) hash_kernel(const unsigned char* buf, uint64_t nbytes,
                                                        unsigned long long* out) {
    uint64_t h = 0;
    const uint64_t nvec = (nbytes + 15) / 16;
    const bool aligned = (reinterpret_cast<uintptr_t>(buf) & 15u) == 0;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint64_t v = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x;
    if (aligned) {
        // main part: four full vectors per thread and iteration, all loads issued before the first hash
        // (eight independent mixing chains per thread); 32-bit word indices while they suffice
        const uint64_t nfull = nbytes / 16;
        const bool k32 = nbytes < (1ull << 35);
        for (; v + 3 * stride < nfull; v += 4 * stride) {
            uint4 x[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) x[j] = ldg_stream(buf + (v + j * stride) * 16);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint64_t k0 = 2 * (v + j * stride);
                if constexpr (LANE2) {
                    const uint64_t g0 = k0 * kGamma;
                    h += splitmix64(g0 ^ pack64(x[j].x, x[j].y)) + splitmix64((g0 + kGamma) ^ pack64(x[j].z, x[j].w));
                } else {
                    h += k32 ? hash_vec_full_k32(x[j], static_cast<uint32_t>(k0)) : hash_vec_full(x[j], k0);
                }
            }
        }
    }
    for (; v < nvec; v += stride) {
        const uint64_t off = v * 16;
        if (aligned && off + 16 <= nbytes && !LANE2) {
            h += hash_vec_full(ldg_stream(buf + off), 2 * v);
        } else {
            // unaligned base or ragged tail: assemble the words byte by byte, zero padded
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            for (int b = 0; b < 16; ++b) {
                if (off + b < nbytes) w[b >> 2] |= static_cast<uint32_t>(buf[off + b]) << (8 * (b & 3));
            }
            const uint64_t rem = nbytes - off;
            if constexpr (LANE2) {
                h += splitmix64((2 * v * kGamma) ^ pack64(w[0], w[1]));
                if (rem > 8) h += splitmix64(((2 * v + 1) * kGamma) ^ pack64(w[2], w[3]));
            } else {
                h += hash_vec(make_uint4(w[0], w[1], w[2], w[3]), 2 * v, rem > 8 ? 2 : 1);
            }
        }
    }
    h = warp_sum_u64(h);
    __shared__ unsigned long long s;
    if (threadIdx.x == 0) s = 0;
    __syncthreads();
    if ((threadIdx.x & 31) == 0 && h) atomicAdd(&s, static_cast<unsigned long long>(h));
    __syncthreads();
    if (threadIdx.x == 0 && s) atomicAdd(out, s);
}

// =============================================================================================
// dense verify
// =============================================================================================
struct DenseParams {
    const unsigned char* ref;
    uint64_t n;                 // elements
    gv_result* results;         // records of this launch's candidates
    unsigned long long* ref_hash;  // nullable
    uint32_t* status;
    float atol, rtol;
    int equal_nan;
    int N;                      // candidates in this launch (<= kMaxPtrs)
    int all_aligned;            // reference and every candidate base are 16-byte aligned
    int rel_regime;             // float dtypes: atol is far below rtol (the tolerance is relative in effect): REL kernel
    const unsigned char* flags; // device, one byte per candidate of this launch: 1 = differs from the reference nearly everywhere
    const unsigned char* cands[kMaxPtrs];
};

// Dense kernel, organisation.
//   * Every warp works on its own: warp-tiles of 512 bytes (one 16-byte vector per lane), tile t
//     belongs to warp (t mod number of warps in the grid). No CTA-wide barrier in steady state.
//   * Reference: the warp's tile is brought into shared memory by one 512-byte bulk async copy (TMA)
//     completing on the warp's own mbarrier, double buffered (the next tile's copy is in flight
//     while the current tile is compared against the chunk). Each lane then holds its vector and the
//     values derived from it in registers for all candidates of the chunk.
//   * Candidates: each lane streams its own 16 bytes of every candidate with asynchronous 16-byte
//     copies into a private ring in shared memory, kRing copies in flight per lane, and reads them
//     back itself -- no registers are spent on data in flight and no barrier on its arrival.
//   * Hash: a candidate vector that is bit-identical to the reference vector has the reference
//     vector's hash terms, so the lane hashes its reference vector once per tile and a 64-bit
//     shared-memory slot per (candidate of the chunk, lane) only collects the corrections
//     hash(c) - hash(r) of the vectors that differ.
//   * Compare: identical vectors are done after the identity test. A sampling pass (classify_kernel)
//     flags the candidates that differ from the reference nearly everywhere; the kernel orders the
//     candidates, cuts them into chunks and runs one of two instances of its loop per chunk: one
//     queues differing vectors per warp and compares them 32 at a time, one per lane (candidates
//     that mostly agree with the reference); the other compares every differing vector in place
//     against values derived from the reference once per tile (chunks of flagged candidates). A
//     second compilation of the kernel (REL), launched when atol is far below rtol, lets that loop
//     settle vectors by the running maximum of the relative error as well.
//   * Accumulators: max |d|, max relative error, counts and the first index go to per-CTA shared
//     accumulators only when they can change them. One block combine and one set of global
//     integer atomics per (CTA, candidate).
constexpr int kWarps = kThreads / 32;
constexpr int kRing = 8;                  // asynchronous copies in flight per lane (power of two)
constexpr int kVisitBlock = 4;            // visits per unrolled block of the dense loop (divides kRing)
constexpr int kWarpTile = 512;            // bytes of one warp-tile

// Queue of differing vectors (one per warp). A candidate vector that differs from the reference
// vector is not compared where it is found: the lane appends (candidate vector, reference vector,
// byte offset | candidate slot, the reference vector's hash terms) to the warp's queue, and whenever
// 32 entries have gathered the warp compares them at once, one entry per lane. Sparse differences
// (a few lanes per visit) thus cost one full-width pass per 32 differing vectors instead of one
// mostly idle pass per visit.
constexpr int kQCap = 64;                           // entries (a power of two, >= 31 pending + 32 new)
constexpr uint32_t kQPlane = kQCap * 16;            // bytes of one plane (candidate / reference / meta)
constexpr size_t kQueueBytes = 3 * size_t(kQPlane);
constexpr int kDenseLanes = 18;                     // a candidate whose sampled tiles average this many differing lanes (of 32) is compared in place

template <int WARPS>
struct DenseSmem {
    static constexpr size_t kRingOff = 0;                                                 // [warp][kRing][32] uint4
    static constexpr size_t kRefOff = kRingOff + size_t(WARPS) * kRing * kWarpTile;       // [warp][2][32] uint4
    static constexpr size_t kSlotOff = kRefOff + size_t(WARPS) * 2 * kWarpTile;           // [warp][kChunk][32] u64
    static constexpr size_t kQueueOff = kSlotOff + size_t(WARPS) * kChunk * 32 * 8;       // [warp][3][kQCap] uint4
    static constexpr size_t kAccOff = kQueueOff + size_t(WARPS) * kQueueBytes;            // CtaAcc[kChunk]
    static constexpr size_t kBarOff = kAccOff + sizeof(CtaAcc) * kChunk;                  // [warp][2] mbarrier
    static constexpr size_t kRefHashOff = kBarOff + size_t(WARPS) * 2 * 8;
    static constexpr size_t kTotal = kRefHashOff + 8;
};

// CTA shape: 8 warps and about 98 KB of shared memory per CTA (ring 32, reference stages 8, hash slots
// 32, queue 24, accumulators 1.3), hence 2 CTAs per SM for every dtype, which leaves each thread up to
// 128 registers.
template <int DT> struct DenseShape {
    static constexpr int kWarpsPerCta = 8;
    static constexpr int kCtasPerSm = 2;
};

// The exact rule for one vector the fast path could not settle; kept out of line so the hot loop
// stays small. Everything it finds goes straight to the CTA accumulators.
template <int DT>
__device__ __noinline__ void settle_vector_exact(uint4 c, RefVec<16 / Traits<DT>::ESZ> r, uint64_t elem0,
                                                 TolF t, CtaAcc* s) {
    Acc a;
    a.clear();
    const uint32_t thr = *reinterpret_cast<volatile unsigned int*>(&s->thr);
    vec_exact_float<DT>(c, r, elem0, t, thr, a);
    push_rare(s, a);
    if (a.cnt) add_count(&s->cnt, a.cnt);
    raise_maxabs(s, a.maxabs);
}
// Two vectors of one flagged float candidate (two tiles of a single-candidate chunk), each against its own
// reference vector: derived values, fast path, exact rule where needed, counts merged for both.
template <int DT, bool REL_OK>
__device__ __noinline__ void compare_pair_float(uint4 c0, uint4 r0, uint4 c1, uint4 r1, TolF tol, CtaAcc* s, uint64_t elem0,
                                                uint64_t elem1) {
    if constexpr (Traits<DT>::IS_FLOAT) {
        constexpr int EPV = 16 / Traits<DT>::ESZ;
        RefVec<EPV> rva, rvb;
        uint32_t fa = 0u, fb = 0u, n0 = 0u, n1 = 0u;
        hoist_ref<DT>(r0, tol, rva, fa);
        hoist_ref<DT>(r1, tol, rvb, fb);
        if (!vec_fast_float<DT, false, REL_OK>(c0, rva, fa, tol, s, elem0, n0)) settle_vector_exact<DT>(c0, rva, elem0, tol, s);
        if (!vec_fast_float<DT, false, REL_OK>(c1, rvb, fb, tol, s, elem1, n1)) settle_vector_exact<DT>(c1, rvb, elem1, tol, s);
        if (__any_sync(0xFFFFFFFFu, (n0 | n1) != 0u)) merge_counts_converged(s, n0 + n1);
    }
}
// One tile of a chunk of one to three flagged float candidates: the reference vector's derived values
// once, then each candidate's vector against them.
template <int DT, bool REL_OK>
__device__ __noinline__ void compare_few_float(uint4 c0, uint4 c1, uint4 c2, uint4 r, int kg, TolF tol, CtaAcc* acc, uint64_t elem0) {
    if constexpr (Traits<DT>::IS_FLOAT) {
        constexpr int EPV = 16 / Traits<DT>::ESZ;
        RefVec<EPV> rv;
        uint32_t flags = 0u;
        hoist_ref<DT>(r, tol, rv, flags);
        const uint4 c[3] = {c0, c1, c2};
#pragma unroll
        for (int u = 0; u < 3; ++u) {
            if (u < kg) {
                uint32_t n = 0u;
                if (!vec_fast_float<DT, false, REL_OK>(c[u], rv, flags, tol, &acc[u], elem0, n)) settle_vector_exact<DT>(c[u], rv, elem0, tol, &acc[u]);
                if (__any_sync(0xFFFFFFFFu, n != 0u)) merge_counts_converged(&acc[u], n);
            }
        }
    }
}
template <int DT>
__device__ __noinline__ void settle_vector_int(uint4 c, uint4 r, uint64_t elem0, CtaAcc* s) {
    Acc a;
    a.clear();
    vec_int<DT>(c, r, elem0, 16 / Traits<DT>::ESZ, a);
    push_rare(s, a);
    if (a.cnt) add_count(&s->cnt, a.cnt);
}

// Compare the n (<= 32) oldest entries of the warp's queue, one per lane; called with the warp
// converged. qbase: shared address of the warp's queue; slots: this lane's column of hash slots;
// acc: the accumulators the entries' slot numbers index.
template <int DT, bool BIGK>
__device__ __forceinline__ void batch_entries(uint32_t qbase, uint32_t head, uint32_t n, uint2* slots, CtaAcc* acc,
                                              const TolF& tol) {
    constexpr int ESZ = Traits<DT>::ESZ;
    const uint32_t lane = threadIdx.x & 31u;
    if (lane < n) {
        const uint32_t at = qbase + ((head + lane) & (kQCap - 1)) * 16u;
        const uint4 c = lds128(at);
        const uint4 r = lds128(at + kQPlane);
        const uint4 m = lds128(at + 2 * kQPlane);
        const uint64_t meta = pack64(m.x, m.y), h_ref = pack64(m.z, m.w);
        const int k = static_cast<int>(m.x & 15u);
        const uint64_t voff = meta & ~uint64_t(15);
        uint64_t h;
        if constexpr (BIGK) {
            h = hash_vec_full(c, voff / 8);
        } else {
            h = hash_vec_full_k32(c, static_cast<uint32_t>(voff / 8));
        }
        const uint2 sl = slots[k * 32];
        const uint64_t hs = pack64(sl.x, sl.y) + (h - h_ref);
        slots[k * 32] = make_uint2(static_cast<uint32_t>(hs), static_cast<uint32_t>(hs >> 32));
        CtaAcc* s = &acc[k];
        // (mismatch counts: one 32-bit shared atomic per lane that found some, add_count -- a vote plus a
        // match over the candidate slots measured slower even when every entry mismatches)
        if constexpr (Traits<DT>::IS_FLOAT) {
            RefVec<16 / ESZ> rv;
            uint32_t rflags = 0u, unused = 0u;
            hoist_ref<DT>(r, tol, rv, rflags);
            if (!vec_fast_float<DT, true>(c, rv, rflags, tol, s, voff / ESZ, unused)) settle_vector_exact<DT>(c, rv, voff / ESZ, tol, s);
        } else {
            Acc a;
            a.clear();
            vec_int<DT>(c, r, voff / ESZ, 16 / ESZ, a);
            push_rare(s, a);
            if (a.cnt) add_count(&s->cnt, a.cnt);
        }
    }
}
template <int DT, bool BIGK>
__device__ __noinline__ void process_batch(uint32_t qbase, uint32_t head, uint32_t n, uint2* slots, CtaAcc* cacc,
                                           TolF tol) {
    batch_entries<DT, BIGK>(qbase, head, n, slots, cacc, tol);
}

// Which candidates differ from the reference nearly everywhere? One CTA per candidate compares a
// sample of its 512-byte tiles (evenly spread) with the reference, bytes only, and writes 1 when on
// average at least kDenseLanes of the 32 vectors of a tile differ. The flag only selects which of
// the dense kernel's two loops handles the candidate; both are correct for any data.
constexpr int kSampleTiles = 64;
__global__ void __launch_bounds__(kThreads) classify_kernel(const __grid_constant__ DenseParams p, uint64_t full_tiles,
                                                            unsigned char* flags) {
    __shared__ unsigned int s_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_total = 0u;
    __syncthreads();
    const unsigned char* cand = p.cands[blockIdx.x];
    const uint64_t S = full_tiles < kSampleTiles ? full_tiles : kSampleTiles;
    unsigned int mine = 0u;
    for (uint64_t i = warp; i < S; i += kThreads / 32) {
        const uint64_t off = (i * full_tiles / S) * kWarpTile + lane * 16;
        const uint4 c = ldg_stream(cand + off);
        const uint4 r = *reinterpret_cast<const uint4*>(p.ref + off);
        const bool differs = (c.x != r.x) || (c.y != r.y) || (c.z != r.z) || (c.w != r.w);
        mine += __popc(__ballot_sync(0xFFFFFFFFu, differs));
    }
    if (lane == 0 && mine) atomicAdd(&s_total, mine);
    __syncthreads();
    if (tid == 0) flags[blockIdx.x] = (S > 0 && s_total >= kDenseLanes * S) ? 1 : 0;
}

// BIGK: word indices of the hash need more than 32 bits (tensors of 32 GiB and more).
// REL: float dtypes, the in-place loop with the fast path's second way to "all close" (the host picks it
// when atol is far below rtol; a kernel of its own so that the other one pays nothing for it).
template <int DT, bool BIGK, bool REL>
__global__ void __launch_bounds__(DenseShape<DT>::kWarpsPerCta * 32, DenseShape<DT>::kCtasPerSm)
dense_kernel(const __grid_constant__ DenseParams p) {
    constexpr int kWarps = DenseShape<DT>::kWarpsPerCta;      // (shadows the 8-warp default of the other kernels)
    using Smem = DenseSmem<kWarps>;
    constexpr int ESZ = Traits<DT>::ESZ;
    constexpr int EPV = 16 / ESZ;
    constexpr bool IS_FLOAT = Traits<DT>::IS_FLOAT;
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    CtaAcc* cacc = reinterpret_cast<CtaAcc*>(smem + Smem::kAccOff);
    unsigned long long* s_refhash = reinterpret_cast<unsigned long long*>(smem + Smem::kRefHashOff);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Smem::kBarOff) + warp * 2;
    unsigned char* ref_stage = smem + Smem::kRefOff + size_t(warp) * 2 * kWarpTile;
    uint2* slots = reinterpret_cast<uint2*>(smem + Smem::kSlotOff) + size_t(warp) * kChunk * 32 + lane;
    const uint32_t ring_base = smem_u32(smem + Smem::kRingOff) + (warp * kRing * 32 + lane) * 16;
    const uint32_t qbase = smem_u32(smem + Smem::kQueueOff) + warp * static_cast<uint32_t>(kQueueBytes);
    const uint32_t lanes_below = (1u << lane) - 1u;
    uint32_t qhead = 0u, qcount = 0u;                       // the warp's queue of differing vectors (warp-uniform)

    const uint64_t nbytes = p.n * ESZ;
    const uint64_t full_tiles = p.all_aligned ? nbytes / kWarpTile : 0;      // tiles the fast loop takes
    const uint64_t all_tiles = (nbytes + kWarpTile - 1) / kWarpTile;
    const uint64_t gw = static_cast<uint64_t>(blockIdx.x) * kWarps + warp;   // this warp in the grid
    const uint64_t GW = static_cast<uint64_t>(gridDim.x) * kWarps;
    const TolF tol = {p.atol, p.rtol, p.equal_nan};

    // Candidates in processing order: those flagged "differs nearly everywhere" last. Chunks of 16 are
    // formed within each class, so every chunk runs one of the two loops below.
    static_assert(kWarps * 32 >= kMaxPtrs, "one thread per candidate");
    __shared__ unsigned char s_list[kMaxPtrs];
    __shared__ int s_wcount[2][kWarps];
    __shared__ __align__(16) const unsigned char* s_cptr[kChunk];
    {
        const bool dn = tid < p.N && p.flags != nullptr && p.flags[tid] != 0;
        const bool sp = tid < p.N && !dn;
        const uint32_t bs = __ballot_sync(0xFFFFFFFFu, sp), bd = __ballot_sync(0xFFFFFFFFu, dn);
        if (lane == 0) { s_wcount[0][warp] = __popc(bs); s_wcount[1][warp] = __popc(bd); }
        __syncthreads();
        int off_s = 0, off_d = 0, tot_s = 0;
        for (int w = 0; w < kWarps; ++w) {
            if (w < warp) { off_s += s_wcount[0][w]; off_d += s_wcount[1][w]; }
            tot_s += s_wcount[0][w];
        }
        if (sp) s_list[off_s + __popc(bs & lanes_below)] = static_cast<unsigned char>(tid);
        if (dn) s_list[tot_s + off_d + __popc(bd & lanes_below)] = static_cast<unsigned char>(tid);
    }
    int n_sparse = 0;
    for (int w = 0; w < kWarps; ++w) n_sparse += s_wcount[0][w];
    // Chunks of the ordered list. A run of candidates is cut into full chunks of 16, then one chunk of 4, 8
    // or 12 (the block loop takes multiples of 4) and one of the last 1 to 3 candidates (a tile-by-tile
    // loop of its own). A chunk takes the in-place loop only when all its candidates are flagged; a chunk holding
    // both classes takes the queueing loop, which is correct (if slower) for flagged candidates too. So
    // when a plain cut would put three or more flagged candidates into such a chunk, the list is cut at
    // the class boundary instead (the unflagged ones up to a multiple of 4, a chunk of 4 across the
    // boundary, then the flagged ones). Small chunks are costly whatever the loop -- the reference's
    // share of the work is spread over fewer candidates -- so this is done only when it pays.
    constexpr int kMaxChunks = 2 * (kMaxPtrs / kChunk) + 8;
    __shared__ unsigned char s_cstart[kMaxChunks], s_csize[kMaxChunks];
    __shared__ int s_nchunks;
    if (tid == 0) {
        int nc = 0;
        auto emit = [&](int start, int n) {
            while (n >= kChunk) { s_cstart[nc] = static_cast<unsigned char>(start); s_csize[nc++] = kChunk; start += kChunk; n -= kChunk; }
            if (n >= 4) { s_cstart[nc] = static_cast<unsigned char>(start); s_csize[nc++] = static_cast<unsigned char>(n & ~3); start += n & ~3; n &= 3; }
            if (n > 0) { s_cstart[nc] = static_cast<unsigned char>(start); s_csize[nc++] = static_cast<unsigned char>(n); }
        };
        const int nd = p.N - n_sparse;
        const int in_last = n_sparse % kChunk;                                  // unflagged candidates in the chunk a plain cut puts across the boundary
        const int flagged_there = in_last ? min(nd, kChunk - in_last) : 0;      // flagged ones it would take along
        if (flagged_there >= 3) {
            const int head = n_sparse & ~3;
            emit(0, head);
            int next = head;
            if (n_sparse & 3) {
                const int size = (n_sparse & 3) + min(nd, 4 - (n_sparse & 3));
                s_cstart[nc] = static_cast<unsigned char>(head);
                s_csize[nc++] = static_cast<unsigned char>(size);
                next = head + size;
            }
            emit(next, p.N - next);
        } else {
            emit(0, p.N);
        }
        s_nchunks = nc;
    }
    __syncthreads();
    const int num_groups = s_nchunks;

    if (lane == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        mbar_fence_init();
    }
    if (tid == 0) *s_refhash = 0;
    if (tid < kChunk) cacc[tid].clear();
    __syncthreads();

    uint32_t phase[2] = {0u, 0u};
    uint64_t my_ref_hash = 0;
    bool timed_out = false;
    // candidate bytes are read exactly once: mark them evict-first in L2 so that they do not push out the
    // reference, which every chunk reads again (+5 % on copies of a reference that fits L2)
    const uint64_t l2pol = l2_evict_first_policy();

    for (int g = 0; g < num_groups; ++g) {
        const int cand0 = s_cstart[g], kg = s_csize[g];       // first entry of the chunk in s_list, its size
        // in-place loop: every candidate of the chunk is flagged, or (a small chunk across the class
        // boundary) at least half of them are -- unflagged candidates rarely differ, and when they do the
        // in-place loop handles them correctly, whereas flagged ones are costly in the queueing loop
        const int flagged_here = max(0, cand0 + kg - max(cand0, n_sparse));
        const bool chunk_dense = 2 * flagged_here >= kg;
        if (tid < kg) s_cptr[tid] = p.cands[s_list[cand0 + tid]];
        __syncthreads();
        for (int k = 0; k < kg; ++k) slots[k * 32] = make_uint2(0u, 0u);

        // ================= fast loop: full warp-tiles, every base 16-byte aligned =================
        // Instances of the same loop: MODE 0 queues every differing vector (candidates that mostly
        // agree with the reference), MODE 1 compares every differing vector in place against values
        // hoisted per tile (candidates that differ nearly everywhere), MODE 2 (the REL kernel's) is MODE 1 with
        // the fast path's second way to "all close" for tolerances that are relative in effect. All are correct
        // for any data.
        auto fast_loop = [&](auto mode_tag) {
            constexpr int MODE = decltype(mode_tag)::value;
            const uint32_t my_tiles = static_cast<uint32_t>(min((full_tiles - gw + GW - 1) / GW, uint64_t(0xFFFFFFFFu)));
            const uint64_t tile_stride = GW * kWarpTile;
            uint64_t voff = gw * kWarpTile + lane * 16;          // this lane's vector in the tensor (current tile)

            // Values derived from the reference vector, computed lazily: only when a candidate
            // vector differs from it (exact copies never pay for them).
            RefVec<IS_FLOAT ? EPV : 1> rv;
            uint32_t force = 0u, rflags = 0u;
            bool hoisted = false, tile_forced = false;
            auto new_tile = [&](const uint4& r) {
                hoisted = false;
                force = 0u;
                if constexpr (IS_FLOAT) {
                    // only a NaN in the reference (without equal_nan) forces identical vectors onto the
                    // compare path; that needs no arithmetic, just the exponent/mantissa test
                    if (!tol.equal_nan) {
                        bool any_nan = false;
                        if constexpr (DT == GV_F32) {
                            any_nan = is_nan_bits(r.x) || is_nan_bits(r.y) || is_nan_bits(r.z) || is_nan_bits(r.w);
                        } else {
                            const uint32_t w[4] = {r.x, r.y, r.z, r.w};
                            constexpr uint32_t kAbs = 0x7FFF7FFFu;
                            constexpr uint32_t kInf = (DT == GV_BF16) ? 0x7F80u : 0x7C00u;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const uint32_t a = w[j] & kAbs;
                                any_nan = any_nan || (a & 0xFFFFu) > kInf || (a >> 16) > kInf;
                            }
                        }
                        force = any_nan ? 0xFFFFFFFFu : 0u;
                    }
                }
                // warp-uniform: does any lane hold such a vector? (keeps the per-lane flag out of the hot path)
                tile_forced = __any_sync(0xFFFFFFFFu, force != 0u);
            };
            // Derive the per-tile values when some lane of the warp first needs them. The decision is
            // warp-uniform (a vote), so the derivation runs once per tile, not once per diverged lane.
            auto ensure_hoisted = [&](const uint4& r) {
                if (!hoisted) {
                    if constexpr (IS_FLOAT) hoist_ref<DT>(r, tol, rv, rflags);
                    hoisted = true;
                }
            };
            auto hoist_now = [&](const uint4& r) {
                if constexpr (IS_FLOAT) hoist_ref<DT>(r, tol, rv, rflags);
            };
            // a candidate vector that is not bit-identical to the reference vector (ensure_hoisted done)
            // (mismatches of float vectors settled on the fast path are added to lane_cnt; the caller
            // merges lane_cnt into the accumulator once the warp has reconverged)
            auto differing = [&](const uint4& c, const uint4& r, int k, uint32_t& lane_cnt) {
                if constexpr (!IS_FLOAT) {
                    settle_vector_int<DT>(c, r, voff / ESZ, &cacc[k]);
                } else {
                    if (!vec_fast_float<DT, false, MODE == 2>(c, rv, rflags, tol, &cacc[k], voff / ESZ, lane_cnt))
                        settle_vector_exact<DT>(c, rv, voff / ESZ, tol, &cacc[k]);
                }
            };
            // Hash of a candidate vector. A vector that is bit-identical to the reference vector has the
            // very hash terms of the reference vector (same words at the same word indices), so the
            // lane only accumulates the reference's terms once per tile (ref_sum) and, per candidate,
            // the *correction* hash(c) - hash(r) of the vectors that differ (slot). At the end of the
            // chunk the candidate's partial is ref_sum + slot. Identical vectors cost no hash at all.
            uint64_t h_ref = 0;        // hash terms of this lane's reference vector (current tile)
            uint64_t ref_sum = 0;      // sum of h_ref over the tiles of this chunk
            // Float chunks of flagged candidates in the block loop: when nearly every vector differs, the identity
            // test decides nothing (a warp runs the compare whenever one of its lanes needs it), so every vector
            // is hashed and compared outright and the slots collect whole hashes, not corrections.
            constexpr bool kEveryVector = MODE != 0 && IS_FLOAT;
            const bool want_ref_hash = g == 0 && p.ref_hash != nullptr;
            uint64_t ref_only = 0;     // the reference's own terms where the slots do not need them
            auto hash_of = [&](const uint4& v) -> uint64_t {
                if constexpr (BIGK) return hash_vec_full(v, voff / 8);
                else return hash_vec_full_k32(v, static_cast<uint32_t>(voff / 8));
            };
            auto correct_slot = [&](const uint4& c, int k) {
                const uint64_t d = hash_of(c) - h_ref;
                const uint2 sl = slots[k * 32];
                const uint64_t h = pack64(sl.x, sl.y) + d;
                slots[k * 32] = make_uint2(static_cast<uint32_t>(h), static_cast<uint32_t>(h >> 32));
            };
            // Append this lane's vector (if it wants a compare) to the warp's queue; bal = ballot of the
            // lanes that do. Compares the 32 oldest entries as soon as 32 have gathered.
            auto enqueue = [&](const uint4& c, const uint4& r, int k, bool want, uint32_t bal) {
                const uint32_t at = qbase + ((qhead + qcount + __popc(bal & lanes_below)) & (kQCap - 1)) * 16u;
                const uint64_t meta = voff | static_cast<uint64_t>(k);
                sts128x3_if(at, kQPlane, c, r, make_uint4(static_cast<uint32_t>(meta), static_cast<uint32_t>(meta >> 32),
                                                          static_cast<uint32_t>(h_ref), static_cast<uint32_t>(h_ref >> 32)), want);
                qcount += __popc(bal);
                if (qcount >= 32u) {
                    __syncwarp();
                    process_batch<DT, BIGK>(qbase, qhead, 32u, slots, cacc, tol);
                    __syncwarp();
                    qhead = (qhead + 32u) & (kQCap - 1);
                    qcount -= 32u;
                }
            };
            // one visit: candidate vector c (already read from the ring) against the held reference.
            // A lane wants a compare when its vector differs, or when the reference holds a NaN that
            // equal_nan does not excuse. Dense differences (kDenseLanes lanes or more) are compared in
            // place against the values hoisted for the tile; sparse ones are queued.
            auto visit = [&](const uint4& c, const uint4& r, int k) {
                const bool differs = (c.x != r.x) || (c.y != r.y) || (c.z != r.z) || (c.w != r.w);
                if (__any_sync(0xFFFFFFFFu, differs) || tile_forced) {
                    const bool want = differs || force != 0u;
                    if constexpr (MODE != 0) {
                        ensure_hoisted(r);
                        uint32_t lane_cnt = 0u;
                        if (differs) correct_slot(c, k);
                        if (want) differing(c, r, k, lane_cnt);
                        if constexpr (IS_FLOAT) {
                            if (__any_sync(0xFFFFFFFFu, lane_cnt != 0u)) merge_counts_converged(&cacc[k], lane_cnt);
                        }
                    } else {
                        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, want);
                        if (bal) enqueue(c, r, k, want, bal);
                    }
                }
            };
            // reference of tile i: wait for its bulk copy, take this lane's vector, start the next copy
            auto next_ref = [&](uint32_t i, uint4& r) -> bool {
                const int b = static_cast<int>(i & 1u);
                bool ok = mbar_wait_bounded(&bars[b], phase[b]);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) return false;
                phase[b] ^= 1u;
                r = *reinterpret_cast<const uint4*>(ref_stage + b * kWarpTile + lane * 16);
                __syncwarp();      // every lane has read buffer b; buffer b^1 was drained one tile ago
                if (lane == 0 && i + 1 < my_tiles) {
                    fence_proxy_async();
                    mbar_expect_tx(&bars[b ^ 1], kWarpTile);
                    bulk_load(ref_stage + (b ^ 1) * kWarpTile, p.ref + (voff - lane * 16) + tile_stride, kWarpTile,
                              &bars[b ^ 1]);
                }
                return true;
            };
            if (lane == 0 && (kg & 3) == 0) {                  // (the loop for 1 to 3 candidates streams the reference itself)
                fence_proxy_async();
                mbar_expect_tx(&bars[0], kWarpTile);
                bulk_load(ref_stage, p.ref + gw * kWarpTile, kWarpTile, &bars[0]);
            }

            if ((kg & 3) == 0) {
                // ---- chunk of 4, 8, 12 or 16 candidates: blocks of U = 4 visits, ring depth 8 = two blocks.
                // The visits of the warp form one sequence (tile by tile, candidate by candidate); while a
                // block is consumed its stages are refilled with the block two further on, which lies in
                // the same tile, the next one or (4 candidates) the one after.
                constexpr int U = kVisitBlock;
#pragma unroll 1
                for (int j = 0; j < kRing; ++j) {
                    const int tt = j / kg, cc = j - tt * kg;
                    if (static_cast<uint32_t>(tt) < my_tiles) cp_async16_hint(ring_base + j * 512u, s_cptr[cc] + voff + tt * tile_stride, l2pol);
                    if ((j % U) == U - 1) cp_async_commit();
                }
                uint32_t vstage = 0u;                      // first stage of the current block: 0 or 4
#pragma unroll 1
                for (uint32_t i = 0; i < my_tiles; ++i) {
                    uint4 r;
                    if (!next_ref(i, r)) { timed_out = true; break; }
                    if constexpr (kEveryVector) {
                        // every candidate vector of this chunk is hashed and compared, identical or not: no
                        // identity test, no shared reference terms; the reference's own hash only if it is asked for
                        hoist_now(r);
                        if (want_ref_hash) ref_only += hash_of(r);
                    } else {
                        h_ref = hash_of(r);
                        ref_sum += h_ref;
                        new_tile(r);
                    }
#pragma unroll 1
                    for (int k0 = 0; k0 < kg; k0 += U) {
                        const uint32_t stage0 = ring_base + vstage * 512u;
                        vstage ^= 4u;
                        int refill = k0 + kRing;           // candidate and tile of the block two further on
                        uint32_t ahead = 0u;
                        if (refill >= kg) { refill -= kg; ahead = 1u; }
                        if (refill >= kg) { refill -= kg; ahead = 2u; }
                        const uint64_t refill_off = voff + ahead * tile_stride;
                        const bool live = i + ahead < my_tiles;
                        // the U refill pointers, two per 128-bit shared load, issued ahead of the wait
                        static_assert(U == 4, "two pointer pairs per block");
                        const uint4 pp0 = lds128(smem_u32(&s_cptr[refill])), pp1 = lds128(smem_u32(&s_cptr[refill + 2]));
                        const unsigned char* const rp[U] = {
                            reinterpret_cast<const unsigned char*>(pack64(pp0.x, pp0.y)), reinterpret_cast<const unsigned char*>(pack64(pp0.z, pp0.w)),
                            reinterpret_cast<const unsigned char*>(pack64(pp1.x, pp1.y)), reinterpret_cast<const unsigned char*>(pack64(pp1.z, pp1.w))};
                        cp_async_wait<kRing / U - 1>();     // the block of U stages issued kRing visits ago has landed
                        uint4 c[U];
#pragma unroll
                        for (int u = 0; u < U; ++u) c[u] = lds128(stage0 + u * 512u);
                        if constexpr (kEveryVector) {
                            uint32_t lane_cnt[U];
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                lane_cnt[u] = 0u;
                                const uint64_t hcand = hash_of(c[u]);
                                const uint2 sl = slots[(k0 + u) * 32];
                                const uint64_t hs = pack64(sl.x, sl.y) + hcand;
                                slots[(k0 + u) * 32] = make_uint2(static_cast<uint32_t>(hs), static_cast<uint32_t>(hs >> 32));
                                differing(c[u], r, k0 + u, lane_cnt[u]);
                            }
                            uint32_t any_cnt = 0u;
#pragma unroll
                            for (int u = 0; u < U; ++u) any_cnt |= lane_cnt[u];
                            if (__any_sync(0xFFFFFFFFu, any_cnt != 0u)) {
#pragma unroll
                                for (int u = 0; u < U; ++u) merge_counts_converged(&cacc[k0 + u], lane_cnt[u]);
                            }
                        } else {
                        // identity test for all U visits; identical vectors are done
                        uint32_t diffmask = 0u;
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            const bool differs = (c[u].x != r.x) || (c[u].y != r.y) || (c[u].z != r.z) || (c[u].w != r.w);
                            diffmask |= differs ? (1u << u) : 0u;
                        }
                        if (__any_sync(0xFFFFFFFFu, diffmask != 0u) || tile_forced) {
                            if constexpr (MODE == 0) {
                                // every visit with a lane that wants a compare appends to the queue
#pragma unroll
                                for (int u = 0; u < U; ++u) {
                                    const bool want = ((diffmask >> u) & 1u) || force != 0u;
                                    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, want);
                                    if (bal) enqueue(c[u], r, k0 + u, want, bal);
                                }
                            } else {
                                // in place, U visits interleaved: hash chain and compare share one block
                                ensure_hoisted(r);
                                uint32_t lane_cnt[U];
#pragma unroll
                                for (int u = 0; u < U; ++u) {
                                    lane_cnt[u] = 0u;
                                    if (diffmask & (1u << u)) {
                                        correct_slot(c[u], k0 + u);
                                        differing(c[u], r, k0 + u, lane_cnt[u]);
                                    } else if (force != 0u) {
                                        differing(c[u], r, k0 + u, lane_cnt[u]);   // identical, but the reference holds a NaN
                                    }
                                }
                                if constexpr (IS_FLOAT) {
                                    // the warp is converged again here; mismatches are rare, so one vote first,
                                    // then one reduction and at most one atomic per visit
                                    uint32_t any_cnt = 0u;
#pragma unroll
                                    for (int u = 0; u < U; ++u) any_cnt |= lane_cnt[u];
                                    if (__any_sync(0xFFFFFFFFu, any_cnt != 0u)) {
#pragma unroll
                                        for (int u = 0; u < U; ++u) merge_counts_converged(&cacc[k0 + u], lane_cnt[u]);
                                    }
                                }
                            }
                        }
                        }
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            if (live) cp_async16_hint(stage0 + u * 512u, rp[u] + refill_off, l2pol);
                        }
                        cp_async_commit();                  // one group per block of U refills
                    }
                    voff += tile_stride;
                }
            } else {
                // ---- the last 1 to 3 candidates (or a call with so few): tile by tile. The reference vector
                // travels through the ring like the candidates, a tile occupies kg + 1 stages, and as many
                // tiles as fit in the ring are in flight (4 for one candidate, else 2); one wait and one
                // commit per tile.
                const uint32_t per = static_cast<uint32_t>(kg) + 1u;
                const uint32_t depth = kg == 1 ? 4u : 2u;
                const uint64_t first_off = voff;                       // this lane's vector in the warp's first tile
                auto issue_tile = [&](uint32_t t, uint32_t into) {
                    if (t < my_tiles) {
                        const uint64_t off = first_off + static_cast<uint64_t>(t) * tile_stride;
                        const uint32_t at = ring_base + into * per * 512u;
                        cp_async16(at, p.ref + off);
                        for (int u = 0; u < kg; ++u) cp_async16_hint(at + (1u + u) * 512u, s_cptr[u] + off, l2pol);
                    }
                    cp_async_commit();
                };
                for (uint32_t t = 0; t < depth; ++t) issue_tile(t, t);
                uint32_t slot = 0u;
                uint32_t i = 0u;
                if (kg == 1) {
                    // One candidate: a warp's iteration is a chain of dependent instructions (the reference's
                    // hash, two votes, the identity test) with nothing to overlap it, so two tiles are taken
                    // per iteration and their reference hashes computed side by side.
#pragma unroll 1
                    for (; i + 2u <= my_tiles; i += 2u) {
                        cp_async_wait<2>();                            // the two oldest tiles have landed
                        const uint32_t at0 = ring_base + slot * 1024u, at1 = at0 + 1024u;     // slot is 0 or 2 here
                        const uint4 r0 = lds128(at0), c0 = lds128(at0 + 512u);
                        const uint4 r1 = lds128(at1), c1 = lds128(at1 + 512u);
                        issue_tile(i + 4u, slot);
                        issue_tile(i + 5u, slot + 1u);
                        slot ^= 2u;
                        if constexpr (kEveryVector) {
                            // a flagged float candidate: both vectors hashed and compared outright, as in the
                            // block loop (whole hashes in the slot, the reference's terms only for ref_hash)
                            uint64_t hc = hash_of(c0);
                            if (want_ref_hash) ref_only += hash_of(r0);
                            voff += tile_stride;
                            hc += hash_of(c1);
                            if (want_ref_hash) ref_only += hash_of(r1);
                            const uint2 sl = slots[0];
                            const uint64_t hs = pack64(sl.x, sl.y) + hc;
                            slots[0] = make_uint2(static_cast<uint32_t>(hs), static_cast<uint32_t>(hs >> 32));
                            compare_pair_float<DT, MODE == 2>(c0, r0, c1, r1, tol, &cacc[0], (voff - tile_stride) / ESZ, voff / ESZ);
                            voff += tile_stride;
                        } else {
                            const uint64_t h0 = hash_of(r0);
                            voff += tile_stride;
                            const uint64_t h1 = hash_of(r1);
                            voff -= tile_stride;
                            ref_sum += h0 + h1;
                            h_ref = h0;
                            new_tile(r0);
                            visit(c0, r0, 0);
                            voff += tile_stride;
                            h_ref = h1;
                            new_tile(r1);
                            visit(c1, r1, 0);
                            voff += tile_stride;
                        }
                    }
                }
#pragma unroll 1
                for (; i < my_tiles; ++i) {
                    if (depth == 4u) cp_async_wait<3>(); else cp_async_wait<1>();
                    const uint32_t at = ring_base + slot * per * 512u;
                    const uint4 r = lds128(at);
                    uint4 c[3];
#pragma unroll
                    for (int u = 0; u < 3; ++u) c[u] = u < kg ? lds128(at + (1u + u) * 512u) : r;
                    issue_tile(i + depth, slot);                       // refill the stages just read
                    slot = slot + 1u == depth ? 0u : slot + 1u;
                    if constexpr (kEveryVector) {
                        // flagged float candidates: every vector hashed and compared outright (see the block loop)
                        if (want_ref_hash) ref_only += hash_of(r);
#pragma unroll
                        for (int u = 0; u < 3; ++u) {
                            if (u < kg) {
                                const uint2 sl = slots[u * 32];
                                const uint64_t hs = pack64(sl.x, sl.y) + hash_of(c[u]);
                                slots[u * 32] = make_uint2(static_cast<uint32_t>(hs), static_cast<uint32_t>(hs >> 32));
                            }
                        }
                        compare_few_float<DT, MODE == 2>(c[0], c[1], c[2], r, kg, tol, cacc, voff / ESZ);
                    } else {
                        h_ref = hash_of(r);
                        ref_sum += h_ref;
                        new_tile(r);
#pragma unroll
                        for (int u = 0; u < 3; ++u)
                            if (u < kg) visit(c[u], r, u);
                    }
                    voff += tile_stride;
                }
            }
            cp_async_wait<0>();
            if (qcount) {                                  // the chunk's accumulators close: drain the queue
                __syncwarp();
                process_batch<DT, BIGK>(qbase, qhead, qcount, slots, cacc, tol);
                __syncwarp();
                qhead = 0u;
                qcount = 0u;
            }
            // every candidate's partial = the reference's terms over this lane's tiles + its corrections
            for (int k = 0; k < kg; ++k) {
                const uint2 sl = slots[k * 32];
                const uint64_t h = pack64(sl.x, sl.y) + ref_sum;
                slots[k * 32] = make_uint2(static_cast<uint32_t>(h), static_cast<uint32_t>(h >> 32));
            }
            if (want_ref_hash) my_ref_hash += ref_sum + ref_only;
            if (timed_out) {
                // flag it; give the copy that may still be in flight a second bounded chance to land
                if (lane == 0) {
                    atomicOr(p.status, kStatusTimeout);
                    (void)mbar_wait_bounded(&bars[0], phase[0]);
                    (void)mbar_wait_bounded(&bars[1], phase[1]);
                }
                __syncwarp();
            }
        };
        if (gw < full_tiles && !timed_out) {
            if (!chunk_dense) {
                fast_loop(std::integral_constant<int, 0>{});
            } else {
                fast_loop(std::integral_constant<int, (IS_FLOAT && REL) ? 2 : 1>{});
            }
        }

        // ================= general loop: ragged tail, or some base not 16-byte aligned =================
        // (synchronous element-sized loads; at most one warp-tile per tensor when bases are aligned)
        for (uint64_t t = full_tiles + gw; t < all_tiles; t += GW) {
            const uint64_t voff = t * kWarpTile + lane * 16;
            const uint64_t rem = voff < nbytes ? nbytes - voff : 0;
            const int nvalid = rem >= 16 ? EPV : static_cast<int>(rem / ESZ);
            if (nvalid > 0) {
                const uint4 r = load_vec_generic<ESZ>(p.ref, voff, nbytes);
                const int nwords = nvalid * ESZ > 8 ? 2 : 1;
                if (g == 0 && p.ref_hash) my_ref_hash += hash_vec(r, voff / 8, nwords);
                for (int k = 0; k < kg; ++k) {
                    const uint4 c = load_vec_generic<ESZ>(s_cptr[k], voff, nbytes);
                    Acc a;
                    a.clear();
                    a.hash = hash_vec(c, voff / 8, nwords);
                    vec_compare<DT>(c, r, voff / ESZ, nvalid, tol, a);
                    const uint2 sl = slots[k * 32];
                    const uint64_t h = pack64(sl.x, sl.y) + a.hash;
                    slots[k * 32] = make_uint2(static_cast<uint32_t>(h), static_cast<uint32_t>(h >> 32));
                    push_rare(&cacc[k], a);
                    if (a.cnt) add_count(&cacc[k].cnt, a.cnt);
                    raise_maxabs(&cacc[k], a.maxabs);
                }
            }
        }

        // ---- end of a chunk: reduce the hash slots once and publish the chunk's records ----
        for (int k = 0; k < kg; ++k) {
            const uint2 sl = slots[k * 32];
            const uint64_t h = warp_sum_u64(pack64(sl.x, sl.y));
            if (lane == 0 && h) atomicAdd(&cacc[k].hash, static_cast<unsigned long long>(h));
        }
        __syncthreads();
        if (tid < kg) push_global(&p.results[s_list[cand0 + tid]], cacc[tid]);
        if (tid < kChunk) cacc[tid].clear();
        __syncthreads();
    }

    if (p.ref_hash) {
        const uint64_t h = warp_sum_u64(my_ref_hash);
        if (lane == 0 && h) atomicAdd(s_refhash, static_cast<unsigned long long>(h));
        __syncthreads();
        if (tid == 0 && *s_refhash) atomicAdd(p.ref_hash, *s_refhash);
    }
}

// =============================================================================================
// ragged verify
// =============================================================================================
struct RaggedParams {
    const unsigned char* ref_base;
    const int64_t* ref_off;     // T+1
    const unsigned char* cand_base;
    const int64_t* cand_off;    // T*N
    const uint8_t* dtypes;      // T
    const int64_t* n_elems;     // T or null
    int64_t T;
    int N;
    gv_result* results;
    uint32_t* status;
    uint32_t* counter;          // work counter of the main kernel (zeroed by the record initialisation)
    int64_t* tile_prefix;       // T+1, workspace
    float atol, rtol;
    int equal_nan;
};

constexpr int kRaggedTile = kWarpTile;      // ragged work is split into the same 512-byte warp-tiles
constexpr int64_t kRaggedMaxBytes = int64_t(1) << 40;   // largest tensor a table entry may describe (1 TiB)
constexpr uint64_t kChunkBig = 256;                     // most work units a warp takes at a time from the global sequence
constexpr int64_t kPartCost = 4;                        // work units charged per tensor on top of its tiles (pointer set-up, tail tile,
                                                        // publishing the records: about what four streamed tiles cost)

// Pre-pass: validates the tables and turns sizes into an exclusive prefix of tile counts.
// One CTA; T is at most a few million in practice (one pass of 1024-wide chunks).
__global__ void __launch_bounds__(1024) ragged_prepass_kernel(RaggedParams p) {
    __shared__ long long s_warp[32];
    __shared__ long long s_carry;
    const int tid = threadIdx.x;
    if (tid == 0) { s_carry = 0; p.tile_prefix[0] = 0; }
    __syncthreads();
    for (int64_t base = 0; base < p.T; base += 1024) {
        const int64_t t = base + tid;
        long long tiles = 0;
        if (t < p.T) {
            const int dt = p.dtypes[t];
            const int esz = elem_size(dt);
            bool good = esz != 0;
            int64_t n = 0;
            if (good) {
                const int64_t ro = p.ref_off[t];
                if (p.n_elems) n = p.n_elems[t];
                else {
                    const int64_t span = p.ref_off[t + 1] - ro;
                    good = good && span >= 0 && span % esz == 0;
                    n = span / esz;
                }
                // sizes beyond kRaggedMaxBytes per tensor are table errors: no device holds such a tensor, and
                // the bound keeps n * esz and the running tile total (T < 2^31 tensors) far from overflow
                good = good && n >= 0 && n <= kRaggedMaxBytes / esz && ro >= 0 && ro % esz == 0;
                for (int j = 0; good && j < p.N; ++j) {
                    const int64_t co = p.cand_off[t * p.N + j];
                    good = co >= 0 && co % esz == 0;
                }
            }
            if (!good) atomicOr(p.status, kStatusBadTable);
            else tiles = (n * esz + kRaggedTile - 1) / kRaggedTile;
            // the table holds WORK units, not tiles: a tensor costs its tiles plus a fixed amount for
            // starting and finishing it (empty and rejected tensors cost nothing and are skipped)
            if (tiles > 0) tiles += kPartCost;
        }
        // inclusive scan of `tiles` over the 1024 threads
        long long x = tiles;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
            if ((tid & 31) >= o) x += y;
        }
        if ((tid & 31) == 31) s_warp[tid >> 5] = x;
        __syncthreads();
        if (tid < 32) {
            long long w = s_warp[tid];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long y = __shfl_up_sync(0xFFFFFFFFu, w, o);
                if (tid >= o) w += y;
            }
            s_warp[tid] = w;
        }
        __syncthreads();
        const long long incl = x + ((tid >> 5) ? s_warp[(tid >> 5) - 1] : 0) + s_carry;
        if (t < p.T) p.tile_prefix[t + 1] = incl;
        __syncthreads();
        if (tid == 1023) s_carry = incl;
        __syncthreads();
    }
}

// Ragged kernel, organisation. The warp-tiles of all tensors form one sequence (tile_prefix); every
// warp of the grid takes one contiguous stretch of it, so it meets only a few tensor boundaries.
// Inside a tensor it works like the dense kernel's general shape: the lane's reference vector is
// held in registers and compared with the same vector of each of the tensor's candidates; the hash
// partials of the current tensor live in per-(candidate, lane) shared-memory slots and the other
// statistics in per-warp shared accumulators, all flushed with integer atomics when the warp leaves
// the tensor. No barrier is used anywhere: warps never share a tensor's accumulators.
// FOUR: the instance for exactly four candidates per tensor keeps slots, accumulators and pointers for four
// candidates only (79 KB per CTA instead of 109). Both instances run 8 warps per CTA and 2 CTAs per SM: more
// warps would need fewer registers than the compare code wants (10 warps at 96 registers: no gain; 11 at
// 80, or 3 CTAs of 7 warps: a third slower).
template <bool FOUR>
struct RaggedSmem {
    static constexpr int kWarpsPerCta = 8;
    static constexpr int kCtasPerSm = 2;
    static constexpr int kCtaThreads = kWarpsPerCta * 32;
    static constexpr int kCands = FOUR ? 4 : kChunk;                                        // candidates handled at a time
    static constexpr size_t kRingOff = 0;                                                   // [warp][kRing][32] uint4
    static constexpr size_t kSlotOff = kRingOff + size_t(kWarpsPerCta) * kRing * kWarpTile;        // [warp][kCands][32] u64
    static constexpr size_t kAccOff = kSlotOff + size_t(kWarpsPerCta) * kCands * 32 * 8;           // [warp][kCands] CtaAcc
    static constexpr size_t kPtrOff = kAccOff + size_t(kWarpsPerCta) * kCands * sizeof(CtaAcc);    // [warp][kCands + 2] reference + candidate pointers
    static constexpr size_t kQueueOff = kPtrOff + size_t(kWarpsPerCta) * (kCands + 2) * 8;         // [warp][3][kQCap] uint4
    static constexpr size_t kRefOff = kQueueOff + size_t(kWarpsPerCta) * kQueueBytes;              // [warp][2][32] uint4 (four-candidate loop)
    static constexpr size_t kMetaOff = kRefOff + size_t(kWarpsPerCta) * 2 * kWarpTile;             // [warp][32] u64: table entries of the current tensor
    static constexpr size_t kTotal = kMetaOff + size_t(kWarpsPerCta) * 32 * 8;
};

// Code size matters in this kernel: the warps of an SM are in different places at the same time (the
// streaming loop, the batch function of one of four dtypes, a tensor's tail), and everything they run
// competes for the instruction cache (ncu: waiting for instructions was the second largest stall; every
// variant that added code to any of these paths lost throughput). So the paths beside the streaming loops
// are written for size: rolled loops and run-time dtype tests instead of one unrolled body per dtype.

// The warp's queue of differing vectors (all of one tensor, hence of one dtype): the n oldest entries, one
// per lane. The hash uses 64-bit word indices (tensors of any size reach this function through the tail path).
template <int DT>
__device__ __forceinline__ void ragged_entry(const uint4& c, const uint4& r, uint64_t voff, const TolF& tol, CtaAcc* s) {
    constexpr int ESZ = Traits<DT>::ESZ;
    if constexpr (Traits<DT>::IS_FLOAT) {
        RefVec<16 / ESZ> rv;
        uint32_t rflags = 0u, unused = 0u;
        hoist_ref<DT>(r, tol, rv, rflags);
        if (!vec_fast_float<DT, true>(c, rv, rflags, tol, s, voff / ESZ, unused)) settle_vector_exact<DT>(c, rv, voff / ESZ, tol, s);
    } else {
        Acc a;
        a.clear();
        vec_int<DT>(c, r, voff / ESZ, 16 / ESZ, a);
        push_rare(s, a);
        if (a.cnt) add_count(&s->cnt, a.cnt);
    }
}
__device__ __noinline__ void ragged_batch(int dt, uint32_t qbase, uint32_t head, uint32_t n, uint2* slots, CtaAcc* wacc,
                                          TolF tol) {
    const uint32_t lane = threadIdx.x & 31u;
    if (lane >= n) return;
    const uint32_t at = qbase + ((head + lane) & (kQCap - 1)) * 16u;
    const uint4 c = lds128(at);
    const uint4 r = lds128(at + kQPlane);
    const uint4 m = lds128(at + 2 * kQPlane);
    const uint64_t meta = pack64(m.x, m.y), h_ref = pack64(m.z, m.w);
    const int k = static_cast<int>(m.x & 15u);
    const uint64_t voff = meta & ~uint64_t(15);
    const uint64_t h = hash_vec_full(c, voff / 8);
    const uint2 sl = slots[k * 32];
    const uint64_t hs = pack64(sl.x, sl.y) + (h - h_ref);
    slots[k * 32] = make_uint2(static_cast<uint32_t>(hs), static_cast<uint32_t>(hs >> 32));
    CtaAcc* s = &wacc[k];
    switch (dt) {
        case GV_F32: ragged_entry<GV_F32>(c, r, voff, tol, s); break;
        case GV_BF16: ragged_entry<GV_BF16>(c, r, voff, tol, s); break;
        case GV_F16: ragged_entry<GV_F16>(c, r, voff, tol, s); break;
        case GV_I32: ragged_entry<GV_I32>(c, r, voff, tol, s); break;
        default: ragged_entry<GV_I64>(c, r, voff, tol, s); break;
    }
}

// Element e of a 16-byte vector of dtype dt, zero-extended raw bits (dynamic indexing: cold code).
__device__ __forceinline__ uint64_t raw_element(const uint4& v, int esz, int e) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (esz == 2) return (w[e >> 1] >> (16 * (e & 1))) & 0xFFFFu;
    if (esz == 4) return w[e];
    return pack64(w[2 * e], w[2 * e + 1]);
}
// A vector that is not complete (the end of a tensor): its nvalid elements one by one through the general
// rule, in one rolled loop for all dtypes; its hash terms go to the slot as they are (no shared terms here).
__device__ __noinline__ void ragged_elements(int dt, uint4 c, uint4 r, uint64_t byte_off, int nvalid, TolF tol, CtaAcc* s,
                                             uint2* slot) {
    Acc a;
    a.clear();
    const int esz = elem_size(dt);
    a.hash = hash_vec(c, byte_off / 8, nvalid * esz > 8 ? 2 : 1);
    const uint64_t elem0 = byte_off / static_cast<uint64_t>(esz);
#pragma unroll 1
    for (int e = 0; e < nvalid; ++e) {
        const uint64_t cr = raw_element(c, esz, e), rr = raw_element(r, esz, e);
        if (dt <= GV_F16) {
            float cf, rf;
            if (dt == GV_F32) { cf = __uint_as_float(static_cast<uint32_t>(cr)); rf = __uint_as_float(static_cast<uint32_t>(rr)); }
            else if (dt == GV_BF16) { cf = __uint_as_float(static_cast<uint32_t>(cr) << 16); rf = __uint_as_float(static_cast<uint32_t>(rr) << 16); }
            else { cf = f16_to_f32(static_cast<uint32_t>(cr)); rf = f16_to_f32(static_cast<uint32_t>(rr)); }
            element_rule<false>(cf, rf, tol, elem0 + e, a);
        } else if (cr != rr) {
            const int64_t cv = dt == GV_I32 ? static_cast<int64_t>(static_cast<int32_t>(cr)) : static_cast<int64_t>(cr);
            const int64_t rv = dt == GV_I32 ? static_cast<int64_t>(static_cast<int32_t>(rr)) : static_cast<int64_t>(rr);
            const uint64_t diff = cv > rv ? static_cast<uint64_t>(cv) - static_cast<uint64_t>(rv)
                                          : static_cast<uint64_t>(rv) - static_cast<uint64_t>(cv);      // exact mod 2^64
            a.cnt += 1;
            a.first = (elem0 + e) < a.first ? (elem0 + e) : a.first;
            a.maxint = diff > a.maxint ? diff : a.maxint;
        }
    }
    const uint2 sl = *slot;
    const uint64_t h = pack64(sl.x, sl.y) + a.hash;
    *slot = make_uint2(static_cast<uint32_t>(h), static_cast<uint32_t>(h >> 32));
    push_rare(s, a);
    if (a.cnt) add_count(&s->cnt, a.cnt);
    raise_maxabs(s, a.maxabs);
}
// A 16-byte vector at byte_off of a tensor of nbytes bytes: one 128-bit load when it is complete and
// aligned, else the elements that exist one by one (rolled), zero fill for the rest.
__device__ __noinline__ uint4 load_vec_slow(int esz, const unsigned char* base, uint64_t byte_off, uint64_t nbytes) {
    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll 1
    for (int b = 0; b < 16; b += esz) {
        const uint64_t o = byte_off + b;
        if (o < nbytes) {
            if (esz == 2) w[b >> 2] |= static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(base + o)) << (8 * (b & 3));
            else if (esz == 4) w[b >> 2] = *reinterpret_cast<const uint32_t*>(base + o);
            else {
                const uint64_t x = *reinterpret_cast<const unsigned long long*>(base + o);
                w[b >> 2] = static_cast<uint32_t>(x);
                w[(b >> 2) + 1] = static_cast<uint32_t>(x >> 32);
            }
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ uint4 load_vec_any(int esz, const unsigned char* base, uint64_t byte_off, uint64_t nbytes) {
    if (byte_off + 16 <= nbytes && ((reinterpret_cast<uintptr_t>(base) + byte_off) & 15u) == 0)
        return *reinterpret_cast<const uint4*>(base + byte_off);
    return load_vec_slow(esz, base, byte_off, nbytes);
}
// NaN anywhere in a reference vector of a float dtype (bit tests only)
__device__ __forceinline__ bool vec_has_nan(int dt, const uint4& r) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    bool any = false;
    if (dt == GV_F32) {
#pragma unroll
        for (int j = 0; j < 4; ++j) any = any || is_nan_bits(w[j]);
    } else if (dt == GV_BF16 || dt == GV_F16) {
        const uint32_t inf = dt == GV_BF16 ? 0x7F80u : 0x7C00u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t a = w[j] & 0x7FFF7FFFu;
            any = any || (a & 0xFFFFu) > inf || (a >> 16) > inf;
        }
    }
    return any;
}
// The streaming loops' version of that test: is any element of the reference vector a NaN OR an infinity?
// (Also sending identical vectors that hold an infinity to the compare path is harmless -- the rule finds
// them equal -- and lets the test run on the multiply-add pipe, which these loops leave idle, instead of the
// logic pipe, which they saturate: x * 0 is a zero for every finite x and a NaN otherwise.)
__device__ __forceinline__ bool vec_has_nonfinite(int dt, const uint4& r) {
    if (dt == GV_F32) {
        float a = __fmul_rn(__uint_as_float(r.x), 0.0f);
        a = __fmaf_rn(__uint_as_float(r.y), 0.0f, a);
        a = __fmaf_rn(__uint_as_float(r.z), 0.0f, a);
        a = __fmaf_rn(__uint_as_float(r.w), 0.0f, a);
        return a != a;
    }
    uint32_t a = 0u;
    if (dt == GV_F16) {
        asm("{ .reg .b32 z;\n\t mov.b32 z, 0;\n\t"
            "fma.rn.f16x2 %0, %1, z, z;\n\t fma.rn.f16x2 %0, %2, z, %0;\n\t"
            "fma.rn.f16x2 %0, %3, z, %0;\n\t fma.rn.f16x2 %0, %4, z, %0; }"
            : "=&r"(a) : "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w));
    } else if (dt == GV_BF16) {
        asm("{ .reg .b32 z;\n\t mov.b32 z, 0;\n\t"
            "fma.rn.bf16x2 %0, %1, z, z;\n\t fma.rn.bf16x2 %0, %2, z, %0;\n\t"
            "fma.rn.bf16x2 %0, %3, z, %0;\n\t fma.rn.bf16x2 %0, %4, z, %0; }"
            : "=&r"(a) : "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w));
    }
    return (a & 0x7FFF7FFFu) != 0u;       // each half is a zero of either sign, or a NaN
}

// Tiles [tile_begin, tile_end) with synchronous loads: the tail tile of a tensor, or every tile of a tensor
// that is not streamed (a base that is not 16-byte aligned, 32 GiB or more). Complete vectors that differ
// from the reference vector go through the warp's queue like those of streamed tiles (same batch function,
// nothing of their own); the one incomplete vector at the end of a tensor goes element by element.
// Returns the sum of the reference's hash terms over the complete vectors it met (the caller adds it to
// every candidate's slot).
__device__ __noinline__ uint64_t ragged_tail(int dt, const unsigned char* ref, uint64_t nbytes, uint64_t tile_begin,
                                             uint64_t tile_end, int kg, uint2* slots, CtaAcc* wacc,
                                             const unsigned char* const* wptr, TolF tol, bool nan_matters, uint32_t qbase) {
    const int esz = elem_size(dt);
    const int lane = threadIdx.x & 31;
    const uint32_t lanes_below = (1u << lane) - 1u;
    uint32_t qhead = 0u, qcount = 0u;
    uint64_t ref_sum = 0;
#pragma unroll 1
    for (uint64_t tile = tile_begin; tile < tile_end; ++tile) {
        const uint64_t voff = tile * kWarpTile + lane * 16;
        const uint64_t rem = voff < nbytes ? nbytes - voff : 0;
        const int nvalid = rem >= 16 ? 16 / esz : static_cast<int>(rem / esz);
        const bool full = rem >= 16;
        uint4 r = make_uint4(0u, 0u, 0u, 0u);
        if (nvalid > 0) r = load_vec_any(esz, ref, voff, nbytes);
        const bool force = nan_matters && full && vec_has_nan(dt, r);
        uint64_t h_ref = 0;
        if (full) {
            h_ref = hash_vec_full(r, voff / 8);
            ref_sum += h_ref;
        }
#pragma unroll 1
        for (int k0 = 0; k0 < kg; k0 += 4) {
            // four candidates' loads are issued together (a tiny tensor is nothing but this function: the
            // loads' latency, not their number, is its cost)
            uint4 cc[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) cc[u] = (k0 + u < kg && nvalid > 0) ? load_vec_any(esz, wptr[k0 + u], voff, nbytes) : r;
#pragma unroll 1
            for (int u = 0; u < 4 && k0 + u < kg; ++u) {
                const int k = k0 + u;
                const uint4 c = u == 0 ? cc[0] : u == 1 ? cc[1] : u == 2 ? cc[2] : cc[3];
                if (nvalid > 0 && !full) ragged_elements(dt, c, r, voff, nvalid, tol, &wacc[k], &slots[k * 32]);
                const bool want = full && ((c.x != r.x) || (c.y != r.y) || (c.z != r.z) || (c.w != r.w) || force);
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, want);
                if (bal == 0u) continue;
                const uint32_t at = qbase + ((qhead + qcount + __popc(bal & lanes_below)) & (kQCap - 1)) * 16u;
                const uint64_t meta = voff | static_cast<uint64_t>(k);
                sts128x3_if(at, kQPlane, c, r, make_uint4(static_cast<uint32_t>(meta), static_cast<uint32_t>(meta >> 32),
                                                          static_cast<uint32_t>(h_ref), static_cast<uint32_t>(h_ref >> 32)), want);
                qcount += __popc(bal);
                if (qcount >= 32u) {
                    __syncwarp();
                    ragged_batch(dt, qbase, qhead, 32u, slots, wacc, tol);
                    __syncwarp();
                    qhead = (qhead + 32u) & (kQCap - 1);
                    qcount -= 32u;
                }
            }
        }
    }
    if (qcount) {
        __syncwarp();
        ragged_batch(dt, qbase, qhead, qcount, slots, wacc, tol);
        __syncwarp();
    }
    return ref_sum;
}

// Tiles [tile_begin, tile_end) of one tensor against kg of its candidates (pointers in wptr).
// Full tiles with 16-byte aligned bases are streamed through the lane's asynchronous-copy ring, so the
// loads of the next tile or two fly while the current one is compared. The ragged tail tile, unaligned
// tensors and tensors of 32 GiB or more (whose hash needs 64-bit word indices, which the streamed loops
// do not carry) use synchronous element-sized loads.
// FOUR: the instance for exactly four candidates per tensor (the usual handful of sampled runs): tile
// by tile, the reference vector in a two-deep stage of its own and the four candidate vectors as one
// block of the ring, two tiles in flight; one wait, one vote and one commit per tile, pointers in
// registers. The other instance takes any number of candidates through one sequence of copies.
template <bool FOUR>
__device__ __noinline__ uint64_t ragged_stream(const RaggedParams& p, int dt, uint64_t tile_begin, uint64_t full_end, int kg,
                                               unsigned char* smem) {
    // (The streamed tiles of one tensor part. Out of line and self-contained -- it takes its pointers from the
    // warp's table in shared memory -- so that its loops get a register allocation that nothing around them,
    // neither the tail code nor the chunk bookkeeping, can disturb. Returns the sum of the reference's hash
    // terms over the tiles it met.)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    using S = RaggedSmem<FOUR>;
    uint2* slots = reinterpret_cast<uint2*>(smem + S::kSlotOff) + size_t(warp) * S::kCands * 32 + lane;
    CtaAcc* wacc = reinterpret_cast<CtaAcc*>(smem + S::kAccOff) + warp * S::kCands;
    const unsigned char* const* wsrc = reinterpret_cast<const unsigned char* const*>(smem + S::kPtrOff) + warp * (S::kCands + 2);
    const uint32_t ring_base = smem_u32(smem + S::kRingOff) + (warp * kRing * 32 + lane) * 16;
    const uint32_t qbase = smem_u32(smem + S::kQueueOff) + warp * static_cast<uint32_t>(kQueueBytes);
    const uint32_t refst_base = smem_u32(smem + S::kRefOff) + (warp * 2 * 32 + lane) * 16;
    const TolF tol = {p.atol, p.rtol, p.equal_nan};
    const bool nan_matters = (dt <= GV_F16) && !p.equal_nan;

    // As in the dense kernel, a vector identical to the reference vector contributes the reference
    // vector's own hash terms: those are summed once per tile (ref_sum), the slots only collect the
    // corrections hash(c) - hash(r) of differing vectors, and ref_sum is added to every slot at the end.
    uint64_t ref_sum = 0;
    // Streamed tiles (the whole warp is present): differing vectors go to the warp's queue and are
    // compared 32 at a time, one per lane, like the dense kernel's sparse visits.
    const uint32_t lanes_below = (1u << lane) - 1u;
    uint32_t qhead = 0u, qcount = 0u;
    auto queued_visit = [&](const uint4& c, const uint4& r, uint64_t h_ref, bool force, uint64_t voff, int k) {
        const bool want = (c.x != r.x) || (c.y != r.y) || (c.z != r.z) || (c.w != r.w) || force;
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, want);
        if (bal == 0u) return;
        {
            const uint32_t at = qbase + ((qhead + qcount + __popc(bal & lanes_below)) & (kQCap - 1)) * 16u;
            const uint64_t meta = voff | static_cast<uint64_t>(k);
            sts128x3_if(at, kQPlane, c, r, make_uint4(static_cast<uint32_t>(meta), static_cast<uint32_t>(meta >> 32),
                                                      static_cast<uint32_t>(h_ref), static_cast<uint32_t>(h_ref >> 32)), want);
        }
        qcount += __popc(bal);
        if (qcount >= 32u) {
            __syncwarp();
            ragged_batch(dt, qbase, qhead, 32u, slots, wacc, tol);
            __syncwarp();
            qhead = (qhead + 32u) & (kQCap - 1);
            qcount -= 32u;
        }
    };

    if constexpr (FOUR) {
        const unsigned char* src_r = wsrc[0] + lane * 16;
        const unsigned char* src_c[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) src_c[u] = wsrc[1 + u] + lane * 16;
        auto issue_tile = [&](uint64_t tile, uint32_t half) {     // half: 0 or 1, which half of the ring / reference stage
            if (tile < full_end) {
                const uint64_t off = tile * kWarpTile;
                cp_async16(refst_base + half * 512u, src_r + off);
#pragma unroll
                for (int u = 0; u < 4; ++u) cp_async16(ring_base + (half * 4u + u) * 512u, src_c[u] + off);
            }
            cp_async_commit();
        };
        issue_tile(tile_begin, 0u);
        issue_tile(tile_begin + 1, 1u);
        uint32_t half = 0u;
#pragma unroll 1
        for (uint64_t tile = tile_begin; tile < full_end; ++tile) {
            const uint64_t voff = tile * kWarpTile + lane * 16;     // (below 32 GiB: word indices fit 32 bits)
            cp_async_wait<1>();                                   // this tile's group has landed
            const uint4 r = lds128(refst_base + half * 512u);
            uint4 c[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) c[u] = lds128(ring_base + (half * 4u + u) * 512u);
            issue_tile(tile + 2, half);                           // refill the stages just read
            half ^= 1u;
            const bool force = nan_matters && vec_has_nonfinite(dt, r);
            const uint64_t h_ref = hash_vec_full_k32(r, static_cast<uint32_t>(voff / 8));
            ref_sum += h_ref;
            // one test for the common case (all four candidate vectors identical to the reference vector)
            uint32_t any_diff = 0u;
#pragma unroll
            for (int u = 0; u < 4; ++u) any_diff |= (c[u].x ^ r.x) | (c[u].y ^ r.y) | (c[u].z ^ r.z) | (c[u].w ^ r.w);
            if (__any_sync(0xFFFFFFFFu, any_diff != 0u || force)) {
#pragma unroll
                for (int u = 0; u < 4; ++u) queued_visit(c[u], r, h_ref, force, voff, u);
            }
        }
    } else {
        // The copies form one sequence: per tile the reference vector, then the kg candidate vectors.
        // The stage a visit has just consumed is refilled at once with the copy kRing places ahead,
        // so consumer and producer share one stage counter. src[0] is the reference, src[1 + k]
        // candidate k (wsrc, one table per warp in shared memory).
        const uint64_t end_off = full_end * kWarpTile;
        uint64_t issue_off = tile_begin * kWarpTile + lane * 16;        // this lane's byte offset of the next copy
        int issue_j = 0;
        auto issue_one = [&](uint32_t stage_addr) {
            if (issue_off < end_off) {
                cp_async16(stage_addr, wsrc[issue_j] + issue_off);
                const bool wrap = issue_j == kg;
                issue_j = wrap ? 0 : issue_j + 1;
                issue_off += wrap ? kWarpTile : 0;
            }
            cp_async_commit();
        };
#pragma unroll 1
        for (int j = 0; j < kRing; ++j) issue_one(ring_base + j * 512u);
        uint32_t stage = 0;
        uint64_t tile = tile_begin;
        if (kg == 1) {
            // One candidate per tensor: two tiles per iteration (four copies of the sequence), the two
            // reference hashes side by side -- a single tile's chain of dependent instructions is too short
            // of parallelism for 16 warps per SM to hide.
#pragma unroll 1
            for (; tile + 2 <= full_end; tile += 2) {
                const uint64_t voff0 = tile * kWarpTile + lane * 16, voff1 = voff0 + kWarpTile;
                cp_async_wait<kRing - 4>();
                const uint32_t at0 = ring_base + stage * 512u, at1 = ring_base + ((stage + 1u) & (kRing - 1)) * 512u;
                const uint32_t at2 = ring_base + ((stage + 2u) & (kRing - 1)) * 512u, at3 = ring_base + ((stage + 3u) & (kRing - 1)) * 512u;
                const uint4 r0 = lds128(at0), c0 = lds128(at1), r1 = lds128(at2), c1 = lds128(at3);
                stage = (stage + 4u) & (kRing - 1);
                issue_one(at0);
                issue_one(at1);
                issue_one(at2);
                issue_one(at3);
                const bool force0 = nan_matters && vec_has_nonfinite(dt, r0), force1 = nan_matters && vec_has_nonfinite(dt, r1);
                const uint64_t h0 = hash_vec_full_k32(r0, static_cast<uint32_t>(voff0 / 8));
                const uint64_t h1 = hash_vec_full_k32(r1, static_cast<uint32_t>(voff1 / 8));
                ref_sum += h0 + h1;
                queued_visit(c0, r0, h0, force0, voff0, 0);
                queued_visit(c1, r1, h1, force1, voff1, 0);
            }
        }
#pragma unroll 1
        for (; tile < full_end; ++tile) {
            const uint64_t voff = tile * kWarpTile + lane * 16;
            cp_async_wait<kRing - 1>();
            uint32_t at = ring_base + stage * 512u;
            const uint4 r = lds128(at);
            stage = (stage + 1u) & (kRing - 1);
            issue_one(at);
            const bool force = nan_matters && vec_has_nonfinite(dt, r);
            const uint64_t h_ref = hash_vec_full_k32(r, static_cast<uint32_t>(voff / 8));
            ref_sum += h_ref;
#pragma unroll 1
            for (int k = 0; k < kg; ++k) {
                cp_async_wait<kRing - 1>();
                at = ring_base + stage * 512u;
                const uint4 c = lds128(at);
                stage = (stage + 1u) & (kRing - 1);
                issue_one(at);
                queued_visit(c, r, h_ref, force, voff, k);
            }
        }
    }
    cp_async_wait<0>();
    if (qcount) {                                   // the tensor's accumulators close: drain the queue
        __syncwarp();
        ragged_batch(dt, qbase, qhead, qcount, slots, wacc, tol);
        __syncwarp();
    }
    return ref_sum;
}

template <bool FOUR>
__device__ __forceinline__ void ragged_stretch(const RaggedParams& p, int dt, const unsigned char* ref, uint64_t n,
                                               uint64_t tile_begin, uint64_t tile_end, int kg, uint2* slots,
                                               CtaAcc* wacc, const unsigned char* const* wsrc, unsigned char* smem) {
    const unsigned char* const* wptr = wsrc + 1;        // wsrc[0] = the reference, wsrc[1 + k] = candidate k
    const int esz = elem_size(dt);
    const uint64_t nbytes = n * esz;
    bool streamed = (reinterpret_cast<uintptr_t>(ref) & 15u) == 0 && nbytes < (1ull << 35);
    for (int k = 0; k < kg; ++k) streamed = streamed && (reinterpret_cast<uintptr_t>(wptr[k]) & 15u) == 0;
    const uint64_t full_end_all = nbytes / kWarpTile;                  // tiles [0, full_end_all) are full
    const uint64_t full_end = streamed ? (tile_end < full_end_all ? tile_end : full_end_all) : tile_begin;
    uint64_t ref_sum = 0;
    if (full_end > tile_begin) ref_sum = ragged_stream<FOUR>(p, dt, tile_begin, full_end, kg, smem);
    // ---- synchronous part: the tail tile, or every tile of a tensor that is not streamed (out of line too) ----
    if (full_end < tile_end) {
        const TolF tol = {p.atol, p.rtol, p.equal_nan};
        const uint32_t qbase = smem_u32(smem + RaggedSmem<FOUR>::kQueueOff) + (threadIdx.x >> 5) * static_cast<uint32_t>(kQueueBytes);
        ref_sum += ragged_tail(dt, ref, nbytes, full_end, tile_end, kg, slots, wacc, wptr, tol, (dt <= GV_F16) && !p.equal_nan, qbase);
    }
    for (int k = 0; k < kg; ++k) {
        const uint2 sl = slots[k * 32];
        const uint64_t h = pack64(sl.x, sl.y) + ref_sum;
        slots[k * 32] = make_uint2(static_cast<uint32_t>(h), static_cast<uint32_t>(h >> 32));
    }
}

// Work distribution of the ragged kernel. The tile sequence of all tensors is cut into chunks: the first
// three quarters into large ones, the rest into small ones. A warp takes chunk `gw` first and further
// chunks from a global counter, so warps whose tiles are costly (data that differs everywhere) simply
// take fewer of them; the large chunks keep the cost of starting a chunk (locating its tensor, refilling
// the copy pipeline, publishing partial records) small, the small ones keep the warps' finishing times
// close. Chunk sizes follow the amount of work: about eight large chunks per warp, at most kChunkBig tiles
// each (a batch of a few thousand tiny tensors is thus spread over all warps, one tile at a time).
struct ChunkPlan {
    uint64_t total, n_big, n_chunks, big_end;
    uint32_t big, small;
    __device__ __forceinline__ ChunkPlan(uint64_t total_tiles, uint64_t warps_in_grid) {
        total = total_tiles;
        const uint64_t want = total_tiles / (8 * warps_in_grid);
        big = static_cast<uint32_t>(want < 1 ? 1 : (want > kChunkBig ? kChunkBig : want));
        small = big / 4 ? big / 4 : 1u;
        n_big = (total_tiles - total_tiles / 4) / big;
        big_end = n_big * big;
        n_chunks = n_big + (total_tiles - big_end + small - 1) / small;
    }
    __device__ __forceinline__ void range(uint64_t c, uint64_t& begin, uint64_t& end) const {
        if (c < n_big) { begin = c * big; end = begin + big; }
        else { begin = big_end + (c - n_big) * small; end = begin + small < total ? begin + small : total; }
    }
};

// The table entries of tensor t, one per lane and all in flight together (a dependent chain of loads per
// tensor is what made batches of tiny tensors slow): lane 0 the tensor's first unit in the work sequence,
// lane 1 its end, lane 2 the dtype, lane 3 the element count (or the next reference offset when counts are
// read off the offsets), lane 4 the reference offset, lanes kMetaCand.. the offsets of its first 16 candidates.
constexpr int kMetaCand = 8;
__device__ __forceinline__ uint64_t load_meta(const RaggedParams& p, int64_t t, int lane) {
    uint64_t v = 0;
    if (t < p.T) {
        if (lane == 0) v = static_cast<uint64_t>(p.tile_prefix[t]);
        else if (lane == 1) v = static_cast<uint64_t>(p.tile_prefix[t + 1]);
        else if (lane == 2) v = p.dtypes[t];
        else if (lane == 3) v = static_cast<uint64_t>(p.n_elems ? p.n_elems[t] : p.ref_off[t + 1]);
        else if (lane == 4) v = static_cast<uint64_t>(p.ref_off[t]);
        else if (lane >= kMetaCand && lane - kMetaCand < (p.N < kChunk ? p.N : kChunk))
            v = static_cast<uint64_t>(p.cand_off[t * p.N + (lane - kMetaCand)]);
    }
    return v;
}

// One tensor's tiles [tile_begin, tile_end) against all its candidates, from pointer set-up to the publication
// of the partial records. Out of line on purpose: the streaming loops inside get a register allocation of
// their own, separate from the chunk bookkeeping of the kernel that calls this.
template <bool FOUR>
__device__ __noinline__ void ragged_part(const RaggedParams& p, int64_t t, uint64_t tile_begin, uint64_t tile_end,
                                         unsigned char* smem) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    using S = RaggedSmem<FOUR>;
    uint2* slots = reinterpret_cast<uint2*>(smem + S::kSlotOff) + size_t(warp) * S::kCands * 32 + lane;
    CtaAcc* wacc = reinterpret_cast<CtaAcc*>(smem + S::kAccOff) + warp * S::kCands;
    const unsigned char** wsrc = reinterpret_cast<const unsigned char**>(smem + S::kPtrOff) + warp * (S::kCands + 2);
    // the tensor's table entries, as the caller's load_meta delivered them (one per lane, now in shared memory)
    const unsigned long long* wmeta = reinterpret_cast<const unsigned long long*>(smem + S::kMetaOff) + warp * 32;
    const int dt = static_cast<int>(wmeta[2]);
    const uint64_t n = p.n_elems ? wmeta[3] : (wmeta[3] - wmeta[4]) / static_cast<uint64_t>(elem_size(dt));
    const unsigned char* ref = p.ref_base + wmeta[4];
    for (int c0 = 0; c0 < p.N; c0 += S::kCands) {
        const int kg = FOUR ? 4 : min(S::kCands, p.N - c0);
        __syncwarp();
        // candidate pointers: the first group's offsets came with the tensor's other table entries (lanes
        // kMetaCand .. kMetaCand + 15 of lane_meta, see load_meta), further groups are read here
        if (c0 == 0) {
            if (lane < kg) wsrc[1 + lane] = p.cand_base + wmeta[kMetaCand + lane];
        } else if (lane < kg) {
            wsrc[1 + lane] = p.cand_base + p.cand_off[t * p.N + c0 + lane];
        }
        if (lane < kg) wacc[lane].clear();
        if (lane == 0) wsrc[0] = ref;
        for (int k = 0; k < kg; ++k) slots[k * 32] = make_uint2(0u, 0u);
        __syncwarp();
        ragged_stretch<FOUR>(p, dt, ref, n, tile_begin, tile_end, kg, slots, wacc, wsrc, smem);
        __syncwarp();
        // leave the tensor (or this group of its candidates): combine and publish
        for (int k = 0; k < kg; ++k) {
            const uint2 sl = slots[k * 32];
            const uint64_t h = warp_sum_u64(pack64(sl.x, sl.y));
            if (lane == 0 && h) wacc[k].hash += h;
        }
        __syncwarp();
        if (lane < kg) push_global(&p.results[t * p.N + c0 + lane], wacc[lane]);
    }
}

template <bool FOUR>
__global__ void __launch_bounds__(RaggedSmem<FOUR>::kCtaThreads, RaggedSmem<FOUR>::kCtasPerSm)
ragged_kernel(const __grid_constant__ RaggedParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    using S = RaggedSmem<FOUR>;
    unsigned long long* wmeta = reinterpret_cast<unsigned long long*>(smem + S::kMetaOff) + warp * 32;
    const uint64_t gw = static_cast<uint64_t>(blockIdx.x) * S::kWarpsPerCta + warp;
    const uint64_t GW = static_cast<uint64_t>(gridDim.x) * S::kWarpsPerCta;
    const ChunkPlan plan(static_cast<uint64_t>(p.tile_prefix[p.T]), GW);
    uint64_t chunk = gw;
    while (chunk < plan.n_chunks) {
        uint32_t next = 0u;
        if (lane == 0) next = atomicAdd(p.counter, 1u);     // reserved now, needed when this chunk is done
        uint64_t begin, end;
        plan.range(chunk, begin, end);

        // tensor holding tile `begin`: last t with tile_prefix[t] <= begin (tensors without tiles are skipped).
        // The warp searches together: 32 probes per round, three rounds for ten thousand tensors.
        int64_t lo = 0, hi = p.T;
        while (hi - lo > 1) {
            const int64_t width = hi - lo;
            const int64_t stride = (width + 31) / 32;
            const int64_t idx = lo + (lane + 1) * stride;
            const bool le = idx < hi && static_cast<uint64_t>(p.tile_prefix[idx]) <= begin;
            const int k = __popc(__ballot_sync(0xFFFFFFFFu, le));     // the prefix is monotone: k leading lanes
            const int64_t nlo = lo + k * stride;
            hi = nlo + stride < hi ? nlo + stride : hi;
            lo = nlo;
        }
        // Walk the tensors of the chunk. A tensor occupies kPartCost + tiles units of the sequence: the first
        // kPartCost stand for the fixed cost of handling it (so chunks of many tiny tensors are not far
        // costlier than chunks of few large ones), the rest are its tiles.
        int64_t t = lo;
        uint64_t item = begin;
        uint64_t meta = load_meta(p, t, lane);
        while (item < end && t < p.T) {         // (t < T always holds for a consistent prefix table; the guard keeps a corrupted one from walking off its end)
            const uint64_t meta_next = load_meta(p, t + 1, lane);       // in flight while tensor t is processed
            const uint64_t t_first = __shfl_sync(0xFFFFFFFFu, meta, 0);
            const uint64_t t_last = __shfl_sync(0xFFFFFFFFu, meta, 1);
            if (t_last > item) {                                    // (else: empty or rejected tensor, no units)
                const uint64_t tiles0 = t_first + kPartCost;        // where the tensor's tiles begin in the sequence
                const uint64_t stop = t_last < end ? t_last : end;
                const uint64_t tile_begin = item > tiles0 ? item - tiles0 : 0;
                const uint64_t tile_end = stop > tiles0 ? stop - tiles0 : 0;
                if (tile_end > tile_begin) {
                    __syncwarp();
                    wmeta[lane] = meta;
                    __syncwarp();
                    ragged_part<FOUR>(p, t, tile_begin, tile_end, smem);
                }
                item = stop;
            }
            meta = meta_next;
            ++t;
        }
        chunk = GW + __shfl_sync(0xFFFFFFFFu, next, 0);
    }
}

}  // namespace gv

// =============================================================================================
// host side: validation, launch configuration, C ABI
// =============================================================================================
namespace {

thread_local char g_last_error[256] = "";

gv_status cuda_fail(cudaError_t e, const char* where) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
    return GV_ERR_CUDA;
}
#define GV_CUDA(call)                                              \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call);      \
    } while (0)

struct DeviceInfo {
    int sm_count = 0;
    bool ready = false;
};
DeviceInfo g_dev[64];

gv_status device_info(int* sm_count) {
    int dev = 0;
    GV_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return GV_ERR_CUDA;
    if (!g_dev[dev].ready) {
        int sms = 0;
        GV_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        g_dev[dev].sm_count = sms;
        g_dev[dev].ready = true;
    }
    *sm_count = g_dev[dev].sm_count;
    return GV_OK;
}

bool tol_valid(const gv_tol* t) {
    // (written so that a NaN fails; above FLT_MAX the binary32 tolerance would be infinite and
    // tol = atol + rtol * |r| a NaN for r = 0)
    const double top = 3.4028234663852886e38;
    return t && t->atol >= 0.0 && t->atol <= top && t->rtol >= 0.0 && t->rtol <= top;
}

template <int DT, bool BIGK, bool REL = false>
gv_status launch_dense_t(const gv::DenseParams& p, int sm_count, cudaStream_t st) {
    constexpr int kWarpsCta = gv::DenseShape<DT>::kWarpsPerCta;
    using S = gv::DenseSmem<kWarpsCta>;
    static int blocks_per_sm[64] = {0};
    int dev = 0;
    GV_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return GV_ERR_CUDA;
    auto kern = gv::dense_kernel<DT, BIGK, REL>;
    if (blocks_per_sm[dev] == 0) {
        GV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(S::kTotal)));
        int b = 0;
        GV_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kern, kWarpsCta * 32, S::kTotal));
        blocks_per_sm[dev] = b > 0 ? b : 1;
    }
    const uint64_t nbytes = p.n * gv::Traits<DT>::ESZ;
    const uint64_t cta_tile = static_cast<uint64_t>(kWarpsCta) * gv::kWarpTile;
    const uint64_t tiles = (nbytes + cta_tile - 1) / cta_tile;
    uint64_t grid = static_cast<uint64_t>(sm_count) * blocks_per_sm[dev];
    if (grid > tiles) grid = tiles;
    if (grid == 0) return GV_OK;
    kern<<<static_cast<unsigned>(grid), kWarpsCta * 32, S::kTotal, st>>>(p);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

gv_status launch_dense(gv_dtype dt, const gv::DenseParams& p, int sm_count, cudaStream_t st) {
    const bool bigk = p.n * static_cast<uint64_t>(gv::elem_size(dt)) >= (1ull << 35);
    if (!bigk && p.rel_regime) {
        switch (dt) {
            case GV_F32: return launch_dense_t<GV_F32, false, true>(p, sm_count, st);
            case GV_BF16: return launch_dense_t<GV_BF16, false, true>(p, sm_count, st);
            case GV_F16: return launch_dense_t<GV_F16, false, true>(p, sm_count, st);
            default: break;
        }
    }
    switch (dt) {
        case GV_F32: return bigk ? launch_dense_t<GV_F32, true>(p, sm_count, st) : launch_dense_t<GV_F32, false>(p, sm_count, st);
        case GV_BF16: return bigk ? launch_dense_t<GV_BF16, true>(p, sm_count, st) : launch_dense_t<GV_BF16, false>(p, sm_count, st);
        case GV_F16: return bigk ? launch_dense_t<GV_F16, true>(p, sm_count, st) : launch_dense_t<GV_F16, false>(p, sm_count, st);
        case GV_I32: return bigk ? launch_dense_t<GV_I32, true>(p, sm_count, st) : launch_dense_t<GV_I32, false>(p, sm_count, st);
        case GV_I64: return bigk ? launch_dense_t<GV_I64, true>(p, sm_count, st) : launch_dense_t<GV_I64, false>(p, sm_count, st);
    }
    return GV_ERR_UNSUPPORTED;
}

// The pre-pass and the main kernel of a ragged call (shared by the two ragged entry points).
template <bool FOUR>
gv_status launch_ragged_t(const gv::RaggedParams& p, int sm_count, cudaStream_t st) {
    using S = gv::RaggedSmem<FOUR>;
    static int blocks_per_sm[64] = {0};
    int dev = 0;
    GV_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return GV_ERR_CUDA;
    auto kern = gv::ragged_kernel<FOUR>;
    if (blocks_per_sm[dev] == 0) {
        GV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(S::kTotal)));
        int b = 0;
        GV_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kern, S::kCtaThreads, S::kTotal));
        blocks_per_sm[dev] = b > 0 ? b : 1;
    }
    const unsigned grid = static_cast<unsigned>(sm_count * blocks_per_sm[dev]);
    kern<<<grid, S::kCtaThreads, S::kTotal, st>>>(p);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}
gv_status launch_ragged(const gv::RaggedParams& p, int sm_count, cudaStream_t st) {
    gv::ragged_prepass_kernel<<<1, 1024, 0, st>>>(p);
    GV_CUDA(cudaGetLastError());
    return p.N == 4 ? launch_ragged_t<true>(p, sm_count, st) : launch_ragged_t<false>(p, sm_count, st);
}

}  // namespace

template <bool LANE2>
gv_status launch_hash(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream) {
    if (!out || (nbytes > 0 && !buf)) return GV_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(out) & 7u) return GV_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int sm_count = 0;
    gv_status rc = device_info(&sm_count);
    if (rc != GV_OK) return rc;
    GV_CUDA(cudaMemsetAsync(out, 0, sizeof(uint64_t), st));
    if (nbytes == 0) return GV_OK;
    const uint64_t nvec = (nbytes + 15) / 16;
    uint64_t grid = (nvec + gv::kThreads - 1) / gv::kThreads;
    const uint64_t cap = static_cast<uint64_t>(sm_count) * 8;
    if (grid > cap) grid = cap;
    gv::hash_kernel<LANE2><<<static_cast<unsigned>(grid), gv::kThreads, 0, st>>>(
        static_cast<const unsigned char*>(buf), nbytes, reinterpret_cast<unsigned long long*>(out));
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}
template <int DT>
gv_status launch_profile(gv::ProfileParams p, uint64_t want_ctas, int sm_count, cudaStream_t st) {
    // one cooperative launch; the grid may not exceed what is resident at once
    static int blocks_per_sm[64] = {0};
    int dev = 0;
    GV_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return GV_ERR_CUDA;
    auto kern = gv::profile_kernel<DT>;
    if (blocks_per_sm[dev] == 0) {
        int b = 0;
        GV_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kern, gv::kProfileThreads, 0));
        blocks_per_sm[dev] = b > 0 ? b : 1;
    }
    uint64_t cap = static_cast<uint64_t>(sm_count) * blocks_per_sm[dev];
    if (cap > gv::kProfileMaxCtas) cap = gv::kProfileMaxCtas;
    const unsigned grid = static_cast<unsigned>(want_ctas < cap ? (want_ctas ? want_ctas : 1) : cap);
    void* args[] = {&p};
    GV_CUDA(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(kern), dim3(grid), dim3(gv::kProfileThreads), args, 0, st));
    return GV_OK;
}

extern "C" {

size_t gv_workspace_bytes(int64_t T, int32_t N) {
    // status word (256 bytes), then either the ragged tile-prefix table (T + 1 entries) or the dense
    // kernel's one classification byte per candidate
    const size_t table = T > 0 ? static_cast<size_t>(T + 1) * sizeof(int64_t) : static_cast<size_t>(N > 0 ? N : 0);
    return 256 + ((table + 255) / 256) * 256;
}

gv_status gv_verify_batch(const void* ref, const void* const* cands, int32_t N, uint64_t n_elems, gv_dtype dt,
                          const gv_tol* tol, gv_result* results, uint64_t* ref_hash, void* workspace,
                          size_t workspace_bytes, void* cuda_stream) {
    if (static_cast<int>(dt) < 0 || static_cast<int>(dt) > GV_I64) return GV_ERR_UNSUPPORTED;
    const int esz = gv::elem_size(dt);
    const bool is_float = dt == GV_F32 || dt == GV_BF16 || dt == GV_F16;
    if (N < 0) return GV_ERR_INVALID_ARG;
    if (N > 0 && (!cands || !results)) return GV_ERR_INVALID_ARG;
    if (n_elems > 0 && !ref) return GV_ERR_INVALID_ARG;
    if (n_elems > (1ull << 60) / esz) return GV_ERR_INVALID_ARG;
    if (is_float && !tol_valid(tol)) return GV_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < gv_workspace_bytes(0, N)) return GV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return GV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ref) % esz) return GV_ERR_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(results) & 7u) return GV_ERR_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(ref_hash) & 7u) return GV_ERR_MISALIGNED;
    for (int32_t j = 0; j < N; ++j) {
        if (n_elems > 0 && !cands[j]) return GV_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(cands[j]) % esz) return GV_ERR_MISALIGNED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int sm_count = 0;
    gv_status rc = device_info(&sm_count);
    if (rc != GV_OK) return rc;

    uint32_t* status = static_cast<uint32_t*>(workspace);
    const uint64_t n_init = static_cast<uint64_t>(N) > 0 ? static_cast<uint64_t>(N) : 1;
    gv::init_results_kernel<<<static_cast<unsigned>((n_init + 255) / 256), 256, 0, st>>>(
        results, static_cast<uint64_t>(N), status, ref_hash);
    GV_CUDA(cudaGetLastError());
    if (n_elems == 0) return GV_OK;

    if (N == 0) {
        if (ref_hash) {
            int grid = sm_count * 8;
            gv::hash_kernel<false><<<grid, gv::kThreads, 0, st>>>(static_cast<const unsigned char*>(ref), n_elems * esz,
                                                           reinterpret_cast<unsigned long long*>(ref_hash));
            GV_CUDA(cudaGetLastError());
        }
        return GV_OK;
    }

    for (int32_t j0 = 0; j0 < N; j0 += gv::kMaxPtrs) {
        gv::DenseParams p;
        p.ref = static_cast<const unsigned char*>(ref);
        p.n = n_elems;
        p.results = results + j0;
        p.ref_hash = j0 == 0 ? reinterpret_cast<unsigned long long*>(ref_hash) : nullptr;
        p.status = status;
        p.atol = is_float ? static_cast<float>(tol->atol) : 0.0f;
        p.rtol = is_float ? static_cast<float>(tol->rtol) : 0.0f;
        p.equal_nan = is_float ? (tol->equal_nan != 0) : 0;
        p.rel_regime = is_float && p.atol < p.rtol * 0.0625f;
        p.N = (N - j0) < gv::kMaxPtrs ? (N - j0) : gv::kMaxPtrs;
        uintptr_t all_bits = reinterpret_cast<uintptr_t>(ref);
        for (int k = 0; k < gv::kMaxPtrs; ++k) {
            p.cands[k] = k < p.N ? static_cast<const unsigned char*>(cands[j0 + k]) : nullptr;
            all_bits |= reinterpret_cast<uintptr_t>(p.cands[k]);
        }
        p.all_aligned = (all_bits & 15u) == 0;
        // one sampling pass decides which candidates take the in-place loop (skipped when the launch is
        // too small for it to pay, below 64 MB of candidates, and when the fast loop cannot run at all:
        // everything then takes the queueing loop)
        unsigned char* flags = static_cast<unsigned char*>(workspace) + 256 + j0;
        const uint64_t full_tiles = p.all_aligned ? n_elems * esz / gv::kWarpTile : 0;
        p.flags = nullptr;
        if (full_tiles >= 64 && full_tiles * gv::kWarpTile * static_cast<uint64_t>(p.N) >= (64ull << 20)) {
            p.flags = flags;
            gv::classify_kernel<<<p.N, gv::kThreads, 0, st>>>(p, full_tiles, flags);
            GV_CUDA(cudaGetLastError());
        }
        rc = launch_dense(dt, p, sm_count, st);
        if (rc != GV_OK) return rc;
    }
    return GV_OK;
}

gv_status gv_verify_ragged(const void* ref_base, const int64_t* ref_off, const void* cand_base,
                           const int64_t* cand_off, const uint8_t* dtypes, const int64_t* n_elems, int64_t T,
                           int32_t N, const gv_tol* tol, gv_result* results, void* workspace,
                           size_t workspace_bytes, void* cuda_stream) {
    if (T < 0 || T > 0x7FFFFFFFll || N < 0) return GV_ERR_INVALID_ARG;
    if (T > 0 && (!ref_base || !ref_off || !dtypes)) return GV_ERR_INVALID_ARG;
    if (T > 0 && N > 0 && (!cand_base || !cand_off || !results)) return GV_ERR_INVALID_ARG;
    if (!tol_valid(tol)) return GV_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < gv_workspace_bytes(T, N)) return GV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return GV_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(ref_off) & 7u) || (reinterpret_cast<uintptr_t>(cand_off) & 7u) ||
        (reinterpret_cast<uintptr_t>(n_elems) & 7u) || (reinterpret_cast<uintptr_t>(results) & 7u))
        return GV_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int sm_count = 0;
    gv_status rc = device_info(&sm_count);
    if (rc != GV_OK) return rc;

    uint32_t* status = static_cast<uint32_t*>(workspace);
    const uint64_t count = static_cast<uint64_t>(T) * static_cast<uint64_t>(N);
    const uint64_t n_init = count > 0 ? count : 1;
    gv::init_results_kernel<<<static_cast<unsigned>((n_init + 255) / 256), 256, 0, st>>>(results, count, status,
                                                                                          nullptr);
    GV_CUDA(cudaGetLastError());
    if (count == 0) return GV_OK;

    gv::RaggedParams p;
    p.ref_base = static_cast<const unsigned char*>(ref_base);
    p.ref_off = ref_off;
    p.cand_base = static_cast<const unsigned char*>(cand_base);
    p.cand_off = cand_off;
    p.dtypes = dtypes;
    p.n_elems = n_elems;
    p.T = T;
    p.N = N;
    p.results = results;
    p.status = status;
    p.counter = status + 1;
    p.tile_prefix = reinterpret_cast<int64_t*>(static_cast<unsigned char*>(workspace) + 256);
    p.atol = static_cast<float>(tol->atol);
    p.rtol = static_cast<float>(tol->rtol);
    p.equal_nan = tol->equal_nan != 0;
    return launch_ragged(p, sm_count, st);
}

// ---------------------------------------------------------------------------------------------
// gv_verify_ragged_noalloc: the ragged verification for callers that have no device memory to lend.
// Its scratch (status word + tile-prefix table) is this fixed array, resident on every GPU that loads
// the library for as long as the process lives.
// ---------------------------------------------------------------------------------------------
#define GV_NOALLOC_SCRATCH_BYTES (256 + (GV_NOALLOC_MAX_TENSORS + 1) * 8)
static __device__ __align__(256) unsigned char g_noalloc_scratch[GV_NOALLOC_SCRATCH_BYTES];

// Device address of g_noalloc_scratch per device. In host code the array's name is only a handle for
// the runtime, not an address a kernel can use; the address is asked for once per device, with that
// device current, the first time the entry point runs there.
static void* g_noalloc_ptr[64] = {nullptr};

gv_status gv_verify_ragged_noalloc(const void* ref_base, const int64_t* ref_off, const void* cand_base,
                                   const int64_t* cand_off, const uint8_t* dtypes, const int64_t* n_elems,
                                   int64_t T, int32_t N, const gv_tol* tol, gv_result* results,
                                   uint32_t* status_out, void* cuda_stream) {
    if (T < 0 || N < 0) return GV_ERR_INVALID_ARG;
    if (T > GV_NOALLOC_MAX_TENSORS) {
        snprintf(g_last_error, sizeof(g_last_error),
                 "gv_verify_ragged_noalloc: T = %lld exceeds GV_NOALLOC_MAX_TENSORS = %d; split the batch or use "
                 "gv_verify_ragged with a caller-provided workspace", static_cast<long long>(T), GV_NOALLOC_MAX_TENSORS);
        return GV_ERR_WORKSPACE;
    }
    if (T > 0 && (!ref_base || !ref_off || !dtypes)) return GV_ERR_INVALID_ARG;
    if (T > 0 && N > 0 && (!cand_base || !cand_off || !results)) return GV_ERR_INVALID_ARG;
    if (!tol_valid(tol)) return GV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ref_off) & 7u) || (reinterpret_cast<uintptr_t>(cand_off) & 7u) ||
        (reinterpret_cast<uintptr_t>(n_elems) & 7u) || (reinterpret_cast<uintptr_t>(results) & 7u) ||
        (reinterpret_cast<uintptr_t>(status_out) & 3u))
        return GV_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int sm_count = 0;
    gv_status rc = device_info(&sm_count);
    if (rc != GV_OK) return rc;
    int dev = 0;
    GV_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return GV_ERR_CUDA;
    if (!g_noalloc_ptr[dev]) {
        void* ptr = nullptr;
        GV_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        g_noalloc_ptr[dev] = ptr;
    }
    unsigned char* scratch = static_cast<unsigned char*>(g_noalloc_ptr[dev]);

    // The array still holds the previous call's status word and table. The status word is cleared by
    // the first kernel below; the table is rewritten in full (entries 0..T) by the pre-pass before the
    // main kernel reads it, so nothing else needs to start from zero.
    uint32_t* status = reinterpret_cast<uint32_t*>(scratch);
    const uint64_t count = static_cast<uint64_t>(T) * static_cast<uint64_t>(N);
    const uint64_t n_init = count > 0 ? count : 1;
    gv::init_results_kernel<<<static_cast<unsigned>((n_init + 255) / 256), 256, 0, st>>>(results, count, status,
                                                                                          nullptr);
    GV_CUDA(cudaGetLastError());
    if (status_out) GV_CUDA(cudaMemsetAsync(status_out, 0, sizeof(uint32_t), st));
    if (count == 0) return GV_OK;

    gv::RaggedParams p;
    p.ref_base = static_cast<const unsigned char*>(ref_base);
    p.ref_off = ref_off;
    p.cand_base = static_cast<const unsigned char*>(cand_base);
    p.cand_off = cand_off;
    p.dtypes = dtypes;
    p.n_elems = n_elems;
    p.T = T;
    p.N = N;
    p.results = results;
    p.status = status_out ? status_out : status;
    p.counter = status + 1;
    p.tile_prefix = reinterpret_cast<int64_t*>(scratch + 256);
    p.atol = static_cast<float>(tol->atol);
    p.rtol = static_cast<float>(tol->rtol);
    p.equal_nan = tol->equal_nan != 0;
    return launch_ragged(p, sm_count, st);
}

gv_status gv_hash(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream) {
    return launch_hash<false>(buf, nbytes, out, cuda_stream);
}
gv_status gv_hash2(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream) {
    return launch_hash<true>(buf, nbytes, out, cuda_stream);
}

static size_t round256(size_t x) { return (x + 255) / 256 * 256; }

// ---- aggregates: pass/fail summary with pass@k, speedup from latency samples ----
gv_status gv_exec_summary(const gv_result* results, int64_t T, int32_t N, int32_t kmax, uint8_t* pass,
                          int32_t* n_pass, double* pass_at_k, void* cuda_stream) {
    if (T < 0 || N < 0 || kmax < 0 || kmax > N || kmax > GV_PASSK_MAX || !n_pass) return GV_ERR_INVALID_ARG;
    if ((N > 0 && !pass) || (kmax > 0 && !pass_at_k) || (T > 0 && N > 0 && !results)) return GV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(results) & 7u) || (reinterpret_cast<uintptr_t>(n_pass) & 3u) ||
        (reinterpret_cast<uintptr_t>(pass_at_k) & 7u))
        return GV_ERR_MISALIGNED;
    gv::exec_summary_kernel<<<1, gv::kStatsThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        results, T, N, kmax, pass, n_pass, pass_at_k);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}
gv_status gv_speedup(const float* ref_lat, const float* gen_lat, int64_t T, int32_t S_ref, int32_t S_gen,
                     float* median_ref, float* median_gen, float* ratio, double* speedup, void* cuda_stream) {
    if (T < 0 || T > 0x7FFFFFFFll || S_ref < 1 || S_gen < 1 || S_ref > GV_SAMPLES_MAX || S_gen > GV_SAMPLES_MAX || !speedup)
        return GV_ERR_INVALID_ARG;
    if (T > 0 && (!ref_lat || !gen_lat || !median_ref || !median_gen || !ratio)) return GV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ref_lat) & 3u) || (reinterpret_cast<uintptr_t>(gen_lat) & 3u) ||
        (reinterpret_cast<uintptr_t>(median_ref) & 3u) || (reinterpret_cast<uintptr_t>(median_gen) & 3u) ||
        (reinterpret_cast<uintptr_t>(ratio) & 3u) || (reinterpret_cast<uintptr_t>(speedup) & 7u))
        return GV_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (T > 0)
        gv::median_ratio_kernel<<<static_cast<unsigned>(T), gv::kStatsThreads, 0, st>>>(ref_lat, gen_lat, S_ref, S_gen,
                                                                                       median_ref, median_gen, ratio);
    gv::speedup_mean_kernel<<<1, 1, 0, st>>>(ratio, T, speedup);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

gv_status gv_mem_efficiency(const float* lat, const uint64_t* bytes, int64_t T, int32_t S, double peak, float* median,
                            double* bandwidth, double* efficiency, double* mean_efficiency, void* cuda_stream) {
    if (T < 0 || T > 0x7FFFFFFFll || S < 1 || S > GV_SAMPLES_MAX || !mean_efficiency) return GV_ERR_INVALID_ARG;
    if (!(peak > 0.0) || !isfinite(peak)) return GV_ERR_INVALID_ARG;
    if (T > 0 && (!lat || !bytes || !median || !bandwidth || !efficiency)) return GV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(lat) & 3u) || (reinterpret_cast<uintptr_t>(median) & 3u) ||
        (reinterpret_cast<uintptr_t>(bytes) & 7u) || (reinterpret_cast<uintptr_t>(bandwidth) & 7u) ||
        (reinterpret_cast<uintptr_t>(efficiency) & 7u) || (reinterpret_cast<uintptr_t>(mean_efficiency) & 7u))
        return GV_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (T > 0)
        gv::mem_efficiency_kernel<<<static_cast<unsigned>(T), gv::kStatsThreads, 0, st>>>(
            lat, reinterpret_cast<const unsigned long long*>(bytes), S, peak, median, bandwidth, efficiency);
    gv::mean_f64_kernel<<<1, 1, 0, st>>>(efficiency, T, mean_efficiency);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}
gv_status gv_accuracy_matrix(const uint8_t* status, int64_t K, int32_t R, int32_t kmax, int32_t* n_call, int32_t* n_exec,
                             double* call_acc, double* exec_acc, void* cuda_stream) {
    if (K < 0 || K > 0x7FFFFFFFll || R < 0 || R > GV_RUNS_MAX || kmax < 0 || kmax > R) return GV_ERR_INVALID_ARG;
    if (K > 0 && (!n_call || !n_exec || (R > 0 && !status))) return GV_ERR_INVALID_ARG;
    if (kmax > 0 && (!call_acc || !exec_acc)) return GV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(n_call) & 3u) || (reinterpret_cast<uintptr_t>(n_exec) & 3u) ||
        (reinterpret_cast<uintptr_t>(call_acc) & 7u) || (reinterpret_cast<uintptr_t>(exec_acc) & 7u))
        return GV_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (K > 0)
        gv::accuracy_counts_kernel<<<static_cast<unsigned>((K + gv::kStatsThreads - 1) / gv::kStatsThreads), gv::kStatsThreads, 0, st>>>(
            status, K, R, n_call, n_exec);
    if (kmax > 0)
        gv::accuracy_at_k_kernel<<<static_cast<unsigned>(kmax), gv::kStatsThreads, 0, st>>>(n_call, n_exec, K, R, call_acc, exec_acc);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

// ---- error profile of one candidate ----
size_t gv_profile_workspace_bytes(void) {
    return 256 + static_cast<size_t>(gv::kProfileMaxCtas) *
                     (sizeof(gv::ProfileWorst) + GV_PROFILE_LIST * sizeof(unsigned long long));
}
gv_status gv_error_profile(const void* ref, const void* cand, uint64_t n_elems, gv_dtype dt, const gv_tol* tol,
                           uint64_t row_len, gv_profile* out, uint32_t* row_mismatch, void* workspace,
                           size_t workspace_bytes, void* cuda_stream) {
    const int esz = gv::elem_size(dt);
    if (esz == 0) return GV_ERR_UNSUPPORTED;
    if (!out || (n_elems > 0 && (!ref || !cand)) || (row_len > 0 && !row_mismatch)) return GV_ERR_INVALID_ARG;
    const bool is_float = dt <= GV_F16;
    if (is_float && !tol_valid(tol)) return GV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ref) % esz) || (reinterpret_cast<uintptr_t>(cand) % esz) ||
        (reinterpret_cast<uintptr_t>(out) & 7u) || (reinterpret_cast<uintptr_t>(row_mismatch) & 3u))
        return GV_ERR_MISALIGNED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u) || workspace_bytes < gv_profile_workspace_bytes())
        return GV_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int sm_count = 0;
    gv_status rc = device_info(&sm_count);
    if (rc != GV_OK) return rc;
    gv::ProfileParams p;
    p.ref = static_cast<const unsigned char*>(ref);
    p.cand = static_cast<const unsigned char*>(cand);
    p.n = n_elems;
    p.atol = is_float ? static_cast<float>(tol->atol) : 0.0f;
    p.rtol = is_float ? static_cast<float>(tol->rtol) : 0.0f;
    p.equal_nan = is_float ? (tol->equal_nan != 0) : 0;
    p.aligned = ((reinterpret_cast<uintptr_t>(ref) | reinterpret_cast<uintptr_t>(cand)) & 15u) == 0;
    p.row_len = row_len;
    p.out = out;
    p.rows = row_mismatch;
    unsigned char* ws = static_cast<unsigned char*>(workspace) + 256;
    p.cta_worst = reinterpret_cast<gv::ProfileWorst*>(ws);
    p.cta_first = reinterpret_cast<unsigned long long*>(ws + static_cast<size_t>(gv::kProfileMaxCtas) * sizeof(gv::ProfileWorst));
    const uint64_t tiles = (n_elems * esz + 511) / 512;
    const uint64_t want = (tiles + gv::kProfileWarps - 1) / gv::kProfileWarps;
    switch (dt) {
        case GV_F32: return launch_profile<GV_F32>(p, want, sm_count, st);
        case GV_BF16: return launch_profile<GV_BF16>(p, want, sm_count, st);
        case GV_F16: return launch_profile<GV_F16>(p, want, sm_count, st);
        case GV_I32: return launch_profile<GV_I32>(p, want, sm_count, st);
        default: return launch_profile<GV_I64>(p, want, sm_count, st);
    }
}

// ---- grouping of duplicate candidates ----
static uint32_t group_slots(int64_t N) {
    uint32_t s = 16;
    while (static_cast<int64_t>(s) < 2 * N) s <<= 1;
    return s;
}
size_t gv_group_workspace_bytes(int64_t N) {
    if (N < 0 || N > GV_GROUP_MAX) return 0;
    return 256 + (N > gv::kGroupFusedMax ? static_cast<size_t>(group_slots(N)) * 8 : 0);
}
gv_status gv_group_candidates(const gv_result* results, int64_t N, int32_t* group_id, int32_t* group_count,
                              int32_t* n_groups, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (N < 0 || (N > 0 && (!results || !group_id))) return GV_ERR_INVALID_ARG;
    if (N > GV_GROUP_MAX) {
        snprintf(g_last_error, sizeof(g_last_error), "gv_group_candidates: N = %lld exceeds GV_GROUP_MAX = %lld",
                 static_cast<long long>(N), static_cast<long long>(GV_GROUP_MAX));
        return GV_ERR_UNSUPPORTED;
    }
    if (reinterpret_cast<uintptr_t>(results) & 15u) return GV_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(group_id) & 3u) || (reinterpret_cast<uintptr_t>(group_count) & 3u) ||
        (reinterpret_cast<uintptr_t>(n_groups) & 3u))
        return GV_ERR_MISALIGNED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u) || workspace_bytes < gv_group_workspace_bytes(N))
        return GV_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    gv::GroupParams p;
    p.results = results;
    p.N = N;
    p.group_id = group_id;
    p.group_count = group_count;
    p.n_groups = n_groups;
    p.status = static_cast<uint32_t*>(workspace);
    p.slots = group_slots(N);
    p.owner = reinterpret_cast<int*>(static_cast<unsigned char*>(workspace) + 256);
    p.min_index = p.owner + p.slots;
    if (N <= gv::kGroupFusedMax) {
        gv::group_fused_kernel<<<1, gv::kGroupThreads, 0, st>>>(p);     // also covers N == 0: clears n_groups and the status
    } else {
        int sm_count = 0;
        gv_status rc = device_info(&sm_count);
        if (rc != GV_OK) return rc;
        const long long want = (static_cast<long long>(p.slots) + gv::kGroupThreads - 1) / gv::kGroupThreads;
        const unsigned grid = static_cast<unsigned>(want < 8LL * sm_count ? want : 8LL * sm_count);
        gv::group_clear_kernel<<<grid, gv::kGroupThreads, 0, st>>>(p);
        gv::group_insert_kernel<<<grid, gv::kGroupThreads, 0, st>>>(p);
        gv::group_finish_kernel<<<grid, gv::kGroupThreads, 0, st>>>(p);
    }
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

size_t gv_host_staging_bytes(uint64_t n_elems, gv_dtype dt, int32_t slab) {
    const int esz = gv::elem_size(dt);
    if (esz == 0 || slab < 1) return 0;
    const size_t tensor = round256(static_cast<size_t>(n_elems) * esz);
    return gv_workspace_bytes(0, slab) + round256(static_cast<size_t>(slab) * sizeof(gv_result)) + 256 +
           tensor * (static_cast<size_t>(slab) + 1);
}

gv_status gv_verify_batch_host(const void* ref_host, const void* const* cands_host, int32_t N, uint64_t n_elems,
                               gv_dtype dt, const gv_tol* tol, gv_result* results_host, uint64_t* ref_hash_host,
                               void* staging, size_t staging_bytes, void* cuda_stream) {
    if (static_cast<int>(dt) < 0 || static_cast<int>(dt) > GV_I64) return GV_ERR_UNSUPPORTED;
    const int esz = gv::elem_size(dt);
    if (N < 0) return GV_ERR_INVALID_ARG;
    if (N > 0 && (!cands_host || !results_host)) return GV_ERR_INVALID_ARG;
    if (n_elems > 0 && !ref_host) return GV_ERR_INVALID_ARG;
    if (n_elems > (1ull << 60) / esz) return GV_ERR_INVALID_ARG;
    if (dt <= GV_F16 && !tol_valid(tol)) return GV_ERR_INVALID_ARG;      // (before the first copy is enqueued)
    if (!staging || (reinterpret_cast<uintptr_t>(staging) & 255u)) return GV_ERR_WORKSPACE;
    if (staging_bytes < gv_host_staging_bytes(n_elems, dt, 1)) return GV_ERR_WORKSPACE;
    for (int32_t j = 0; j < N; ++j)
        if (n_elems > 0 && !cands_host[j]) return GV_ERR_INVALID_ARG;
    // largest slab that fits
    const size_t tensor = round256(static_cast<size_t>(n_elems) * esz);
    int32_t slab = 1;
    while (slab < N && slab < gv::kMaxPtrs && gv_host_staging_bytes(n_elems, dt, slab + 1) <= staging_bytes) ++slab;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned char* base = static_cast<unsigned char*>(staging);
    const size_t ws_bytes = gv_workspace_bytes(0, slab);
    void* ws = base;
    gv_result* d_res = reinterpret_cast<gv_result*>(base + ws_bytes);
    uint64_t* d_hash = reinterpret_cast<uint64_t*>(base + ws_bytes + round256(static_cast<size_t>(slab) * sizeof(gv_result)));
    unsigned char* d_ref = reinterpret_cast<unsigned char*>(d_hash) + 256;
    unsigned char* d_cand = d_ref + tensor;
    const size_t tbytes = static_cast<size_t>(n_elems) * esz;

    if (tbytes) GV_CUDA(cudaMemcpyAsync(d_ref, ref_host, tbytes, cudaMemcpyHostToDevice, st));
    const void* ptrs[gv::kMaxPtrs];
    bool first = true;
    for (int32_t j0 = 0; j0 < N || first; j0 += slab) {
        const int32_t m = (N - j0) < slab ? (N - j0) : slab;
        for (int32_t k = 0; k < m; ++k) {
            ptrs[k] = d_cand + static_cast<size_t>(k) * tensor;
            if (tbytes)
                GV_CUDA(cudaMemcpyAsync(d_cand + static_cast<size_t>(k) * tensor, cands_host[j0 + k], tbytes,
                                        cudaMemcpyHostToDevice, st));
        }
        gv_status rc = gv_verify_batch(d_ref, ptrs, m, n_elems, dt, tol, d_res, (first && ref_hash_host) ? d_hash : nullptr,
                                       ws, ws_bytes, st);
        if (rc != GV_OK) return rc;
        if (m > 0)
            GV_CUDA(cudaMemcpyAsync(results_host + j0, d_res, static_cast<size_t>(m) * sizeof(gv_result),
                                    cudaMemcpyDeviceToHost, st));
        if (first && ref_hash_host)
            GV_CUDA(cudaMemcpyAsync(ref_hash_host, d_hash, sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
        first = false;
        if (N == 0) break;
    }
    GV_CUDA(cudaStreamSynchronize(st));
    return GV_OK;
}

// Diagnostic: drives the bounded device-side wait to its limit on purpose. One warp arms an mbarrier
// in its own shared memory for a transfer that is never started, polls it through the same bounded
// wait the verify kernels use (with a limit of a few hundred polls, a few milliseconds at most),
// records the expiry in the status word and returns. Nothing traps, faults or waits without limit;
// the context stays usable.
gv_status gv_selftest_wait_expiry(void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u) || workspace_bytes < 256) return GV_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    gv::wait_expiry_kernel<<<1, 32, 0, st>>>(static_cast<uint32_t*>(workspace));
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

// Diagnostic: what a read-only stream reaches on this device (the verify kernels only read their inputs,
// while the usual copy benchmark reads and writes).
gv_status gv_selftest_read_sum(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream) {
    if (!out || (nbytes > 0 && !buf)) return GV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(buf) & 15u) || (nbytes & 15u) || (reinterpret_cast<uintptr_t>(out) & 7u)) return GV_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int sm_count = 0;
    gv_status rc = device_info(&sm_count);
    if (rc != GV_OK) return rc;
    GV_CUDA(cudaMemsetAsync(out, 0, sizeof(uint64_t), st));
    const uint64_t nvec = nbytes / 16;
    if (nvec == 0) return GV_OK;
    uint64_t grid = (nvec + gv::kThreads - 1) / gv::kThreads;
    const uint64_t cap = static_cast<uint64_t>(sm_count) * 8;
    if (grid > cap) grid = cap;
    gv::read_sum_kernel<<<static_cast<unsigned>(grid), gv::kThreads, 0, st>>>(static_cast<const uint4*>(buf), nvec,
                                                                             reinterpret_cast<unsigned long long*>(out));
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

gv_status gv_check(const void* workspace, void* cuda_stream) {
    if (!workspace) return GV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint32_t word = 0;
    GV_CUDA(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st));
    GV_CUDA(cudaStreamSynchronize(st));
    if (word & gv::kStatusTimeout) return GV_ERR_DEVICE_TIMEOUT;
    if (word & gv::kStatusBadTable) return GV_ERR_BAD_TABLE;
    if (word & gv::kStatusGroupOverflow) return GV_ERR_DEVICE_TIMEOUT;      // a bounded probe gave up
    return GV_OK;
}

const char* gv_status_string(gv_status s) {
    switch (s) {
        case GV_OK: return "ok";
        case GV_ERR_INVALID_ARG: return "invalid argument";
        case GV_ERR_UNSUPPORTED: return "unsupported dtype";
        case GV_ERR_MISALIGNED: return "misaligned pointer";
        case GV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GV_ERR_CUDA: return "CUDA runtime error";
        case GV_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case GV_ERR_BAD_TABLE: return "inconsistent ragged tables";
    }
    return "unknown status";
}

const char* gv_last_cuda_error(void) { return g_last_error; }

uint32_t gv_version(void) { return (0u << 16) | (1u << 8) | 0u; }

}  // extern "C"
