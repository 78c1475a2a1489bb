// gv_kernels.cu -- kernels and C ABI of the batched output verifier (sm_100a).
//
// Hot path (one call of gv_verify_batch): init records -> one persistent kernel in which every
// CTA walks its share of reference tiles once per chunk of candidates. The reference tile is
// brought into shared memory by a 1-D bulk async copy (TMA) completing on an mbarrier, double
// buffered so the next tile arrives while the current one is compared against the chunk; each
// thread then keeps its slice of the tile in registers and streams the same slice of every
// candidate of the chunk with 128-bit loads. Per (thread, candidate) partials (hash, mismatch
// count, max |d|) live in conflict-free shared-memory slots for the whole lifetime of the chunk,
// so the warp/block reduction and the global integer atomics happen once per CTA and candidate,
// not once per tile.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "gv.h"
#include "gv_device.cuh"

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

// =============================================================================================
// gv_hash
// =============================================================================================
__global__ void __launch_bounds__(kThreads) hash_kernel(const unsigned char* buf, uint64_t nbytes,
                                                        unsigned long long* out) {
    uint64_t h = 0;
    const uint64_t nvec = (nbytes + 15) / 16;
    const bool aligned = (reinterpret_cast<uintptr_t>(buf) & 15u) == 0;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t v = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x; v < nvec; v += stride) {
        const uint64_t off = v * 16;
        if (aligned && off + 16 <= nbytes) {
            h += hash_vec_full(ldg_stream(buf + off), 2 * v);
        } else {
            // unaligned base or ragged tail: assemble the words byte by byte, zero padded
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            for (int b = 0; b < 16; ++b) {
                if (off + b < nbytes) w[b >> 2] |= static_cast<uint32_t>(buf[off + b]) << (8 * (b & 3));
            }
            const uint64_t rem = nbytes - off;
            h += hash_vec(make_uint4(w[0], w[1], w[2], w[3]), 2 * v, rem > 8 ? 2 : 1);
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
    const unsigned char* cands[kMaxPtrs];
};

// Shared-memory layout of the dense kernel (dynamic):
//   [0, 2*TILE)                     two reference tile buffers (bulk-copy destinations, 128-B aligned)
//   then uint4 slots[kChunk][kThreads]   per (candidate, thread): hash lo, hash hi, count, max|d| bits
//   then CtaAcc acc[kChunk], two mbarriers
template <int V>
struct DenseSmem {
    static constexpr int TILE = kThreads * 16 * V;
    static constexpr size_t kSlots = 2 * TILE;
    static constexpr size_t kAcc = kSlots + sizeof(uint4) * kChunk * kThreads;
    static constexpr size_t kBar = kAcc + sizeof(CtaAcc) * kChunk;
    static constexpr size_t kRefHash = kBar + 2 * sizeof(uint64_t);
    static constexpr size_t kTotal = kRefHash + sizeof(unsigned long long);
};

template <int DT, int V>
__global__ void __launch_bounds__(kThreads) dense_kernel(const __grid_constant__ DenseParams p) {
    constexpr int ESZ = Traits<DT>::ESZ;
    constexpr int EPV = 16 / ESZ;
    constexpr int TILE = DenseSmem<V>::TILE;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* ref_buf = smem;
    uint4* slots = reinterpret_cast<uint4*>(smem + DenseSmem<V>::kSlots);
    CtaAcc* cacc = reinterpret_cast<CtaAcc*>(smem + DenseSmem<V>::kAcc);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + DenseSmem<V>::kBar);
    unsigned long long* s_refhash = reinterpret_cast<unsigned long long*>(smem + DenseSmem<V>::kRefHash);

    const int tid = threadIdx.x;
    const uint64_t nbytes = p.n * ESZ;
    const uint64_t num_tiles = (nbytes + TILE - 1) / TILE;
    const uint64_t my_tiles = blockIdx.x < num_tiles ? (num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int num_groups = (p.N + kChunk - 1) / kChunk;
    const uint64_t num_items = my_tiles * num_groups;
    const bool ref_aligned = (reinterpret_cast<uintptr_t>(p.ref) & 15u) == 0;
    const TolF tol = {p.atol, p.rtol, p.equal_nan};

    if (tid == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        mbar_fence_init();
        *s_refhash = 0;
    }
    __syncthreads();
    if (num_items == 0) return;

    // item s of this CTA = (group s / my_tiles, tile blockIdx.x + (s % my_tiles) * gridDim.x)
    auto tile_of = [&](uint64_t s) { return blockIdx.x + (s % my_tiles) * static_cast<uint64_t>(gridDim.x); };
    auto tile_bytes = [&](uint64_t t) {
        const uint64_t rem = nbytes - t * TILE;
        return static_cast<uint32_t>(rem < TILE ? rem : TILE);
    };
    // a tile can be fetched by the bulk copy when source and size are multiples of 16 bytes
    auto tma_ok = [&](uint64_t t) { return ref_aligned && (tile_bytes(t) & 15u) == 0; };
    auto issue = [&](uint64_t s) {          // called by thread 0 only
        const uint64_t t = tile_of(s);
        if (tma_ok(t)) {
            const uint32_t bytes = tile_bytes(t);
            fence_proxy_async();
            mbar_expect_tx(&bars[s & 1], bytes);
            bulk_load(ref_buf + (s & 1) * TILE, p.ref + t * TILE, bytes, &bars[s & 1]);
        }
    };

    if (tid == 0) issue(0);
    uint32_t phase[2] = {0u, 0u};
    uint64_t my_ref_hash = 0;
    int aborted_buf = -1;      // >= 0: a wait expired on this buffer's barrier

    for (uint64_t s = 0; s < num_items; ++s) {
        const int g = static_cast<int>(s / my_tiles);
        const int kg = min(kChunk, p.N - g * kChunk);
        const uint64_t t = tile_of(s);
        const uint32_t tb = tile_bytes(t);
        const int b = static_cast<int>(s & 1);
        unsigned char* rbuf = ref_buf + b * TILE;

        if (s % my_tiles == 0) {
            // new chunk of candidates: start its accumulators from the identities
            for (int k = 0; k < kg; ++k) slots[k * kThreads + tid] = make_uint4(0u, 0u, 0u, 0u);
            if (tid < kChunk) cacc[tid].clear();
            // (made visible by the barrier below, before any rare-path atomic can touch them)
        }

        // ---- reference tile: wait for the bulk copy, or fetch it with ordinary loads ----
        bool ok = true;
        if (tma_ok(t)) {
            ok = mbar_wait_bounded(&bars[b], phase[b]);
            if (ok) phase[b] ^= 1u;
        } else {
            // ragged tail / unaligned reference: element-sized loads, zero fill to the tile end
            for (uint32_t o = tid * ESZ; o < static_cast<uint32_t>(TILE); o += kThreads * ESZ) {
                if (ESZ == 2) {
                    *reinterpret_cast<unsigned short*>(rbuf + o) =
                        o < tb ? *reinterpret_cast<const unsigned short*>(p.ref + t * TILE + o) : static_cast<unsigned short>(0);
                } else if (ESZ == 4) {
                    *reinterpret_cast<uint32_t*>(rbuf + o) =
                        o < tb ? *reinterpret_cast<const uint32_t*>(p.ref + t * TILE + o) : 0u;
                } else {
                    *reinterpret_cast<unsigned long long*>(rbuf + o) =
                        o < tb ? *reinterpret_cast<const unsigned long long*>(p.ref + t * TILE + o) : 0ull;
                }
            }
            __syncthreads();
        }
        uint4 r[V];
        if (ok) {
#pragma unroll
            for (int v = 0; v < V; ++v) r[v] = *reinterpret_cast<const uint4*>(rbuf + (v * kThreads + tid) * 16);
        }
        ok = __syncthreads_and(ok ? 1 : 0) != 0;       // also: everyone has read its slice of rbuf
        if (!ok) { aborted_buf = b; break; }
        if (tid == 0 && s + 1 < num_items) issue(s + 1);   // next tile lands in the other buffer meanwhile

        // per-vector geometry of this thread
        uint64_t voff[V];      // byte offset of the vector in the tensor
        int nvalid[V];         // elements of the vector that exist
        bool full[V];
#pragma unroll
        for (int v = 0; v < V; ++v) {
            voff[v] = t * TILE + static_cast<uint64_t>(v * kThreads + tid) * 16;
            const uint64_t rem = voff[v] < nbytes ? nbytes - voff[v] : 0;
            nvalid[v] = rem >= 16 ? EPV : static_cast<int>(rem / ESZ);
            full[v] = rem >= 16;
        }

        if (g == 0 && p.ref_hash) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (nvalid[v] > 0) my_ref_hash += hash_vec(r[v], voff[v] / 8, nvalid[v] * ESZ > 8 ? 2 : 1);
            }
        }

        // ---- stream the candidates of the chunk ----
        auto fetch = [&](int k, uint4 (&dst)[V]) {
            const unsigned char* cp = p.cands[g * kChunk + k];
            const bool cal = (reinterpret_cast<uintptr_t>(cp) & 15u) == 0;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (cal && full[v]) dst[v] = ldg_stream(cp + voff[v]);
                else if (nvalid[v] > 0) dst[v] = load_vec_generic<ESZ>(cp, voff[v], nbytes);
                else dst[v] = make_uint4(0u, 0u, 0u, 0u);
            }
        };
        constexpr int PF = (V == 1) ? 4 : 2;        // candidates fetched ahead
        uint4 pre[PF][V];
#pragma unroll
        for (int q = 0; q < PF; ++q) {
            if (q < kg) fetch(q, pre[q]);
        }
        for (int k0 = 0; k0 < kg; k0 += PF) {
#pragma unroll
            for (int q = 0; q < PF; ++q) {
                const int k = k0 + q;
                if (k < kg) {
                    uint4 cur[V];
#pragma unroll
                    for (int v = 0; v < V; ++v) cur[v] = pre[q][v];
                    if (k + PF < kg) fetch(k + PF, pre[q]);
                    Acc a;
                    a.clear();
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        if (nvalid[v] > 0) {
                            a.hash += full[v] ? hash_vec_full(cur[v], voff[v] / 8)
                                              : hash_vec(cur[v], voff[v] / 8, nvalid[v] * ESZ > 8 ? 2 : 1);
                            vec_compare<DT>(cur[v], r[v], voff[v] / ESZ, nvalid[v], tol, a);
                        }
                    }
                    uint4 sl = slots[k * kThreads + tid];
                    const uint64_t h = pack64(sl.x, sl.y) + a.hash;
                    sl.x = static_cast<uint32_t>(h);
                    sl.y = static_cast<uint32_t>(h >> 32);
                    sl.z += a.cnt;
                    sl.w = a.maxabs > sl.w ? a.maxabs : sl.w;
                    slots[k * kThreads + tid] = sl;
                    push_rare(&cacc[k], a);
                }
            }
        }

        // ---- end of a chunk: reduce the slots once and publish ----
        if ((s + 1) % my_tiles == 0) {
            for (int k = 0; k < kg; ++k) {
                const uint4 sl = slots[k * kThreads + tid];
                const uint64_t h = warp_sum_u64(pack64(sl.x, sl.y));
                const uint64_t c = warp_sum_u64(static_cast<uint64_t>(sl.z));
                const uint32_t m = __reduce_max_sync(0xFFFFFFFFu, sl.w);
                if ((tid & 31) == 0) {
                    if (h) atomicAdd(&cacc[k].hash, static_cast<unsigned long long>(h));
                    if (c) atomicAdd(&cacc[k].cnt, static_cast<unsigned long long>(c));
                    if (m) atomicMax(&cacc[k].maxabs, m);
                }
            }
            __syncthreads();
            if (tid < kg) push_global(&p.results[g * kChunk + tid], cacc[tid]);
            __syncthreads();        // records pushed before the next chunk clears the accumulators
        }
    }

    if (aborted_buf >= 0) {
        // flag the timeout, give the one copy still in flight a second bounded chance to land
        // (its destination is this CTA's shared memory), then leave
        if (tid == 0) {
            atomicOr(p.status, kStatusTimeout);
            (void)mbar_wait_bounded(&bars[aborted_buf], phase[aborted_buf]);
        }
        __syncthreads();
        return;
    }
    if (p.ref_hash) {
        const uint64_t h = warp_sum_u64(my_ref_hash);
        if ((tid & 31) == 0 && h) atomicAdd(s_refhash, static_cast<unsigned long long>(h));
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
    int64_t* tile_prefix;       // T+1, workspace
    float atol, rtol;
    int equal_nan;
};

constexpr int kRaggedV = 4;                                  // 16-byte vectors per thread per tile
constexpr int kRaggedTile = kThreads * 16 * kRaggedV;        // 16 KiB

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
                good = good && n >= 0 && ro >= 0 && ro % esz == 0;
                for (int j = 0; good && j < p.N; ++j) {
                    const int64_t co = p.cand_off[t * p.N + j];
                    good = co >= 0 && co % esz == 0;
                }
            }
            if (!good) atomicOr(p.status, kStatusBadTable);
            else tiles = (n * esz + kRaggedTile - 1) / kRaggedTile;
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

// One tile of one tensor against its N candidates; block-wide reduction per candidate.
template <int DT>
__device__ __forceinline__ void ragged_tile(const RaggedParams& p, int64_t t, uint64_t tile, uint64_t n,
                                            const unsigned char* ref, const unsigned char* rbuf,
                                            CtaAcc* cacc) {
    constexpr int ESZ = Traits<DT>::ESZ;
    constexpr int EPV = 16 / ESZ;
    constexpr int V = kRaggedV;
    const int tid = threadIdx.x;
    const uint64_t nbytes = n * ESZ;
    const TolF tol = {p.atol, p.rtol, p.equal_nan};
    (void)ref;

    uint4 r[V];
    uint64_t voff[V];
    int nvalid[V];
    bool full[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        r[v] = *reinterpret_cast<const uint4*>(rbuf + (v * kThreads + tid) * 16);
        voff[v] = tile * kRaggedTile + static_cast<uint64_t>(v * kThreads + tid) * 16;
        const uint64_t rem = voff[v] < nbytes ? nbytes - voff[v] : 0;
        nvalid[v] = rem >= 16 ? EPV : static_cast<int>(rem / ESZ);
        full[v] = rem >= 16;
    }
    for (int j = 0; j < p.N; ++j) {
        const unsigned char* cp = p.cand_base + p.cand_off[t * p.N + j];
        const bool cal = (reinterpret_cast<uintptr_t>(cp) & 15u) == 0;
        uint4 c[V];
#pragma unroll
        for (int v = 0; v < V; ++v) {
            if (cal && full[v]) c[v] = ldg_stream(cp + voff[v]);
            else if (nvalid[v] > 0) c[v] = load_vec_generic<ESZ>(cp, voff[v], nbytes);
            else c[v] = make_uint4(0u, 0u, 0u, 0u);
        }
        Acc a;
        a.clear();
#pragma unroll
        for (int v = 0; v < V; ++v) {
            if (nvalid[v] > 0) {
                a.hash += full[v] ? hash_vec_full(c[v], voff[v] / 8)
                                  : hash_vec(c[v], voff[v] / 8, nvalid[v] * ESZ > 8 ? 2 : 1);
                vec_compare<DT>(c[v], r[v], voff[v] / ESZ, nvalid[v], tol, a);
            }
        }
        // CTA-wide combine for candidate j (slot j % 2 so the next candidate need not wait)
        CtaAcc* s = &cacc[j & 1];
        const uint64_t h = warp_sum_u64(a.hash);
        const uint32_t c32 = __reduce_add_sync(0xFFFFFFFFu, a.cnt);
        const uint32_t m = __reduce_max_sync(0xFFFFFFFFu, a.maxabs);
        if ((tid & 31) == 0) {
            if (h) atomicAdd(&s->hash, static_cast<unsigned long long>(h));
            if (c32) atomicAdd(&s->cnt, static_cast<unsigned long long>(c32));
            if (m) atomicMax(&s->maxabs, m);
        }
        push_rare(s, a);
        __syncthreads();
        if (tid == 0) {
            push_global(&p.results[t * p.N + j], *s);
            s->clear();
        }
        // the slot is reused two candidates later; the barrier of the next iteration orders that
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads) ragged_kernel(const __grid_constant__ RaggedParams p) {
    __shared__ __align__(128) unsigned char rbuf[kRaggedTile];
    __shared__ CtaAcc cacc[2];
    __shared__ uint64_t bar;
    const int tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
        cacc[0].clear();
        cacc[1].clear();
    }
    __syncthreads();
    const int64_t total = p.tile_prefix[p.T];
    uint32_t phase = 0;
    for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
        // tensor of this item: last t with tile_prefix[t] <= item
        int64_t lo = 0, hi = p.T;          // invariant: tile_prefix[lo] <= item < tile_prefix[hi]
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (p.tile_prefix[mid] <= item) lo = mid; else hi = mid;
        }
        const int64_t t = lo;
        const uint64_t tile = static_cast<uint64_t>(item - p.tile_prefix[t]);
        const int dt = p.dtypes[t];
        const int esz = elem_size(dt);
        const uint64_t n = p.n_elems ? static_cast<uint64_t>(p.n_elems[t])
                                     : static_cast<uint64_t>(p.ref_off[t + 1] - p.ref_off[t]) / esz;
        const unsigned char* ref = p.ref_base + p.ref_off[t];
        const uint64_t nbytes = n * esz;
        const uint64_t rem = nbytes - tile * kRaggedTile;
        const uint32_t tb = static_cast<uint32_t>(rem < kRaggedTile ? rem : kRaggedTile);
        const unsigned char* src = ref + tile * kRaggedTile;

        bool ok = true;
        if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0 && (tb & 15u) == 0) {
            if (tid == 0) {
                fence_proxy_async();
                mbar_expect_tx(&bar, tb);
                bulk_load(rbuf, src, tb, &bar);
            }
            // (bytes of rbuf beyond tb keep stale contents; vectors there have no valid element)
            ok = mbar_wait_bounded(&bar, phase);
            if (ok) phase ^= 1u;
        } else {
            for (uint32_t o = tid * esz; o < static_cast<uint32_t>(kRaggedTile); o += kThreads * esz) {
                if (esz == 2)
                    *reinterpret_cast<unsigned short*>(rbuf + o) =
                        o < tb ? *reinterpret_cast<const unsigned short*>(src + o) : static_cast<unsigned short>(0);
                else if (esz == 4)
                    *reinterpret_cast<uint32_t*>(rbuf + o) = o < tb ? *reinterpret_cast<const uint32_t*>(src + o) : 0u;
                else
                    *reinterpret_cast<unsigned long long*>(rbuf + o) =
                        o < tb ? *reinterpret_cast<const unsigned long long*>(src + o) : 0ull;
            }
        }
        ok = __syncthreads_and(ok ? 1 : 0) != 0;
        if (!ok) {
            if (tid == 0) {
                atomicOr(p.status, kStatusTimeout);
                (void)mbar_wait_bounded(&bar, phase);
            }
            __syncthreads();
            return;
        }
        switch (dt) {
            case GV_F32: ragged_tile<GV_F32>(p, t, tile, n, ref, rbuf, cacc); break;
            case GV_BF16: ragged_tile<GV_BF16>(p, t, tile, n, ref, rbuf, cacc); break;
            case GV_F16: ragged_tile<GV_F16>(p, t, tile, n, ref, rbuf, cacc); break;
            case GV_I32: ragged_tile<GV_I32>(p, t, tile, n, ref, rbuf, cacc); break;
            default: ragged_tile<GV_I64>(p, t, tile, n, ref, rbuf, cacc); break;
        }
        // ragged_tile ends with a barrier: rbuf may be overwritten by the next item
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
    return t && isfinite(t->atol) && isfinite(t->rtol) && t->atol >= 0.0 && t->rtol >= 0.0;
}

template <int DT, int V>
gv_status launch_dense_t(const gv::DenseParams& p, int sm_count, cudaStream_t st) {
    using S = gv::DenseSmem<V>;
    static int blocks_per_sm[64] = {0};
    int dev = 0;
    GV_CUDA(cudaGetDevice(&dev));
    auto kern = gv::dense_kernel<DT, V>;
    if (blocks_per_sm[dev] == 0) {
        GV_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(S::kTotal)));
        int b = 0;
        GV_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kern, gv::kThreads, S::kTotal));
        blocks_per_sm[dev] = b > 0 ? b : 1;
    }
    const uint64_t nbytes = p.n * gv::Traits<DT>::ESZ;
    const uint64_t tiles = (nbytes + S::TILE - 1) / S::TILE;
    uint64_t grid = static_cast<uint64_t>(sm_count) * blocks_per_sm[dev];
    if (grid > tiles) grid = tiles;
    if (grid == 0) return GV_OK;
    kern<<<static_cast<unsigned>(grid), gv::kThreads, S::kTotal, st>>>(p);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

gv_status launch_dense(gv_dtype dt, const gv::DenseParams& p, int sm_count, cudaStream_t st) {
    switch (dt) {
        case GV_F32: return launch_dense_t<GV_F32, 2>(p, sm_count, st);
        case GV_BF16: return launch_dense_t<GV_BF16, 1>(p, sm_count, st);
        case GV_F16: return launch_dense_t<GV_F16, 1>(p, sm_count, st);
        case GV_I32: return launch_dense_t<GV_I32, 2>(p, sm_count, st);
        case GV_I64: return launch_dense_t<GV_I64, 2>(p, sm_count, st);
    }
    return GV_ERR_UNSUPPORTED;
}

}  // namespace

extern "C" {

size_t gv_workspace_bytes(int64_t T, int32_t N) {
    (void)N;
    const size_t table = T > 0 ? static_cast<size_t>(T + 1) * sizeof(int64_t) : 0;
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
            gv::hash_kernel<<<grid, gv::kThreads, 0, st>>>(static_cast<const unsigned char*>(ref), n_elems * esz,
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
        p.N = (N - j0) < gv::kMaxPtrs ? (N - j0) : gv::kMaxPtrs;
        for (int k = 0; k < gv::kMaxPtrs; ++k)
            p.cands[k] = k < p.N ? static_cast<const unsigned char*>(cands[j0 + k]) : nullptr;
        rc = launch_dense(dt, p, sm_count, st);
        if (rc != GV_OK) return rc;
    }
    return GV_OK;
}

gv_status gv_verify_ragged(const void* ref_base, const int64_t* ref_off, const void* cand_base,
                           const int64_t* cand_off, const uint8_t* dtypes, const int64_t* n_elems, int64_t T,
                           int32_t N, const gv_tol* tol, gv_result* results, void* workspace,
                           size_t workspace_bytes, void* cuda_stream) {
    if (T < 0 || N < 0) return GV_ERR_INVALID_ARG;
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
    p.tile_prefix = reinterpret_cast<int64_t*>(static_cast<unsigned char*>(workspace) + 256);
    p.atol = static_cast<float>(tol->atol);
    p.rtol = static_cast<float>(tol->rtol);
    p.equal_nan = tol->equal_nan != 0;
    gv::ragged_prepass_kernel<<<1, 1024, 0, st>>>(p);
    GV_CUDA(cudaGetLastError());

    static int blocks_per_sm[64] = {0};
    int dev = 0;
    GV_CUDA(cudaGetDevice(&dev));
    if (blocks_per_sm[dev] == 0) {
        int b = 0;
        GV_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, gv::ragged_kernel, gv::kThreads, 0));
        blocks_per_sm[dev] = b > 0 ? b : 1;
    }
    const unsigned grid = static_cast<unsigned>(sm_count * blocks_per_sm[dev]);
    gv::ragged_kernel<<<grid, gv::kThreads, 0, st>>>(p);
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

gv_status gv_hash(const void* buf, uint64_t nbytes, uint64_t* out, void* cuda_stream) {
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
    gv::hash_kernel<<<static_cast<unsigned>(grid), gv::kThreads, 0, st>>>(
        static_cast<const unsigned char*>(buf), nbytes, reinterpret_cast<unsigned long long*>(out));
    GV_CUDA(cudaGetLastError());
    return GV_OK;
}

static size_t round256(size_t x) { return (x + 255) / 256 * 256; }

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

gv_status gv_check(const void* workspace, void* cuda_stream) {
    if (!workspace) return GV_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    uint32_t word = 0;
    GV_CUDA(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st));
    GV_CUDA(cudaStreamSynchronize(st));
    if (word & gv::kStatusTimeout) return GV_ERR_DEVICE_TIMEOUT;
    if (word & gv::kStatusBadTable) return GV_ERR_BAD_TABLE;
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
