// Grouping of duplicate candidates: device code.
//
// Candidates whose 64-byte result records are identical byte for byte (same content hash, same
// statistics) form one group; the group's representative is its member with the smallest index.
// The paper samples many generation runs per reference in parallel (Section 4.2, parallel
// scaling), which yields identical candidates; the content hash in each record exists so that they
// can be recognised. N is small next to the tensors (hundreds to thousands of records), so this is
// latency-bound work: an open-addressing table keyed by a mix of the whole record, one thread per
// record, integer atomics only. The result does not depend on the order in which threads arrive.
#pragma once
#include <stdint.h>

#include "gv.h"

namespace gv {

constexpr int kGroupEmpty = -1;
constexpr int kGroupThreads = 256;
constexpr int kGroupFusedMax = 2048;                 // records a single CTA groups with its table in shared memory
constexpr int kGroupFusedSlots = 2 * kGroupFusedMax; // power of two, load factor <= 1/2
constexpr uint32_t kStatusGroupOverflow = 4u;        // a probe sequence found no slot (cannot happen at load <= 1/2)

struct GroupParams {
    const gv_result* results;
    long long N;
    int* group_id;       // N
    int* group_count;    // N or null
    int* n_groups;       // 1 or null
    int* owner;          // table: index of the record that claimed the slot, or kGroupEmpty
    int* min_index;      // table: smallest index among the records that joined the slot
    unsigned int slots;  // power of two
    uint32_t* status;
};

__device__ __forceinline__ uint4 group_ld(const gv_result* r, int q) {
    return reinterpret_cast<const uint4*>(r)[q];
}
__device__ __forceinline__ bool group_same_record(const gv_result* a, const gv_result* b) {
    bool same = true;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint4 x = group_ld(a, q), y = group_ld(b, q);
        same = same && x.x == y.x && x.y == y.y && x.z == y.z && x.w == y.w;
    }
    return same;
}
// where a record starts probing: every word of the record takes part
__device__ __forceinline__ uint32_t group_start_slot(const gv_result* r, uint32_t slots) {
    uint64_t x = 0x9E3779B97F4A7C15ull;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint4 v = group_ld(r, q);
        x = (x ^ (static_cast<uint64_t>(v.y) << 32 | v.x)) * 0xBF58476D1CE4E5B9ull;
        x ^= x >> 31;
        x = (x ^ (static_cast<uint64_t>(v.w) << 32 | v.z)) * 0x94D049BB133111EBull;
        x ^= x >> 29;
    }
    return static_cast<uint32_t>(x) & (slots - 1u);
}

// Record j finds the slot of its group (claiming an empty one if it is the first to arrive) and
// lowers the slot's smallest index to j. Returns the slot, or -1 if the bounded probe gave up.
__device__ __forceinline__ int group_insert(const gv_result* results, int j, int* owner, int* min_index,
                                            uint32_t slots) {
    const gv_result* mine = results + j;
    uint32_t s = group_start_slot(mine, slots);
    for (uint32_t probe = 0; probe < slots; ++probe) {
        int o = *reinterpret_cast<volatile int*>(&owner[s]);
        if (o == kGroupEmpty) {
            const int prev = atomicCAS(&owner[s], kGroupEmpty, j);
            o = prev == kGroupEmpty ? j : prev;
        }
        if (o == j || group_same_record(results + o, mine)) {
            atomicMin(&min_index[s], j);
            return static_cast<int>(s);
        }
        s = (s + 1u) & (slots - 1u);
    }
    return -1;
}
__device__ __forceinline__ void group_finish(const GroupParams& p, int j, int slot, const int* min_index) {
    if (slot < 0) {
        atomicOr(p.status, kStatusGroupOverflow);
        p.group_id[j] = j;
        return;
    }
    const int g = min_index[slot];
    p.group_id[j] = g;
    if (p.group_count) atomicAdd(&p.group_count[g], 1);
    if (p.n_groups && g == j) atomicAdd(p.n_groups, 1);
}

// N <= kGroupFusedMax: one CTA, table in shared memory, one launch.
__global__ void __launch_bounds__(kGroupThreads) group_fused_kernel(GroupParams p) {
    __shared__ int s_owner[kGroupFusedSlots];
    __shared__ int s_min[kGroupFusedSlots];
    const int tid = threadIdx.x;
    const int N = static_cast<int>(p.N);
    for (int s = tid; s < kGroupFusedSlots; s += kGroupThreads) { s_owner[s] = kGroupEmpty; s_min[s] = 0x7FFFFFFF; }
    for (int j = tid; j < N; j += kGroupThreads) if (p.group_count) p.group_count[j] = 0;
    if (tid == 0) { if (p.n_groups) *p.n_groups = 0; *p.status = 0u; }
    __syncthreads();
    constexpr int kPer = kGroupFusedMax / kGroupThreads;
    int slot_of[kPer];
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int j = tid + i * kGroupThreads;
        slot_of[i] = j < N ? group_insert(p.results, j, s_owner, s_min, kGroupFusedSlots) : 0;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int j = tid + i * kGroupThreads;
        if (j < N) group_finish(p, j, slot_of[i], s_min);
    }
}

// Larger N: table in the workspace, three grid-wide phases as three launches.
__global__ void __launch_bounds__(kGroupThreads) group_clear_kernel(GroupParams p) {
    const long long i = static_cast<long long>(blockIdx.x) * kGroupThreads + threadIdx.x;
    const long long stride = static_cast<long long>(gridDim.x) * kGroupThreads;
    for (long long s = i; s < p.slots; s += stride) { p.owner[s] = kGroupEmpty; p.min_index[s] = 0x7FFFFFFF; }
    if (p.group_count) for (long long j = i; j < p.N; j += stride) p.group_count[j] = 0;
    if (i == 0) { if (p.n_groups) *p.n_groups = 0; *p.status = 0u; }
}
__global__ void __launch_bounds__(kGroupThreads) group_insert_kernel(GroupParams p) {
    const long long i = static_cast<long long>(blockIdx.x) * kGroupThreads + threadIdx.x;
    const long long stride = static_cast<long long>(gridDim.x) * kGroupThreads;
    for (long long j = i; j < p.N; j += stride)      // the slot is parked in group_id until the last phase
        p.group_id[j] = group_insert(p.results, static_cast<int>(j), p.owner, p.min_index, p.slots);
}
__global__ void __launch_bounds__(kGroupThreads) group_finish_kernel(GroupParams p) {
    const long long i = static_cast<long long>(blockIdx.x) * kGroupThreads + threadIdx.x;
    const long long stride = static_cast<long long>(gridDim.x) * kGroupThreads;
    for (long long j = i; j < p.N; j += stride) group_finish(p, static_cast<int>(j), p.group_id[j], p.min_index);
}

}  // namespace gv
