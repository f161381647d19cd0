// Device-side helpers: Philox4x32-10, the per-batch id table, warp scans.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#define MG_OUT_SLOT_BASE 65536  // first draw slot of the outgoing direction (incoming + outgoing sampling)
#define MG_SLOT_BITS 24  // per-batch id-table slots are addressed with 24 bits (<= 16M slots)

// Where a node's base representation lives: its partition, and its row in the feature buffer (rows of one node each,
// slot after slot).  Partitions are contiguous equal id ranges unless a partition-id array was given.
struct FeatGeom {
    const int32_t* slot_of_part;    // device [n_parts]; -1 = not resident
    const uint8_t* part_of_node;    // device [n_nodes], or null: partition = id / part_size
    const int32_t* local_of_node;   // device [n_nodes], or null: the node's rank inside its partition (partition-id array given)
    uint32_t part_size;             // rows per slot: ceil(n_nodes / n_parts), or the largest partition's population
    int32_t identity;               // 1: the buffer is the whole table in node order, row = node id
};

__device__ __forceinline__ uint32_t feat_part(const FeatGeom& g, int32_t v) {
    return g.part_of_node ? (uint32_t)g.part_of_node[v] : (uint32_t)v / g.part_size;
}
__device__ __forceinline__ bool feat_resident(const FeatGeom& g, int32_t v) { return g.slot_of_part[feat_part(g, v)] >= 0; }
// row of node v in the buffer (v must be resident)
__device__ __forceinline__ int64_t feat_row(const FeatGeom& g, int32_t v) {
    if (g.identity) return v;
    if (g.part_of_node) return (int64_t)g.slot_of_part[g.part_of_node[v]] * g.part_size + g.local_of_node[v];
    const uint32_t p = (uint32_t)v / g.part_size;
    return (int64_t)g.slot_of_part[p] * g.part_size + ((uint32_t)v - p * g.part_size);
}

// Philox4x32-10 (Salmon et al., SC'11); the draw of (seed, node, hop, slot) is word slot % 4
// of the block with counter (node, 0, hop, slot / 4) and key (seed low, seed high).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

__device__ __forceinline__ uint32_t draw_word(uint64_t seed, uint32_t node, uint32_t hop, uint32_t slot) {
    uint32_t o[4];
    philox4x32_10(node, 0u, hop, slot >> 2, (uint32_t)seed, (uint32_t)(seed >> 32), o);
    const uint32_t s = slot & 3u;
    return s == 0 ? o[0] : (s == 1 ? o[1] : (s == 2 ? o[2] : o[3]));
}

// first probe slot of `id` in a table of `size` slots (any size: multiplicative hash, then multiply-high)
__device__ __forceinline__ uint32_t table_hash(int32_t id, int32_t size) {
    return __umulhi((uint32_t)id * 0x9E3779B1u, (uint32_t)size);
}

// Insert `id` into the open-addressing table `keys` (table_size slots, -1 = empty).
// Returns the slot; *is_new tells whether this call created the entry.  Returns -1 when the
// table is full (the caller raises ST_CAP_TABLE).
__device__ __forceinline__ int32_t table_insert(int32_t* keys, int32_t table_size, int32_t id, bool* is_new) {
    uint32_t slot = table_hash(id, table_size);
    for (int32_t probe = 0; probe < table_size; ++probe) {
        const int32_t old = atomicCAS(&keys[slot], -1, id);
        if (old == -1) { *is_new = true; return (int32_t)slot; }
        if (old == id) { *is_new = false; return (int32_t)slot; }
        slot = slot + 1u == (uint32_t)table_size ? 0u : slot + 1u;
    }
    *is_new = false;
    return -1;
}

__device__ __forceinline__ int32_t table_find(const int32_t* keys, int32_t table_size, int32_t id) {
    uint32_t slot = table_hash(id, table_size);
    for (int32_t probe = 0; probe < table_size; ++probe) {
        const int32_t cur = keys[slot];
        if (cur == id) return (int32_t)slot;
        if (cur == -1) return -1;
        slot = slot + 1u == (uint32_t)table_size ? 0u : slot + 1u;
    }
    return -1;
}

// largest j in [0, n) with arr[j] <= x, for a non-decreasing arr with arr[0] <= x
__device__ __forceinline__ int upper_segment(const int32_t* arr, int n, int32_t x) {
    int lo = 0, hi = n;  // invariant: arr[lo] <= x, (hi == n or arr[hi] > x)
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (arr[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}
