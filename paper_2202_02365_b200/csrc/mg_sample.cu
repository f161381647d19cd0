// DENSE multi-hop sampling (Algorithm 1) for many independent mini-batches per pass.
//
// Layout kept on the device (hop-major, sampling order):
//   nodes[]     hop 0 = the targets of all batches, hop h+1 = the deltas found from hop h,
//               inside a hop batch after batch, inside a batch ascending id (targets: caller order)
//   ent_off[]   for each sampled node its first entry in ent_nbrs / ent_repr (same order as nodes)
//   ent_repr[]  the neighbour's LOCAL row: its position in the batch's node list taken in
//               sampling order (targets first).  In that order the rows layer l needs are the
//               prefix [0, N_l) of the batch, which is what Algorithm 2 achieves by cutting the
//               front of node_ids in the paper's (reversed) order.
// The paper's arrays are produced from this by mg_dense_view.
//
// Every kernel sizes itself from counters in device memory (DenseHeader), so a k-hop sample is
// issued without a host round trip per hop; the host reads the header once at the end.

#include <stdarg.h>

#include <algorithm>
#include <cstdlib>

#include "mg_device.cuh"
#include "mg_internal.cuh"

namespace {

constexpr int kThreads = 256;

// -------------------------------------------------------------------------------------
// generic exclusive scan over a device-sized range (three kernels, no inter-block waits)
// -------------------------------------------------------------------------------------
constexpr int kScanTile = 2048;  // 256 threads x 8

struct ScanRange {       // all device pointers
    const int32_t* lo;   // range is data[*lo .. *hi)
    const int32_t* hi;
    const int32_t* base; // value added to every output (nullable)
};

__device__ __forceinline__ uint32_t block_excl_scan_256(uint32_t v, uint32_t* smem /*>= 9*/, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t inc = warp_incl_scan(v);
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < 8 ? smem[lane] : 0u;
        const uint32_t wi = warp_incl_scan(w);
        if (lane < 8) smem[lane] = wi - w;
        if (lane == 7) smem[8] = wi;
    }
    __syncthreads();
    const uint32_t res = inc - v + smem[warp];
    *total = smem[8];
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(kThreads) k_scan_reduce(const uint32_t* data, ScanRange r, uint32_t* tile_sums) {
    __shared__ uint32_t sm[9];
    const int32_t lo = *r.lo, n = *r.hi - lo;
    const int ntiles = (n + kScanTile - 1) / kScanTile;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        uint32_t s = 0;
        const int start = t * kScanTile + threadIdx.x * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (start + j < n) s += data[lo + start + j];
        uint32_t total;
        block_excl_scan_256(s, sm, &total);
        if (threadIdx.x == 0) tile_sums[t] = total;
    }
}

// what the scan of a hop's entry counts also does once the total is known: close the hop's entry range, check the arena
struct HopClose {
    DenseHeader* hdr;      // null: a plain scan
    int hop;
    int32_t* ent_off;
    int64_t cap_entries;
};

// single block: exclusive scan of the tile sums in place; total (plus base) to *total_out
__global__ void __launch_bounds__(1024) k_scan_tiles(uint32_t* tile_sums, ScanRange r, uint32_t* total_out, HopClose hc) {
    __shared__ uint32_t warp_tot[33];
    const int n = *r.hi - *r.lo;
    const int ntiles = (n + kScanTile - 1) / kScanTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t carry = 0;
    for (int start = 0; start < ntiles; start += 1024) {
        const int i = start + threadIdx.x;
        const uint32_t v = i < ntiles ? tile_sums[i] : 0u;
        const uint32_t inc = warp_incl_scan(v);
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const uint32_t w = warp_tot[lane];
            const uint32_t wi = warp_incl_scan(w);
            warp_tot[lane] = wi - w;
            if (lane == 31) warp_tot[32] = wi;
        }
        __syncthreads();
        if (i < ntiles) tile_sums[i] = carry + warp_tot[warp] + inc - v;
        carry += warp_tot[32];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const uint32_t end = carry + (r.base ? (uint32_t)*r.base : 0u);
        if (total_out) *total_out = end;
        if (hc.hdr && !hc.hdr->status) {
            if ((int64_t)end > hc.cap_entries) atomicOr(&hc.hdr->status, ST_CAP_ENTRIES);
            else {
                hc.hdr->ent_base[hc.hop + 1] = (int32_t)end;
                hc.ent_off[hc.hdr->hop_base[hc.hop + 1]] = (int32_t)end;   // (past the range the scan's last kernel writes)
                hc.hdr->n_new = 0;
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) k_scan_down(uint32_t* data, ScanRange r, const uint32_t* tile_sums) {
    __shared__ uint32_t sm[9];
    const int32_t lo = *r.lo, n = *r.hi - lo;
    const uint32_t base = r.base ? (uint32_t)*r.base : 0u;
    const int ntiles = (n + kScanTile - 1) / kScanTile;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        uint32_t v[8], s = 0;
        const int start = t * kScanTile + threadIdx.x * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            v[j] = (start + j < n) ? data[lo + start + j] : 0u;
            s += v[j];
        }
        uint32_t total;
        uint32_t run = block_excl_scan_256(s, sm, &total) + tile_sums[t] + base;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (start + j < n) data[lo + start + j] = run;
            run += v[j];
        }
    }
}

// -------------------------------------------------------------------------------------
// hop 0: targets
// -------------------------------------------------------------------------------------
struct TableGeom {
    int32_t size;   // slots per batch (any size)
};

// The host-known part of a sample (header, target offsets, per-batch row tables, seeds) is read straight from mapped
// pinned memory by a kernel instead of being copied by a copy engine: a copy engine may be busy for a long time with
// a partition that is being swapped in, and the sample would wait behind it.
__global__ void __launch_bounds__(kThreads)
k_stage_in(const int32_t* __restrict__ stage, int32_t n_hdr, int32_t n_off, int32_t n_cum, int32_t n_seed_words, int32_t seed_at,
           int32_t* hdr, int32_t* node_off, int32_t* cum, int32_t* seeds) {
    const int32_t total = n_hdr + n_off + n_cum + n_seed_words;
    for (int32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        int32_t j = i;
        if (j < n_hdr) hdr[j] = stage[j];
        else if ((j -= n_hdr) < n_off) node_off[j] = stage[n_hdr + j];
        else if ((j -= n_off) < n_cum) cum[j] = stage[n_hdr + n_off + j];
        else seeds[j - n_cum] = stage[seed_at + (j - n_cum)];
    }
}

__global__ void __launch_bounds__(kThreads) k_copy_i32(const int32_t* __restrict__ src, int32_t* dst, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) dst[i] = src[i];
}

__global__ void __launch_bounds__(kThreads)
k_init_targets(DenseHeader* hdr, const int32_t* __restrict__ targets,
               const int32_t* __restrict__ tgt_off, int32_t B, int32_t* nodes, int32_t* node_batch,
               int32_t* hkeys, int32_t* hvals, TableGeom tg, int64_t n_nodes, FeatGeom feat) {
    const int32_t n_total = hdr->hop_base[1];   // read on the device: the launch does not depend on the number of targets
    for (int32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_total; i += gridDim.x * blockDim.x) {
        const int b = upper_segment(tgt_off, B + 1, i);
        const int32_t v = targets[i];
        nodes[i] = v;
        node_batch[i] = b;
        if (v < 0 || (int64_t)v >= n_nodes) { atomicOr(&hdr->status, ST_RANGE); continue; }
        if (!feat_resident(feat, v)) { atomicOr(&hdr->status, ST_NONRESIDENT); continue; }
        bool is_new;
        const int32_t slot = table_insert(hkeys + (int64_t)b * tg.size, tg.size, v, &is_new);
        if (slot < 0) { atomicOr(&hdr->status, ST_CAP_TABLE); continue; }
        if (!is_new) { atomicOr(&hdr->status, ST_DUPLICATE); continue; }
        hvals[(int64_t)b * tg.size + slot] = i - tgt_off[b];
    }
}

// -------------------------------------------------------------------------------------
// per hop: degree -> count, (scan), pick + id-table insert, (sort), place, relabel
// -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
k_count(const DenseHeader* hdr, int hop, int32_t fanout, const int32_t* __restrict__ nodes,
        const int64_t* __restrict__ row_off, int32_t* ent_off, int64_t* node_r0, uint32_t* node_deg,
        const int64_t* __restrict__ row_off_out, int64_t* node_r0_out, uint32_t* node_deg_out) {
    if (hdr->status) return;
    const int32_t lo = hdr->hop_base[hop], hi = hdr->hop_base[hop + 1];
    for (int32_t i = lo + blockIdx.x * blockDim.x + threadIdx.x; i < hi; i += gridDim.x * blockDim.x) {
        const int32_t v = nodes[i];
        const int64_t r0 = row_off[v];
        const int64_t d = row_off[v + 1] - r0;
        int32_t n = (int32_t)(d < (int64_t)fanout ? d : (int64_t)fanout);
        node_r0[i] = r0;        // the one random look-up of the row bounds; k_pick reads these coalesced
        node_deg[i] = (uint32_t)d;
        if (row_off_out) {      // incoming + outgoing sampling: up to `fanout` of each list
            const int64_t q0 = row_off_out[v];
            const int64_t dq = row_off_out[v + 1] - q0;
            n += (int32_t)(dq < (int64_t)fanout ? dq : (int64_t)fanout);
            node_r0_out[i] = q0;
            node_deg_out[i] = (uint32_t)dq;
        }
        ent_off[i] = n;
    }
}

struct PickArgs {
    DenseHeader* hdr;
    int hop;
    int32_t fanout;
    const int32_t* nodes;
    const int32_t* node_batch;
    const int64_t* node_r0;
    const uint32_t* node_deg;
    const int32_t* row_nbrs;
    const int32_t* ent_off;
    int32_t* ent_nbrs;
    int32_t* ent_repr;  // receives the batch id of the entry (k_insert turns it into the id-table slot)
    const uint64_t* seeds;
    // second direction of incoming + outgoing sampling: its picks follow the first direction's min(degree, fanout)
    // entries of the node and its draws use slots slot_base + t
    const uint32_t* pre_deg;   // nullptr for the first (or only) direction
    uint32_t slot_base;
};

// first entry of node i's picks in this launch's direction
__device__ __forceinline__ int32_t pick_base(const PickArgs& a, int32_t i) {
    int32_t out0 = a.ent_off[i];
    if (a.pre_deg) {
        const uint32_t d0 = a.pre_deg[i];
        out0 += (int32_t)(d0 < (uint32_t)a.fanout ? d0 : (uint32_t)a.fanout);
    }
    return out0;
}

// A pick goes to its place in the entry arena; ent_repr carries the batch id until k_insert replaces it.
__device__ __forceinline__ void store_pick(const PickArgs& a, bool valid, int32_t b, int32_t u, int32_t out_pos) {
    if (!valid) return;
    a.ent_nbrs[out_pos] = u;
    a.ent_repr[out_pos] = b;
}

// G lanes per node, fanout <= G <= 32; a warp holds 32 / G nodes (G need not divide 32: the lanes left over idle, and
// G = 5 or 10 keeps 30 lanes busy where the next power of two keeps 20).
template <int G>
__global__ void __launch_bounds__(kThreads) k_pick(PickArgs a) {
    if (a.hdr->status) return;
    constexpr int kPerWarp = 32 / G;
    constexpr int kGroups = (kThreads / 32) * kPerWarp;
    const int32_t lo = a.hdr->hop_base[a.hop], hi = a.hdr->hop_base[a.hop + 1];
    const int lane = threadIdx.x & 31;
    const int grp = lane / G;                     // group inside the warp (== kPerWarp: a left-over lane)
    const int gl = lane - grp * G;                // lane inside the group
    const int gshift = grp * G;                   // first warp lane of the group
    const uint32_t gmask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << gshift);
    const int32_t f = a.fanout;
    for (int32_t base = lo + blockIdx.x * kGroups; base < hi; base += gridDim.x * kGroups) {
        const int32_t i = base + (threadIdx.x >> 5) * kPerWarp + grp;
        const bool node_ok = grp < kPerWarp && i < hi;
        int32_t v = 0, b = 0, out0 = 0;
        int64_t r0 = 0, d = 0;
        if (node_ok) {
            v = a.nodes[i];
            b = a.node_batch[i];
            out0 = pick_base(a, i);
            r0 = a.node_r0[i];
            d = (int64_t)a.node_deg[i];
        }
        bool valid = false;
        int32_t u = 0, pos = 0;
        const bool floyd = node_ok && d > (int64_t)f;
        // Floyd's subset algorithm: slot t draws x in [0, d-f+t]; it keeps x unless an earlier slot
        // already holds x, in which case it keeps d-f+t.  Draws are independent of each other, so
        // all lanes draw at once and only the "already held" test runs slot by slot.
        uint32_t x = 0xFFFFFFFFu, jt = 0, pick = 0xFFFFFFFFu;
        if (floyd && gl < f) {
            jt = (uint32_t)(d - f) + (uint32_t)gl;
            x = __umulhi(draw_word(a.seeds[b], (uint32_t)v, (uint32_t)a.hop, a.slot_base + (uint32_t)gl), jt + 1u);
        }
        for (int t = 0; t < f; ++t) {
            const uint32_t xt = __shfl_sync(0xFFFFFFFFu, x, gshift + t);
            const uint32_t hit = __ballot_sync(0xFFFFFFFFu, gl < t && pick == xt) & gmask;
            if (gl == t) pick = hit ? jt : xt;
        }
        // rank of this lane's position among the f picks (they are distinct); every lane of the warp
        // takes part in the shuffles, whatever its node needs
        int rank = 0;
        for (int t = 0; t < f; ++t) {
            const uint32_t pt = __shfl_sync(0xFFFFFFFFu, pick, gshift + t);
            rank += (pt < pick) ? 1 : 0;
        }
        if (floyd) {
            if (gl < f) {
                valid = true;
                u = a.row_nbrs[r0 + (int64_t)pick];
                pos = out0 + rank;
            }
        } else if (node_ok && (int64_t)gl < d) {
            valid = true;
            u = a.row_nbrs[r0 + gl];
            pos = out0 + gl;
        }
        store_pick(a, valid, b, u, pos);
    }
}

// Any fanout up to MG_MAX_FANOUT: one warp per node, picks staged in shared memory.
__global__ void __launch_bounds__(kThreads) k_pick_wide(PickArgs a) {
    extern __shared__ uint32_t sm_dyn[];  // per warp: x[f], pick[f]
    if (a.hdr->status) return;
    constexpr int kWarps = kThreads / 32;
    const int32_t lo = a.hdr->hop_base[a.hop], hi = a.hdr->hop_base[a.hop + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t f = a.fanout;
    uint32_t* xs = sm_dyn + (size_t)warp * 2 * f;
    uint32_t* picks = xs + f;
    const int rounds = (f + 31) / 32;
    for (int32_t base = lo + blockIdx.x * kWarps; base < hi; base += gridDim.x * kWarps) {
        const int32_t i = base + warp;
        const bool node_ok = i < hi;
        int32_t v = 0, b = 0, out0 = 0;
        int64_t r0 = 0, d = 0;
        if (node_ok) {
            v = a.nodes[i];
            b = a.node_batch[i];
            out0 = pick_base(a, i);
            r0 = a.node_r0[i];
            d = (int64_t)a.node_deg[i];
        }
        const bool floyd = node_ok && d > (int64_t)f;
        if (floyd) {
            for (int t = lane; t < f; t += 32) {
                const uint32_t jt = (uint32_t)(d - f) + (uint32_t)t;
                xs[t] = __umulhi(draw_word(a.seeds[b], (uint32_t)v, (uint32_t)a.hop, a.slot_base + (uint32_t)t), jt + 1u);
            }
            __syncwarp();
            for (int t = 0; t < f; ++t) {
                const uint32_t xt = xs[t];
                bool hit = false;
                for (int s = lane; s < t; s += 32) hit |= (picks[s] == xt);
                const bool any = __any_sync(0xFFFFFFFFu, hit);
                if (lane == 0) picks[t] = any ? ((uint32_t)(d - f) + (uint32_t)t) : xt;
                __syncwarp();
            }
        }
        for (int rd = 0; rd < rounds; ++rd) {
            const int t = rd * 32 + lane;
            bool valid = false;
            int32_t u = 0, pos = 0;
            if (floyd && t < f) {
                const uint32_t p = picks[t];
                int rank = 0;
                for (int s = 0; s < f; ++s) rank += (picks[s] < p) ? 1 : 0;
                valid = true;
                u = a.row_nbrs[r0 + (int64_t)p];
                pos = out0 + rank;
            } else if (node_ok && !floyd && (int64_t)t < d) {
                valid = true;
                u = a.row_nbrs[r0 + t];
                pos = out0 + t;
            }
            store_pick(a, valid, b, u, pos);
        }
        __syncwarp();
    }
}

// Deduplication: every entry's neighbour id goes into its batch's id table.  One thread owns eight
// entries; their first-probe compare-and-swaps are issued back to back (eight atomics in flight per
// thread), collisions are resolved afterwards.  The keys of the ids that were new are appended to the
// list with one global atomic per 2048 entries.
struct InsertArgs {
    DenseHeader* hdr;
    int hop;
    const int32_t* ent_nbrs;
    int32_t* ent_repr;   // in: batch id; out: the node's row (new node) or -1 - (batch * table_size + slot)
    int32_t* hkeys;
    TableGeom tg;
    uint64_t* newlist;
    int64_t cap_new;
    int id_bits;
    // outermost hop only: rows are handed out at insert time
    int32_t k;
    const int32_t* cum;          // [B][k+2]
    int32_t* hvals;
    uint32_t* batch_cnt;         // [B] new nodes of the hop per mini-batch, zero before the launch
    int32_t max_nodes_per_batch;
};

constexpr int kInsertPerThread = 4;
constexpr int kInsertSpan = 16;   // mini-batches a block's chunk of entries may touch on the fast path

// New nodes are not sorted on the device: nothing the path computes depends on the order of ids inside a delta (the
// paper's arrays, with ascending ids, are an export: mg_dense_batch_perm).  A new node takes the next free row of its
// mini-batch right here -- a count per mini-batch in shared memory, one global atomic per (block, mini-batch) --,
// its table value is written at once, and its list entry carries (mini-batch, id, rank in the hop).
__global__ void __launch_bounds__(kThreads) k_insert(InsertArgs a) {
    constexpr bool OUTER = true;
    __shared__ uint32_t warp_tot[kThreads / 32 + 1];
    __shared__ uint32_t block_base;
    __shared__ uint32_t span_cnt[kInsertSpan], span_base[kInsertSpan];
    __shared__ int32_t first_batch;
    if (a.hdr->status) return;
    const int32_t lo = a.hdr->ent_base[a.hop], hi = a.hdr->ent_base[a.hop + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kChunk = kThreads * kInsertPerThread;
    for (int32_t base = lo + blockIdx.x * kChunk; base < hi; base += gridDim.x * kChunk) {
        int32_t u[kInsertPerThread], b[kInsertPerThread], old[kInsertPerThread];
        uint32_t slot[kInsertPerThread];
#pragma unroll
        for (int j = 0; j < kInsertPerThread; ++j) {
            const int32_t e = base + j * kThreads + threadIdx.x;
            u[j] = -1; b[j] = 0; old[j] = 0; slot[j] = 0;
            if (e < hi) { u[j] = a.ent_nbrs[e]; b[j] = a.ent_repr[e]; }
        }
#pragma unroll
        for (int j = 0; j < kInsertPerThread; ++j)
            if (u[j] >= 0) {
                slot[j] = table_hash(u[j], a.tg.size);
                old[j] = atomicCAS(&a.hkeys[(int64_t)b[j] * a.tg.size + slot[j]], -1, u[j]);
            }
        uint32_t n_mine = 0, new_bits = 0;
#pragma unroll
        for (int j = 0; j < kInsertPerThread; ++j) {
            if (u[j] < 0) continue;
            bool fresh = old[j] == -1;
            if (!fresh && old[j] != u[j]) {   // first slot taken by another id: linear probing
                int32_t* keys = a.hkeys + (int64_t)b[j] * a.tg.size;
                int32_t probe = 1;
                for (; probe < a.tg.size; ++probe) {
                    slot[j] = slot[j] + 1u == (uint32_t)a.tg.size ? 0u : slot[j] + 1u;
                    const int32_t o = atomicCAS(&keys[slot[j]], -1, u[j]);
                    if (o == -1) { fresh = true; break; }
                    if (o == u[j]) break;
                }
                if (probe >= a.tg.size) { atomicOr(&a.hdr->status, ST_CAP_TABLE); slot[j] = 0; }
            }
            // an entry that found its node already in the table gets the node's row later (k_relabel): it leaves
            // -1 - (table index) behind; the entry of a new node gets its row below
            if (fresh) { new_bits |= 1u << j; ++n_mine; }
            else a.ent_repr[base + j * kThreads + threadIdx.x] = -1 - (b[j] * a.tg.size + (int32_t)slot[j]);
        }
        // block-wide exclusive scan of the per-thread counts, one global atomic for the block
        const uint32_t inc = warp_incl_scan(n_mine);
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t run = 0;
            for (int w = 0; w < kThreads / 32; ++w) { const uint32_t t = warp_tot[w]; warp_tot[w] = run; run += t; }
            block_base = run ? atomicAdd(&a.hdr->n_new, run) : 0u;
        }
        __syncthreads();
        int64_t pos = (int64_t)block_base + warp_tot[warp] + inc - n_mine;
        uint32_t rank[kInsertPerThread];
        if (OUTER) {
            // entries are ordered by mini-batch, so a chunk touches a short run of them
            if (threadIdx.x == 0) first_batch = b[0];   // thread 0's first item is the chunk's first entry
            if (threadIdx.x < kInsertSpan) span_cnt[threadIdx.x] = 0;
            __syncthreads();
            const int32_t b0 = first_batch;
#pragma unroll
            for (int j = 0; j < kInsertPerThread; ++j) {
                rank[j] = 0;
                if (new_bits & (1u << j)) {
                    const int32_t bb = b[j] - b0;
                    rank[j] = bb < kInsertSpan ? atomicAdd(&span_cnt[bb], 1u) : atomicAdd(&a.batch_cnt[b[j]], 1u);
                }
            }
            __syncthreads();
            if (threadIdx.x < kInsertSpan && span_cnt[threadIdx.x])
                span_base[threadIdx.x] = atomicAdd(&a.batch_cnt[b0 + threadIdx.x], span_cnt[threadIdx.x]);
            __syncthreads();
#pragma unroll
            for (int j = 0; j < kInsertPerThread; ++j)
                if (new_bits & (1u << j)) {
                    const int32_t bb = b[j] - b0;
                    if (bb < kInsertSpan) rank[j] += span_base[bb];
                    const int64_t row = (int64_t)a.cum[b[j] * (a.k + 2) + a.hop + 1] + rank[j];
                    if (row < a.max_nodes_per_batch) a.hvals[(int64_t)b[j] * a.tg.size + slot[j]] = (int32_t)row;
                    else atomicOr(&a.hdr->status, ST_CAP_TABLE);
                    a.ent_repr[base + j * kThreads + threadIdx.x] = (int32_t)row;   // final: no table read for this entry
                }
        }
#pragma unroll
        for (int j = 0; j < kInsertPerThread; ++j)
            if (new_bits & (1u << j)) {
                const uint64_t key = (uint64_t)(OUTER ? rank[j] : slot[j]) | ((uint64_t)(uint32_t)u[j] << MG_SLOT_BITS) |
                                     ((uint64_t)(uint32_t)b[j] << (MG_SLOT_BITS + a.id_bits));
                if (pos < a.cap_new) a.newlist[pos] = key;
                else atomicOr(&a.hdr->status, ST_CAP_NODES);
                ++pos;
            }
        __syncthreads();
    }
}

// -------------------------------------------------------------------------------------
// Last hop: deduplication in shared memory
// -------------------------------------------------------------------------------------
// The last hop has most of the entries (12.9M of 16.6M on the bench) and its new nodes are never looked up again, so
// it does not go through the id tables in global memory.  The ids of a mini-batch are split by hash into nb buckets.
// k_bucket_entries: block (mini-batch, r) takes the r-th share of the mini-batch's entries and the r-th share of the
// nodes it already has (hops 0..hop) and writes both grouped by bucket (a counting sort inside the block): (id, entry)
// pairs and (id, row) pairs, with the groups' bounds.
// k_dedupe_last: block (mini-batch, bucket) holds the bucket's id table (keys and rows, S slots) in shared memory.  It
// enters its bucket's earlier nodes, then its bucket's entries from every share (dense), ranks its new nodes (a scan over
// the table, no atomics), takes a run of the mini-batch's rows and of the list of new nodes with ONE global atomic
// each, and gives every entry its node's row.
// (measured on the bench's last hop: 512 threads x 13,312 slots x 32 buckets and 512 x 6,656 x 64 take the same time)
constexpr int kDedupThreads = 1024;
constexpr int kDedupMaxSlots = 26624;    // 208 KiB of keys + rows per block
constexpr int kDedupMaxBuckets = 16;
constexpr int kBucketThreads = 512;

struct DedupArgs {
    DenseHeader* hdr;
    int hop;
    int32_t B, k, nb, S;
    const int32_t* nodes;
    const int32_t* node_off;    // [hop + 1][B + 1] valid
    const int32_t* ent_off;
    const int32_t* ent_nbrs;
    int32_t* ent_repr;
    int2* pairs;                // [entries of the hop] (id, entry), grouped by (mini-batch, share, bucket); from
                                // node_pairs0 on: (id, row) of the earlier nodes, grouped the same way
    int32_t* share_off;         // [2][B][nb][nb + 1] group bounds (positions in pairs): entries, then earlier nodes
    const int32_t* cum;         // [B][k + 2]
    uint32_t* batch_cnt;        // [B] new nodes of the hop per mini-batch, zero before the launch
    uint64_t* newlist;
    int64_t cap_new;
    int id_bits;
    int32_t max_nodes_per_batch;
    int64_t node_pairs0;
};

// bucket and first slot of an id: one multiplicative hash, the bucket from its top, the slot from what is left
__device__ __forceinline__ uint32_t dedup_bucket(int32_t id, uint32_t nb) { return __umulhi((uint32_t)id * 0x9E3779B1u, nb); }
__device__ __forceinline__ uint32_t dedup_slot(int32_t id, uint32_t nb, uint32_t S) {
    return __umulhi((uint32_t)id * 0x9E3779B1u * nb, S);
}

__global__ void __launch_bounds__(kBucketThreads) k_bucket_entries(DedupArgs a) {
    constexpr int kWarps = kBucketThreads / 32;
    __shared__ uint32_t cnt[kWarps][kDedupMaxBuckets];
    __shared__ uint32_t base[kDedupMaxBuckets + 1];
    __shared__ int32_t hop_lo[MG_MAX_HOPS + 1], hop_row0[MG_MAX_HOPS + 2];
    if (a.hdr->status) return;
    const uint32_t nb = (uint32_t)a.nb;
    const int32_t b = (int32_t)(blockIdx.x / nb);
    const uint32_t r = blockIdx.x % nb;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x <= (unsigned)a.hop) hop_lo[threadIdx.x] = a.node_off[threadIdx.x * (a.B + 1) + b];
    if (threadIdx.x <= (unsigned)a.hop + 1) hop_row0[threadIdx.x] = a.cum[b * (a.k + 2) + threadIdx.x];
    __syncthreads();
    // pass 0: the entries of the hop; pass 1: the nodes the mini-batch already has, item t = the node of row t
    for (int pass = 0; pass < 2; ++pass) {
        int64_t first, last, out0;
        if (pass == 0) {
            first = a.ent_off[a.node_off[a.hop * (a.B + 1) + b]];
            last = a.ent_off[a.node_off[a.hop * (a.B + 1) + b + 1]];
            out0 = first;
        } else {
            first = 0;
            last = hop_row0[a.hop + 1];
            out0 = a.node_pairs0;   // this mini-batch's node pairs follow those of the mini-batches before it
            for (int j = 0; j <= a.hop; ++j) out0 += hop_lo[j] - a.node_off[j * (a.B + 1)];
        }
        const int32_t len = (int32_t)((last - first + nb - 1) / nb);
        const int32_t s_lo = (int32_t)min(last, first + (int64_t)r * len);
        const int32_t s_hi = (int32_t)min(last, (int64_t)s_lo + len);
        auto id_at = [&](int32_t i) -> int32_t {
            if (pass == 0) return a.ent_nbrs[i];
            int j = 0;
            while (j < a.hop && hop_row0[j + 1] <= i) ++j;
            return a.nodes[hop_lo[j] + (i - hop_row0[j])];
        };
        for (int i = threadIdx.x; i < kWarps * kDedupMaxBuckets; i += kBucketThreads) (&cnt[0][0])[i] = 0;
        __syncthreads();
        // (four loads in flight per thread: the walk is latency-bound otherwise)
        for (int32_t e0 = s_lo + (int32_t)threadIdx.x; e0 < s_hi; e0 += 4 * kBucketThreads) {
            int32_t id[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) id[u] = e0 + u * kBucketThreads < s_hi ? id_at(e0 + u * kBucketThreads) : -1;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (e0 + u * kBucketThreads < s_hi) atomicAdd(&cnt[warp][dedup_bucket(id[u], nb)], 1u);
        }
        __syncthreads();
        if (threadIdx.x < nb) {   // this bucket's pairs of the share: warp after warp
            uint32_t run = 0;
            for (int w = 0; w < kWarps; ++w) { const uint32_t c = cnt[w][threadIdx.x]; cnt[w][threadIdx.x] = run; run += c; }
            base[threadIdx.x] = run;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t run = 0;
            for (uint32_t q = 0; q < nb; ++q) { const uint32_t c = base[q]; base[q] = run; run += c; }
            base[nb] = run;
        }
        __syncthreads();
        const int64_t dst0 = out0 + (s_lo - first);
        if (threadIdx.x <= nb)
            a.share_off[(((int64_t)pass * a.B + b) * nb + r) * (nb + 1) + threadIdx.x] = (int32_t)(dst0 + base[threadIdx.x]);
        for (int32_t e0 = s_lo + (int32_t)threadIdx.x; e0 < s_hi; e0 += 4 * kBucketThreads) {
            int32_t id[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) id[u] = e0 + u * kBucketThreads < s_hi ? id_at(e0 + u * kBucketThreads) : -1;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int32_t e = e0 + u * kBucketThreads;
                if (e >= s_hi) continue;
                const uint32_t q = dedup_bucket(id[u], nb);
                a.pairs[dst0 + base[q] + atomicAdd(&cnt[warp][q], 1u)] = make_int2(id[u], e);
            }
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kDedupThreads) k_dedupe_last(DedupArgs a) {
    extern __shared__ int32_t dedup_sm[];
    __shared__ uint32_t row_base, list_base, warp_tot[kDedupThreads / 32];
    __shared__ int32_t run_lo[2][kDedupMaxBuckets], run_start[2][kDedupMaxBuckets + 1];
    if (a.hdr->status) return;
    const uint32_t S = (uint32_t)a.S, nb = (uint32_t)a.nb;
    int32_t* keys = dedup_sm;
    int32_t* vals = dedup_sm + S;
    const int32_t b = (int32_t)(blockIdx.x / nb);
    const uint32_t bucket = blockIdx.x % nb;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint32_t i = threadIdx.x; i < S; i += kDedupThreads) keys[i] = -1;
    if (threadIdx.x < 2 * nb) {   // this bucket's runs of pairs, one per share: entries [0], earlier nodes [1] ...
        const uint32_t which = threadIdx.x / nb, r = threadIdx.x % nb;
        const int32_t* so = a.share_off + (((int64_t)which * a.B + b) * nb + r) * (nb + 1) + bucket;
        run_lo[which][r] = so[0];
        run_start[which][r + 1] = so[1] - so[0];
    }
    __syncthreads();
    if (threadIdx.x < 2) {   // ... and their lengths' prefix
        int32_t run = 0;
        for (uint32_t r = 0; r < nb; ++r) { const int32_t c = run_start[threadIdx.x][r + 1]; run_start[threadIdx.x][r] = run; run += c; }
        run_start[threadIdx.x][nb] = run;
    }
    __syncthreads();
    auto pair_at = [&](int which, int32_t i) -> int2* {   // i-th pair of the bucket: which share's run it falls in (run_start ascends)
        uint32_t lo = 0, hi = nb;                           // run_start[lo] <= i < run_start[hi]
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (run_start[which][mid] <= i) lo = mid; else hi = mid;
        }
        return a.pairs + run_lo[which][lo] + (i - run_start[which][lo]);
    };
    // the nodes the mini-batch already has (this bucket's): rows = positions
    {
        const int32_t n_old = run_start[1][nb];
        for (int32_t i0 = threadIdx.x; i0 < n_old; i0 += 4 * kDedupThreads) {
            int2 it[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) it[u] = *pair_at(1, min(i0 + u * kDedupThreads, n_old - 1));
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (i0 + u * kDedupThreads >= n_old) continue;
                const int32_t id = it[u].x;
                uint32_t s = dedup_slot(id, nb, S), probe = 0;
                for (; probe < S; ++probe) {
                    const int32_t old = atomicCAS(&keys[s], -1, id);
                    if (old == -1) { vals[s] = it[u].y; break; }
                    if (old == id) { atomicOr(&a.hdr->status, ST_DUPLICATE); break; }   // only targets can repeat
                    s = s + 1u == S ? 0u : s + 1u;
                }
                if (probe >= S) atomicOr(&a.hdr->status, ST_CAP_TABLE);
            }
        }
    }
    __syncthreads();
    // this bucket's entries: enter the id, leave its slot in place of the id
    const int32_t n_pairs = run_start[0][nb];
    for (int32_t i0 = threadIdx.x; i0 < n_pairs; i0 += 4 * kDedupThreads) {
        int2* pp[4];
        int32_t id[4], old[4];
        uint32_t s[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {   // four loads, then four first-probe compare-and-swaps, in flight per thread
            const int32_t i = i0 + u * kDedupThreads;
            pp[u] = pair_at(0, min(i, n_pairs - 1));
            id[u] = i < n_pairs ? pp[u]->x : -1;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            s[u] = dedup_slot(id[u], nb, S);
            old[u] = id[u] >= 0 ? atomicCAS(&keys[s[u]], -1, id[u]) : id[u];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (id[u] < 0) continue;
            bool fresh = old[u] == -1;
            if (!fresh && old[u] != id[u]) {   // first slot taken by another id: linear probing
                uint32_t probe = 1;
                for (; probe < S; ++probe) {
                    s[u] = s[u] + 1u == S ? 0u : s[u] + 1u;
                    const int32_t o = atomicCAS(&keys[s[u]], -1, id[u]);
                    if (o == -1) { fresh = true; break; }
                    if (o == id[u]) break;
                }
                if (probe >= S) { atomicOr(&a.hdr->status, ST_CAP_TABLE); s[u] = 0; fresh = false; }
            }
            if (fresh) vals[s[u]] = -1;   // new: ranked below
            pp[u]->x = (int32_t)s[u];
        }
    }
    __syncthreads();
    // rank the new nodes of this block's table, take a run of the mini-batch's rows and of the list of new nodes
    uint32_t mine = 0;
    for (uint32_t i = threadIdx.x; i < S; i += kDedupThreads) mine += (keys[i] != -1 && vals[i] < 0) ? 1u : 0u;
    const uint32_t inc = warp_incl_scan(mine);
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const uint32_t w = lane < kDedupThreads / 32 ? warp_tot[lane] : 0u;
        const uint32_t wi = warp_incl_scan(w);
        if (lane < kDedupThreads / 32) warp_tot[lane] = wi - w;
        if (lane == 31) {
            row_base = wi ? atomicAdd(&a.batch_cnt[b], wi) : 0u;
            list_base = wi ? atomicAdd(&a.hdr->n_new, wi) : 0u;
        }
    }
    __syncthreads();
    const int32_t first_row = a.cum[b * (a.k + 2) + a.hop + 1];
    uint32_t rk = warp_tot[warp] + inc - mine;
    for (uint32_t i = threadIdx.x; i < S; i += kDedupThreads) {
        if (keys[i] == -1 || vals[i] >= 0) continue;
        const uint32_t rank = row_base + rk;
        const int64_t row = (int64_t)first_row + rank;
        if (row >= a.max_nodes_per_batch) atomicOr(&a.hdr->status, ST_CAP_TABLE);
        vals[i] = (int32_t)row;
        const int64_t pos = (int64_t)list_base + rk;
        if (pos < a.cap_new)
            a.newlist[pos] = (uint64_t)rank | ((uint64_t)(uint32_t)keys[i] << MG_SLOT_BITS) |
                             ((uint64_t)(uint32_t)b << (MG_SLOT_BITS + a.id_bits));
        else atomicOr(&a.hdr->status, ST_CAP_NODES);
        ++rk;
    }
    __syncthreads();
    // every entry of the bucket gets its node's row
    for (int32_t i0 = threadIdx.x; i0 < n_pairs; i0 += 4 * kDedupThreads) {
        int2 p[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) p[u] = *pair_at(0, min(i0 + u * kDedupThreads, n_pairs - 1));
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (i0 + u * kDedupThreads < n_pairs) a.ent_repr[p[u].y] = vals[p[u].x];
    }
}

// -------------------------------------------------------------------------------------
// radix sort of the new-node list on bits [lo_bit, lo_bit + bits) of the composite key
// -------------------------------------------------------------------------------------
constexpr int kSortKeysPerThread = 16;
constexpr int kSortTile = kThreads * kSortKeysPerThread;  // 4096
constexpr int kRadixBits = 9;                              // 34 key bits (27 id + 7 batch) take four passes
constexpr int kBins = 1 << kRadixBits;
constexpr int kBinsPerThread = kBins / kThreads;


// A tile of a segmented sort: a run of at most kSortTile keys of one segment.  Its histogram sits with its segment's
// (digit-major inside the segment), so that one exclusive scan over all histograms in segment order gives every
// (segment, digit, tile) its place in the output, where segment follows segment.
struct SegTile {
    int32_t in0;      // first key of the tile in the input of the first pass (the segments lie elsewhere there)
    int32_t out0;     // first key of the tile in every pass's output and the later passes' input
    int32_t count;
    int32_t hist0;    // index of the tile's count of digit 0
    int32_t stride;   // distance between its counts of consecutive digits: the segment's tiles
};

// (tiles == nullptr: one segment, tile t = keys [t * kSortTile, ...), histograms digit-major over all tiles)
__global__ void __launch_bounds__(kThreads)
k_radix_hist(const uint64_t* __restrict__ keys, const SortParams* sp, int shift, uint32_t* hist,
             const SegTile* __restrict__ tiles, bool first_pass) {
    __shared__ uint32_t sh[kBins];
    const int32_t n = sp->n, ntiles = sp->ntiles;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
#pragma unroll
        for (int q = 0; q < kBinsPerThread; ++q) sh[threadIdx.x + q * kThreads] = 0;
        __syncthreads();
        int32_t tb = t * kSortTile, tn = min(kSortTile, n - tb), h0 = t, hs = ntiles;
        if (tiles) { const SegTile st = tiles[t]; tb = first_pass ? st.in0 : st.out0; tn = st.count; h0 = st.hist0; hs = st.stride; }
#pragma unroll 4
        for (int j = 0; j < kSortKeysPerThread; ++j) {
            const int32_t l = j * kThreads + threadIdx.x;
            if (l < tn) atomicAdd(&sh[(uint32_t)(keys[tb + l] >> shift) & (kBins - 1)], 1u);
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kBinsPerThread; ++q) {
            const int bin = threadIdx.x + q * kThreads;
            hist[(size_t)h0 + (size_t)bin * hs] = sh[bin];
        }
        __syncthreads();
    }
}

// One stable counting pass.  A tile's keys are ranked per digit (warp by warp, 32 keys at a time with
// match_any), laid out digit by digit in shared memory, and written from there, so that every run of
// equal digits leaves the SM as consecutive addresses.
__global__ void __launch_bounds__(kThreads)
k_radix_scatter(const uint64_t* __restrict__ keys, uint64_t* __restrict__ out, const SortParams* sp, int shift,
                const uint32_t* __restrict__ hist_scanned, const SegTile* __restrict__ tiles, bool first_pass) {
    extern __shared__ __align__(16) uint8_t sort_smem[];
    uint64_t* stage = reinterpret_cast<uint64_t*>(sort_smem);                          // [kSortTile]
    uint32_t (*cnt)[kBins] = reinterpret_cast<uint32_t (*)[kBins]>(stage + kSortTile);   // [warps][kBins]
    uint32_t* tile_base = reinterpret_cast<uint32_t*>(cnt + kThreads / 32);             // [kBins] first slot of a digit in the tile
    uint32_t* glob_base = tile_base + kBins;                                            // [kBins] first output position
    __shared__ uint32_t warp_tot[kThreads / 32];
    const int32_t n = sp->n, ntiles = sp->ntiles;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kThreads / 32;
    constexpr int kPerWarp = kSortTile / kWarps;  // 512 consecutive keys per warp
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        for (int w = 0; w < kWarps; ++w)
#pragma unroll
            for (int q = 0; q < kBinsPerThread; ++q) cnt[w][threadIdx.x + q * kThreads] = 0;
        __syncthreads();
        uint64_t key[kSortKeysPerThread];
        uint32_t rank[kSortKeysPerThread];
        int32_t tb = t * kSortTile, tile_n = min(kSortTile, n - tb), h0 = t, hs = ntiles;
        if (tiles) { const SegTile st = tiles[t]; tb = first_pass ? st.in0 : st.out0; tile_n = st.count; h0 = st.hist0; hs = st.stride; }
        const int32_t wl = warp * kPerWarp;   // the warp's first key inside the tile
#pragma unroll
        for (int r = 0; r < kSortKeysPerThread; ++r) {
            const bool ok = wl + r * 32 + lane < tile_n;
            key[r] = ok ? keys[tb + wl + r * 32 + lane] : 0ull;
            const uint32_t dg = ok ? ((uint32_t)(key[r] >> shift) & (kBins - 1)) : 0xFFFFFFFFu;
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, dg);
            const int leader = __ffs(peers) - 1;
            uint32_t old = 0;
            if (ok && lane == leader) {
                old = cnt[warp][dg];
                cnt[warp][dg] = old + __popc(peers);
            }
            old = __shfl_sync(0xFFFFFFFFu, old, leader);
            rank[r] = old + __popc(peers & ((1u << lane) - 1u));
            __syncwarp();
        }
        __syncthreads();
        // per digit: prefix over the warps, total in the tile; then an exclusive scan over the digits
        uint32_t mine[kBinsPerThread], sum = 0;
#pragma unroll
        for (int q = 0; q < kBinsPerThread; ++q) {
            const int bin = threadIdx.x * kBinsPerThread + q;   // consecutive bins per thread: scan order = bin order
            uint32_t run = 0;
            for (int w = 0; w < kWarps; ++w) { const uint32_t c = cnt[w][bin]; cnt[w][bin] = run; run += c; }
            mine[q] = run;
            sum += run;
        }
        const uint32_t inc = warp_incl_scan(sum);
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        uint32_t before = inc - sum;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
#pragma unroll
        for (int q = 0; q < kBinsPerThread; ++q) {
            const int bin = threadIdx.x * kBinsPerThread + q;
            tile_base[bin] = before;
            glob_base[bin] = hist_scanned[(size_t)h0 + (size_t)bin * hs];
            before += mine[q];
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSortKeysPerThread; ++r) {
            if (wl + r * 32 + lane < tile_n) {
                const uint32_t dg = (uint32_t)(key[r] >> shift) & (kBins - 1);
                stage[tile_base[dg] + cnt[warp][dg] + rank[r]] = key[r];
            }
        }
        __syncthreads();
        for (int32_t i = threadIdx.x; i < tile_n; i += kThreads) {
            const uint64_t kx = stage[i];
            const uint32_t dg = (uint32_t)(kx >> shift) & (kBins - 1);
            out[glob_base[dg] + ((uint32_t)i - tile_base[dg])] = kx;
        }
        __syncthreads();
    }
}

constexpr size_t kScatterSmem = (size_t)kSortTile * 8 + (size_t)(kThreads / 32) * kBins * 4 + 2 * (size_t)kBins * 4;

// -------------------------------------------------------------------------------------
// place the sorted new nodes as the next hop
// -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
k_relabel(const DenseHeader* hdr, int hop, const int32_t* __restrict__ hvals, int32_t* ent_repr) {
    if (hdr->status) return;
    const int32_t lo = hdr->ent_base[hop], hi = hdr->ent_base[hop + 1];
    for (int32_t e = lo + blockIdx.x * blockDim.x + threadIdx.x; e < hi; e += gridDim.x * blockDim.x) {
        const int32_t v = ent_repr[e];
        if (v < 0) ent_repr[e] = hvals[-1 - v];   // entries of nodes that were new got their row at insert time
    }
}

// End of a hop (one block): the node arena's next bound, then per-batch counts -> node offsets of the next hop and the
// batches' row totals
__global__ void __launch_bounds__(1024)
k_outer_offsets(DenseHeader* hdr, int hop, int32_t B, int32_t k, const uint32_t* __restrict__ batch_cnt, int32_t* node_off_next,
                int32_t* cum, int32_t max_nodes_per_batch, int64_t cap_nodes) {
    __shared__ uint32_t warp_tot[33];
    if (hdr->status) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t start = hdr->hop_base[hop + 1];
    const int64_t end = (int64_t)start + hdr->n_new;
    if (end > cap_nodes) { if (threadIdx.x == 0) atomicOr(&hdr->status, ST_CAP_NODES); return; }
    if (threadIdx.x == 0) hdr->hop_base[hop + 2] = (int32_t)end;
    uint32_t carry = 0;
    for (int s0 = 0; s0 < B; s0 += 1024) {
        const int b = s0 + threadIdx.x;
        const uint32_t v = b < B ? batch_cnt[b] : 0u;
        const uint32_t inc = warp_incl_scan(v);
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const uint32_t w = warp_tot[lane];
            const uint32_t wi = warp_incl_scan(w);
            warp_tot[lane] = wi - w;
            if (lane == 31) warp_tot[32] = wi;
        }
        __syncthreads();
        if (b < B) {
            node_off_next[b] = start + (int32_t)(carry + warp_tot[warp] + inc - v);
            const int32_t rows = cum[b * (k + 2) + hop + 1] + (int32_t)v;
            cum[b * (k + 2) + hop + 2] = rows;
            if (rows > max_nodes_per_batch) atomicOr(&hdr->status, ST_CAP_TABLE);
        }
        carry += warp_tot[32];
        __syncthreads();
    }
    if (threadIdx.x == 0) node_off_next[B] = start + (int32_t)carry;
}

// Outermost hop: list entry (mini-batch, id, rank) -> the node's place in its mini-batch's run
__global__ void __launch_bounds__(kThreads)
k_place_nodes_outer(const DenseHeader* hdr, const uint64_t* __restrict__ list, int id_bits, const int32_t* __restrict__ node_off_next,
                    int32_t* nodes, int32_t* node_batch) {
    if (hdr->status) return;
    const int32_t n = (int32_t)hdr->n_new;
    const uint64_t id_mask = (1ull << id_bits) - 1ull;
    for (int32_t j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
        const uint64_t key = list[j];
        const int32_t b = (int32_t)(key >> (MG_SLOT_BITS + id_bits));
        const int32_t at = node_off_next[b] + (int32_t)(key & ((1u << MG_SLOT_BITS) - 1u));
        nodes[at] = (int32_t)((key >> MG_SLOT_BITS) & id_mask);
        node_batch[at] = b;
    }
}

// one block: packed row bases of every layer and the per-batch entry bounds of every hop; then the sample's summary
// (header, per-batch tables) for the host, stored straight into mapped pinned memory.  A copy engine is not used on
// purpose: a large output copy of a forward pass may be queued on it, and the host would wait for that copy before it
// learned the sample's sizes.  (After an error the summary still goes out: it carries the status word.)
__global__ void __launch_bounds__(1024)
k_finalize(DenseHeader* hdr, int32_t B, int32_t k, const int32_t* cum, const int32_t* node_off,
           const int32_t* __restrict__ ent_off, int32_t* rowbase, int32_t* ent_hop, int32_t n_hdr, int32_t* out) {
    __shared__ uint32_t warp_tot[33];
    const bool bad = hdr->status != 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int l = 0; l <= k && !bad; ++l) {
        uint32_t carry = 0;
        for (int start = 0; start < B; start += 1024) {
            const int b = start + threadIdx.x;
            const uint32_t v = b < B ? (uint32_t)cum[b * (k + 2) + (k - l + 1)] : 0u;
            const uint32_t inc = warp_incl_scan(v);
            if (lane == 31) warp_tot[warp] = inc;
            __syncthreads();
            if (warp == 0) {
                const uint32_t w = warp_tot[lane];
                const uint32_t wi = warp_incl_scan(w);
                warp_tot[lane] = wi - w;
                if (lane == 31) warp_tot[32] = wi;
            }
            __syncthreads();
            if (b < B) rowbase[l * (B + 1) + b] = (int32_t)(carry + warp_tot[warp] + inc - v);
            carry += warp_tot[32];
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            rowbase[l * (B + 1) + B] = (int32_t)carry;
            hdr->rows_total[l] = (int32_t)carry;
        }
    }
    for (int h = 0; h < k && !bad; ++h)
        for (int b = threadIdx.x; b <= B; b += blockDim.x)
            ent_hop[h * (B + 1) + b] = ent_off[node_off[h * (B + 1) + b]];
    __syncthreads();   // (one block: its own writes above are what the summary reads)
    const int32_t n_cum = B * (k + 2), n_off = (k + 1) * (B + 1), n_ent = k * (B + 1);
    const int32_t total = n_hdr + n_cum + 2 * n_off + n_ent;
    const volatile int32_t* h32 = reinterpret_cast<const volatile int32_t*>(hdr);
    for (int32_t i = threadIdx.x; i < total; i += blockDim.x) {
        int32_t j = i, v;
        if (j < n_hdr) v = j < (int32_t)(sizeof(DenseHeader) / 4) ? h32[j] : 0;
        else if ((j -= n_hdr) < n_cum) v = cum[j];
        else if ((j -= n_cum) < n_off) v = node_off[j];
        else if ((j -= n_off) < n_off) v = rowbase[j];
        else v = ent_hop[j - n_off];
        out[i] = v;
    }
}


// -------------------------------------------------------------------------------------
// export to the paper's layout (mg_dense_view)
// -------------------------------------------------------------------------------------
// The device keeps every delta in discovery order.  The paper's arrays list the ids of a delta in ascending order
// (targets in the caller's order), so an export goes through a permutation of the mini-batch's local rows:
// perm[c] = local row of canonical row c, inv[l] = canonical row of local row l.
struct BatchGeom {
    int32_t k, V, n_targets;
    int32_t cum[MG_MAX_HOPS + 2];      // local row base per hop
    int32_t node_off[MG_MAX_HOPS + 1]; // first node of the mini-batch's run in each hop
};

__device__ __forceinline__ int hop_of_row(const BatchGeom& g, int32_t l) {
    int h = 0;
    while (h < g.k && l >= g.cum[h + 1]) ++h;
    return h;
}

// keys (canonical delta, id, local row) of the rows of hops >= 1
__global__ void __launch_bounds__(kThreads)
k_perm_keys(BatchGeom g, const int32_t* __restrict__ nodes, int id_bits, uint64_t* keys) {
    const int32_t n = g.V - g.n_targets;
    for (int32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const int32_t l = g.n_targets + i;
        const int h = hop_of_row(g, l);
        const int32_t id = nodes[g.node_off[h] + (l - g.cum[h])];
        keys[i] = ((uint64_t)(g.k - h) << (MG_SLOT_BITS + id_bits)) | ((uint64_t)(uint32_t)id << MG_SLOT_BITS) | (uint64_t)l;
    }
}

__global__ void __launch_bounds__(kThreads)
k_perm_fill(BatchGeom g, const uint64_t* __restrict__ sorted, int32_t* perm, int32_t* inv) {
    const int32_t n = g.V - g.n_targets;
    for (int32_t c = blockIdx.x * blockDim.x + threadIdx.x; c < g.V; c += gridDim.x * blockDim.x) {
        // deltas k-1 .. 0 (hops >= 1) come first in the sorted keys; the targets keep the caller's order at the end
        const int32_t l = c < n ? (int32_t)(sorted[c] & ((1u << MG_SLOT_BITS) - 1u)) : c - n;
        perm[c] = l;
        inv[l] = c;
    }
}

struct ExportArgs {
    BatchGeom g;
    int32_t n0;                       // |Delta_0|: canonical rows below n0 have no sampled neighbours
    int32_t nio[MG_MAX_HOPS + 2];     // canonical node_id_offsets
    const int32_t *nodes, *ent_off, *ent_nbrs, *ent_repr, *perm, *inv;
    int32_t *o_node_ids, *o_nio, *o_nbrs, *o_nbr_off, *o_repr;
};

// node ids in canonical order; the sampled nodes' entry counts go to o_nbr_off (scanned next)
__global__ void __launch_bounds__(kThreads) k_export_nodes(ExportArgs a) {
    const int32_t tid = blockIdx.x * blockDim.x + threadIdx.x;
    if (tid <= a.g.k + 1) a.o_nio[tid] = a.nio[tid];
    for (int32_t c = tid; c < a.g.V; c += gridDim.x * blockDim.x) {
        const int32_t l = a.perm[c];
        const int h = hop_of_row(a.g, l);
        const int32_t idx = a.g.node_off[h] + (l - a.g.cum[h]);
        a.o_node_ids[c] = a.nodes[idx];
        if (c >= a.n0) a.o_nbr_off[c - a.n0] = a.ent_off[idx + 1] - a.ent_off[idx];
    }
}

// in-place exclusive scan of data[0, n), total to data[n] (one block)
__global__ void __launch_bounds__(1024) k_export_scan(int32_t* data, int32_t n) {
    __shared__ uint32_t warp_tot[33];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t carry = 0;
    for (int s0 = 0; s0 < n; s0 += 1024) {
        const int i = s0 + threadIdx.x;
        const uint32_t v = i < n ? (uint32_t)data[i] : 0u;
        const uint32_t inc = warp_incl_scan(v);
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const uint32_t w = warp_tot[lane];
            const uint32_t wi = warp_incl_scan(w);
            warp_tot[lane] = wi - w;
            if (lane == 31) warp_tot[32] = wi;
        }
        __syncthreads();
        if (i < n) data[i] = (int32_t)(carry + warp_tot[warp] + inc - v);
        carry += warp_tot[32];
        __syncthreads();
    }
    if (threadIdx.x == 0) data[n] = (int32_t)carry;
}

// nbrs and repr_map: the entries of canonical node c start at o_nbr_off[c - n0]
__global__ void __launch_bounds__(kThreads) k_export_entries(ExportArgs a) {
    for (int32_t c = a.n0 + blockIdx.x * blockDim.x + threadIdx.x; c < a.g.V; c += gridDim.x * blockDim.x) {
        const int32_t l = a.perm[c];
        const int h = hop_of_row(a.g, l);
        const int32_t idx = a.g.node_off[h] + (l - a.g.cum[h]);
        const int32_t e0 = a.ent_off[idx], e1 = a.ent_off[idx + 1];
        const int32_t o0 = a.o_nbr_off[c - a.n0];
        for (int32_t e = e0; e < e1; ++e) {
            a.o_nbrs[o0 + (e - e0)] = a.ent_nbrs[e];
            a.o_repr[o0 + (e - e0)] = a.inv[a.ent_repr[e]];
        }
    }
}

// -------------------------------------------------------------------------------------
// export of every mini-batch at once (mg_dense_export_many): the canonical DENSE ordering for the whole sample
// -------------------------------------------------------------------------------------
// One sort orders all nodes of the sample by (mini-batch, delta, id); a node's position in that order is its row in
// the packed canonical node list (mini-batch after mini-batch, each [Delta_0 .. Delta_k]).  Targets keep the caller's
// order: their "id" field is their position.
struct ExportManyArgs {
    int32_t B, k, n_nodes_total, pay_bits, id_bits;
    int32_t hop_base[MG_MAX_HOPS + 2];
    const int32_t *nodes, *node_batch, *node_off, *cum, *rowbase0, *ent_off, *ent_nbrs, *ent_repr;
    int32_t *o_node_ids, *o_nio, *o_nbrs, *o_repr, *o_nbr_off, *inv;
    uint32_t* cnt;   // per canonical row: entry count, then (scanned) its first entry in the packed entry list
};

__device__ __forceinline__ int hop_of_arena(const ExportManyArgs& a, int32_t i) {
    int h = 0;
    while (h < a.k && i >= a.hop_base[h + 1]) ++h;
    return h;
}

// The segments of the export's sort in output order -- mini-batch after mini-batch, inside it the farthest delta
// first -- cut into tiles: where a tile's keys lie in the arenas (hop-major), where in the output, and where its
// histogram goes.  One block; also the sort's parameters and the range of the entry-count scan.
__global__ void __launch_bounds__(1024) k_export_tiles(ExportManyArgs a, SegTile* tiles, SortParams* sp, int32_t* range) {
    __shared__ int32_t warp_t[32], warp_n[32];
    __shared__ int32_t carry_t, carry_n;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { carry_t = 0; carry_n = 0; }
    __syncthreads();
    const int32_t n_seg = a.B * (a.k + 1);
    for (int32_t s0 = 0; s0 < n_seg; s0 += 1024) {
        const int32_t s = s0 + (int32_t)threadIdx.x;
        int32_t in0 = 0, len = 0;
        if (s < n_seg) {
            const int32_t b = s / (a.k + 1), h = a.k - s % (a.k + 1);
            in0 = a.node_off[h * (a.B + 1) + b];
            len = a.node_off[h * (a.B + 1) + b + 1] - in0;
        }
        const int32_t nt = (len + kSortTile - 1) / kSortTile;
        const int32_t it = (int32_t)warp_incl_scan((uint32_t)nt), in = (int32_t)warp_incl_scan((uint32_t)len);
        if (lane == 31) { warp_t[warp] = it; warp_n[warp] = in; }
        __syncthreads();
        int32_t t0 = carry_t + it - nt, o0 = carry_n + in - len;
        for (int w = 0; w < warp; ++w) { t0 += warp_t[w]; o0 += warp_n[w]; }
        for (int32_t t = 0; t < nt; ++t) {
            SegTile st;
            st.in0 = in0 + t * kSortTile;
            st.out0 = o0 + t * kSortTile;
            st.count = min(kSortTile, len - t * kSortTile);
            st.hist0 = t0 * kBins + t;
            st.stride = nt;
            tiles[t0 + t] = st;
        }
        __syncthreads();
        if (threadIdx.x == 1023) { carry_t = t0 + nt; carry_n = o0 + len; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        sp->zero = 0; sp->n = a.n_nodes_total; sp->ntiles = carry_t; sp->hist_len = kBins * carry_t;
        range[0] = 0; range[1] = a.n_nodes_total;
    }
}

__global__ void __launch_bounds__(kThreads) k_export_keys(ExportManyArgs a, uint64_t* keys) {
    for (int32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < a.n_nodes_total; i += gridDim.x * blockDim.x) {
        const int h = hop_of_arena(a, i);
        const int32_t b = a.node_batch[i];
        const uint32_t id = h == 0 ? (uint32_t)(i - a.node_off[b]) : (uint32_t)a.nodes[i];
        keys[i] = ((uint64_t)id << a.pay_bits) | (uint64_t)(uint32_t)i;   // sorted inside its (mini-batch, delta) segment
    }
    // node_id_offsets of every mini-batch
    for (int32_t t = blockIdx.x * blockDim.x + threadIdx.x; t < a.B; t += gridDim.x * blockDim.x) {
        const int32_t* cum = a.cum + (int64_t)t * (a.k + 2);
        int32_t run = 0;
        a.o_nio[(int64_t)t * (a.k + 2)] = 0;
        a.o_nbr_off[a.rowbase0[t] + t] = 0;   // (an empty mini-batch has this terminal entry only)
        for (int j = 0; j <= a.k; ++j) { run += cum[a.k - j + 1] - cum[a.k - j]; a.o_nio[(int64_t)t * (a.k + 2) + j + 1] = run; }
    }
}

__global__ void __launch_bounds__(kThreads) k_export_place(ExportManyArgs a, const uint64_t* __restrict__ sorted) {
    const uint64_t pay_mask = (1ull << a.pay_bits) - 1ull;
    for (int32_t c = blockIdx.x * blockDim.x + threadIdx.x; c < a.n_nodes_total; c += gridDim.x * blockDim.x) {
        const uint64_t key = sorted[c];
        const int32_t i = (int32_t)(key & pay_mask);
        a.inv[i] = c;
        // the key carries the node id (for the targets their position: they keep the caller's order)
        a.o_node_ids[c] = i < a.hop_base[1] ? a.nodes[i] : (int32_t)((key >> a.pay_bits) & ((1ull << a.id_bits) - 1ull));
        a.cnt[c] = i < a.hop_base[a.k] ? (uint32_t)(a.ent_off[i + 1] - a.ent_off[i]) : 0u;   // the farthest delta has no entries
    }
}

// 8 lanes per sampled node: its entries go to their place in the packed canonical entry list, neighbours translated to
// canonical rows of the mini-batch; the node's offset (relative to its mini-batch) goes to nbr_offsets
__global__ void __launch_bounds__(kThreads) k_export_many_entries(ExportManyArgs a) {
    const int gl = threadIdx.x & 7;
    const int32_t n_sampled = a.hop_base[a.k];
    for (int32_t i = (blockIdx.x * blockDim.x + threadIdx.x) >> 3; i < n_sampled; i += (gridDim.x * blockDim.x) >> 3) {
        const int32_t b = a.node_batch[i];
        const int32_t c = a.inv[i];
        const int32_t row0 = a.rowbase0[b];                        // first packed row of the mini-batch
        const int32_t* cum = a.cum + (int64_t)b * (a.k + 2);
        const int32_t n0 = cum[a.k + 1] - cum[a.k];                // |Delta_0|
        const uint32_t o0 = a.cnt[c], batch_e0 = a.cnt[row0];
        const int32_t e0 = a.ent_off[i], n = a.ent_off[i + 1] - e0;
        if (gl == 0) {
            int32_t* off = a.o_nbr_off + row0 + b;                 // the mini-batch's nbr_offsets: |sampled| + 1 entries
            off[c - row0 - n0] = (int32_t)(o0 - batch_e0);
            if (c + 1 == a.rowbase0[b + 1]) off[c + 1 - row0 - n0] = (int32_t)(o0 - batch_e0) + n;   // terminal entry
        }
        for (int32_t j = gl; j < n; j += 8) {
            const int32_t l = a.ent_repr[e0 + j];                  // the neighbour's local row in the mini-batch
            int h = 0;
            while (h < a.k && l >= cum[h + 1]) ++h;
            const int32_t ai = a.node_off[h * (a.B + 1) + b] + (l - cum[h]);
            a.o_nbrs[o0 + j] = a.ent_nbrs[e0 + j];
            a.o_repr[o0 + j] = a.inv[ai] - row0;
        }
    }
}

int ilog2_ceil(int64_t x) {
    int b = 0;
    while (((int64_t)1 << b) < x) ++b;
    return b;
}

}  // namespace

// ---------------------------------------------------------------------------------------
// generic pieces other translation units use
// ---------------------------------------------------------------------------------------
size_t mg_sort_hist_elems(int64_t max_keys) { return (size_t)kBins * ((max_keys + kSortTile - 1) / kSortTile) + kBins; }
void mg_sort_params_host(SortParams* sp, int64_t n) {
    sp->zero = 0; sp->n = (int32_t)n; sp->ntiles = (int32_t)((n + kSortTile - 1) / kSortTile); sp->hist_len = kBins * sp->ntiles;
}
size_t mg_scan_tmp_elems(int64_t max_elems) { return (size_t)((max_elems + kScanTile - 1) / kScanTile) + 16; }

static void sample_kernel_attributes();

// LSD radix sort of 64-bit keys on bits [lo_bit, lo_bit + bits); sp (device) holds the key count.
// Keys start in buf[0]; *res_buf tells which buffer holds the result.
// With a tile table (seg_tiles, SegTile per tile; sp->ntiles tiles): a sort inside segments -- the first pass reads
// every segment where its tiles say and all passes write segment after segment.
void mg_sort_u64(mg_ctx* ctx, uint64_t* const buf[2], const SortParams* sp, int lo_bit, int bits, uint32_t* hist,
                 uint32_t* scan_tmp, int* res_buf, const void* seg_tiles) {
    const SegTile* tiles = static_cast<const SegTile*>(seg_tiles);
    cudaStream_t st = ctx->stream;
    const int grid = mg_grid(ctx, 8);
    const int passes = (bits + kRadixBits - 1) / kRadixBits;
    ScanRange r{&sp->zero, &sp->hist_len, nullptr};
    sample_kernel_attributes();
    int cur = 0;
    for (int p = 0; p < passes; ++p) {
        const int shift = lo_bit + kRadixBits * p;
        k_radix_hist<<<grid, kThreads, 0, st>>>(buf[cur], sp, shift, hist, tiles, p == 0);
        k_scan_reduce<<<grid, kThreads, 0, st>>>(hist, r, scan_tmp);
        k_scan_tiles<<<1, 1024, 0, st>>>(scan_tmp, r, nullptr, HopClose{nullptr, 0, nullptr, 0});
        k_scan_down<<<grid, kThreads, 0, st>>>(hist, r, scan_tmp);
        k_radix_scatter<<<grid, kThreads, kScatterSmem, st>>>(buf[cur], buf[cur ^ 1], sp, shift, hist, tiles, p == 0);
        cur ^= 1;
    }
    ctx->launches += 5 * passes;
    *res_buf = cur;
}

// in-place exclusive scan of data[*lo .. *hi) (+ *base); total (+ *base) to *total_out (nullable)
void mg_scan_u32(mg_ctx* ctx, uint32_t* data, const int32_t* lo, const int32_t* hi, const int32_t* base,
                 uint32_t* scan_tmp, uint32_t* total_out) {
    cudaStream_t st = ctx->stream;
    const int grid = mg_grid(ctx, 8);
    ScanRange r{lo, hi, base};
    k_scan_reduce<<<grid, kThreads, 0, st>>>(data, r, scan_tmp);
    k_scan_tiles<<<1, 1024, 0, st>>>(scan_tmp, r, total_out, HopClose{nullptr, 0, nullptr, 0});
    k_scan_down<<<grid, kThreads, 0, st>>>(data, r, scan_tmp);
    ctx->launches += 3;
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
template <typename T>
static int dev_realloc(mg_ctx* ctx, T** p, size_t elems) {
    if (*p) cudaFree(*p);
    *p = nullptr;
    if (cudaMalloc((void**)p, std::max<size_t>(elems, 1) * sizeof(T)) != cudaSuccess) {
        cudaGetLastError();
        *p = nullptr;
        return mg_fail(ctx, MG_ERR_OOM, "device allocation of %zu bytes failed", elems * sizeof(T));
    }
    return MG_OK;
}

static int dense_alloc(mg_ctx* ctx, mg_dense* d, int32_t B, int32_t k, int64_t cap_nodes, int64_t cap_entries,
                       int32_t table_size, int32_t smem_nb) {
    int rc;
    if (!d->hdr && (rc = dev_realloc(ctx, &d->hdr, 1))) return rc;
    // sort scratch: a tile per 4096 keys, and one more per (mini-batch, delta) segment for the export's segmented sort
    const int64_t want_sort_tiles = (std::max(cap_nodes, d->cap_nodes) + kSortTile - 1) / kSortTile + (int64_t)B * (k + 1);
    const bool grow_sort = d->cap_nodes < cap_nodes || d->cap_sort_tiles < want_sort_tiles;
    if (d->cap_nodes < cap_nodes) {
        d->cap_nodes = 0;
        if ((rc = dev_realloc(ctx, &d->nodes, (size_t)cap_nodes))) return rc;
        if ((rc = dev_realloc(ctx, &d->node_batch, (size_t)cap_nodes))) return rc;
        if ((rc = dev_realloc(ctx, &d->ent_off, (size_t)cap_nodes + 1))) return rc;
        if ((rc = dev_realloc(ctx, &d->node_r0, (size_t)cap_nodes))) return rc;
        if ((rc = dev_realloc(ctx, &d->node_deg, (size_t)cap_nodes))) return rc;
        d->cap_nodes_out = 0;
        if ((rc = dev_realloc(ctx, &d->newlist[0], (size_t)cap_nodes))) return rc;
        if ((rc = dev_realloc(ctx, &d->newlist[1], (size_t)cap_nodes))) return rc;
        d->cap_nodes = cap_nodes;
    }
    if (grow_sort) {
        d->cap_sort_tiles = 0;
        const int64_t sort_tiles = want_sort_tiles;
        const int64_t scan_tiles = std::max<int64_t>((d->cap_nodes + kScanTile - 1) / kScanTile,
                                                     (kBins * sort_tiles + kScanTile - 1) / kScanTile);
        d->scan_tmp_elems = (size_t)scan_tiles + 16;
        if ((rc = dev_realloc(ctx, &d->scan_tmp, d->scan_tmp_elems))) return rc;
        d->sort_hist_elems = (size_t)kBins * sort_tiles + kBins;
        if ((rc = dev_realloc(ctx, &d->sort_hist, d->sort_hist_elems))) return rc;
        SegTile* tiles = static_cast<SegTile*>(d->seg_tiles);
        if ((rc = dev_realloc(ctx, &tiles, (size_t)sort_tiles + 1))) { d->seg_tiles = nullptr; return rc; }
        d->seg_tiles = tiles;
        d->cap_sort_tiles = sort_tiles;
    }
    if (d->cap_entries < cap_entries) {
        d->cap_entries = 0;
        if ((rc = dev_realloc(ctx, &d->ent_nbrs, (size_t)cap_entries))) return rc;
        if ((rc = dev_realloc(ctx, &d->ent_repr, (size_t)cap_entries))) return rc;
        d->cap_entries = cap_entries;
        d->cap_pairs = 0;
    }
    if (smem_nb > 0) {
        if (d->cap_pairs < d->cap_entries + d->cap_nodes) {   // (id, entry) of the last hop's entries, then (id, row) of the earlier nodes
            d->cap_pairs = 0;
            if ((rc = dev_realloc(ctx, &d->pairs, (size_t)(d->cap_entries + d->cap_nodes)))) return rc;
            d->cap_pairs = d->cap_entries + d->cap_nodes;
        }
        const int64_t need_share = 2 * (int64_t)B * smem_nb * (smem_nb + 1);
        if (d->cap_share < need_share) {
            d->cap_share = 0;
            if ((rc = dev_realloc(ctx, &d->share_off, (size_t)need_share))) return rc;
            d->cap_share = need_share;
        }
    }
    if (ctx->sample_inout && d->cap_nodes_out < d->cap_nodes) {
        d->cap_nodes_out = 0;
        if ((rc = dev_realloc(ctx, &d->node_r0_out, (size_t)d->cap_nodes))) return rc;
        if ((rc = dev_realloc(ctx, &d->node_deg_out, (size_t)d->cap_nodes))) return rc;
        d->cap_nodes_out = d->cap_nodes;
    }
    const int64_t need_table = (int64_t)B * table_size;
    if (d->alloc_table < need_table) {
        d->alloc_table = 0;
        if ((rc = dev_realloc(ctx, &d->hkeys, (size_t)need_table))) return rc;
        if ((rc = dev_realloc(ctx, &d->hvals, (size_t)need_table))) return rc;
        d->alloc_table = need_table;
    }
    const int64_t need_b = (int64_t)(MG_MAX_HOPS + 2) * (B + 1);
    if (d->alloc_batches < need_b) {
        d->alloc_batches = 0;
        if ((rc = dev_realloc(ctx, &d->node_off, (size_t)need_b))) return rc;
        if ((rc = dev_realloc(ctx, &d->cum, (size_t)need_b))) return rc;
        if ((rc = dev_realloc(ctx, &d->rowbase, (size_t)need_b))) return rc;
        if ((rc = dev_realloc(ctx, &d->d_ent_hop, (size_t)need_b))) return rc;
        if ((rc = dev_realloc(ctx, &d->d_seeds, (size_t)need_b))) return rc;
        if ((rc = dev_realloc(ctx, &d->batch_cnt, (size_t)need_b))) return rc;
        d->alloc_batches = need_b;
    }
    d->k = k;
    d->n_batches = B;
    d->table_size = table_size;
    return MG_OK;
}

static const char* status_text(uint32_t st) {
    if (st & ST_RANGE) return "a target id is outside [0, n_nodes)";
    if (st & ST_NONRESIDENT) return "a target lies in a partition that is not resident";
    if (st & ST_DUPLICATE) return "a batch lists a target twice";
    if (st & ST_CAP_ENTRIES) return "neighbour capacity (max_entries_total) exceeded";
    if (st & ST_CAP_NODES) return "node capacity (max_nodes_total) exceeded";
    if (st & ST_CAP_TABLE) return "per-batch node capacity (max_nodes_per_batch) exceeded";
    return "internal invariant violated";
}

static int status_code(uint32_t st) {
    if (st & ST_RANGE) return MG_ERR_ARG;
    if (st & ST_NONRESIDENT) return MG_ERR_NONRESIDENT;
    if (st & ST_DUPLICATE) return MG_ERR_DUPLICATE;
    if (st & (ST_CAP_ENTRIES | ST_CAP_NODES | ST_CAP_TABLE)) return MG_ERR_CAPACITY;
    return MG_ERR_CUDA;
}

// All sampling work is queued on the library's sampling stream, so that it can overlap a forward pass that is
// running on the context's stream.  The sampling stream first waits for whatever the caller had queued on the
// context's stream (e.g. the kernel that produced device-resident targets).
static int sample_begin_impl(mg_ctx* ctx, const int32_t* targets, int targets_on_device,
                             const int64_t* target_offsets, int32_t n_batches, const int32_t* fanouts,
                             int32_t k, const uint64_t* seeds, const mg_sample_caps* caps, mg_dense** out);

extern "C" int mg_sample_many_begin(mg_ctx* ctx, const int32_t* targets, int targets_on_device,
                                    const int64_t* target_offsets, int32_t n_batches, const int32_t* fanouts,
                                    int32_t k, const uint64_t* seeds, const mg_sample_caps* caps, mg_dense** out) {
    if (!ctx) return MG_ERR_ARG;
    cudaStream_t user = ctx->stream;
    if (cudaEventRecord(ctx->ev_user, user) == cudaSuccess) cudaStreamWaitEvent(ctx->sample_stream, ctx->ev_user, 0);
    ctx->stream = ctx->sample_stream;     // every helper launches on ctx->stream
    const int rc = sample_begin_impl(ctx, targets, targets_on_device, target_offsets, n_batches, fanouts, k, seeds, caps, out);
    ctx->stream = user;
    return rc;
}

extern "C" int mg_sample_many_end(mg_ctx* ctx, mg_dense* d) {
    if (!ctx) return MG_ERR_ARG;
    if (!d) return mg_fail(ctx, MG_ERR_ARG, "null mg_dense");
    if (!d->pending) return mg_fail(ctx, MG_ERR_STATE, "no sample in flight on this mg_dense");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    d->pending = false;
    MG_CUDA(ctx, cudaEventSynchronize(d->ev_sampled));
    const int B = d->n_batches, k = d->k;
    const int32_t* p = d->h_pinned;
    memcpy(&d->h_hdr, p, sizeof(DenseHeader)); p += (sizeof(DenseHeader) + 3) / 4;
    d->h_cum.assign(p, p + (size_t)B * (k + 2)); p += (size_t)B * (k + 2);
    d->h_node_off.assign(p, p + (size_t)(k + 1) * (B + 1)); p += (size_t)(k + 1) * (B + 1);
    d->h_rowbase.assign(p, p + (size_t)(k + 1) * (B + 1)); p += (size_t)(k + 1) * (B + 1);
    d->h_ent_hop.assign(p, p + (size_t)k * (B + 1));
    if (d->h_hdr.status) return mg_fail(ctx, status_code(d->h_hdr.status), "%s", status_text(d->h_hdr.status));
    d->valid = true;
    d->perm_batch = -1;
    return MG_OK;
}

extern "C" int mg_sample_many(mg_ctx* ctx, const int32_t* targets, int targets_on_device,
                              const int64_t* target_offsets, int32_t n_batches, const int32_t* fanouts,
                              int32_t k, const uint64_t* seeds, const mg_sample_caps* caps, mg_dense** out) {
    const int rc = mg_sample_many_begin(ctx, targets, targets_on_device, target_offsets, n_batches, fanouts, k, seeds, caps, out);
    if (rc) return rc;
    return mg_sample_many_end(ctx, *out);
}


// dynamic shared-memory limits of the sampler's kernels, set once (not inside a stream capture)
static void sample_kernel_attributes() {
    static bool done = false;
    if (done) return;
    cudaFuncSetAttribute(k_radix_scatter, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScatterSmem);
    cudaFuncSetAttribute(k_dedupe_last, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kDedupMaxSlots * 2 * sizeof(int32_t)));
    cudaFuncSetAttribute(k_pick_wide, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)((size_t)(kThreads / 32) * 2 * MG_MAX_FANOUT * sizeof(uint32_t)));
    done = true;
}

static int sample_begin_impl(mg_ctx* ctx, const int32_t* targets, int targets_on_device,
                             const int64_t* target_offsets, int32_t n_batches, const int32_t* fanouts,
                             int32_t k, const uint64_t* seeds, const mg_sample_caps* caps, mg_dense** out) {
    if (!ctx) return MG_ERR_ARG;
    if (!out || !target_offsets || !fanouts || !seeds) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (n_batches <= 0 || n_batches > MG_MAX_BATCHES) return mg_fail(ctx, MG_ERR_ARG, "n_batches must be in [1, %d]", MG_MAX_BATCHES);
    if (k <= 0 || k > MG_MAX_HOPS) return mg_fail(ctx, MG_ERR_ARG, "k must be in [1, %d]", MG_MAX_HOPS);
    for (int h = 0; h < k; ++h)
        if (fanouts[h] <= 0 || fanouts[h] > MG_MAX_FANOUT) return mg_fail(ctx, MG_ERR_ARG, "fanouts must be in [1, %d]", MG_MAX_FANOUT);
    if (!ctx->row_off) return mg_fail(ctx, MG_ERR_STATE, "no graph loaded");
    if (!ctx->view_off) return mg_fail(ctx, MG_ERR_NONRESIDENT, "no partition is resident");
    const bool inout = ctx->sample_inout;
    if (inout && !ctx->view_off_out) return mg_fail(ctx, MG_ERR_STATE, "no outgoing edge list loaded");
    if (target_offsets[0] != 0) return mg_fail(ctx, MG_ERR_ARG, "target_offsets[0] must be 0");
    for (int b = 0; b < n_batches; ++b)
        if (target_offsets[b + 1] < target_offsets[b]) return mg_fail(ctx, MG_ERR_ARG, "target_offsets must be non-decreasing");
    const int64_t T = target_offsets[n_batches];
    if (T > 0 && !targets) return mg_fail(ctx, MG_ERR_ARG, "null targets");
    if (T >= (1ll << 31)) return mg_fail(ctx, MG_ERR_ARG, "too many targets");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));

    // capacities: worst case unless the caller bounds them
    const int64_t N = ctx->n_nodes;
    int64_t worst_nodes_total = 0, worst_entries_total = 0, worst_nodes_batch = 0;
    for (int b = 0; b < n_batches; ++b) {
        double level = (double)(target_offsets[b + 1] - target_offsets[b]);  // nodes that can be new at this hop
        double nodes = level, entries = 0;
        for (int h = 0; h < k; ++h) {
            level = std::min(level, (double)N) * fanouts[h] * (ctx->sample_inout ? 2 : 1);
            entries += level;
            nodes += level;
        }
        const int64_t nb = (int64_t)std::min(nodes, (double)N);
        worst_nodes_total += nb;
        worst_entries_total += (int64_t)std::min(entries, 4.0e18);
        worst_nodes_batch = std::max(worst_nodes_batch, nb);
    }
    // Worst-case bounds follow the number of targets: they are rounded up on a geometric grid (steps of 1/8), so
    // that calls of similar size share allocations, table size and the captured graph.
    auto grid_up = [](int64_t v) {
        int64_t q = 1024;
        while (q < v) q += std::max<int64_t>(q / 8, 1);
        return q >= (1ll << 31) - 1 ? v : q;   // never round a legal bound out of range
    };
    int64_t cap_nodes = (caps && caps->max_nodes_total > 0) ? caps->max_nodes_total : grid_up(worst_nodes_total);
    int64_t cap_entries = (caps && caps->max_entries_total > 0) ? caps->max_entries_total : grid_up(worst_entries_total);
    int64_t cap_batch = (caps && caps->max_nodes_per_batch > 0) ? caps->max_nodes_per_batch : worst_nodes_batch;
    if (!(caps && caps->max_nodes_per_batch > 0)) cap_batch = std::min<int64_t>(grid_up(cap_batch), std::max<int64_t>(N, 1));
    cap_nodes = std::max<int64_t>({cap_nodes, T, 1});   // even an empty call needs its (one-element) arrays
    cap_batch = std::max<int64_t>(cap_batch, 1);
    for (int b = 0; b < n_batches; ++b) cap_batch = std::max<int64_t>(cap_batch, target_offsets[b + 1] - target_offsets[b]);
    if (cap_nodes >= (1ll << 31) - 1 || cap_entries >= (1ll << 31) - 1)
        return mg_fail(ctx, MG_ERR_CAPACITY, "capacities must stay below 2^31 (nodes %lld, entries %lld): pass tighter mg_sample_caps or fewer batches",
                       (long long)cap_nodes, (long long)cap_entries);
    // id table of a mini-batch: 1.625 slots per node it may hold (load factor <= 0.62 for linear probing), any size:
    // its traffic is random 32-byte sectors, so every slot that is not needed costs DRAM bandwidth
    // (sized below, once it is known whether the last hop goes through it)
    // The last hop is deduplicated in shared memory (k_bucket_entries, k_dedupe_last) when a mini-batch's nodes fit the
    // tables of a few blocks: S slots per block, filled to 92 % at most when the mini-batch is at its capacity (the
    // buckets of a hash differ by a per cent or so at these sizes), nb blocks per mini-batch.
    const int32_t dedup_slots = (int32_t)std::min<int64_t>(kDedupMaxSlots, (cap_batch + cap_batch / 4 + 64 + 1023) / 1024 * 1024);
    const int64_t dedup_nb = (cap_batch + (cap_batch * 7 + 79) / 80 + dedup_slots - 1) / dedup_slots;
    const bool smem_last = dedup_nb <= kDedupMaxBuckets && dedup_nb * n_batches < (1ll << 24) && cap_entries + cap_nodes < (1ll << 31) &&
                           !getenv("MG_GLOBAL_TABLES");
    // With the last hop deduplicated in shared memory the global tables only ever hold the nodes that are sampled from
    // (targets and the inner deltas): a caller who bounds those gets tables several times smaller.
    int64_t table_nodes = cap_batch;
    if (smem_last && caps && caps->max_inner_nodes_per_batch > 0) {
        table_nodes = std::min<int64_t>(cap_batch, caps->max_inner_nodes_per_batch);
        for (int b = 0; b < n_batches; ++b) table_nodes = std::max<int64_t>(table_nodes, target_offsets[b + 1] - target_offsets[b]);
    }
    const int64_t want_slots = std::max<int64_t>(16, (table_nodes + table_nodes / 2 + table_nodes / 8 + 7) / 8 * 8);
    if (want_slots > (1ll << MG_SLOT_BITS)) return mg_fail(ctx, MG_ERR_CAPACITY, "max_nodes_per_batch above %d", (int)((1ll << MG_SLOT_BITS) * 8 / 13));
    const int32_t table_size = (int32_t)want_slots;
    if ((int64_t)table_size * n_batches >= (1ll << 31))
        return mg_fail(ctx, MG_ERR_CAPACITY, "n_batches x id-table size must stay below 2^31: pass a smaller max_nodes_per_batch or fewer batches");
    const int id_bits = std::max(1, ilog2_ceil(N));
    const int b_bits = std::max(1, ilog2_ceil(n_batches));
    if (MG_SLOT_BITS + id_bits + b_bits > 64) return mg_fail(ctx, MG_ERR_ARG, "id and batch bits do not fit the sort key");

    mg_dense* d = *out;
    const bool created = (d == nullptr);
    if (created) { d = new mg_dense(); d->ctx = ctx; d->device = ctx->device; }
    else if (d->ctx != ctx) return mg_fail(ctx, MG_ERR_ARG, "mg_dense belongs to another context");
    d->valid = false;
    d->pending = false;
    d->export_valid = false;
    if (d->ev_read_done) MG_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, d->ev_read_done, 0));
    int rc = dense_alloc(ctx, d, n_batches, k, cap_nodes, std::max<int64_t>(cap_entries, 1), table_size, smem_last ? (int32_t)dedup_nb : 0);
    if (rc) { if (created) mg_dense_free(d); return rc; }
    *out = d;
    for (int h = 0; h < k; ++h) d->fanouts[h] = fanouts[h];
    d->n_targets_total = T;
    d->resident_serial = ctx->resident_serial;
    d->slot_of_part_at_sample = ctx->slot_of_part;

    cudaStream_t st = ctx->stream;
    const int B = n_batches;
    const TableGeom tg{table_size};

    // Host-known part of the header, the per-batch tables and the seeds go through a pinned staging block of the
    // sample handle, so that the device work below reads nothing but fixed addresses: it can then be captured once
    // in a CUDA graph and replayed for every later call with the same shape.
    const size_t n_stage_ints = (sizeof(DenseHeader) + 3) / 4 + (size_t)(B + 1) + (size_t)B * (k + 2) + 2 * (size_t)B + 2;
    if (d->h_stage_ints < n_stage_ints) {
        if (d->h_stage) cudaFreeHost(d->h_stage);
        d->h_stage = nullptr; d->h_stage_ints = 0;
        if (cudaHostAlloc((void**)&d->h_stage, n_stage_ints * sizeof(int32_t), cudaHostAllocMapped) != cudaSuccess ||
            cudaHostGetDevicePointer((void**)&d->h_stage_dev, d->h_stage, 0) != cudaSuccess) {
            cudaGetLastError();
            return mg_fail(ctx, MG_ERR_OOM, "pinned host allocation failed");
        }
        d->h_stage_ints = n_stage_ints;
    }
    DenseHeader* st_hdr = reinterpret_cast<DenseHeader*>(d->h_stage);
    int32_t* st_off = d->h_stage + (sizeof(DenseHeader) + 3) / 4;
    int32_t* st_cum = st_off + (B + 1);
    uint64_t* st_seeds = reinterpret_cast<uint64_t*>(d->h_stage + (((sizeof(DenseHeader) + 3) / 4 + (size_t)(B + 1) + (size_t)B * (k + 2) + 1) & ~(size_t)1));
    memset(st_hdr, 0, sizeof(DenseHeader));
    st_hdr->hop_base[0] = 0;
    st_hdr->hop_base[1] = (int32_t)T;
    memset(st_cum, 0, sizeof(int32_t) * (size_t)B * (k + 2));
    for (int b = 0; b <= B; ++b) st_off[b] = (int32_t)target_offsets[b];
    for (int b = 0; b < B; ++b) st_cum[(size_t)b * (k + 2) + 1] = st_off[b + 1] - st_off[b];
    memcpy(st_seeds, seeds, sizeof(uint64_t) * B);

    // the summary's landing place (mapped pinned memory)
    const size_t n_ints = (sizeof(DenseHeader) + 3) / 4 + (size_t)B * (k + 2) + 2 * (size_t)(k + 1) * (B + 1) + (size_t)k * (B + 1);
    if (d->h_pinned_ints < n_ints) {
        if (d->h_pinned) cudaFreeHost(d->h_pinned);
        d->h_pinned = nullptr; d->h_pinned_ints = 0;
        if (cudaHostAlloc((void**)&d->h_pinned, n_ints * sizeof(int32_t), cudaHostAllocMapped) != cudaSuccess ||
            cudaHostGetDevicePointer((void**)&d->h_pinned_dev, d->h_pinned, 0) != cudaSuccess) {
            cudaGetLastError();
            return mg_fail(ctx, MG_ERR_OOM, "pinned host allocation failed");
        }
        d->h_pinned_ints = n_ints;
    }
    sample_kernel_attributes();

    // the targets are staged in newlist[1] (outside the graph: their source changes from call to call)
    if (T > 0) {
        if (targets_on_device) {
            k_copy_i32<<<std::max(1, std::min(mg_grid(ctx, 2), (int)((T + kThreads - 1) / kThreads))), kThreads, 0, st>>>(targets, (int32_t*)d->newlist[1], T);
            ctx->launches++;
        } else {
            MG_CUDA(ctx, cudaMemcpyAsync(d->newlist[1], targets, sizeof(int32_t) * T, cudaMemcpyHostToDevice, st));
        }
    }
    const int32_t* tgt_dev = (const int32_t*)d->newlist[1];

    // ---- everything the device does for this sample ----
    auto enqueue = [&]() -> int {
    {
        ProfScope ps(ctx, PH_SAMPLE_INIT, 1);
        static_assert(sizeof(DenseHeader) % 4 == 0, "the header is staged as 32-bit words");
        k_stage_in<<<4, kThreads, 0, st>>>(d->h_stage_dev, (int32_t)(sizeof(DenseHeader) / 4), B + 1, B * (k + 2), 2 * B,
                                          (int32_t)(reinterpret_cast<int32_t*>(st_seeds) - d->h_stage), reinterpret_cast<int32_t*>(d->hdr),
                                          d->node_off, d->cum, reinterpret_cast<int32_t*>(d->d_seeds));
        ctx->launches++;
        MG_CUDA(ctx, cudaMemsetAsync(d->hkeys, 0xFF, sizeof(int32_t) * (size_t)B * table_size, st));
        {
            k_init_targets<<<mg_grid(ctx, 4), kThreads, 0, st>>>(d->hdr, tgt_dev, d->node_off, B, d->nodes,
                                                               d->node_batch, d->hkeys, d->hvals, tg, ctx->n_nodes, mg_feat_geom(ctx));
            ctx->launches++;
        }
    }

    // new nodes per (hop, mini-batch)
    uint32_t* batch_cnt = d->batch_cnt;
    MG_CUDA(ctx, cudaMemsetAsync(batch_cnt, 0, sizeof(uint32_t) * (size_t)k * B, st));
    uint32_t* scan_total = (uint32_t*)(d->scan_tmp + d->scan_tmp_elems - 4);
    const int grid = mg_grid(ctx, 8);
    for (int h = 0; h < k; ++h) {
        const int32_t f = fanouts[h];
        {
            ProfScope ps(ctx, PH_SAMPLE_COUNT, 1);
            k_count<<<grid, kThreads, 0, st>>>(d->hdr, h, f, d->nodes, ctx->view_off, d->ent_off, d->node_r0, d->node_deg,
                                               inout ? ctx->view_off_out : nullptr, d->node_r0_out, d->node_deg_out);
        }
        {
            ProfScope ps(ctx, PH_SAMPLE_SCAN, 3);
            // (the scan's middle kernel also closes the hop's entry range: ent_base, the sentinel offset, the arena check)
            const ScanRange sr{&d->hdr->hop_base[h], &d->hdr->hop_base[h + 1], &d->hdr->ent_base[h]};
            k_scan_reduce<<<grid, kThreads, 0, st>>>((uint32_t*)d->ent_off, sr, (uint32_t*)d->scan_tmp);
            k_scan_tiles<<<1, 1024, 0, st>>>((uint32_t*)d->scan_tmp, sr, scan_total, HopClose{d->hdr, h, d->ent_off, d->cap_entries});
            k_scan_down<<<grid, kThreads, 0, st>>>((uint32_t*)d->ent_off, sr, (uint32_t*)d->scan_tmp);
            ctx->launches += 3;
        }
        {
            ProfScope ps(ctx, PH_SAMPLE_PICK, 1);
            for (int dir = 0; dir < (inout ? 2 : 1); ++dir) {
                PickArgs a{d->hdr, h, f, d->nodes, d->node_batch, dir ? d->node_r0_out : d->node_r0, dir ? d->node_deg_out : d->node_deg,
                           dir ? ctx->view_nbrs_out : ctx->view_nbrs, d->ent_off, d->ent_nbrs, d->ent_repr, d->d_seeds,
                           dir ? d->node_deg : nullptr, dir ? (uint32_t)MG_OUT_SLOT_BASE : 0u};
                // the narrowest group that holds the fanout among those that waste at most two lanes of a warp
                if (f <= 2) k_pick<2><<<grid, kThreads, 0, st>>>(a);
                else if (f == 3) k_pick<3><<<grid, kThreads, 0, st>>>(a);
                else if (f == 4) k_pick<4><<<grid, kThreads, 0, st>>>(a);
                else if (f == 5) k_pick<5><<<grid, kThreads, 0, st>>>(a);
                else if (f == 6) k_pick<6><<<grid, kThreads, 0, st>>>(a);
                else if (f <= 8) k_pick<8><<<grid, kThreads, 0, st>>>(a);
                else if (f <= 10) k_pick<10><<<grid, kThreads, 0, st>>>(a);
                else if (f <= 16) k_pick<16><<<grid, kThreads, 0, st>>>(a);
                else if (f <= 32) k_pick<32><<<grid, kThreads, 0, st>>>(a);
                else {
                    const size_t wide_smem = (size_t)(kThreads / 32) * 2 * f * sizeof(uint32_t);   // 64 KiB at the largest fanout
                    k_pick_wide<<<grid, kThreads, wide_smem, st>>>(a);
                }
                if (dir) ctx->launches++;
            }
            if (smem_last && h == k - 1) {
                DedupArgs da{d->hdr, h, B, k, (int32_t)dedup_nb, dedup_slots, d->nodes, d->node_off, d->ent_off, d->ent_nbrs,
                             d->ent_repr, d->pairs, d->share_off, d->cum, batch_cnt + (size_t)h * B, d->newlist[0], d->cap_nodes,
                             id_bits, (int32_t)cap_batch, d->cap_entries};
                k_bucket_entries<<<(unsigned)(B * dedup_nb), kBucketThreads, 0, st>>>(da);
                k_dedupe_last<<<(unsigned)(B * dedup_nb), kDedupThreads, (size_t)dedup_slots * 2 * sizeof(int32_t), st>>>(da);
                ctx->launches += 2;
            } else {
                InsertArgs ia{d->hdr, h, d->ent_nbrs, d->ent_repr, d->hkeys, tg, d->newlist[0], d->cap_nodes, id_bits,
                              k, d->cum, d->hvals, batch_cnt + (size_t)h * B, (int32_t)cap_batch};
                // many short blocks: measured on the bench's last hop, 0.94 ms at 32 blocks per SM against 1.08 ms at 8
                // (blocks past the end of the entries return at once)
                const int igrid = mg_grid(ctx, 32);
                k_insert<<<igrid, kThreads, 0, st>>>(ia);
                ctx->launches++;
            }
        }
        {
            // rows were handed out at insert time, in discovery order: per-batch counts -> offsets, then every list
            // entry (mini-batch, id, rank) goes to its place.  No sort, no second pass over the id tables.
            ProfScope ps(ctx, PH_SAMPLE_PLACE, 2);
            int32_t* off_next = d->node_off + (size_t)(h + 1) * (B + 1);
            k_outer_offsets<<<1, 1024, 0, st>>>(d->hdr, h, B, k, batch_cnt + (size_t)h * B, off_next, d->cum, (int32_t)cap_batch, d->cap_nodes);
            k_place_nodes_outer<<<grid, kThreads, 0, st>>>(d->hdr, d->newlist[0], id_bits, off_next, d->nodes, d->node_batch);
            ctx->launches += 2;
        }
        if (!(smem_last && h == k - 1)) {   // (the last hop's shared-memory kernel leaves final rows)
            ProfScope ps(ctx, PH_SAMPLE_RELABEL, 1);
            k_relabel<<<grid, kThreads, 0, st>>>(d->hdr, h, d->hvals, d->ent_repr);
            ctx->launches++;
        }
        ctx->launches += 1 + 1;  // count, pick
    }
    {
        ProfScope ps(ctx, PH_SAMPLE_FINAL, 1);
        // (the summary goes to pinned host memory behind the kernels; mg_sample_many_end waits for it)
        static_assert(sizeof(DenseHeader) % 4 == 0, "the header is copied as 32-bit words");
        k_finalize<<<1, 1024, 0, st>>>(d->hdr, B, k, d->cum, d->node_off, d->ent_off, d->rowbase, d->d_ent_hop,
                                       (int32_t)((sizeof(DenseHeader) + 3) / 4), d->h_pinned_dev);
        ctx->launches++;
    }
    MG_CUDA(ctx, cudaGetLastError());
    return MG_OK;
    };   // enqueue

    // Replay the captured graph when nothing that the device work depends on has changed since it was captured;
    // capture it (again) otherwise.  Profiling runs the launches one by one (its events do not belong in a graph).
    SampleSignature sig;
    memset(&sig, 0, sizeof(sig));
    sig.B = B; sig.k = k; sig.T = 0; sig.table_size = table_size; sig.cap_batch = cap_batch;   // (the device work does not depend on T)
    sig.cap_nodes = d->cap_nodes; sig.cap_entries = d->cap_entries; sig.n_nodes = ctx->n_nodes; sig.part_size = ctx->part_size;
    sig.inout = (inout ? 1 : 0) | (smem_last ? 2 + 4 * dedup_nb : 0);
    for (int h = 0; h < k; ++h) sig.fanouts[h] = fanouts[h];
    const void* ptrs[] = {d->hdr, d->nodes, d->node_batch, d->ent_off, d->node_r0, d->node_deg, d->newlist[0], d->newlist[1],
                          d->scan_tmp, d->sort_hist, d->ent_nbrs, d->ent_repr, d->hkeys, d->hvals, d->node_off, d->cum, d->rowbase,
                          d->d_ent_hop, d->d_seeds, d->h_stage_dev, d->h_pinned_dev, ctx->view_off, ctx->view_nbrs, ctx->d_slot_of_part, st, ctx->d_part_of_node,
                          inout ? (const void*)ctx->view_off_out : nullptr, inout ? (const void*)ctx->view_nbrs_out : nullptr,
                          d->node_r0_out, d->node_deg_out, d->pairs, d->share_off};
    static_assert(sizeof(ptrs) <= sizeof(sig.ptrs), "signature too small");
    memcpy(sig.ptrs, ptrs, sizeof(ptrs));
    const bool use_graph = ctx->sample_graphs && !ctx->prof_on && !getenv("MG_NO_SAMPLE_GRAPH");
    if (use_graph) {
        if (!d->graph_exec || memcmp(&sig, &d->graph_sig, sizeof(sig)) != 0) {
            if (d->graph_exec) { cudaGraphExecDestroy(d->graph_exec); d->graph_exec = nullptr; }
            const int64_t launches0 = ctx->launches;
            MG_CUDA(ctx, cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
            const int erc = enqueue();
            cudaGraph_t graph = nullptr;
            const cudaError_t ce = cudaStreamEndCapture(st, &graph);
            d->graph_launches = ctx->launches - launches0;
            ctx->launches = launches0;
            if (erc || ce != cudaSuccess || !graph) {
                if (graph) cudaGraphDestroy(graph);
                cudaGetLastError();
                return erc ? erc : mg_fail(ctx, MG_ERR_CUDA, "capture of the sampler failed: %s", cudaGetErrorString(ce));
            }
            const cudaError_t ie = cudaGraphInstantiate(&d->graph_exec, graph, 0);
            cudaGraphDestroy(graph);
            if (ie != cudaSuccess) { d->graph_exec = nullptr; cudaGetLastError(); return mg_fail(ctx, MG_ERR_CUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(ie)); }
            d->graph_sig = sig;
        }
        MG_CUDA(ctx, cudaGraphLaunch(d->graph_exec, st));
        ctx->launches += d->graph_launches;
    } else {
        const int erc = enqueue();
        if (erc) return erc;
    }
    if (!d->ev_sampled) MG_CUDA(ctx, cudaEventCreateWithFlags(&d->ev_sampled, cudaEventDisableTiming));
    MG_CUDA(ctx, cudaEventRecord(d->ev_sampled, st));
    d->pending = true;
    return MG_OK;
}

extern "C" int mg_sample(mg_ctx* ctx, const int32_t* targets, int targets_on_device, int32_t n_targets,
                         const int32_t* fanouts, int32_t k, uint64_t seed, const mg_sample_caps* caps, mg_dense** out) {
    if (!ctx) return MG_ERR_ARG;
    if (n_targets < 0) return mg_fail(ctx, MG_ERR_ARG, "negative n_targets");
    const int64_t off[2] = {0, n_targets};
    return mg_sample_many(ctx, targets, targets_on_device, off, 1, fanouts, k, &seed, caps, out);
}

extern "C" int mg_dense_counts(const mg_dense* d, int32_t* n_batches, int32_t* k, int64_t* nodes_per_hop,
                               int64_t* entries_per_hop) {
    if (!d) return MG_ERR_ARG;
    if (!d->valid) return MG_ERR_STATE;
    const int B = d->n_batches, K = d->k;
    if (n_batches) *n_batches = B;
    if (k) *k = K;
    if (nodes_per_hop)
        for (int b = 0; b < B; ++b)
            for (int h = 0; h <= K; ++h)
                nodes_per_hop[(size_t)b * (K + 1) + h] = d->h_cum[(size_t)b * (K + 2) + h + 1] - d->h_cum[(size_t)b * (K + 2) + h];
    if (entries_per_hop)
        for (int b = 0; b < B; ++b)
            for (int h = 0; h < K; ++h)
                entries_per_hop[(size_t)b * K + h] = d->h_ent_hop[(size_t)h * (B + 1) + b + 1] - d->h_ent_hop[(size_t)h * (B + 1) + b];
    return MG_OK;
}


static void batch_geom(const mg_dense* d, int b, BatchGeom* g) {
    const int k = d->k, B = d->n_batches;
    memset(g, 0, sizeof(*g));
    g->k = k;
    for (int h = 0; h <= k + 1; ++h) g->cum[h] = d->h_cum[(size_t)b * (k + 2) + h];
    for (int h = 0; h <= k; ++h) g->node_off[h] = d->h_node_off[(size_t)h * (B + 1) + b];
    g->V = g->cum[k + 1];
    g->n_targets = g->cum[1];
}

// perm / inv of mini-batch b (device arrays owned by d, valid until the next call for another batch or sample)
int mg_dense_batch_perm(mg_ctx* ctx, mg_dense* d, int b, const int32_t** perm, const int32_t** inv) {
    BatchGeom g;
    batch_geom(d, b, &g);
    int rc = mg_ensure(ctx, &d->perm_buf, &d->perm_elems, 2 * (size_t)g.V + 8);
    if (rc) return rc;
    *perm = d->perm_buf;
    *inv = d->perm_buf + g.V;
    if (d->perm_batch == b) return MG_OK;
    d->perm_batch = -1;
    cudaStream_t st = ctx->stream;
    if (d->export_pending) MG_CUDA(ctx, cudaStreamWaitEvent(st, d->ev_exported, 0));   // the export uses the same sort scratch
    const int32_t n = g.V - g.n_targets;
    const int id_bits = std::max(1, ilog2_ceil(ctx->n_nodes)), hop_bits = std::max(1, ilog2_ceil(g.k + 1));
    const int grid = std::max(1, std::min(mg_grid(ctx, 4), (g.V + kThreads - 1) / kThreads));
    int res = 0;
    if (n > 0) {
        SortParams* sp = (SortParams*)(d->scan_tmp + d->scan_tmp_elems - 8);   // tail of the scratch block, as in the sampler
        SortParams h_sp;
        mg_sort_params_host(&h_sp, n);
        MG_CUDA(ctx, cudaMemcpyAsync(sp, &h_sp, sizeof(h_sp), cudaMemcpyHostToDevice, st));
        k_perm_keys<<<grid, kThreads, 0, st>>>(g, d->nodes, id_bits, d->newlist[0]);
        mg_sort_u64(ctx, d->newlist, sp, MG_SLOT_BITS, id_bits + hop_bits, d->sort_hist, (uint32_t*)d->scan_tmp, &res);
        ctx->launches++;
    }
    if (g.V > 0) {
        k_perm_fill<<<grid, kThreads, 0, st>>>(g, d->newlist[res], d->perm_buf, d->perm_buf + g.V);
        ctx->launches++;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(st));   // h_sp is a stack variable
    d->perm_batch = b;
    return MG_OK;
}

extern "C" int mg_dense_view(mg_ctx* ctx, mg_dense* d, int32_t batch, mg_dense_arrays* out) {
    if (!ctx) return MG_ERR_ARG;
    if (!d || !out) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (!d->valid) return mg_fail(ctx, MG_ERR_STATE, "mg_dense holds no completed sample");
    if (batch < 0 || batch >= d->n_batches) return mg_fail(ctx, MG_ERR_ARG, "batch out of range");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    const int k = d->k, B = d->n_batches, b = batch;
    ExportArgs a;
    memset(&a, 0, sizeof(a));
    batch_geom(d, b, &a.g);
    int rc = mg_dense_batch_perm(ctx, d, b, &a.perm, &a.inv);
    if (rc) return rc;
    // canonical Delta_j = hop k - j
    a.nio[0] = 0;
    for (int j = 0; j <= k; ++j) a.nio[j + 1] = a.nio[j] + (a.g.cum[k - j + 1] - a.g.cum[k - j]);
    a.n0 = a.nio[1];
    int32_t n_entries = 0;
    for (int h = 0; h < k; ++h) n_entries += d->h_ent_hop[(size_t)h * (B + 1) + b + 1] - d->h_ent_hop[(size_t)h * (B + 1) + b];
    const int32_t n_s = a.g.V - a.n0;
    const size_t need = (size_t)a.g.V + (k + 2) + 2 * (size_t)n_entries + (size_t)n_s + 1 + 16;
    rc = mg_ensure(ctx, &d->exp_buf, &d->exp_elems, need);
    if (rc) return rc;
    a.nodes = d->nodes; a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
    a.o_node_ids = d->exp_buf;
    a.o_nio = a.o_node_ids + a.g.V;
    a.o_nbrs = a.o_nio + (k + 2);
    a.o_nbr_off = a.o_nbrs + n_entries;
    a.o_repr = a.o_nbr_off + n_s + 1;
    const int grid = std::max(1, std::min(mg_grid(ctx, 4), (a.g.V + kThreads - 1) / kThreads));
    k_export_nodes<<<grid, kThreads, 0, ctx->stream>>>(a);
    k_export_scan<<<1, 1024, 0, ctx->stream>>>(a.o_nbr_off, n_s);
    if (n_s > 0) k_export_entries<<<grid, kThreads, 0, ctx->stream>>>(a);
    ctx->launches += 3;
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    out->k = k;
    out->n_nodes = a.g.V;
    out->n_sampled = n_s;
    out->n_entries = n_entries;
    out->node_ids = a.o_node_ids;
    out->node_id_offsets = a.o_nio;
    out->nbrs = a.o_nbrs;
    out->nbr_offsets = a.o_nbr_off;
    out->repr_map = a.o_repr;
    return MG_OK;
}

// Layout of the export buffer (int32 elements), from the sample's capacities so that it is allocated once per handle.
struct ExportLayout { size_t node_ids, nio, nbrs, repr, nbr_off, inv, cnt, total; };
static ExportLayout export_layout(const mg_dense* d) {
    ExportLayout L;
    const size_t cn = (size_t)d->cap_nodes, ce = (size_t)d->cap_entries, B = (size_t)d->n_batches;
    size_t at = 0;
    L.node_ids = at; at += cn;
    L.nio = at; at += B * (MG_MAX_HOPS + 2);
    L.nbrs = at; at += ce;
    L.repr = at; at += ce;
    L.nbr_off = at; at += cn + B + 1;
    L.inv = at; at += cn;
    L.cnt = at; at += cn + 1;
    L.total = at + 16;
    return L;
}

extern "C" int mg_dense_export_many(mg_ctx* ctx, mg_dense* d) {
    if (!ctx) return MG_ERR_ARG;
    if (!d) return mg_fail(ctx, MG_ERR_ARG, "null mg_dense");
    if (d->ctx != ctx) return mg_fail(ctx, MG_ERR_ARG, "mg_dense belongs to another context");
    if (d->pending) return mg_fail(ctx, MG_ERR_STATE, "a sample is in flight on this mg_dense: call mg_sample_many_end first");
    if (!d->valid) return mg_fail(ctx, MG_ERR_STATE, "mg_dense holds no completed sample");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    const int k = d->k, B = d->n_batches;
    const int32_t n_total = d->h_hdr.hop_base[k + 1];
    const int id_bits = std::max({1, ilog2_ceil(ctx->n_nodes), ilog2_ceil(d->n_targets_total + 1)});
    const int pay_bits = std::max(1, ilog2_ceil((int64_t)n_total + 1));
    if (id_bits + pay_bits > 64)
        return mg_fail(ctx, MG_ERR_CAPACITY, "sample too large for a one-pass export (%d key bits): export fewer mini-batches per sample", id_bits + pay_bits);
    if ((int64_t)(n_total + kSortTile - 1) / kSortTile + (int64_t)B * (k + 1) > d->cap_sort_tiles)
        return mg_fail(ctx, MG_ERR_STATE, "the sort scratch of this mg_dense is too small for its sample");
    const ExportLayout L = export_layout(d);
    int rc = mg_ensure(ctx, &d->expm_buf, &d->expm_elems, L.total);
    if (rc) return rc;
    if (!d->ev_exported) MG_CUDA(ctx, cudaEventCreateWithFlags(&d->ev_exported, cudaEventDisableTiming));
    // on the sampling stream: behind the sample (and a later sample into d behind this), beside the layers
    cudaStream_t user = ctx->stream;
    cudaStream_t st = ctx->sample_stream;
    ExportManyArgs a;
    memset(&a, 0, sizeof(a));
    a.B = B; a.k = k; a.n_nodes_total = n_total; a.pay_bits = pay_bits; a.id_bits = id_bits;
    for (int h = 0; h <= k + 1; ++h) a.hop_base[h] = d->h_hdr.hop_base[h];
    a.nodes = d->nodes; a.node_batch = d->node_batch; a.node_off = d->node_off; a.cum = d->cum; a.rowbase0 = d->rowbase;
    a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
    a.o_node_ids = d->expm_buf + L.node_ids; a.o_nio = d->expm_buf + L.nio; a.o_nbrs = d->expm_buf + L.nbrs;
    a.o_repr = d->expm_buf + L.repr; a.o_nbr_off = d->expm_buf + L.nbr_off; a.inv = d->expm_buf + L.inv;
    a.cnt = reinterpret_cast<uint32_t*>(d->expm_buf + L.cnt);
    d->export_valid = false;
    if (n_total > 0) {
        SortParams* sp = (SortParams*)(d->scan_tmp + d->scan_tmp_elems - 8);
        int32_t* range = d->scan_tmp + d->scan_tmp_elems - 12;
        const int grid = mg_grid(ctx, 8);
        ctx->stream = st;   // the sort and scan helpers (and the phase events) use ctx->stream
        {
        ProfScope ps(ctx, PH_SAMPLE_SORT, 0);
        k_export_tiles<<<1, 1024, 0, st>>>(a, static_cast<SegTile*>(d->seg_tiles), sp, range);
        k_export_keys<<<grid, kThreads, 0, st>>>(a, d->newlist[0]);
        int res = 0;
        mg_sort_u64(ctx, d->newlist, sp, pay_bits, id_bits, d->sort_hist, (uint32_t*)d->scan_tmp, &res, d->seg_tiles);
        k_export_place<<<grid, kThreads, 0, st>>>(a, d->newlist[res]);
        mg_scan_u32(ctx, a.cnt, &range[0], &range[1], nullptr, (uint32_t*)d->scan_tmp, nullptr);
        k_export_many_entries<<<grid, kThreads, 0, st>>>(a);
        }
        ctx->stream = user;
        ctx->launches += 4;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaEventRecord(d->ev_exported, st));
    d->export_pending = true;
    d->export_valid = true;
    d->perm_batch = -1;   // the per-batch permutation shares the sort scratch
    return MG_OK;
}

extern "C" int mg_dense_export_view(mg_ctx* ctx, mg_dense* d, int32_t batch, mg_dense_arrays* out) {
    if (!ctx) return MG_ERR_ARG;
    if (!d || !out) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (!d->valid || !d->export_valid) return mg_fail(ctx, MG_ERR_STATE, "no export of this sample: call mg_dense_export_many first");
    if (batch < 0 || batch >= d->n_batches) return mg_fail(ctx, MG_ERR_ARG, "batch out of range");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    if (d->export_pending) { MG_CUDA(ctx, cudaEventSynchronize(d->ev_exported)); d->export_pending = false; }
    const int k = d->k, B = d->n_batches, b = batch;
    const ExportLayout L = export_layout(d);
    const int32_t row0 = d->h_rowbase[b], V = d->h_rowbase[b + 1] - row0;
    const int32_t n0 = d->h_cum[(size_t)b * (k + 2) + k + 1] - d->h_cum[(size_t)b * (k + 2) + k];
    int64_t e_before = 0, e_mine = 0;
    for (int h = 0; h < k; ++h) {
        // entries are packed mini-batch after mini-batch in the export
        for (int bb = 0; bb < b; ++bb) e_before += d->h_ent_hop[(size_t)h * (B + 1) + bb + 1] - d->h_ent_hop[(size_t)h * (B + 1) + bb];
        e_mine += d->h_ent_hop[(size_t)h * (B + 1) + b + 1] - d->h_ent_hop[(size_t)h * (B + 1) + b];
    }
    out->k = k;
    out->n_nodes = V;
    out->n_sampled = V - n0;
    out->n_entries = (int32_t)e_mine;
    out->node_ids = d->expm_buf + L.node_ids + row0;
    out->node_id_offsets = d->expm_buf + L.nio + (size_t)b * (k + 2);
    out->nbrs = d->expm_buf + L.nbrs + e_before;
    out->repr_map = d->expm_buf + L.repr + e_before;
    out->nbr_offsets = d->expm_buf + L.nbr_off + row0 + b;
    return MG_OK;
}

extern "C" int mg_dense_free(mg_dense* d) {
    if (!d) return MG_OK;
    cudaSetDevice(d->device);
    if (d->ctx && d->ctx->last_fwd_dense == d) d->ctx->last_fwd_dense = nullptr;
    cudaFree(d->hdr); cudaFree(d->nodes); cudaFree(d->node_batch); cudaFree(d->ent_off); cudaFree(d->node_r0); cudaFree(d->node_deg); cudaFree(d->node_r0_out); cudaFree(d->node_deg_out); cudaFree(d->pairs); cudaFree(d->share_off);
    cudaFree(d->ent_nbrs); cudaFree(d->ent_repr); cudaFree(d->node_off); cudaFree(d->cum);
    cudaFree(d->rowbase); cudaFree(d->hkeys); cudaFree(d->hvals); cudaFree(d->newlist[0]);
    cudaFree(d->newlist[1]); cudaFree(d->d_seeds); cudaFree(d->batch_cnt); cudaFree(d->scan_tmp); cudaFree(d->sort_hist); cudaFree(d->seg_tiles);
    cudaFree(d->exp_buf); cudaFree(d->perm_buf); cudaFree(d->d_ent_hop); cudaFree(d->expm_buf);
    if (d->ev_exported) cudaEventDestroy(d->ev_exported);
    if (d->h_pinned) cudaFreeHost(d->h_pinned);
    if (d->h_stage) cudaFreeHost(d->h_stage);
    if (d->graph_exec) cudaGraphExecDestroy(d->graph_exec);
    if (d->ev_sampled) cudaEventDestroy(d->ev_sampled);
    if (d->ev_read_done) cudaEventDestroy(d->ev_read_done);
    delete d;
    return MG_OK;
}
