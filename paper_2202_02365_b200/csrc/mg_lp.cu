// Link prediction: shared uniform negatives per chunk, the batch's target union, and DistMult
// scoring (the decoder of the paper's link-prediction configuration, Section 7.1).

#include <algorithm>
#include <cstdlib>

#include "mg_device.cuh"
#include "mg_internal.cuh"
#include "mg_tcgen05.cuh"

namespace {

constexpr int kThreads = 256;

// The target union of a batch = the distinct ids among sources, destinations and negatives, ascending.  It is taken
// with a bit per node: every id sets its bit (k_lp_mark, which also draws the negatives), the words' population counts
// are scanned, a word's set bits are written out from its prefix on (k_lp_emit), and the row of an id is its word's prefix
// plus the set bits below it (k_lp_index); counts and prefixes are kept per group of 32 words, so the scan runs over
// n_nodes / 1024 values.  Seven short launches, none of them a sort.
// Origins: [0, E) sources, [E, 2E) destinations, [2E, 2E + C * negs) negatives.
__global__ void __launch_bounds__(kThreads)
k_lp_mark(const int32_t* __restrict__ src, const int32_t* __restrict__ dst, int64_t E, int32_t n_chunks, int32_t negs,
          uint64_t seed, const int64_t* __restrict__ res_prefix, int32_t n_parts, int64_t n_resident, int64_t n_nodes, FeatGeom feat,
          const int64_t* __restrict__ part_start, const int32_t* __restrict__ nodes_by_part, int32_t* neg_ids, uint32_t* bitmap,
          uint32_t* status) {
    const int64_t total = 2 * E + (int64_t)n_chunks * negs;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int32_t id;
        if (i < 2 * E) {
            id = i < E ? src[i] : dst[i - E];
            if (id < 0 || (int64_t)id >= n_nodes) { atomicOr(status, ST_RANGE); id = 0; }
            else if (!feat_resident(feat, id)) atomicOr(status, ST_NONRESIDENT);
        } else {
            const int64_t j = i - 2 * E;
            const uint32_t c = (uint32_t)(j / negs), t = (uint32_t)(j % negs);
            uint32_t o[4];
            philox4x32_10(c, t, 0xFFFFFFFFu, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), o);
            // index among the resident nodes, counted in ascending partition order
            const int64_t r = (int64_t)(((unsigned __int128)o[0] * (unsigned __int128)(uint64_t)n_resident) >> 32);
            int p = 0;
            while (p + 1 < n_parts && res_prefix[p + 1] <= r) ++p;
            // (partitions are id ranges, or, with a partition-id array, listed in nodes_by_part in ascending id)
            id = nodes_by_part ? nodes_by_part[part_start[p] + (r - res_prefix[p])] : (int32_t)(part_start[p] + (r - res_prefix[p]));
            neg_ids[j] = id;
        }
        atomicOr(&bitmap[(uint32_t)id >> 5], 1u << (id & 31));
    }
}

// population count of every group of 32 words (1,024 nodes): the scan then runs over n_words / 32 counts
constexpr int kLpGroup = 32;
__global__ void __launch_bounds__(kThreads) k_lp_popc(const uint32_t* __restrict__ bitmap, int32_t n_words, int32_t n_groups, uint32_t* counts) {
    const int lane = threadIdx.x & 31;
    const int32_t warps = gridDim.x * (kThreads / 32);
    for (int32_t g = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); g < n_groups; g += warps) {
        const int32_t w = g * kLpGroup + lane;
        uint32_t c = w < n_words ? __popc(bitmap[w]) : 0u;
        for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
        if (lane == 0) counts[g] = c;
    }
}

// after the exclusive scan of the group counts: the ids of the set bits, ascending (a warp per group: lane = word)
__global__ void __launch_bounds__(kThreads)
k_lp_emit(const uint32_t* __restrict__ bitmap, const uint32_t* __restrict__ prefix, int32_t n_words, int32_t n_groups, int32_t* targets) {
    const int lane = threadIdx.x & 31;
    const int32_t warps = gridDim.x * (kThreads / 32);
    for (int32_t g = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5); g < n_groups; g += warps) {
        const int32_t w = g * kLpGroup + lane;
        uint32_t bits = w < n_words ? bitmap[w] : 0u;
        if (!__any_sync(0xFFFFFFFFu, bits != 0u)) continue;
        const uint32_t c = __popc(bits);
        uint32_t at = prefix[g] + warp_incl_scan(c) - c;
        while (bits) {
            const int bpos = __ffs(bits) - 1;
            targets[at++] = w * 32 + bpos;
            bits &= bits - 1;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
k_lp_index(const int32_t* __restrict__ src, const int32_t* __restrict__ dst, const int32_t* __restrict__ neg_ids, int64_t E,
           int64_t total, int64_t n_nodes, const uint32_t* __restrict__ bitmap, const uint32_t* __restrict__ prefix,
           int32_t* src_idx, int32_t* dst_idx, int32_t* neg_idx, const uint32_t* status, const int32_t* n_targets, int32_t* host_words) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {   // the call's two results, straight into mapped host memory
        host_words[0] = (int32_t)*status;
        host_words[1] = *n_targets;
    }
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int32_t id = i < E ? src[i] : (i < 2 * E ? dst[i - E] : neg_ids[i - 2 * E]);
        if (id < 0 || (int64_t)id >= n_nodes) id = 0;   // (as k_lp_mark: the call fails with the range error anyway)
        const uint32_t w = (uint32_t)id >> 5;
        // the group's prefix, the set bits of the group's words before this one, the set bits below the id in its word
        uint32_t rank = prefix[w / kLpGroup] + __popc(bitmap[w] & ((1u << (id & 31)) - 1u));
        for (uint32_t v = w - w % kLpGroup; v < w; ++v) rank += __popc(bitmap[v]);
        if (i < E) src_idx[i] = (int32_t)rank;
        else if (i < 2 * E) dst_idx[i - E] = (int32_t)rank;
        else neg_idx[i - 2 * E] = (int32_t)rank;
    }
}

// pos[i] = sum_d h[s_i, d] * rel[r_i, d] * h[o_i, d]; one warp per edge, fixed summation order
__global__ void __launch_bounds__(kThreads)
k_distmult_pos(const float* __restrict__ h, const float* __restrict__ rel_emb, const int32_t* __restrict__ src_idx,
               const int32_t* __restrict__ dst_idx, const int32_t* __restrict__ rel, int64_t E, int dim, float* pos) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
    for (int64_t i = blockIdx.x * (int64_t)(kThreads / 32) + (threadIdx.x >> 5); i < E; i += warps) {
        const float* hs = h + (int64_t)src_idx[i] * dim;
        const float* ho = h + (int64_t)dst_idx[i] * dim;
        const float* r = rel_emb + (int64_t)rel[i] * dim;
        float s = 0.f;
        for (int d = lane; d < dim; d += 32) s = fmaf(hs[d] * r[d], ho[d], s);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (lane == 0) pos[i] = s;
    }
}

// neg[i, t] = sum_d (h[a_i, d] * rel[r_i, d]) * h[neg_{c(i), t}, d], a = source (destination side
// corrupted) or destination (source side corrupted).  Tiles of 64 edges x 64 negatives inside one
// chunk; both operands are gathered into shared memory.
struct NegArgs {
    const float* h;
    const float* rel_emb;
    const int32_t* keep_idx;  // src_idx when the destination is corrupted, dst_idx otherwise
    const int32_t* rel;
    const int32_t* neg_idx;   // [n_chunks, negs]
    int64_t E;
    int32_t n_chunks, negs, dim, tiles_per_chunk;
    float* out;               // [E, negs]
};

__global__ void __launch_bounds__(256) k_distmult_neg(NegArgs a) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    __shared__ int32_t a_row[BM], a_rel[BM], b_row[BN];
    const int c = blockIdx.x / a.tiles_per_chunk;
    const int tile = blockIdx.x % a.tiles_per_chunk;
    // chunk c holds the edges i with floor(i * n_chunks / E) == c
    const int64_t lo = ((int64_t)c * a.E + a.n_chunks - 1) / a.n_chunks;
    const int64_t hi = ((int64_t)(c + 1) * a.E + a.n_chunks - 1) / a.n_chunks;
    const int64_t m0 = lo + (int64_t)tile * BM;
    if (m0 >= hi) return;
    const int n0 = blockIdx.y * BN;
    if (threadIdx.x < BM) {
        const int64_t i = m0 + threadIdx.x;
        a_row[threadIdx.x] = i < hi ? a.keep_idx[i] : -1;
        a_rel[threadIdx.x] = i < hi ? a.rel[i] : 0;
    } else if (threadIdx.x < BM + BN) {
        const int t = n0 + (threadIdx.x - BM);
        b_row[threadIdx.x - BM] = t < a.negs ? a.neg_idx[(int64_t)c * a.negs + t] : -1;
    }
    __syncthreads();
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < a.dim; k0 += BK) {
        for (int i = threadIdx.x; i < BM * BK; i += 256) {
            const int mm = i / BK, kk = i % BK;
            float v = 0.f;
            if (a_row[mm] >= 0 && k0 + kk < a.dim)
                v = a.h[(int64_t)a_row[mm] * a.dim + k0 + kk] * a.rel_emb[(int64_t)a_rel[mm] * a.dim + k0 + kk];
            As[kk][mm] = v;
        }
        for (int i = threadIdx.x; i < BN * BK; i += 256) {
            const int nn = i / BK, kk = i % BK;
            Bs[kk][nn] = (b_row[nn] >= 0 && k0 + kk < a.dim) ? a.h[(int64_t)b_row[nn] * a.dim + k0 + kk] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = As[kk][ty * 4 + i]; bv[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= hi) continue;
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < a.negs) a.out[m * a.negs + n] = acc[i][j];
        }
    }
}

// ---- tensor-core negative scoring ------------------------------------------------------------
// The right operand -- the chunk's negatives h[neg], rounded to TF32 -- is the same for every 128-edge tile of a chunk:
// k_stage_negs writes it once per call as ready-made operand images (blocks of up to 128 negatives, K-major slices of
// 32 columns, 128-byte swizzle), a few MB that stay in L2, and the scoring kernel fetches a block with one bulk copy
// per slice.
// One CTA of the scoring kernel owns 128 edges of one chunk and one corrupted side.  The left operand rows
// h[keep] (*) rel[r] are gathered once (eight warps), rounded to TF32 and written K-major with the 128-byte swizzle.
// Then, block by block: one thread streams the operand images (two buffers), one thread issues the tcgen05 MMAs (fp32
// accumulator in tensor memory, two buffers), and eight epilogue warps -- four from the start, four more once the left
// operand is in place -- store the scores as coalesced row segments.  The score matrix (4 bytes per (edge, negative))
// is the bulk of the traffic; the contraction itself is small.  Every wait is bounded.
constexpr int kTcGatherWarps = 8, kTcEpilogueWarps = 8;   // warps 4..7 gather first and store afterwards
constexpr int kTcFirstGatherWarp = 4;
constexpr int kTcMmaWarp = kTcFirstGatherWarp + kTcGatherWarps;   // 12
constexpr int kTcCopyWarp = kTcMmaWarp + 1;                       // 13
constexpr int kTcThreads = (kTcCopyWarp + 1) * 32;                // 448
constexpr int kTcMaxSlices = 4;   // dim <= 128
constexpr int kTcBlockN = 128;    // negatives per block

struct NegTcArgs {
    NegArgs base;
    int32_t n_slices, bn_max, tmem_cols;
    const uint8_t* b_images;   // [n_chunks][n_blocks][n_slices][bn_max x 128 bytes]
    uint32_t* error;
};

__device__ __forceinline__ size_t swz_off(int row, int slot) {   // 16-byte slot of a 128-byte row, 8-row groups
    return (size_t)(row >> 3) * 1024 + (size_t)(row & 7) * 128 + (size_t)((slot ^ (row & 7)) << 4);
}

// operand images of the negatives: item = (chunk, block, row of the block, 16-byte slot of the row)
__global__ void __launch_bounds__(kThreads)
k_stage_negs(const float* __restrict__ h, const int32_t* __restrict__ neg_idx, int32_t n_chunks, int32_t negs, int32_t dim,
             int32_t n_slices, int32_t bn_max, uint8_t* images) {
    const int n_slots = n_slices * 8;
    const int n_blocks = (negs + bn_max - 1) / bn_max;
    const int64_t total = (int64_t)n_chunks * n_blocks * bn_max * n_slots;
    const size_t slice_bytes = (size_t)bn_max * 128;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int q = (int)(i % n_slots);
        const int r = (int)((i / n_slots) % bn_max);
        const int64_t cb = i / ((int64_t)n_slots * bn_max);   // chunk * n_blocks + block
        const int n = (int)(cb % n_blocks) * bn_max + r;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (n < negs && q * 4 < dim) {
            const int32_t src = neg_idx[(cb / n_blocks) * negs + n];
            const float4 x = __ldg(reinterpret_cast<const float4*>(h + (int64_t)src * dim) + q);
            v = make_float4(tc::to_tf32(x.x), tc::to_tf32(x.y), tc::to_tf32(x.z), tc::to_tf32(x.w));
        }
        *reinterpret_cast<float4*>(images + ((size_t)cb * n_slices + (q >> 3)) * slice_bytes + swz_off(r, q & 7)) = v;
    }
}

__global__ void __launch_bounds__(kTcThreads, 1) k_distmult_neg_tc(NegTcArgs ta) {
    using namespace tc;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t a_full, b_full[2], b_empty[2], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int32_t a_row[128], a_rel[128];
    __shared__ __align__(16) float out_stage[kTcEpilogueWarps][32 * 32];
    const NegArgs& a = ta.base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* a_smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);   // n_slices x 16 KiB
    const size_t b_slice_bytes = (size_t)ta.bn_max * 128;
    const size_t b_buf_bytes = (size_t)ta.n_slices * b_slice_bytes;
    uint8_t* b_smem = a_smem + (size_t)ta.n_slices * 16384;                          // 2 x n_slices x bn_max x 128 B

    const int c = blockIdx.x / a.tiles_per_chunk, tile = blockIdx.x % a.tiles_per_chunk;
    const int64_t lo = ((int64_t)c * a.E + a.n_chunks - 1) / a.n_chunks;
    const int64_t hi = ((int64_t)(c + 1) * a.E + a.n_chunks - 1) / a.n_chunks;
    const int64_t m0 = lo + (int64_t)tile * 128;
    const int n_blocks = (a.negs + ta.bn_max - 1) / ta.bn_max;
    const int n_slots = ta.n_slices * 8;                  // 16-byte slots per operand row
    constexpr int kGatherThreads = kTcGatherWarps * 32, kGatherUnroll = 8;

    if (threadIdx.x == 0) {
        mbar_init(&a_full, kTcGatherWarps);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1);
            mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], kTcEpilogueWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kTcMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)ta.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x < 128) {
        const int64_t i = m0 + threadIdx.x;
        a_row[threadIdx.x] = i < hi ? a.keep_idx[i] : -1;
        a_rel[threadIdx.x] = i < hi ? a.rel[i] : 0;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t acc_stride = (uint32_t)(ta.tmem_cols / 2);

    if (warp >= kTcFirstGatherWarp && warp < kTcMmaWarp) {
        // ---------------- gather warps: the left operand, once ----------------
        const int gt = threadIdx.x - kTcFirstGatherWarp * 32;
        // (all loads of a round are issued before the first use: the gathers are latency-bound otherwise)
        for (int i0 = gt; i0 < 128 * n_slots; i0 += kGatherThreads * kGatherUnroll) {
            float4 hv[kGatherUnroll], rv[kGatherUnroll];
#pragma unroll
            for (int u = 0; u < kGatherUnroll; ++u) {
                const int i = min(i0 + u * kGatherThreads, 128 * n_slots - 1);
                const int r = i / n_slots, q = i % n_slots;
                const bool on = a_row[r] >= 0 && q * 4 < a.dim;
                // an absent row reads row 0 (always valid) and is zeroed below: no branch around the loads
                hv[u] = __ldg(reinterpret_cast<const float4*>(a.h + (int64_t)(on ? a_row[r] : 0) * a.dim) + (on ? q : 0));
                rv[u] = __ldg(reinterpret_cast<const float4*>(a.rel_emb + (int64_t)(on ? a_rel[r] : 0) * a.dim) + (on ? q : 0));
            }
#pragma unroll
            for (int u = 0; u < kGatherUnroll; ++u) {
                const int i = i0 + u * kGatherThreads;
                if (i >= 128 * n_slots) continue;
                const int r = i / n_slots, q = i % n_slots;
                const bool on = a_row[r] >= 0 && q * 4 < a.dim;
                const float4 v = on ? make_float4(to_tf32(hv[u].x * rv[u].x), to_tf32(hv[u].y * rv[u].y), to_tf32(hv[u].z * rv[u].z),
                                                  to_tf32(hv[u].w * rv[u].w))
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4*>(a_smem + (size_t)(q >> 3) * 16384 + swz_off(r, q & 7)) = v;
            }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&a_full);
    }
    if (warp < kTcEpilogueWarps) {
        // ---------------- epilogue: tensor memory -> coalesced row segments of the score matrix ----------------
        // warp w reads the accumulator rows 32 (w % 4) .. + 31 (its quarter of tensor memory) and takes every second
        // 32-column slice of them
        bool ok = true;
        const int quarter = warp & 3, half = warp >> 2;
        const int64_t row0 = m0 + quarter * 32;
        const bool vec4 = a.negs % 4 == 0 && (reinterpret_cast<uintptr_t>(a.out) & 15) == 0;   // rows start 16-byte aligned
        for (int j = 0; j < n_blocks && ok; ++j) {
            const int buf = j & 1;
            const int n0 = j * ta.bn_max;
            const int bn = min(ta.bn_max, (a.negs - n0 + 15) / 16 * 16);
            if (!mbar_wait(&acc_full[buf], (j >> 1) & 1)) { if (lane == 0) atomicExch(ta.error, 21u); ok = false; break; }
            tc_fence_after();
            for (int c0 = 32 * half; c0 < bn; c0 += 64) {
                uint32_t v[32];
                tmem_ld_32(tmem_base + buf * acc_stride + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row0 < hi) {
                    float* st = out_stage[warp];
                    const int rows = (int)min((int64_t)32, hi - row0);
                    if (vec4) {
                        // lane = row: its 8 16-byte pieces go to slots piece ^ (row % 8) of a 128-byte row; then 8 lanes
                        // store one row's 128 bytes, 4 rows per instruction
                        uint8_t* sb = reinterpret_cast<uint8_t*>(st);
#pragma unroll
                        for (int p = 0; p < 8; ++p)
                            *reinterpret_cast<float4*>(sb + lane * 128 + ((p ^ (lane & 7)) << 4)) =
                                make_float4(__uint_as_float(v[4 * p]), __uint_as_float(v[4 * p + 1]), __uint_as_float(v[4 * p + 2]),
                                            __uint_as_float(v[4 * p + 3]));
                        __syncwarp();
                        const int p = lane & 7;
                        const int n = n0 + c0 + 4 * p;
#pragma unroll
                        for (int r4 = 0; r4 < 32; r4 += 4) {
                            const int rr = r4 + (lane >> 3);
                            if (rr < rows && n < a.negs)
                                *reinterpret_cast<float4*>(a.out + (row0 + rr) * a.negs + n) =
                                    *reinterpret_cast<const float4*>(sb + rr * 128 + ((p ^ (rr & 7)) << 4));
                        }
                    } else {
                        // lane = row: column q of the row goes to word q ^ row, so that writes (one column, 32 rows) and
                        // reads (one row, 32 columns) both touch 32 banks
#pragma unroll
                        for (int q = 0; q < 32; ++q) st[lane * 32 + (q ^ lane)] = __uint_as_float(v[q]);
                        __syncwarp();
                        const int n = n0 + c0 + lane;
                        if (n < a.negs)
                            for (int rr = 0; rr < rows; ++rr) a.out[(row0 + rr) * a.negs + n] = st[rr * 32 + (lane ^ rr)];
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    } else if (warp == kTcCopyWarp) {
        // ---------------- operand images of the negatives: one bulk copy per slice ----------------
        if (lane == 0) {
            bool ok = true;
            const uint8_t* images = ta.b_images + (size_t)c * n_blocks * b_buf_bytes;
            int issued = 0;
            for (int j = 0; j < n_blocks && ok; ++j) {
                const int buf = j & 1;
                if (j >= 2 && !mbar_wait(&b_empty[buf], ((j >> 1) - 1) & 1)) { atomicExch(ta.error, 22u); ok = false; break; }
                mbar_expect_tx(&b_full[buf], (uint32_t)b_buf_bytes);
                for (int sl = 0; sl < ta.n_slices; ++sl)
                    bulk_load(b_smem + (size_t)buf * b_buf_bytes + (size_t)sl * b_slice_bytes,
                              images + (size_t)j * b_buf_bytes + (size_t)sl * b_slice_bytes, (uint32_t)b_slice_bytes, &b_full[buf]);
                issued = j + 1;
            }
            // nothing of this CTA's may be in flight when it ends: the last copy into each buffer has landed
            for (int j = max(0, issued - 2); j < issued; ++j)
                if (!mbar_wait(&b_full[j & 1], (j >> 1) & 1)) atomicExch(ta.error, 26u);
        }
        __syncwarp();
    } else if (warp == kTcMmaWarp) {
        // ---------------- MMA issue ----------------
        if (lane == 0) {
            bool ok = mbar_wait(&a_full, 0);
            if (!ok) atomicExch(ta.error, 23u);
            for (int j = 0; j < n_blocks && ok; ++j) {
                const int buf = j & 1;
                const int n0 = j * ta.bn_max;
                const int bn = min(ta.bn_max, (a.negs - n0 + 15) / 16 * 16);
                if (!mbar_wait(&b_full[buf], (j >> 1) & 1)) { atomicExch(ta.error, 24u); ok = false; break; }
                if (j >= 2 && !mbar_wait(&acc_empty[buf], ((j >> 1) - 1) & 1)) { atomicExch(ta.error, 25u); ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
                const uint8_t* bb = b_smem + (size_t)buf * b_buf_bytes;
                for (int sl = 0; sl < ta.n_slices; ++sl) {
                    const uint64_t da = smem_desc_sw128(smem_u32(a_smem + (size_t)sl * 16384));
                    const uint64_t db = smem_desc_sw128(smem_u32(bb + (size_t)sl * b_slice_bytes));
                    const int k_steps = min(4, (a.dim - 32 * sl + 7) / 8);   // columns past dim are zero: skipped
                    for (int kk = 0; kk < k_steps; ++kk)
                        mma_tf32(tmem_base + buf * acc_stride, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (sl | kk) ? 1u : 0u);
                }
                mma_commit(&b_empty[buf]);
                mma_commit(&acc_full[buf]);
            }
        }
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kTcMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)ta.tmem_cols) : "memory");
    }
}

}  // namespace

extern "C" int mg_lp_free(mg_lp_batch* lp) {
    if (!lp) return MG_OK;
    cudaSetDevice(lp->device);
    mg_ctx* ctx = lp->ctx;
    // the block becomes the context's spare (the next mg_lp_prepare takes it) unless the spare is already larger
    if (ctx && lp->block && lp->block_bytes > ctx->lp_spare_bytes) {
        cudaFree(ctx->lp_spare);
        ctx->lp_spare = lp->block; ctx->lp_spare_bytes = lp->block_bytes;
    } else {
        cudaFree(lp->block);
    }
    delete lp;
    return MG_OK;
}

extern "C" int mg_lp_prepare(mg_ctx* ctx, const int32_t* src, const int32_t* rel, const int32_t* dst, int64_t n_edges,
                             int32_t n_chunks, int32_t negs, uint64_t seed, mg_lp_batch** out) {
    if (!ctx) return MG_ERR_ARG;
    if (!out || !src || !rel || !dst) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (n_edges <= 0 || n_chunks <= 0 || negs < 0 || n_chunks > n_edges) return mg_fail(ctx, MG_ERR_ARG, "need n_edges >= n_chunks >= 1 and negs >= 0");
    if (!ctx->row_off) return mg_fail(ctx, MG_ERR_STATE, "no graph loaded");
    if (ctx->n_resident_nodes <= 0) return mg_fail(ctx, MG_ERR_STATE, "no resident partition");
    const int64_t total = 2 * n_edges + (int64_t)n_chunks * negs;
    if (total >= (1ll << 31)) return mg_fail(ctx, MG_ERR_ARG, "batch too large");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->stream;
    mg_lp_batch* lp = new mg_lp_batch();
    lp->ctx = ctx; lp->device = ctx->device; lp->n_edges = n_edges; lp->n_chunks = n_chunks; lp->negs = negs;

    const size_t n_neg = (size_t)std::max<int64_t>((int64_t)n_chunks * negs, 1);
    const int64_t n_words = (ctx->n_nodes + 31) / 32;
    const int64_t n_groups = (n_words + kLpGroup - 1) / kLpGroup;
    const size_t scan_elems = mg_scan_tmp_elems(n_groups);
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    // scratch: one block of the context that only grows
    const size_t ws_bytes = 2 * up(4 * (size_t)n_edges) + up(4 * (size_t)n_words) + up(4 * (size_t)n_groups) + up(4 * scan_elems) + 3 * 256;
    if (ctx->lp_ws_bytes < ws_bytes) {
        cudaFree(ctx->lp_ws);
        ctx->lp_ws = nullptr; ctx->lp_ws_bytes = 0;
        if (cudaMalloc((void**)&ctx->lp_ws, ws_bytes + ws_bytes / 4) != cudaSuccess) {
            cudaGetLastError(); delete lp;
            return mg_fail(ctx, MG_ERR_OOM, "allocation of the link-prediction scratch failed");
        }
        ctx->lp_ws_bytes = ws_bytes + ws_bytes / 4;
    }
    char* w = ctx->lp_ws;
    auto take = [&](size_t b) { char* p = w; w += up(b); return p; };
    int32_t* d_src = (int32_t*)take(4 * (size_t)n_edges);
    int32_t* d_dst = (int32_t*)take(4 * (size_t)n_edges);
    uint32_t* bitmap = (uint32_t*)take(4 * (size_t)n_words);
    uint32_t* prefix = (uint32_t*)take(4 * (size_t)n_groups);
    uint32_t* scan_tmp = (uint32_t*)take(4 * scan_elems);
    uint32_t* d_status = (uint32_t*)take(4);
    int32_t* d_nt = (int32_t*)take(4);
    if (!ctx->lp_words) {
        if (cudaHostAlloc((void**)&ctx->lp_words, 2 * sizeof(int32_t), cudaHostAllocMapped) != cudaSuccess ||
            cudaHostGetDevicePointer((void**)&ctx->lp_words_dev, ctx->lp_words, 0) != cudaSuccess ||
            cudaMalloc((void**)&ctx->lp_range, 2 * sizeof(int32_t)) != cudaSuccess) {
            cudaGetLastError(); delete lp;
            return mg_fail(ctx, MG_ERR_OOM, "allocation of the link-prediction scratch failed");
        }
    }
    if (ctx->lp_range_words != n_words) {   // (once per graph)
        const int32_t h_range[2] = {0, (int32_t)n_groups};
        if (cudaMemcpy(ctx->lp_range, h_range, sizeof(h_range), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaGetLastError(); delete lp;
            return mg_fail(ctx, MG_ERR_CUDA, "copy failed");
        }
        ctx->lp_range_words = n_words;
    }
    const int32_t* d_range = ctx->lp_range;
    // results: one block, taken from the context's spare when that is large enough
    const size_t blk_bytes = up(4 * (size_t)total) + 3 * up(4 * (size_t)n_edges) + 2 * up(4 * n_neg);
    if (ctx->lp_spare && ctx->lp_spare_bytes >= blk_bytes) {
        lp->block = ctx->lp_spare; lp->block_bytes = ctx->lp_spare_bytes;
        ctx->lp_spare = nullptr; ctx->lp_spare_bytes = 0;
    } else if (cudaMalloc((void**)&lp->block, blk_bytes) != cudaSuccess) {
        cudaGetLastError(); delete lp;
        return mg_fail(ctx, MG_ERR_OOM, "allocation of the link-prediction batch failed");
    } else {
        lp->block_bytes = blk_bytes;
    }
    w = lp->block;
    lp->targets = (int32_t*)take(4 * (size_t)total);
    lp->src_idx = (int32_t*)take(4 * (size_t)n_edges);
    lp->dst_idx = (int32_t*)take(4 * (size_t)n_edges);
    lp->rel = (int32_t*)take(4 * (size_t)n_edges);
    lp->neg_ids = (int32_t*)take(4 * n_neg);
    lp->neg_idx = (int32_t*)take(4 * n_neg);
    auto cleanup = [&]() {};

    cudaMemcpyAsync(d_src, src, 4 * n_edges, cudaMemcpyHostToDevice, st);
    cudaMemcpyAsync(d_dst, dst, 4 * n_edges, cudaMemcpyHostToDevice, st);
    cudaMemcpyAsync(lp->rel, rel, 4 * n_edges, cudaMemcpyHostToDevice, st);
    cudaMemsetAsync(d_status, 0, 4, st);
    cudaMemsetAsync(bitmap, 0, 4 * (size_t)n_words, st);
    const int grid = mg_grid(ctx, 4);
    k_lp_mark<<<grid, kThreads, 0, st>>>(d_src, d_dst, n_edges, n_chunks, negs, seed, ctx->d_res_prefix, ctx->n_parts,
                                         ctx->n_resident_nodes, ctx->n_nodes, mg_feat_geom(ctx), ctx->d_part_start, ctx->d_nodes_by_part,
                                         lp->neg_ids, bitmap, d_status);
    k_lp_popc<<<grid, kThreads, 0, st>>>(bitmap, (int32_t)n_words, (int32_t)n_groups, prefix);
    mg_scan_u32(ctx, prefix, d_range, d_range + 1, nullptr, scan_tmp, reinterpret_cast<uint32_t*>(d_nt));
    k_lp_emit<<<grid, kThreads, 0, st>>>(bitmap, prefix, (int32_t)n_words, (int32_t)n_groups, lp->targets);
    k_lp_index<<<grid, kThreads, 0, st>>>(d_src, d_dst, lp->neg_ids, n_edges, total, ctx->n_nodes, bitmap, prefix, lp->src_idx,
                                          lp->dst_idx, lp->neg_idx, d_status, d_nt, ctx->lp_words_dev);
    ctx->launches += 4;
    cudaError_t e = cudaStreamSynchronize(st);
    const uint32_t h_status = e == cudaSuccess ? (uint32_t)ctx->lp_words[0] : 0u;
    lp->n_targets = e == cudaSuccess ? ctx->lp_words[1] : 0;
    if (e == cudaSuccess) e = cudaGetLastError();
    cleanup();
    if (e != cudaSuccess) { mg_lp_free(lp); return mg_cuda_fail(ctx, e, "mg_lp_prepare"); }
    if (h_status & ST_RANGE) { mg_lp_free(lp); return mg_fail(ctx, MG_ERR_ARG, "an edge endpoint is outside [0, n_nodes)"); }
    if (h_status & ST_NONRESIDENT) { mg_lp_free(lp); return mg_fail(ctx, MG_ERR_NONRESIDENT, "an edge endpoint lies in a partition that is not resident"); }
    *out = lp;
    return MG_OK;
}

extern "C" int mg_lp_view(const mg_lp_batch* lp, int32_t* n_targets, const int32_t** targets, const int32_t** src_idx,
                          const int32_t** dst_idx, const int32_t** neg_ids, const int32_t** neg_idx) {
    if (!lp) return MG_ERR_ARG;
    if (n_targets) *n_targets = lp->n_targets;
    if (targets) *targets = lp->targets;
    if (src_idx) *src_idx = lp->src_idx;
    if (dst_idx) *dst_idx = lp->dst_idx;
    if (neg_ids) *neg_ids = lp->neg_ids;
    if (neg_idx) *neg_idx = lp->neg_idx;
    return MG_OK;
}

extern "C" int mg_distmult_score(mg_ctx* ctx, const mg_lp_batch* lp, const float* h_dev, int32_t dim, const float* rel_emb_dev,
                                 int32_t n_relations, int corrupt, int gemm_precision, float* pos_out, float* neg_dst_out, float* neg_src_out) {
    if (!ctx) return MG_ERR_ARG;
    if (!lp || !h_dev || !rel_emb_dev || !pos_out) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (dim <= 0 || n_relations <= 0) return mg_fail(ctx, MG_ERR_ARG, "dim and n_relations must be positive");
    if (gemm_precision != MG_GEMM_TF32 && gemm_precision != MG_GEMM_FP32) return mg_fail(ctx, MG_ERR_ARG, "unknown gemm precision");
    if ((corrupt & MG_CORRUPT_DST) && lp->negs > 0 && !neg_dst_out) return mg_fail(ctx, MG_ERR_ARG, "null neg_dst_out");
    if ((corrupt & MG_CORRUPT_SRC) && lp->negs > 0 && !neg_src_out) return mg_fail(ctx, MG_ERR_ARG, "null neg_src_out");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->stream;
    ProfScope ps(ctx, PH_DISTMULT, 3);
    k_distmult_pos<<<mg_grid(ctx, 8), kThreads, 0, st>>>(h_dev, rel_emb_dev, lp->src_idx, lp->dst_idx, lp->rel, lp->n_edges, dim, pos_out);
    ctx->launches++;
    if (lp->negs > 0) {
        const int64_t max_chunk = (lp->n_edges + lp->n_chunks - 1) / lp->n_chunks;
        NegArgs a;
        a.h = h_dev; a.rel_emb = rel_emb_dev; a.rel = lp->rel; a.neg_idx = lp->neg_idx; a.E = lp->n_edges;
        a.n_chunks = lp->n_chunks; a.negs = lp->negs; a.dim = dim;
        a.tiles_per_chunk = (int32_t)((max_chunk + 63) / 64);
        const bool tensor = gemm_precision == MG_GEMM_TF32 && dim % 4 == 0 && dim <= 32 * kTcMaxSlices;
        if (tensor) {
            NegTcArgs ta;
            ta.n_slices = (dim + 31) / 32;
            ta.bn_max = std::min(kTcBlockN, (lp->negs + 15) / 16 * 16);
            int cols = 32;
            while (cols < ta.bn_max) cols <<= 1;
            ta.tmem_cols = 2 * cols;   // two accumulator buffers
            ta.error = ctx->d_flags;
            a.tiles_per_chunk = (int32_t)((max_chunk + 127) / 128);
            // operand images of the negatives (context scratch, grow-only)
            const int n_blocks = (lp->negs + ta.bn_max - 1) / ta.bn_max;
            const size_t image_bytes = (size_t)lp->n_chunks * n_blocks * ta.n_slices * ta.bn_max * 128;
            if (ctx->dm_images_bytes < image_bytes) {
                cudaFree(ctx->dm_images);
                ctx->dm_images = nullptr; ctx->dm_images_bytes = 0;
                if (cudaMalloc((void**)&ctx->dm_images, image_bytes) != cudaSuccess) {
                    cudaGetLastError();
                    return mg_fail(ctx, MG_ERR_OOM, "device allocation of %zu bytes failed", image_bytes);
                }
                ctx->dm_images_bytes = image_bytes;
            }
            k_stage_negs<<<mg_grid(ctx, 8), kThreads, 0, st>>>(h_dev, lp->neg_idx, lp->n_chunks, lp->negs, dim, ta.n_slices, ta.bn_max,
                                                             (uint8_t*)ctx->dm_images);
            ctx->launches++;
            ta.b_images = (const uint8_t*)ctx->dm_images;
            const size_t smem = (size_t)ta.n_slices * 16384 + 2 * (size_t)ta.n_slices * ta.bn_max * 128 + 1024;
            MG_CUDA(ctx, cudaFuncSetAttribute(k_distmult_neg_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            const unsigned blocks = (unsigned)(a.tiles_per_chunk * lp->n_chunks);
            if (corrupt & MG_CORRUPT_DST) {
                a.keep_idx = lp->src_idx; a.out = neg_dst_out; ta.base = a;
                k_distmult_neg_tc<<<blocks, kTcThreads, smem, st>>>(ta);
                ctx->launches++;
            }
            if (corrupt & MG_CORRUPT_SRC) {
                a.keep_idx = lp->dst_idx; a.out = neg_src_out; ta.base = a;
                k_distmult_neg_tc<<<blocks, kTcThreads, smem, st>>>(ta);
                ctx->launches++;
            }
        } else {
        dim3 grid((unsigned)(a.tiles_per_chunk * lp->n_chunks), (unsigned)((lp->negs + 63) / 64));
        if (corrupt & MG_CORRUPT_DST) {
            a.keep_idx = lp->src_idx; a.out = neg_dst_out;
            k_distmult_neg<<<grid, 256, 0, st>>>(a);
            ctx->launches++;
        }
        if (corrupt & MG_CORRUPT_SRC) {
            a.keep_idx = lp->dst_idx; a.out = neg_src_out;
            k_distmult_neg<<<grid, 256, 0, st>>>(a);
            ctx->launches++;
        }
        }
    }
    MG_CUDA(ctx, cudaGetLastError());
    return MG_OK;
}
