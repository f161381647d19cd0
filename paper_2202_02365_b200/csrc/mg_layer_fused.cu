// One GraphSage layer over DENSE as a single persistent kernel (Algorithm 3 with the mean
// aggregator, fused with the layer's linear maps):
//
//     H^l[r] = act([ self_r | mean_r ] . [W_self ; W_nbr] + b)
//
// The [self | mean] operand never goes to global memory.  Producer warps gather the rows a tile of
// 128 output rows needs (layer 1: base representations straight from the partition buffer; later
// layers: rows of H^{l-1}), reduce each segment in entry order, round to TF32 and write 32-float
// K slices directly into 128-byte-swizzled shared-memory stages.  One thread issues tcgen05.mma
// kind::tf32 against weight slices that a TMA thread streams from L2 (no multicast); the fp32
// accumulator lives in tensor memory, double-buffered so that the epilogue of one tile (bias,
// ReLU, store) overlaps the gather and MMAs of the next.  Tiles are handed out round-robin in
// packed row order, so all SMs work on the same mini-batch at a time and its rows stay in L2.
// Every mbarrier wait is bounded; on a time-out the role records a code and stops.

#include <cuda_fp16.h>

#include <algorithm>
#include <cstdlib>

#include "mg_device.cuh"
#include "mg_internal.cuh"
#include "mg_tcgen05.cuh"

using namespace tc;

namespace {

constexpr int BM = 128;               // output rows per tile
constexpr int KC = 32;                // floats per K slice (one 128-byte swizzle row)
// Warp roles, laid out so that every role fills whole warpgroups (four consecutive warps):
//   warps 0..15   producers (gather + segment mean)         four warpgroups
//   warps 16..19  epilogue (tensor memory -> global)        one warpgroup
//   warp 20 TMA (weights), warp 21 MMA + tensor memory, warps 22..23 planners: one warpgroup
// Every thread has 80 registers (768 x 80 = 61,440 of the SM's 65,536).  A build option moves registers between the
// warpgroups with `setmaxnreg` (-DMG_FUSED_SETMAXNREG=1 -DMG_FUSED_MAXNREG=72 -DMG_REG_PROD=80 -DMG_REG_EPI=56
// -DMG_REG_CTL=56: the CTA then leaves room for a 256-thread block of the sampler beside it); it is off because every
// such configuration measured 15 % slower in the first layer than the plain one.
constexpr int kProducerWarps = 16;
constexpr int kFirstProducerWarp = 0;
constexpr int kFirstEpilogueWarp = 16;
constexpr int kTmaWarp = 20, kMmaWarp = 21;
constexpr int kPlannerWarps = 2;
constexpr int kFirstPlannerWarp = 22;
constexpr int kFusedThreads = (kFirstPlannerWarp + kPlannerWarps) * 32;  // 768
#ifndef MG_FUSED_MAXNREG
#define MG_FUSED_MAXNREG 80
#endif
#ifndef MG_FUSED_SETMAXNREG
#define MG_FUSED_SETMAXNREG 0
#endif
constexpr int kMaxStages = 8;
constexpr int kGroupCols = 128;                  // input columns whose (self, mean) slices the producers fill together (TF32 operands)
// With half-precision base representations the first layer can run its GEMM in kind::f16 (fp16 operands, fp32
// accumulate): a 128-byte slice row then holds 64 columns, a lane's 16 bytes are 8 columns, a group is 256 columns,
// and the same number of MMAs covers twice the K.  Everything else (slices per group, swizzle, stages, barriers) is
// the same, so the element-size dependent constants come from one place:
template <bool F16> struct Geo {
    static constexpr int kKC = F16 ? 64 : 32;        // columns per K slice (one 128-byte swizzle row)
    static constexpr int kLaneCols = F16 ? 8 : 4;    // columns of a group one lane owns (16 bytes of operand)
    static constexpr int kGroup = 32 * kLaneCols;    // columns per group
};
constexpr int kRowsInFlight = 2;                 // rows a producer warp builds at the same time
constexpr int kBlockRows = kProducerWarps * kRowsInFlight;   // 32: rows of a tile the producers build in one round
constexpr int kBlocksPerTile = BM / kBlockRows;              // 4
constexpr int kPlanSlots = kBlocksPerTile;                   // planned row blocks in shared memory (one tile's worth)
constexpr int HM = BM / 2;                                   // rows of a half tile: the unit the MMAs work on
constexpr int kBlocksPerHalf = kBlocksPerTile / 2;
constexpr int kAccBufs = 4;                                  // accumulator buffers in tensor memory (two tiles' halves)
constexpr int kSlicesPerGroup = 2 * kGroupCols / KC;         // 8 K slices: (self, mean) x four 32-column blocks
constexpr int kUnroll = 5;                       // neighbour rows per output row fetched before the first add
static_assert(kUnroll == 5, "the first-round table is read as four + one source rows");
constexpr uint32_t kABytes = BM * KC * 4;  // 16 KiB per A stage

struct FusedArgs {
    // DENSE (device arrays of the sample)
    int32_t B, k, layer;
    const int32_t* rowbase_out;  // [B+1] of layer l
    const int32_t* rowbase_in;   // [B+1] of layer l-1
    const int32_t* cum;          // [B][k+2]
    const int32_t* node_off;     // [k+1][B+1]
    const int32_t* nodes;
    const int32_t* ent_off;
    const int32_t* ent_nbrs;
    const int32_t* ent_repr;
    const int4* row_meta;        // [M] (self source row, first entry, entry count, first H^{l-1} row of the batch)
    // input rows
    const float* h_prev;         // layers >= 2: [rows of layer l-1, d_in]
    const char* src_base;        // layer 1: the feature buffer; later layers: h_prev
    uint32_t src_row_bytes;      // (32-bit: the row address is then one wide multiply-add)
    FeatGeom feat;               // layer 1: where a node's row lives in the partition buffer
    int32_t safe_src;            // a source row that is always valid to read (rows past the end load it)
    // shapes
    int32_t d_in, d_in_pad;      // d_in_pad = d_in rounded up to 32; K = 2 * d_in_pad
    int32_t N, BN;               // output width and its MMA tile width (multiple of 16, <= 256)
    int64_t row_lo;              // first packed output row this launch computes
    int64_t M;                   // one past its last packed output row
    int32_t sa, sb;              // A and B stages
    const void* w_rows;          // weights-in-tensor-memory form: the padded weight matrix [N][2 * d_in_pad] (fp32 or fp16), K order of the slices
    int32_t tmem_cols;
    int32_t relu;
    int32_t sum_aggr;            // neighbour term = sum of the sampled neighbours instead of their mean
    int32_t out_f16;             // the output rows are stored as fp16 (an intermediate layer of a model that keeps them so)
    const float* bias;
    float* out;                  // [M, N]
    uint32_t* error;
};

constexpr int kTsMaxEntriesPerRow = 8;   // layers with more entries per output row than this stream their weights
constexpr int kLaneEntries = 32;   // rows up to this long are translated by their own lane of the planner warp
constexpr int kKeyCap = 704;    // source-row indices of a row block's entries cached in shared memory (22 per row: what still fits the 196 KB carve-out)

// What a producer needs to build one output row: x = source row of the row's own representation; y = first
// entry and z = number of entries in the sample's entry arrays (z < 0: row past the end); w = first cached
// source-row index of the row when the block's entries fit the cache, else (layers >= 2) the first row of the
// mini-batch in H^{l-1}.
typedef int4 RowMeta;

// Source row of an entry.  Layer 1: the feature-buffer row of node `key` (its partition's slot);
// later layers: row of H^{l-1}.  The address is src_base + row * src_row_bytes.
template <bool FIRST>
__device__ __forceinline__ int32_t source_row(const FusedArgs& a, int32_t in_base, int32_t key) {
    if (FIRST) return (int32_t)feat_row(a.feat, key);
    return in_base + key;
}

// A lane's piece of a source row, as 16 bytes of registers: four fp32 values (fp16 sources widened exactly), or,
// for fp16 operands (F16), eight fp16 values as they are in memory.
template <bool HALF, bool F16>
__device__ __forceinline__ uint4 load_piece(const char* p) {
    if (F16) return __ldg(reinterpret_cast<const uint4*>(p));
    if (HALF) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(p));
        const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        return make_uint4(__float_as_uint(lo.x), __float_as_uint(lo.y), __float_as_uint(hi.x), __float_as_uint(hi.y));
    }
    return __ldg(reinterpret_cast<const uint4*>(p));
}

// fp32 running sum of a lane's piece over a row's entries, and the operand forms of the result and of the self row
template <bool F16> struct PieceSum;
template <> struct PieceSum<false> {
    float a[4];
    __device__ __forceinline__ void zero() { a[0] = a[1] = a[2] = a[3] = 0.f; }
    __device__ __forceinline__ void add(const uint4& r) {
        a[0] += __uint_as_float(r.x); a[1] += __uint_as_float(r.y); a[2] += __uint_as_float(r.z); a[3] += __uint_as_float(r.w);
    }
    __device__ __forceinline__ uint4 operand(float scale) const {   // rounded to nearest TF32
        return make_uint4(__float_as_uint(to_tf32(a[0] * scale)), __float_as_uint(to_tf32(a[1] * scale)),
                          __float_as_uint(to_tf32(a[2] * scale)), __float_as_uint(to_tf32(a[3] * scale)));
    }
    static __device__ __forceinline__ uint4 self_operand(const uint4& r) {
        return make_uint4(__float_as_uint(to_tf32(__uint_as_float(r.x))), __float_as_uint(to_tf32(__uint_as_float(r.y))),
                          __float_as_uint(to_tf32(__uint_as_float(r.z))), __float_as_uint(to_tf32(__uint_as_float(r.w))));
    }
};
template <> struct PieceSum<true> {
    float a[8];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = 0.f;
    }
    __device__ __forceinline__ void add(const uint4& r) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            a[2 * i] += f.x; a[2 * i + 1] += f.y;
        }
    }
    __device__ __forceinline__ uint4 operand(float scale) const {   // rounded to nearest fp16 (the 10-bit mantissa TF32 keeps)
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __half2 h = __floats2half2_rn(a[2 * i] * scale, a[2 * i + 1] * scale);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    static __device__ __forceinline__ uint4 self_operand(const uint4& r) { return r; }   // fp16 rows are operands as they are
};

// TS: the weights stay in tensor memory for the whole kernel and are the MMAs' first operand (M = 256 output columns over
// the pair, a CTA's 128 in its 128 lanes, K <= 256 columns), the gathered rows the second (N = 128: a half tile of either
// CTA); the accumulator is the transposed output, [output column][row].  Nothing is streamed per half tile then -- with
// the weights in shared memory a half tile waits for eight 16 KB slices through a two-stage ring (4 us of latency).
template <bool FIRST, bool HALF, bool F16, bool TS = false>
__global__ void __cluster_dims__(2, 1, 1) __maxnreg__(MG_FUSED_MAXNREG)
k_sage_layer_fused(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_out, FusedArgs a) {
    constexpr int KCE = Geo<F16>::kKC, GC = Geo<F16>::kGroup, LC = Geo<F16>::kLaneCols;
    extern __shared__ uint8_t smem_raw[];
    // a_ready and acc_empty are used in the leader CTA only (both CTAs arrive there); a_free, b_empty and acc_full
    // exist in both CTAs and are signalled in both by the leader's commits; b_full counts both halves' bytes in
    // the leader.
    __shared__ uint64_t a_ready[2], a_free[2], b_full[kMaxStages], b_empty[kMaxStages];   // a_*: one per half tile
    __shared__ uint64_t acc_full[kAccBufs], acc_empty[kAccBufs];
    __shared__ uint64_t w_ready;   // TS, leader only: both CTAs' weights are in tensor memory
    __shared__ uint32_t tmem_slot;
    __shared__ uint64_t plan_full[kPlanSlots], plan_empty[kPlanSlots];
    __shared__ RowMeta meta[kPlanSlots][kBlockRows];
    __shared__ int32_t src_rows[kPlanSlots][kKeyCap];
    __shared__ int32_t plan_total[kPlanSlots];   // entries of the block, or -1 when they do not fit the cache
    // source rows of each row's first kUnroll entries, padded with the row's own source row: the first round of
    // gathers then needs no selects
    __shared__ __align__(16) int32_t first_rows[kPlanSlots][kBlockRows][8];
    __shared__ __align__(1024) float out_stage[4][32 * 32];   // per epilogue warp: one 32 x 32 slice, 128-byte swizzled, for the TMA store

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();      // 0: leader of the pair (issues the MMAs), 1: its peer
    const bool leader = rank == 0;
    const uint32_t pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int half_n = a.BN / 2;                  // weight rows (output columns) this CTA stages
    const uint32_t b_bytes = (uint32_t)half_n * 128;   // one 128-byte slice row per staged output column
    uint8_t* a_base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* b_base = a_base + (size_t)a.sa * kABytes;
    const int n_chunks = 2 * a.d_in_pad / KCE;
    const int64_t n_tiles = (a.M - a.row_lo + BM - 1) / BM;
    const int64_t n_tile_pairs = (n_tiles + 1) / 2;
    // iteration `it` of this pair works on tile pair (pair + it * n_pairs): the leader on its even tile, the peer
    // on the odd one (which may lie past the end: then all its rows are padding)
    const uint32_t my_iters = pair < n_tile_pairs ? (uint32_t)((n_tile_pairs - pair + n_pairs - 1) / n_pairs) : 0u;
    auto tile_of = [&](uint32_t it) -> int64_t { return 2 * ((int64_t)pair + (int64_t)it * n_pairs) + rank; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(&a_ready[s], 2 * kProducerWarps); mbar_init(&a_free[s], 1); }
        for (int s = 0; s < a.sb; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); }
        for (int s = 0; s < kAccBufs; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 2 * 4); }
        mbar_init(&w_ready, 2 * 4);   // the four loading warps of both CTAs
        for (int s = 0; s < kPlanSlots; ++s) { mbar_init(&plan_full[s], 1); mbar_init(&plan_empty[s], kProducerWarps); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_out) : "memory");
    }
    if (warp == kMmaWarp) {
        // the same warp of both CTAs allocates the pair's tensor memory
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();       // barriers of both CTAs are initialised before anyone arrives on a remote one
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t acc_stride = (uint32_t)(a.tmem_cols / kAccBufs);  // columns per accumulator buffer (a multiple of 32)
    constexpr uint32_t kTsAcc0 = 256, kTsAccCols = 128;              // TS: weights in columns [0, 256), two accumulators behind them
    if constexpr (TS) {
        if (warp >= kFirstEpilogueWarp && warp < kTmaWarp) {   // (the warps that may touch lanes 32 q .. 32 q + 31)
            const int q = warp & 3;
            const int n = (int)rank * 128 + q * 32 + lane;     // this lane's output column = its row of the weights
            const int K = F16 ? a.d_in_pad : 2 * a.d_in_pad;   // 32-bit words per row of the weights (two fp16 values per word)
            const float4* wrow = reinterpret_cast<const float4*>(static_cast<const uint32_t*>(a.w_rows) + (size_t)min(n, a.N - 1) * K);
            for (int k0 = 0; k0 < K; k0 += 32) {
                uint32_t v[32];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float4 x = n < a.N ? __ldg(wrow + k0 / 4 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
                    v[4 * j] = __float_as_uint(x.x); v[4 * j + 1] = __float_as_uint(x.y);
                    v[4 * j + 2] = __float_as_uint(x.z); v[4 * j + 3] = __float_as_uint(x.w);
                }
                tmem_st_32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)k0, v);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            // only the leader's MMA thread waits for the weights: planners and gather warps start at once
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (leader) mbar_arrive(&w_ready);
                else mbar_arrive_cluster(mapa_u32(smem_u32(&w_ready), 0));
            }
        }
    }
    const int n_groups = (a.d_in_pad + GC - 1) / GC;

    // (Build option) registers move from the epilogue's and the control warpgroup to the producers': each warpgroup
    // executes its one setmaxnreg at the head of its own branch, so that the compiler budgets the branch with it (the
    // decreases never wait, the increases wait for them; the static_assert keeps the sum within the launch allocation).
#define MG_STR2(x) #x
#define MG_STR(x) MG_STR2(x)
#if MG_FUSED_SETMAXNREG
#define MG_REG_SET(n) do { if ((n) < MG_FUSED_MAXNREG) asm volatile("setmaxnreg.dec.sync.aligned.u32 " MG_STR(n) ";" ::: "memory"); \
                           else if ((n) > MG_FUSED_MAXNREG) asm volatile("setmaxnreg.inc.sync.aligned.u32 " MG_STR(n) ";" ::: "memory"); } while (0)
#else
#define MG_REG_SET(n)
#endif
#ifndef MG_REG_PROD
#define MG_REG_PROD 80
#define MG_REG_EPI 56
#define MG_REG_CTL 56
#endif
    static_assert(MG_FUSED_SETMAXNREG == 0 || 16 * MG_REG_PROD + 4 * MG_REG_EPI + 4 * MG_REG_CTL <= 24 * MG_FUSED_MAXNREG,
                  "the warpgroups' registers must fit what the CTA was launched with");
    if (warp >= kTmaWarp) {
    MG_REG_SET(MG_REG_CTL);
    if (warp == kTmaWarp && !TS) {
        // ---------------- weight slices: each CTA stages its half of the output columns (TMA from L2) ----------------
        if (lane == 0) {
            uint32_t cnt = 0;
            bool ok = true;
            // the weight slices of a group are streamed once per half tile, in the order the MMAs consume them
            for (uint32_t it = 0; it < my_iters && ok; ++it)
                for (int grp = 0; grp < n_groups && ok; ++grp)
                    for (int h = 0; h < 2 && ok; ++h) {
                        const int gch = min(kSlicesPerGroup, n_chunks - grp * kSlicesPerGroup);
                        for (int c = 0; c < gch; ++c, ++cnt) {
                            const int s = cnt % a.sb;
                            if (cnt >= (uint32_t)a.sb && !mbar_wait(&b_empty[s], ((cnt / a.sb) - 1) & 1)) { atomicExch(a.error, 11u); ok = false; break; }
                            if (leader) mbar_expect_tx(&b_full[s], 2 * b_bytes);   // both halves are counted on the leader's barrier
                            tma_load_2d_pair(b_base + (size_t)s * b_bytes, &map_w, mapa_u32(smem_u32(&b_full[s]), 0),
                                             (grp * kSlicesPerGroup + c) * KCE, (int)rank * half_n);
                        }
                    }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ---------------- MMA issue: one thread of the leader, for both CTAs ----------------
        if (TS && lane == 0 && leader) {
            // M = 256 output columns over the pair, N = 128 rows (a half tile of each CTA), fp32 accumulate, K-major
            const uint32_t idesc = (1u << 4) | ((F16 ? 0u : 2u) << 7) | ((F16 ? 0u : 2u) << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
            bool ok = mbar_wait(&w_ready, 0);
            if (!ok) atomicExch(a.error, 18u);
            tc_fence_after();
            for (uint32_t it = 0; it < my_iters && ok; ++it)
                for (int h = 0; h < 2 && ok; ++h) {
                    const uint32_t hu = it * 2 + h, buf = hu & 1;
                    if (hu >= 2 && !mbar_wait(&acc_empty[buf], ((hu >> 1) - 1) & 1)) { atomicExch(a.error, 12u); ok = false; break; }
                    tc_fence_after();
                    if (!mbar_wait(&a_ready[h], it & 1)) { atomicExch(a.error, 13u); ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + kTsAcc0 + buf * kTsAccCols;
                    for (int c = 0; c < n_chunks; ++c) {
                        const uint64_t db = smem_desc_sw128(smem_u32(a_base + (size_t)c * kABytes + (size_t)h * (HM * 128)));
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {   // 32 bytes of every slice row = 8 columns of the weights per instruction
                            if (F16) mma_f16_pair_ts(d_tmem, tmem_base + (uint32_t)(c * 32 + kk * 8), db + (uint64_t)(kk * 2), idesc, (c | kk) ? 1u : 0u);
                            else mma_tf32_pair_ts(d_tmem, tmem_base + (uint32_t)(c * 32 + kk * 8), db + (uint64_t)(kk * 2), idesc, (c | kk) ? 1u : 0u);
                        }
                    }
                    mma_commit_pair(&a_free[h]);
                    mma_commit_pair(&acc_full[buf]);
                }
        }
        if (!TS && lane == 0 && leader) {
            // M = 128 over the pair: 64 rows (a half tile) of each CTA per instruction
            // fp32 accumulate; operands TF32 (format 2) or fp16 (format 0), both K-major
            const uint32_t idesc = (1u << 4) | ((F16 ? 0u : 2u) << 7) | ((F16 ? 0u : 2u) << 10) | ((uint32_t)(a.BN >> 3) << 17) |
                                   ((uint32_t)((2 * HM) >> 4) << 24);
            uint32_t cnt = 0;
            bool ok = true;
            for (uint32_t it = 0; it < my_iters && ok; ++it)
                for (int grp = 0; grp < n_groups && ok; ++grp)
                    for (int h = 0; h < 2 && ok; ++h) {
                        const uint32_t hu = it * 2 + h;                       // half tiles of this CTA, in order
                        const uint32_t buf = hu % kAccBufs;
                        const uint32_t s_h = it * (uint32_t)n_groups + grp;   // fills of half h's stage rows so far
                        if (grp == 0) {
                            if (hu >= (uint32_t)kAccBufs && !mbar_wait(&acc_empty[buf], ((hu / kAccBufs) - 1) & 1)) { atomicExch(a.error, 12u); ok = false; break; }
                            tc_fence_after();
                        }
                        // both CTAs' producers have filled the half's rows of this group's K slices
                        if (!mbar_wait(&a_ready[h], s_h & 1)) { atomicExch(a.error, 13u); ok = false; break; }
                        const uint32_t d_tmem = tmem_base + buf * acc_stride;
                        const int gch = min(kSlicesPerGroup, n_chunks - grp * kSlicesPerGroup);
                        for (int c = 0; c < gch; ++c, ++cnt) {
                            const int sb = cnt % a.sb;
                            if (!mbar_wait(&b_full[sb], (cnt / a.sb) & 1)) { atomicExch(a.error, 13u); ok = false; break; }
                            tc_fence_after();
                            const uint64_t da = smem_desc_sw128(smem_u32(a_base + (size_t)c * kABytes + (size_t)h * (HM * 128)));
                            const uint64_t db = smem_desc_sw128(smem_u32(b_base + (size_t)sb * b_bytes));
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) {   // 32 bytes of every slice row per instruction: K = 8 (TF32) or 16 (fp16)
                                if (F16) mma_f16_pair(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (grp | c | kk) ? 1u : 0u);
                                else mma_tf32_pair(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (grp | c | kk) ? 1u : 0u);
                            }
                            mma_commit_pair(&b_empty[sb]);
                        }
                        if (!ok) break;
                        mma_commit_pair(&a_free[h]);    // one commit frees the half's rows of all the group's stages
                        if (grp == n_groups - 1) mma_commit_pair(&acc_full[buf]);
                    }
        }
        __syncwarp();
    } else {
        // ---------------- planners: row blocks of 32 rows, prepared ahead of the producers ----------------
        // A planner warp takes every kPlannerWarps-th row block: lane = row.  It reads the rows' metadata, scans the
        // entry counts, and translates the block's entries to source rows in shared memory, so that the producers'
        // gathers depend on nothing but shared memory.
        // (with the weights in tensor memory nothing is streamed and the weight warp is a third planner)
        constexpr int kPlanners = TS ? kPlannerWarps + 1 : kPlannerWarps;
        const int plw = warp == kTmaWarp ? kPlannerWarps : warp - kFirstPlannerWarp;
        const int32_t* keys = FIRST ? a.ent_nbrs : a.ent_repr;
        bool ok = true;
        for (uint32_t q = plw; ok; q += kPlanners) {
            if (q / kBlocksPerTile >= my_iters) break;
            const int64_t t = tile_of(q / kBlocksPerTile);   // past the end for the peer of an odd last tile: all padding
            const int slot = q % kPlanSlots;
            if (q >= (uint32_t)kPlanSlots && !mbar_wait(&plan_empty[slot], ((q / kPlanSlots) - 1) & 1)) {
                if (lane == 0) atomicExch(a.error, 17u);
                ok = false;
            }
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            const int64_t r = a.row_lo + t * BM + (q % kBlocksPerTile) * kBlockRows + lane;
            int4 rm = make_int4(a.safe_src, 0, -1, 0);
            if (r < a.M) rm = __ldg(a.row_meta + r);   // (self source row, first entry, count, first H^{l-1} row of the batch)
            const int32_t end = (int32_t)warp_incl_scan((uint32_t)max(rm.z, 0));   // end of the row's cached entries
            const int32_t total = __shfl_sync(0xFFFFFFFFu, end, 31);
            const bool cached = total <= kKeyCap;
            const int32_t in_base = rm.w, koff = end - max(rm.z, 0);
            meta[slot][lane] = make_int4(rm.x, rm.y, rm.z, cached ? koff : in_base);
            const int32_t zmax = (int32_t)__reduce_max_sync(0xFFFFFFFFu, (uint32_t)max(rm.z, 0));
            if (cached && zmax <= kLaneEntries) {
                // short rows (the usual case): every lane translates its own row's entries, kUnroll loads in flight
                // (the entries of consecutive rows are consecutive, so the lanes' loads share their cache lines)
                for (int32_t i0 = 0; i0 < zmax; i0 += kUnroll) {
                    int32_t key[kUnroll];
#pragma unroll
                    for (int u = 0; u < kUnroll; ++u) key[u] = i0 + u < rm.z ? __ldg(keys + rm.y + i0 + u) : 0;
#pragma unroll
                    for (int u = 0; u < kUnroll; ++u)
                        if (i0 + u < rm.z) src_rows[slot][koff + i0 + u] = source_row<FIRST>(a, in_base, key[u]);
                }
            } else if (cached) {
                // entry j belongs to the first row whose end exceeds j
                for (int32_t j0 = 0; j0 < total; j0 += 32 * 4) {
                    int32_t key[4], base[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int32_t j = j0 + u * 32 + lane;
                        int lo = 0, hi = 31;
#pragma unroll
                        for (int s = 0; s < 5; ++s) {
                            const int mid = (lo + hi) >> 1;
                            const int32_t e = __shfl_sync(0xFFFFFFFFu, end, mid);
                            if (lo < hi) { if (e > j) hi = mid; else lo = mid + 1; }
                        }
                        const int32_t e0 = __shfl_sync(0xFFFFFFFFu, rm.y, lo), k0 = __shfl_sync(0xFFFFFFFFu, koff, lo);
                        base[u] = __shfl_sync(0xFFFFFFFFu, in_base, lo);
                        key[u] = j < total ? __ldg(keys + e0 + (j - k0)) : 0;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int32_t j = j0 + u * 32 + lane;
                        if (j < total) src_rows[slot][j] = source_row<FIRST>(a, base[u], key[u]);
                    }
                }
            }
            if (lane == 0) plan_total[slot] = cached ? total : -1;
            __syncwarp();
            if (cached) {
                // lane = row: its first kUnroll source rows, padded with its own source row
                int32_t fr[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) fr[j] = (j < kUnroll && j < rm.z) ? src_rows[slot][koff + j] : rm.x;
                fr[5] = __float_as_int(rm.z > 0 ? (a.sum_aggr ? 1.f : 1.f / (float)rm.z) : 0.f);   // the mean's factor (1 for a sum)
                *reinterpret_cast<int4*>(&first_rows[slot][lane][0]) = make_int4(fr[0], fr[1], fr[2], fr[3]);
                *reinterpret_cast<int4*>(&first_rows[slot][lane][4]) = make_int4(fr[4], fr[5], fr[6], fr[7]);
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(&plan_full[slot]);
        }
    }
    } else if (warp >= kFirstEpilogueWarp) {
    MG_REG_SET(MG_REG_EPI);
    {
        // ---------------- epilogue: tensor memory -> bias, ReLU -> global ----------------
        // A half tile's accumulator: rows 0..63 of output columns [0, BN/2) in lanes 0..63, the same rows of columns
        // [BN/2, BN) in lanes 64..127.  Warp quadrant q reads lanes 32q..32q+31.
        const int lane_group = warp & 3;
        const int col_base = (lane_group >> 1) * half_n;
        const int n_cols = half_n;
        bool ok = true;
        if constexpr (TS) {
            // The accumulator of a half-tile pair: lane = output column (this CTA's 128), column j = row j of the
            // leader's half tile (j < 64) or row j - 64 of the peer's.  A warp turns 32 x 32 pieces round through its
            // staging tile (lane = column of the box, 128-byte swizzle) and stores them with TMA.
            const int n0 = (int)rank * 128 + lane_group * 32;
            const float bias_n = n0 + lane < a.N ? __ldg(a.bias + n0 + lane) : 0.f;
            uint8_t* stage = reinterpret_cast<uint8_t*>(out_stage[lane_group]);
            for (uint32_t hu = 0; hu < 2 * my_iters && ok; ++hu) {
                const uint32_t buf = hu & 1;
                if (!mbar_wait(&acc_full[buf], (hu >> 1) & 1)) { if (lane == 0) atomicExch(a.error, 14u); ok = false; break; }
                tc_fence_after();
                for (int g = 0; g < 4; ++g) {
                    uint32_t v[32];
                    tmem_ld_32(tmem_base + kTsAcc0 + buf * kTsAccCols + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)(g * 32), v);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    const int64_t t = 2 * ((int64_t)pair + (int64_t)(hu >> 1) * n_pairs) + (g >> 1);   // the tile of CTA g / 2
                    const int64_t row0 = a.row_lo + t * BM + (hu & 1) * HM + (g & 1) * 32;
                    if (row0 >= a.M || n0 >= a.N) continue;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the previous box has left the tile
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float o = __uint_as_float(v[j]) + bias_n;
                        if (a.relu) o = fmaxf(o, 0.f);
                        if (a.out_f16) *reinterpret_cast<__half*>(stage + j * 64 + lane * 2) = __float2half_rn(o);   // (boxes of 32 fp16 columns, not swizzled)
                        else *reinterpret_cast<float*>(stage + j * 128 + (((lane >> 2) ^ (j & 7)) << 4) + ((lane & 3) << 2)) = o;
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        // rows past the end of the layer and columns past its width are clipped by the tensor map
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                     ::"l"(&map_out), "r"(smem_u32(stage)), "r"(n0), "r"((int)row0) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (leader) mbar_arrive(&acc_empty[buf]);
                    else mbar_arrive_cluster(mapa_u32(smem_u32(&acc_empty[buf]), 0));
                }
            }
        }
        for (uint32_t hu = 0; !TS && hu < 2 * my_iters && ok; ++hu) {
            const int64_t t = tile_of(hu >> 1);
            const uint32_t buf = hu % kAccBufs;
            if (!mbar_wait(&acc_full[buf], (hu / kAccBufs) & 1)) { if (lane == 0) atomicExch(a.error, 14u); ok = false; break; }
            tc_fence_after();
            const int64_t row0 = a.row_lo + t * BM + (hu & 1) * HM + (lane_group & 1) * 32;
            uint8_t* stage = reinterpret_cast<uint8_t*>(out_stage[lane_group]);
            // 16 accumulator columns at a time (few registers); two such steps fill one 32-column fp32 box of the TMA
            // store, four a 64-column fp16 box
            for (int c0 = 0; c0 < n_cols; c0 += 16) {
                uint32_t v[16];
                tmem_ld_16(tmem_base + buf * acc_stride + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int ncol0 = col_base + c0;   // first output column of this step
                if (row0 >= a.M || ncol0 >= a.N) continue;
                if (a.out_f16) {
                    // fp16 output (widths that are multiples of 128 only): 128 bytes per row and box, so a row of the next
                    // layer's input is again fetched in 512-byte requests
                    const int pbase = (c0 & 63) >> 3;    // first 16-byte piece (8 columns) of this step in the box's rows
                    if (pbase == 0) {
                        // the previous box's TMA store must have read the staging tile before it is rewritten
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                    }
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const int n = ncol0 + 8 * c;
                        const float4 b0 = __ldg(reinterpret_cast<const float4*>(a.bias + n)), b1 = __ldg(reinterpret_cast<const float4*>(a.bias + n + 4));
                        float o[8] = {__uint_as_float(v[8 * c]) + b0.x, __uint_as_float(v[8 * c + 1]) + b0.y, __uint_as_float(v[8 * c + 2]) + b0.z,
                                      __uint_as_float(v[8 * c + 3]) + b0.w, __uint_as_float(v[8 * c + 4]) + b1.x, __uint_as_float(v[8 * c + 5]) + b1.y,
                                      __uint_as_float(v[8 * c + 6]) + b1.z, __uint_as_float(v[8 * c + 7]) + b1.w};
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const __half2 h = a.relu ? __floats2half2_rn(fmaxf(o[2 * i], 0.f), fmaxf(o[2 * i + 1], 0.f)) : __floats2half2_rn(o[2 * i], o[2 * i + 1]);
                            w[i] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                        *reinterpret_cast<uint4*>(stage + lane * 128 + (((pbase + c) ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    if (pbase == 6) {
                        fence_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                         ::"l"(&map_out), "r"(smem_u32(stage)), "r"(ncol0 - 48), "r"((int)row0) : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                    }
                } else if ((c0 & ~31) + 32 <= n_cols) {
                    const int pbase = (c0 & 31) >> 2;    // 0 or 4: first 16-byte piece (4 columns) of this step
                    if (pbase == 0) {
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                    }
                    // lane = row of the box; 16-byte piece c of the row goes to piece c ^ (row % 8) (128-byte swizzle)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int n = ncol0 + 4 * c;
                        float4 o = make_float4(__uint_as_float(v[4 * c]), __uint_as_float(v[4 * c + 1]),
                                               __uint_as_float(v[4 * c + 2]), __uint_as_float(v[4 * c + 3]));
                        if (n < a.N) {
                            const float4 bb = __ldg(reinterpret_cast<const float4*>(a.bias + n));
                            o.x += bb.x; o.y += bb.y; o.z += bb.z; o.w += bb.w;
                        }
                        if (a.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                        *reinterpret_cast<float4*>(stage + lane * 128 + (((pbase + c) ^ (lane & 7)) << 4)) = o;
                    }
                    if (pbase == 4) {
                        fence_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            // rows past the end of the layer and columns past its width are clipped by the tensor map
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                         ::"l"(&map_out), "r"(smem_u32(stage)), "r"(ncol0 - 16), "r"((int)row0) : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                    }
                } else {
                    // the ragged end of the half (BN / 2 is not a multiple of 32): lane = row, plain stores
                    const int64_t row = row0 + lane;
                    if (row < a.M) {
                        float* orow = a.out + row * a.N;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int n = ncol0 + 4 * c;
                            if (c0 + 4 * c < n_cols && n < a.N) {
                                const float4 bb = __ldg(reinterpret_cast<const float4*>(a.bias + n));
                                float4 o = make_float4(__uint_as_float(v[4 * c]) + bb.x, __uint_as_float(v[4 * c + 1]) + bb.y,
                                                       __uint_as_float(v[4 * c + 2]) + bb.z, __uint_as_float(v[4 * c + 3]) + bb.w);
                                if (a.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                                *reinterpret_cast<float4*>(orow + n) = o;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {   // this accumulator buffer of this CTA is drained: tell the leader's MMA thread
                if (leader) mbar_arrive(&acc_empty[buf]);
                else mbar_arrive_cluster(mapa_u32(smem_u32(&acc_empty[buf]), 0));
            }
        }
    }
    } else {
    MG_REG_SET(MG_REG_PROD);
    {
        // ---------------- producers: gather + segment mean -> swizzled A slices ----------------
        // K slices come in groups of eight: (self, mean) pairs for four consecutive 32-column blocks, i.e. 128
        // columns of the input rows.  A tile is built in rounds of 32 rows (a row block, planned ahead by the
        // planner warps): a warp builds two rows per round from whole 512-byte row segments (lane L owns columns
        // 4L..4L+3 of the group) and keeps 2 x (1 + kUnroll) loads in flight per lane -- memory-level parallelism
        // comes from registers.  Each lane scatters its 16-byte pieces into the group's stages: slice pair L / 8,
        // slot L % 8.  Producer warps only meet at the mbarriers, never at a block-wide barrier.
        const int pw = warp - kFirstProducerWarp;     // 0 .. kProducerWarps-1
        const int gl = lane & 7;                      // 16-byte slot inside a 128-byte slice row
        bool ok = true;
        for (uint32_t it = 0; it < my_iters; ++it) {
            for (int grp = 0; grp < n_groups; ++grp) {
                const uint32_t s_h = it * (uint32_t)n_groups + (uint32_t)grp;   // fills of each half's stage rows so far
                const int pairs = min(GC / KCE, (a.d_in_pad - grp * GC) / KCE);   // slice pairs in this group
                const int col = grp * GC + lane * LC;
                const bool lane_on = (lane >> 3) < pairs;
                const bool col_ok = lane_on && col < a.d_in;
                const char* src = a.src_base + (size_t)col * (HALF ? 2 : 4);
                for (int blk = 0; blk < kBlocksPerTile; ++blk) {
                    const int h = blk / kBlocksPerHalf;               // the half tile this block belongs to
                    const uint32_t q = it * kBlocksPerTile + blk;     // row block counter of this CTA
                    const int slot = q % kPlanSlots;
                    if (grp == 0 && ok && !mbar_wait(&plan_full[slot], (q / kPlanSlots) & 1)) {
                        if (lane == 0) atomicExch(a.error, 16u);
                        ok = false;
                    }
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    const bool cached = plan_total[slot] >= 0;
                    const int32_t* rows_of = src_rows[slot];
                    const int brow = pw * kRowsInFlight;              // this warp's first row inside the block
                    RowMeta mq[kRowsInFlight];
                    uint4 selfv[kRowsInFlight], meanv[kRowsInFlight];   // the two operand pieces of each row
                    PieceSum<F16> acc[kRowsInFlight];
                    int top = 0;
#pragma unroll
                    for (int q2 = 0; q2 < kRowsInFlight; ++q2) {
                        mq[q2] = meta[slot][brow + q2];
                        selfv[q2] = make_uint4(0u, 0u, 0u, 0u);
                        meanv[q2] = selfv[q2];
                        acc[q2].zero();
                        top = max(top, mq[q2].z);
                    }
                    if (col_ok && ok) {
#pragma unroll
                        for (int q2 = 0; q2 < kRowsInFlight; ++q2)
                            selfv[q2] = load_piece<HALF, F16>(src + (size_t)(uint32_t)mq[q2].x * (size_t)a.src_row_bytes);
                        if (cached) {
                            // Every load is issued unconditionally: a slot past the end of a row's entries re-reads
                            // the row's own representation (a cache hit) and is not added.  Branch-free code is what
                            // lets all loads of a round be in flight together.  First round: the planner has laid
                            // out the kUnroll source rows per row, padding included.
                            {
                                uint4 v[kRowsInFlight][kUnroll];
#pragma unroll
                                for (int q2 = 0; q2 < kRowsInFlight; ++q2) {
                                    const int4 f4 = *reinterpret_cast<const int4*>(first_rows[slot][brow + q2]);
                                    const int32_t f5 = first_rows[slot][brow + q2][4];
                                    v[q2][0] = load_piece<HALF, F16>(src + (size_t)(uint32_t)f4.x * (size_t)a.src_row_bytes);
                                    v[q2][1] = load_piece<HALF, F16>(src + (size_t)(uint32_t)f4.y * (size_t)a.src_row_bytes);
                                    v[q2][2] = load_piece<HALF, F16>(src + (size_t)(uint32_t)f4.z * (size_t)a.src_row_bytes);
                                    v[q2][3] = load_piece<HALF, F16>(src + (size_t)(uint32_t)f4.w * (size_t)a.src_row_bytes);
                                    v[q2][4] = load_piece<HALF, F16>(src + (size_t)(uint32_t)f5 * (size_t)a.src_row_bytes);
                                }
#pragma unroll
                                for (int j = 0; j < kUnroll; ++j)   // entry order
#pragma unroll
                                    for (int q2 = 0; q2 < kRowsInFlight; ++q2)
                                        if (j < mq[q2].z) acc[q2].add(v[q2][j]);
                            }
                            for (int e = kUnroll; e < top; e += kUnroll) {
                                uint4 v[kRowsInFlight][kUnroll];
#pragma unroll
                                for (int j = 0; j < kUnroll; ++j)
#pragma unroll
                                    for (int q2 = 0; q2 < kRowsInFlight; ++q2) {
                                        const bool live = e + j < mq[q2].z;
                                        const int32_t sr = rows_of[live ? mq[q2].w + e + j : 0];
                                        v[q2][j] = load_piece<HALF, F16>(src + (size_t)(uint32_t)(live ? sr : mq[q2].x) * (size_t)a.src_row_bytes);
                                    }
#pragma unroll
                                for (int j = 0; j < kUnroll; ++j)   // entry order
#pragma unroll
                                    for (int q2 = 0; q2 < kRowsInFlight; ++q2)
                                        if (e + j < mq[q2].z) acc[q2].add(v[q2][j]);   // warp-uniform: predicated adds, not a branch around a load
                            }
                        } else {
                            // a row block with more entries than the shared-memory cache holds: plain per-entry loop
                            const int32_t* keys = FIRST ? a.ent_nbrs : a.ent_repr;
#pragma unroll
                            for (int q2 = 0; q2 < kRowsInFlight; ++q2)
                                for (int e = 0; e < mq[q2].z; ++e) {
                                    const int32_t sr = source_row<FIRST>(a, mq[q2].w, __ldg(keys + mq[q2].y + e));
                                    acc[q2].add(load_piece<HALF, F16>(src + (size_t)(uint32_t)sr * (size_t)a.src_row_bytes));
                                }
                        }
#pragma unroll
                        for (int q2 = 0; q2 < kRowsInFlight; ++q2) {
                            const float inv = cached ? __int_as_float(first_rows[slot][brow + q2][5])
                                                     : (mq[q2].z > 0 ? (a.sum_aggr ? 1.f : 1.f / (float)mq[q2].z) : 0.f);
                            meanv[q2] = acc[q2].operand(inv);
                            selfv[q2] = PieceSum<F16>::self_operand(selfv[q2]);
                        }
                    }
                    if (grp == n_groups - 1) {
                        // the block's plan has been read for the last time: its slot may be planned again
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&plan_empty[slot]);
                    }
                    if (blk % kBlocksPerHalf == 0) {
                        // the half's rows of the stages must have been read by the MMAs of their previous fill (one
                        // commit frees them all); those MMAs ran while the other half was gathered, and the loads
                        // above are already in flight while this waits
                        if (ok && s_h >= 1 && !mbar_wait(&a_free[h], (s_h - 1) & 1)) {
                            if (lane == 0) atomicExch(a.error, 15u);
                            ok = false;
                        }
                        ok = __all_sync(0xFFFFFFFFu, ok);
                    }
                    if (ok && lane_on) {
                        // K-major, 128-byte swizzle: 16-byte slot gl of row r lands in slot gl ^ (r % 8)
                        const uint32_t s_self = 2 * (lane >> 3), s_mean = 2 * (lane >> 3) + 1;   // the group's slice = its stage
                        uint8_t* stage_self = a_base + (size_t)s_self * kABytes;
                        uint8_t* stage_mean = a_base + (size_t)s_mean * kABytes;
#pragma unroll
                        for (int q2 = 0; q2 < kRowsInFlight; ++q2) {
                            const int row = blk * kBlockRows + brow + q2;
                            const size_t off = (size_t)(row >> 3) * 1024 + (size_t)(row & 7) * 128 + (size_t)((gl ^ (row & 7)) << 4);
                            *reinterpret_cast<uint4*>(stage_self + off) = selfv[q2];
                            *reinterpret_cast<uint4*>(stage_mean + off) = meanv[q2];
                        }
                    }
                    if (blk % kBlocksPerHalf == kBlocksPerHalf - 1) {
                        // this warp's rows of the half are in place: tell the leader's MMA thread
                        fence_async_smem();
                        __syncwarp();
                        if (ok && lane == 0) {
                            if (leader) mbar_arrive(&a_ready[h]);
                            else mbar_arrive_cluster(mapa_u32(smem_u32(&a_ready[h]), 0));
                        }
                    }
                }
            }
        }
    }
    }
    if (warp >= kFirstEpilogueWarp && warp < kTmaWarp && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    tc_fence_before();
    cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while the other may still signal or read it
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

// Pre-pass: for every output row of the layer, where its own representation lives and which
// entries it aggregates.  One thread per row, full occupancy; the fused kernel then needs a single
// coalesced load per row instead of a chain of dependent look-ups.
template <bool FIRST>
__global__ void __launch_bounds__(256) k_layer_rows(FusedArgs a, int4* __restrict__ row_meta) {
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; r < a.M; r += (int64_t)gridDim.x * blockDim.x) {
        const int b = upper_segment(a.rowbase_out, a.B + 1, (int32_t)r);
        const int32_t l = (int32_t)r - a.rowbase_out[b];
        const int32_t* cum = a.cum + b * (a.k + 2);
        int h = 0;
        while (h < a.k - a.layer && l >= cum[h + 1]) ++h;
        const int32_t idx = a.node_off[h * (a.B + 1) + b] + (l - cum[h]);
        const int32_t e0 = a.ent_off[idx];
        const int32_t in_base = FIRST ? 0 : a.rowbase_in[b];
        row_meta[r] = make_int4(source_row<FIRST>(a, in_base, FIRST ? a.nodes[idx] : l), e0, a.ent_off[idx + 1] - e0, in_base);
    }
}

// slice order of the fused kernel: groups of kGroup input columns; inside a group (self, mean) pairs of kKC-column blocks
template <bool F16>
__global__ void k_pack_weights(const float* __restrict__ w_cat /*[2 d_in, N]*/, void* __restrict__ w_pad_t /*[N, 2 d_in_pad]*/,
                               int d_in, int d_in_pad, int N) {
    constexpr int KCE = Geo<F16>::kKC, GC = Geo<F16>::kGroup;
    const int K = 2 * d_in_pad;
    const int64_t total = (int64_t)N * K;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i / K), kx = (int)(i % K);
        const int slice = kx / KCE;
        int grp = 0, rem = slice, pairs = min(GC / KCE, d_in_pad / KCE);
        while (rem >= 2 * pairs) { rem -= 2 * pairs; ++grp; pairs = min(GC / KCE, (d_in_pad - grp * GC) / KCE); }
        const int part = rem & 1;
        const int col = grp * GC + (rem >> 1) * KCE + (kx % KCE);
        const float w = col < d_in ? w_cat[(int64_t)(part * d_in + col) * N + n] : 0.f;
        if (F16) reinterpret_cast<__half*>(w_pad_t)[i] = __float2half_rn(w);
        else reinterpret_cast<float*>(w_pad_t)[i] = to_tf32(w);
    }
}

// row-major [rows, K] fp16 matrix, boxes of 64 halves x box_rows, 128-byte swizzle, zero fill
// the same matrix in boxes of 32 halves x 32 rows, not swizzled (the transposed epilogue's fp16 stores)
static bool make_map_f16_box32(CUtensorMap* map, const void* base, int64_t rows, int K) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {32u, 32u};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
static bool make_map_f16(CUtensorMap* map, const void* base, int64_t rows, int K, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// K-major, zero-padded, TF32-rounded copy of [W_self ; W_nbr] for the fused layer kernel
int mg_pack_layer_weights(mg_ctx* ctx, const float* w_cat_dev, float* w_pad_t_dev, int d_in, int N) {
    const int d_in_pad = (d_in + KC - 1) / KC * KC;
    k_pack_weights<false><<<mg_grid(ctx, 2), 256, 0, ctx->stream>>>(w_cat_dev, w_pad_t_dev, d_in, d_in_pad, N);
    ctx->launches++;
    return MG_OK;
}

// The same rounded to fp16 (64-column slices), [N, 2 * roundup64(d_in)] halves: the first layer's weights when the base
// representations are fp16 and the layer's GEMM runs on fp16 operands
int mg_pack_layer_weights_f16(mg_ctx* ctx, const float* w_cat_dev, void* w_pad_h_dev, int d_in, int N) {
    const int d_in_pad = (d_in + 63) / 64 * 64;
    k_pack_weights<true><<<mg_grid(ctx, 2), 256, 0, ctx->stream>>>(w_cat_dev, w_pad_h_dev, d_in, d_in_pad, N);
    ctx->launches++;
    return MG_OK;
}

bool mg_layer_fused_supported(int d_in, int d_out) { return d_out <= 256 && d_out % 4 == 0 && d_in % 4 == 0; }

static void fill_args(mg_ctx* ctx, const mg_dense* d, int layer, int d_in, int d_out, FusedArgs* pa) {
    FusedArgs& a = *pa;
    const int B = d->n_batches;
    a.B = B; a.k = d->k; a.layer = layer;
    a.rowbase_out = d->rowbase + (size_t)layer * (B + 1);
    a.rowbase_in = d->rowbase + (size_t)(layer - 1) * (B + 1);
    a.cum = d->cum; a.node_off = d->node_off; a.nodes = d->nodes;
    a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
    a.feat = mg_feat_geom(ctx);
    a.d_in = d_in;
    a.d_in_pad = (d_in + KC - 1) / KC * KC;
    a.N = d_out;
    a.BN = (d_out + 15) / 16 * 16;
    a.row_lo = 0;
    a.M = d->h_hdr.rows_total[layer];
    a.error = ctx->d_flags;
}

// Pre-pass of one layer: row_meta[r] for every packed output row r of the layer.
int mg_layer_rows(mg_ctx* ctx, const mg_dense* d, int layer, int d_in, int d_out, int4* row_meta) {
    FusedArgs a;
    memset(&a, 0, sizeof(a));
    fill_args(ctx, d, layer, d_in, d_out, &a);
    if (a.M <= 0) return MG_OK;
    if (layer == 1) k_layer_rows<true><<<mg_grid(ctx, 8), 256, 0, ctx->stream>>>(a, row_meta);
    else k_layer_rows<false><<<mg_grid(ctx, 8), 256, 0, ctx->stream>>>(a, row_meta);
    ctx->launches++;
    return MG_OK;
}

// Runs layer `layer` (1-based) for the packed output rows [row_lo, row_hi).  h_prev and h_out are indexed by
// GLOBAL packed row (callers that keep only a window of a layer pass pointers shifted accordingly).
int mg_layer_fused(mg_ctx* ctx, const mg_dense* d, int layer, int d_in, int d_out, const float* w_pad_t, const float* bias,
                   const float* h_prev, float* h_out, int flags, const int4* row_meta, int64_t row_lo, int64_t row_hi,
                   int64_t safe_src_row, const void* w_pad_h, int in_f16, int out_f16) {
    if (row_hi <= row_lo) return MG_OK;
    FusedArgs a;
    memset(&a, 0, sizeof(a));
    fill_args(ctx, d, layer, d_in, d_out, &a);
    a.row_lo = row_lo;
    a.M = row_hi;
    a.row_meta = row_meta;
    a.safe_src = (int32_t)safe_src_row;
    a.h_prev = h_prev;
    a.src_base = layer == 1 ? ctx->slots : reinterpret_cast<const char*>(h_prev);
    a.src_row_bytes = layer == 1 ? (uint32_t)ctx->row_bytes : (uint32_t)d_in * (in_f16 ? 2u : 4u);
    a.out_f16 = out_f16;
    a.relu = flags & 1;
    a.sum_aggr = (flags >> 1) & 1;
    a.bias = bias; a.out = h_out;
    // fp16 operands: first layer over fp16 base representations, mean aggregator (a sum of fp16 values may leave the
    // fp16 range), weights given in fp16 form (the caller withholds them when they do not suit fp16)
    // (later layers: in_f16 says that H^{l-1} was stored as fp16; the caller only does that with fp16 weights at hand)
    const bool f16 = (layer == 1 ? ctx->feat_dtype == MG_DTYPE_F16 : in_f16 != 0) && w_pad_h && !a.sum_aggr;
    if (layer > 1 && in_f16 && !f16) return mg_fail(ctx, MG_ERR_STATE, "fp16 layer input without fp16 operands");
    if (out_f16 && d_out % 128 != 0) return mg_fail(ctx, MG_ERR_STATE, "fp16 layer outputs need widths that are multiples of 128");
    const int kce = f16 ? 64 : KC;
    a.d_in_pad = (d_in + kce - 1) / kce * kce;
    int stride = 32;
    while (stride < a.BN / 2) stride <<= 1;
    a.tmem_cols = kAccBufs * stride;   // accumulator buffers of half tiles: BN / 2 columns each, a power of two >= 32
    const int b_bytes = (a.BN / 2) * 128;       // each CTA of a pair stages half of the output columns
    const int n_chunks = 2 * a.d_in_pad / kce;
    a.sa = std::min(8, n_chunks);   // one group of (self, mean) slice pairs: 128 input columns
    // A shallow weight ring (32 KB) on purpose: with 128 KB of A stages the CTA then fits the 196 KB shared-memory
    // carve-out, which leaves the gathers twice the L1 (measured: layer 1 of the bench 2.92 -> 2.75 ms).
    a.sb = std::max(2, std::min({kMaxStages, n_chunks, (32 * 1024) / b_bytes}));
    // weights in tensor memory: TF32 operands, fp32 output, all of K in 256 columns, at most 256 output columns
    // ... and rows with few entries: a half tile of long rows is gathered for longer than its weight slices take to
    // arrive, so the stream costs nothing there, while the transposed epilogue does (measured: 5.3 entries per row,
    // 2.03 -> 1.92 ms with the weights in tensor memory; 20 per row, 0.83 -> 0.90 ms)
    const int64_t layer_entries = d->h_hdr.ent_base[d->k - layer + 1], layer_rows = d->h_hdr.rows_total[layer];
    const bool ts = n_chunks <= 8 && d_out <= 256 && layer_entries <= kTsMaxEntriesPerRow * layer_rows && !getenv("MG_FUSED_NO_TS");
    if (ts) { a.tmem_cols = 512; a.sb = 0; a.w_rows = f16 ? (const void*)w_pad_h : (const void*)w_pad_t; }
    const size_t smem = (size_t)a.sa * kABytes + (size_t)a.sb * b_bytes + 1024;
    CUtensorMap mw;
    if (!(f16 ? make_map_f16(&mw, w_pad_h, d_out, 2 * a.d_in_pad, a.BN / 2) : make_map_f32(&mw, w_pad_t, d_out, 2 * a.d_in_pad, a.BN / 2)))
        return mg_fail(ctx, MG_ERR_CUDA, "cuTensorMapEncodeTiled failed for the layer weights");
    // output [row_hi rows, d_out] fp32, 32 x 32 boxes, 128-byte swizzle; rows are global packed rows, so a window's
    // shifted base pointer works unchanged (rows below row_lo are never stored)
    CUtensorMap mo;
    if (!(out_f16 ? (ts ? make_map_f16_box32(&mo, h_out, row_hi, d_out) : make_map_f16(&mo, h_out, row_hi, d_out, 32))
                  : make_map_f32(&mo, h_out, row_hi, d_out, 32)))
        return mg_fail(ctx, MG_ERR_CUDA, "cuTensorMapEncodeTiled failed for the layer output");
    const bool first = layer == 1, half = first && ctx->feat_dtype == MG_DTYPE_F16;
    auto kern = first ? (f16 ? k_sage_layer_fused<true, true, true> : half ? k_sage_layer_fused<true, true, false> : k_sage_layer_fused<true, false, false>)
                      : (f16 ? k_sage_layer_fused<false, true, true> : k_sage_layer_fused<false, false, false>);
    if (ts) kern = first ? (f16 ? k_sage_layer_fused<true, true, true, true> : half ? k_sage_layer_fused<true, true, false, true> : k_sage_layer_fused<true, false, false, true>)
                         : (f16 ? k_sage_layer_fused<false, true, true, true> : k_sage_layer_fused<false, false, false, true>);
    MG_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t n_tiles = (row_hi - row_lo + BM - 1) / BM;
    const int grid = 2 * (int)std::min<int64_t>((n_tiles + 1) / 2, ctx->n_sms / 2);   // CTA pairs
    kern<<<grid, kFusedThreads, smem, ctx->stream>>>(mw, mo, a);
    ctx->launches++;
    MG_CUDA(ctx, cudaGetLastError());
    return MG_OK;
}
