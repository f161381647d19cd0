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

#include "mg_device.cuh"
#include "mg_internal.cuh"
#include "mg_tcgen05.cuh"

using namespace tc;

namespace {

constexpr int BM = 128;               // output rows per tile
constexpr int KC = 32;                // floats per K slice (one 128-byte swizzle row)
constexpr int kProducerWarps = 16;
constexpr int kFirstProducerWarp = 6; // warp 0 TMA, warp 1 MMA + tensor memory, warps 2..5 epilogue
constexpr int kFusedThreads = (kFirstProducerWarp + kProducerWarps) * 32;  // 704
constexpr int kMaxStages = 8;
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
    // input rows
    const float* h_prev;         // layers >= 2: [rows of layer l-1, d_in]
    const char* slots;           // layer 1: partition buffer
    const int32_t* slot_of_part;
    int64_t slot_bytes, row_bytes;
    uint32_t part_size;
    // shapes
    int32_t d_in, d_in_pad;      // d_in_pad = d_in rounded up to 32; K = 2 * d_in_pad
    int32_t N, BN;               // output width and its MMA tile width (multiple of 16, <= 256)
    int64_t M;                   // packed output rows of the layer
    int32_t sa, sb;              // A and B stages
    int32_t tmem_cols;
    int32_t relu;
    const float* bias;
    float* out;                  // [M, N]
    uint32_t* error;
};

struct RowMeta {      // what a producer needs to build one output row
    int64_t self_off; // layer 1: node id of the row; later layers: row index into h_prev
    int64_t in_base;  // later layers: first h_prev row of the row's mini-batch
    int32_t e0, cnt;  // entries of the row
};

template <bool FIRST>
__device__ __forceinline__ const char* input_row(const FusedArgs& a, int64_t in_base, int32_t key) {
    if (FIRST) {
        const uint32_t p = (uint32_t)key / a.part_size;
        return a.slots + (int64_t)a.slot_of_part[p] * a.slot_bytes + (int64_t)((uint32_t)key - p * a.part_size) * a.row_bytes;
    }
    return reinterpret_cast<const char*>(a.h_prev + (in_base + key) * a.d_in);
}

// 4 consecutive values of a row starting at column col (a multiple of 4)
template <bool HALF>
__device__ __forceinline__ float4 load4(const char* row, int col) {
    if (HALF) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(row + (size_t)col * 2));
        const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        return make_float4(lo.x, lo.y, hi.x, hi.y);
    }
    return __ldg(reinterpret_cast<const float4*>(row + (size_t)col * 4));
}

template <bool FIRST, bool HALF>
__global__ void __launch_bounds__(kFusedThreads, 1)
k_sage_layer_fused(const __grid_constant__ CUtensorMap map_w, FusedArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t a_full[kMaxStages], a_empty[kMaxStages], b_full[kMaxStages], b_empty[kMaxStages];
    __shared__ uint64_t acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ RowMeta meta[BM];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t b_bytes = (uint32_t)a.BN * KC * 4;
    uint8_t* a_base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* b_base = a_base + (size_t)a.sa * kABytes;
    const int n_chunks = 2 * a.d_in_pad / KC;
    const int self_chunks = a.d_in_pad / KC;
    const int64_t n_tiles = (a.M + BM - 1) / BM;

    if (threadIdx.x == 0) {
        for (int s = 0; s < a.sa; ++s) { mbar_init(&a_full[s], kProducerWarps); mbar_init(&a_empty[s], 1); }
        for (int s = 0; s < a.sb; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t acc_stride = (uint32_t)(a.tmem_cols / 2);  // columns per accumulator buffer (a multiple of 32)

    if (warp == 0) {
        // ---------------- weight slices: TMA from L2 ----------------
        if (lane == 0) {
            uint32_t cnt = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                for (int c = 0; c < n_chunks; ++c, ++cnt) {
                    const int s = cnt % a.sb;
                    if (cnt >= (uint32_t)a.sb && !mbar_wait(&b_empty[s], ((cnt / a.sb) - 1) & 1)) { atomicExch(a.error, 11u); ok = false; break; }
                    mbar_expect_tx(&b_full[s], b_bytes);
                    tma_load_2d(b_base + (size_t)s * b_bytes, &map_w, &b_full[s], c * KC, 0);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issue ----------------
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(a.BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            uint32_t cnt = 0, it = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
                const uint32_t buf = it & 1;
                if (it >= 2 && !mbar_wait(&acc_empty[buf], ((it >> 1) - 1) & 1)) { atomicExch(a.error, 12u); ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * acc_stride;
                for (int c = 0; c < n_chunks; ++c, ++cnt) {
                    const int sa = cnt % a.sa, sb = cnt % a.sb;
                    if (!mbar_wait(&a_full[sa], (cnt / a.sa) & 1) || !mbar_wait(&b_full[sb], (cnt / a.sb) & 1)) {
                        atomicExch(a.error, 13u); ok = false; break;
                    }
                    tc_fence_after();
                    const uint64_t da = smem_desc_sw128(smem_u32(a_base + (size_t)sa * kABytes));
                    const uint64_t db = smem_desc_sw128(smem_u32(b_base + (size_t)sb * b_bytes));
#pragma unroll
                    for (int kk = 0; kk < KC / 8; ++kk)
                        mma_tf32(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (c | kk) ? 1u : 0u);
                    mma_commit(&a_empty[sa]);
                    mma_commit(&b_empty[sb]);
                }
                mma_commit(&acc_full[buf]);
            }
        }
        __syncwarp();
    } else if (warp < kFirstProducerWarp) {
        // ---------------- epilogue: tensor memory -> bias, ReLU -> global ----------------
        const int lane_group = warp & 3;
        uint32_t it = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++it) {
            const uint32_t buf = it & 1;
            if (!mbar_wait(&acc_full[buf], (it >> 1) & 1)) { if (lane == 0) atomicExch(a.error, 14u); ok = false; break; }
            tc_fence_after();
            const int64_t row = t * BM + lane_group * 32 + lane;
            for (int c0 = 0; c0 < a.BN; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32(tmem_base + buf * acc_stride + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row < a.M) {
                    float* orow = a.out + row * a.N + c0;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const int n = c0 + j;
                        if (n < a.N) {
                            const float4 bb = __ldg(reinterpret_cast<const float4*>(a.bias + n));
                            float4 o = make_float4(__uint_as_float(v[j]) + bb.x, __uint_as_float(v[j + 1]) + bb.y,
                                                   __uint_as_float(v[j + 2]) + bb.z, __uint_as_float(v[j + 3]) + bb.w);
                            if (a.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                            *reinterpret_cast<float4*>(orow + j) = o;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    } else {
        // ---------------- producers: gather + segment mean -> swizzled A slices ----------------
        const int pw = warp - kFirstProducerWarp;     // 0 .. kProducerWarps-1
        const int ptid = threadIdx.x - kFirstProducerWarp * 32;
        const int g = lane >> 3, gl = lane & 7;       // 4 rows per warp at a time, 8 lanes x float4 per row slice
        constexpr int kRowsPerWarp = BM / kProducerWarps;  // 8
        uint32_t cnt = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
            // row metadata of the tile, once
            asm volatile("bar.sync 1, %0;" ::"r"(kProducerWarps * 32) : "memory");   // previous tile's readers are done
            if (ptid < BM) {
                const int64_t r = t * BM + ptid;
                RowMeta mm;
                mm.self_off = 0; mm.in_base = 0; mm.e0 = 0; mm.cnt = -1;   // cnt < 0: row past the end
                if (r < a.M) {
                    const int b = upper_segment(a.rowbase_out, a.B + 1, (int32_t)r);
                    const int32_t l = (int32_t)r - a.rowbase_out[b];
                    const int32_t* cum = a.cum + b * (a.k + 2);
                    int h = 0;
                    while (h < a.k - a.layer && l >= cum[h + 1]) ++h;
                    const int32_t idx = a.node_off[h * (a.B + 1) + b] + (l - cum[h]);
                    mm.e0 = a.ent_off[idx];
                    mm.cnt = a.ent_off[idx + 1] - mm.e0;
                    mm.in_base = FIRST ? 0 : (int64_t)a.rowbase_in[b];
                    mm.self_off = FIRST ? (int64_t)a.nodes[idx] : (int64_t)l;
                }
                meta[ptid] = mm;
            }
            asm volatile("bar.sync 1, %0;" ::"r"(kProducerWarps * 32) : "memory");
            for (int c = 0; c < n_chunks; ++c, ++cnt) {
                const int s = cnt % a.sa;
                if (ok && cnt >= (uint32_t)a.sa && !mbar_wait(&a_empty[s], ((cnt / a.sa) - 1) & 1)) {
                    if (lane == 0) atomicExch(a.error, 15u);
                    ok = false;
                }
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) continue;   // keep the named barriers balanced, do no more work
                uint8_t* stage = a_base + (size_t)s * kABytes;
                const bool is_self = c < self_chunks;
                const int col = (is_self ? c : c - self_chunks) * KC + gl * 4;
                const bool col_ok = col < a.d_in;
#pragma unroll
                for (int rr = 0; rr < kRowsPerWarp; rr += 4) {
                    const int row = pw * kRowsPerWarp + rr + g;
                    const RowMeta mm = meta[row];
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (mm.cnt >= 0 && col_ok) {
                        if (is_self) {
                            acc = load4<HALF>(input_row<FIRST>(a, mm.in_base, (int32_t)mm.self_off), col);
                        } else if (mm.cnt > 0) {
                            const int32_t* keys = (FIRST ? a.ent_nbrs : a.ent_repr) + mm.e0;
                            int e = 0;
                            for (; e + 4 <= mm.cnt; e += 4) {   // four rows in flight, summed in entry order
                                const float4 v0 = load4<HALF>(input_row<FIRST>(a, mm.in_base, __ldg(keys + e)), col);
                                const float4 v1 = load4<HALF>(input_row<FIRST>(a, mm.in_base, __ldg(keys + e + 1)), col);
                                const float4 v2 = load4<HALF>(input_row<FIRST>(a, mm.in_base, __ldg(keys + e + 2)), col);
                                const float4 v3 = load4<HALF>(input_row<FIRST>(a, mm.in_base, __ldg(keys + e + 3)), col);
                                acc.x += v0.x; acc.y += v0.y; acc.z += v0.z; acc.w += v0.w;
                                acc.x += v1.x; acc.y += v1.y; acc.z += v1.z; acc.w += v1.w;
                                acc.x += v2.x; acc.y += v2.y; acc.z += v2.z; acc.w += v2.w;
                                acc.x += v3.x; acc.y += v3.y; acc.z += v3.z; acc.w += v3.w;
                            }
                            for (; e < mm.cnt; ++e) {
                                const float4 v0 = load4<HALF>(input_row<FIRST>(a, mm.in_base, __ldg(keys + e)), col);
                                acc.x += v0.x; acc.y += v0.y; acc.z += v0.z; acc.w += v0.w;
                            }
                            const float inv = 1.f / (float)mm.cnt;
                            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
                        }
                        acc.x = to_tf32(acc.x); acc.y = to_tf32(acc.y); acc.z = to_tf32(acc.z); acc.w = to_tf32(acc.w);
                    }
                    // K-major, 128-byte swizzle: 16-byte slot gl of row `row` lands in slot gl ^ (row % 8)
                    uint8_t* dst = stage + (size_t)(row >> 3) * 1024 + (size_t)(row & 7) * 128 + (size_t)((gl ^ (row & 7)) << 4);
                    *reinterpret_cast<float4*>(dst) = acc;
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_full[s]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

__global__ void k_pack_weights(const float* __restrict__ w_cat /*[2 d_in, N]*/, float* __restrict__ w_pad_t /*[N, 2 d_in_pad]*/,
                               int d_in, int d_in_pad, int N) {
    const int K = 2 * d_in_pad;
    const int64_t total = (int64_t)N * K;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i / K), kx = (int)(i % K);
        const int part = kx / d_in_pad, col = kx % d_in_pad;
        w_pad_t[i] = col < d_in ? to_tf32(w_cat[(int64_t)(part * d_in + col) * N + n]) : 0.f;
    }
}

}  // namespace

// K-major, zero-padded, TF32-rounded copy of [W_self ; W_nbr] for the fused layer kernel
int mg_pack_layer_weights(mg_ctx* ctx, const float* w_cat_dev, float* w_pad_t_dev, int d_in, int N) {
    const int d_in_pad = (d_in + KC - 1) / KC * KC;
    k_pack_weights<<<mg_grid(ctx, 2), 256, 0, ctx->stream>>>(w_cat_dev, w_pad_t_dev, d_in, d_in_pad, N);
    ctx->launches++;
    return MG_OK;
}

bool mg_layer_fused_supported(int d_in, int d_out) { return d_out <= 256 && d_out % 4 == 0 && d_in % 4 == 0; }

// Runs layer `layer` (1-based) of the model over all mini-batches of the sample.
int mg_layer_fused(mg_ctx* ctx, const mg_dense* d, int layer, int d_in, int d_out, const float* w_pad_t, const float* bias,
                   const float* h_prev, float* h_out, bool relu) {
    const int64_t M = d->h_hdr.rows_total[layer];
    if (M <= 0) return MG_OK;
    const int B = d->n_batches;
    FusedArgs a;
    a.B = B; a.k = d->k; a.layer = layer;
    a.rowbase_out = d->rowbase + (size_t)layer * (B + 1);
    a.rowbase_in = d->rowbase + (size_t)(layer - 1) * (B + 1);
    a.cum = d->cum; a.node_off = d->node_off; a.nodes = d->nodes;
    a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
    a.h_prev = h_prev;
    a.slots = ctx->slots; a.slot_of_part = ctx->d_slot_of_part;
    a.slot_bytes = ctx->slot_bytes; a.row_bytes = ctx->row_bytes; a.part_size = (uint32_t)ctx->part_size;
    a.d_in = d_in;
    a.d_in_pad = (d_in + KC - 1) / KC * KC;
    a.N = d_out;
    a.BN = (d_out + 15) / 16 * 16;
    a.M = M;
    a.relu = relu ? 1 : 0;
    a.bias = bias; a.out = h_out; a.error = ctx->d_flags;
    int stride = 32;
    while (stride < a.BN) stride <<= 1;
    a.tmem_cols = 2 * stride;   // two accumulator buffers, each a power of two >= 32 columns
    const int b_bytes = a.BN * KC * 4;
    const int n_chunks = 2 * a.d_in_pad / KC;
    a.sa = std::min(kMaxStages, std::max(2, std::min(n_chunks, 5)));
    a.sb = std::max(2, std::min({kMaxStages, n_chunks, (int)((212 * 1024 - a.sa * (int)kABytes) / b_bytes)}));
    const size_t smem = (size_t)a.sa * kABytes + (size_t)a.sb * b_bytes + 1024;
    CUtensorMap mw;
    if (!make_map_f32(&mw, w_pad_t, d_out, 2 * a.d_in_pad, a.BN))
        return mg_fail(ctx, MG_ERR_CUDA, "cuTensorMapEncodeTiled failed for the layer weights");
    const bool first = layer == 1, half = first && ctx->feat_dtype == MG_DTYPE_F16;
    auto kern = first ? (half ? k_sage_layer_fused<true, true> : k_sage_layer_fused<true, false>) : k_sage_layer_fused<false, false>;
    MG_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024));
    const int64_t n_tiles = (M + BM - 1) / BM;
    const int grid = (int)std::min<int64_t>(n_tiles, ctx->n_sms);
    kern<<<grid, kFusedThreads, smem, ctx->stream>>>(mw, a);
    ctx->launches++;
    MG_CUDA(ctx, cudaGetLastError());
    return MG_OK;
}
