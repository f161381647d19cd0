// TF32 tensor-core GEMM for the GraphSage linear layers on sm_100a:
//     out[M, N] = act(x[M, K] . w_t[N, K]^T + bias)
// x is the [self | mean] staging matrix (K-major), w_t the K-major copy of [W_self; W_nbr].
// Both operands are already rounded to the nearest TF32 value by their producers.
//
// One CTA computes a 128 x BN tile (BN = N rounded up to 16, at most 256; wider outputs use
// several N tiles).  A producer thread streams 32-float K slices of both operands into a ring
// of 128-byte-swizzled shared-memory stages with TMA (no multicast); one thread issues
// tcgen05.mma kind::tf32 with the fp32 accumulator in tensor memory; four epilogue warps read
// the accumulator with tcgen05.ld, add the bias, apply ReLU and store.  Two CTAs fit on an SM,
// so one tile's epilogue overlaps the other's main loop.  Every mbarrier wait is bounded: on a
// time-out the kernel records an error code, still frees its tensor memory and returns.

#include <cuda.h>

#include <algorithm>

#include "mg_internal.cuh"
#include "mg_tcgen05.cuh"

namespace {

constexpr int BM = 128;
constexpr int BK = 32;                       // floats per stage row = 128 bytes = one swizzle row
constexpr int kGemmThreads = 192;            // warp 0 TMA, warp 1 MMA + TMEM, warps 2..5 epilogue

using namespace tc;

struct GemmParams {
    float* out;
    const float* bias;
    int64_t M;
    int32_t N, K, BN, stages, tmem_cols, relu;
    int32_t kt_per_slice;   // split-K: blockIdx.z owns this many 32-wide K steps and ADDS its product to out (0 = whole K, plain store)
    int32_t mn_major;       // 1: the operands are stored [K, M] and [K, N] (the contraction runs over their rows)
    uint32_t* error;  // device word: 0 = ok, else the role that gave up waiting
};

__global__ void __launch_bounds__(kGemmThreads)
k_gemm_tf32(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[8], empty_bar[8], acc_bar;
    __shared__ uint32_t tmem_slot;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t m0 = (int64_t)blockIdx.x * BM;
    const int n0 = blockIdx.y * p.BN;
    const int kt_all = (p.K + BK - 1) / BK;
    const int kt_first = p.kt_per_slice ? (int)blockIdx.z * p.kt_per_slice : 0;
    const int kt_total = p.kt_per_slice ? min(p.kt_per_slice, kt_all - kt_first) : kt_all;   // K steps of this CTA
    const uint32_t a_bytes = BM * BK * 4, b_bytes = (uint32_t)p.BN * BK * 4;
    uint8_t* stage_base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t stage_bytes = a_bytes + b_bytes;  // both multiples of 1024

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&acc_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int kt = 0; kt < kt_total; ++kt) {
                const int s = kt % p.stages;
                if (kt >= p.stages && !mbar_wait(&empty_bar[s], ((kt / p.stages) - 1) & 1)) { atomicExch(p.error, 1u); break; }
                uint8_t* sa = stage_base + (size_t)s * stage_bytes;
                mbar_expect_tx(&full_bar[s], stage_bytes);
                if (p.mn_major) {   // boxes of 32 K rows x 32 floats of M (or N): the tile's 32-float blocks one after the other
                    for (int j = 0; j < BM / 32; ++j)
                        tma_load_2d(sa + j * (BK * 128), &map_a, &full_bar[s], (int)m0 + 32 * j, (kt_first + kt) * BK);
                    for (int j = 0; j < p.BN / 32; ++j)
                        tma_load_2d(sa + a_bytes + j * (BK * 128), &map_b, &full_bar[s], n0 + 32 * j, (kt_first + kt) * BK);
                    continue;
                }
                tma_load_2d(sa, &map_a, &full_bar[s], (kt_first + kt) * BK, (int)m0);
                tma_load_2d(sa + a_bytes, &map_b, &full_bar[s], (kt_first + kt) * BK, n0);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: fp32 accumulator, TF32 x TF32, both K-major, M = 128, N = BN
            // (bits 15 and 16: the operand's M / N dimension is the contiguous one)
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(p.BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24) |
                                   (p.mn_major ? (1u << 15) | (1u << 16) : 0u);
            bool ok = true;
            for (int kt = 0; kt < kt_total && ok; ++kt) {
                const int s = kt % p.stages;
                if (!mbar_wait(&full_bar[s], (kt / p.stages) & 1)) { atomicExch(p.error, 2u); ok = false; break; }
                tc_fence_after();
                const uint32_t sa = smem_u32(stage_base + (size_t)s * stage_bytes);
                if (p.mn_major) {
                    const uint64_t da = smem_desc_sw128_mn(sa, BK * 128), db = smem_desc_sw128_mn(sa + a_bytes, BK * 128);
#pragma unroll
                    for (int kk = 0; kk < BK / 8; ++kk)   // 8 K rows of every box = 1024 bytes further on
                        mma_tf32(tmem_base, da + (uint64_t)(kk * 64), db + (uint64_t)(kk * 64), idesc, (kt | kk) ? 1u : 0u);
                } else {
                    const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + a_bytes);
#pragma unroll
                    for (int kk = 0; kk < BK / 8; ++kk)   // one instruction consumes 8 TF32 values (32 bytes) of K
                        mma_tf32(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (kt | kk) ? 1u : 0u);
                }
                mma_commit(&empty_bar[s]);   // the stage may be refilled once these MMAs have read it
            }
            mma_commit(&acc_bar);            // accumulator complete (arrives even after a time-out)
        }
        __syncwarp();
    } else {
        const bool ok = mbar_wait(&acc_bar, 0);
        if (!ok && lane == 0) atomicExch(p.error, 3u);
        tc_fence_after();
        const int lane_group = warp & 3;                 // tensor-memory lanes this warp may read
        const int64_t row0 = m0 + lane_group * 32;
        // the operand ring is idle once the accumulator is complete: its first 17 KiB serve as the four
        // warps' transpose buffers for coalesced stores
        float* out_stage = reinterpret_cast<float*>(stage_base);
        if (ok) {
            for (int c0 = 0; c0 < p.BN; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32(tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row0 >= p.M) continue;
                if (p.kt_per_slice) add_slice_coalesced(v, out_stage + lane_group * (32 * 33), p.out, row0, p.M, p.N, n0 + c0);
                else store_slice_coalesced(v, out_stage + lane_group * (32 * 33), p.bias, p.out, row0, p.M, p.N, n0 + c0, p.relu != 0);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

}  // namespace

static int gemm_tf32_launch(mg_ctx* ctx, const float* x, const float* w_t, const float* bias, float* out, int64_t M, int N, int K,
                            bool relu, int kt_per_slice, bool mn_major = false) {
    if (M <= 0) return MG_OK;
    if ((mn_major ? M : K) % 4 != 0 || N % 4 != 0) return mg_fail(ctx, MG_ERR_ARG, "GEMM sizes must be multiples of 4");
    GemmParams p;
    p.out = out; p.bias = bias; p.M = M; p.N = N; p.K = K; p.relu = relu ? 1 : 0; p.error = ctx->d_flags;
    p.kt_per_slice = kt_per_slice;
    p.mn_major = mn_major ? 1 : 0;
    p.BN = mn_major ? std::min(256, (N + 31) / 32 * 32) : std::min(256, (N + 15) / 16 * 16);
    p.tmem_cols = 32;
    while (p.tmem_cols < p.BN) p.tmem_cols <<= 1;
    const int stage_bytes = BM * BK * 4 + p.BN * BK * 4;
    const int kt = kt_per_slice ? std::min(kt_per_slice, (K + BK - 1) / BK) : (K + BK - 1) / BK;
    p.stages = std::max(1, std::min({kt, 8, (96 * 1024) / stage_bytes}));
    const size_t smem = (size_t)p.stages * stage_bytes + 1024;
    CUtensorMap ma, mb;
    if (mn_major ? (!make_map_f32(&ma, x, K, (int)M, BK, true) || !make_map_f32(&mb, w_t, K, N, BK, true))
                 : (!make_map_f32(&ma, x, M, K, BM) || !make_map_f32(&mb, w_t, N, K, p.BN)))
        return mg_fail(ctx, MG_ERR_CUDA, "cuTensorMapEncodeTiled failed (M %lld N %d K %d)", (long long)M, N, K);
    static bool attr_set = false;
    if (!attr_set) {
        MG_CUDA(ctx, cudaFuncSetAttribute(k_gemm_tf32, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
        attr_set = true;
    }
    dim3 grid((unsigned)((M + BM - 1) / BM), (unsigned)((N + p.BN - 1) / p.BN),
              kt_per_slice ? (unsigned)(((K + BK - 1) / BK + kt_per_slice - 1) / kt_per_slice) : 1u);
    k_gemm_tf32<<<grid, kGemmThreads, smem, ctx->stream>>>(ma, mb, p);
    ctx->launches++;
    MG_CUDA(ctx, cudaGetLastError());
    return MG_OK;
}

int mg_gemm_tf32(mg_ctx* ctx, const float* x, const float* w_t, const float* bias, float* out, int64_t M, int N, int K,
                 bool relu) {
    return gemm_tf32_launch(ctx, x, w_t, bias, out, M, N, K, relu, 0);
}

// out[M, N] += x[K, M]^T . g[K, N], both operands as they lie in memory (rows = the contraction, far longer than M and
// N: weight gradients), the contraction split over CTAs (kt_per_slice steps of 32 rows each; atomic adds, any order).
// M and N are multiples of 4; rows past K and columns past M, N read as zeros.
int mg_gemm_tf32_splitk_add_rows(mg_ctx* ctx, const float* x, const float* g, float* out, int M, int N, int64_t K, int kt_per_slice) {
    if (K >= (1ll << 31)) return mg_fail(ctx, MG_ERR_ARG, "too many rows for one product");
    return gemm_tf32_launch(ctx, x, g, nullptr, out, M, N, (int)K, false, std::max(1, kt_per_slice), true);
}

// After the stream has drained: MG_ERR_TIMEOUT if a GEMM gave up on a barrier (the word is cleared).
int mg_gemm_tf32_status(mg_ctx* ctx) {
    uint32_t flag = 0;
    MG_CUDA(ctx, cudaMemcpy(&flag, ctx->d_flags, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    if (!flag) return MG_OK;
    cudaMemset(ctx->d_flags, 0, sizeof(uint32_t));
    return mg_fail(ctx, MG_ERR_TIMEOUT, "tensor-core GEMM gave up waiting on a barrier (role %u)", flag);
}
