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

namespace {

constexpr int BM = 128;
constexpr int BK = 32;                       // floats per stage row = 128 bytes = one swizzle row
constexpr int kGemmThreads = 192;            // warp 0 TMA, warp 1 MMA + TMEM, warps 2..5 epilogue
constexpr long long kWaitCycles = 2000000000ll;  // ~1 s: far beyond any legitimate wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// false = gave up
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > kWaitCycles) return false;
    return true;
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// shared-memory matrix descriptor: K-major rows of 128 bytes, 128-byte swizzle, groups of 8 rows
// 1024 bytes apart (the layout TMA writes with CU_TENSOR_MAP_SWIZZLE_128B and a 32-float box).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);   // start address
    d |= (uint64_t)1 << 16;                         // leading byte offset (unused with swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                         // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                         // 128-byte swizzle
    return d;
}

__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_ld_32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

struct GemmParams {
    float* out;
    const float* bias;
    int64_t M;
    int32_t N, K, BN, stages, tmem_cols, relu;
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
    const int kt_total = (p.K + BK - 1) / BK;
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
                tma_load_2d(sa, &map_a, &full_bar[s], kt * BK, (int)m0);
                tma_load_2d(sa + a_bytes, &map_b, &full_bar[s], kt * BK, n0);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: fp32 accumulator, TF32 x TF32, both K-major, M = 128, N = BN
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(p.BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            bool ok = true;
            for (int kt = 0; kt < kt_total && ok; ++kt) {
                const int s = kt % p.stages;
                if (!mbar_wait(&full_bar[s], (kt / p.stages) & 1)) { atomicExch(p.error, 2u); ok = false; break; }
                tc_fence_after();
                const uint32_t sa = smem_u32(stage_base + (size_t)s * stage_bytes);
                const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + a_bytes);
#pragma unroll
                for (int kk = 0; kk < BK / 8; ++kk)   // one instruction consumes 8 TF32 values (32 bytes) of K
                    mma_tf32(tmem_base, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (kt | kk) ? 1u : 0u);
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
        const int64_t row = m0 + lane_group * 32 + lane;
        if (ok) {
            for (int c0 = 0; c0 < p.BN; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32(tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row < p.M) {
                    float* orow = p.out + row * p.N + n0 + c0;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const int n = n0 + c0 + j;
                        if (c0 + j < p.BN && n < p.N) {
                            float4 o;
                            o.x = __uint_as_float(v[j]) + p.bias[n];
                            o.y = __uint_as_float(v[j + 1]) + p.bias[n + 1];
                            o.z = __uint_as_float(v[j + 2]) + p.bias[n + 2];
                            o.w = __uint_as_float(v[j + 3]) + p.bias[n + 3];
                            if (p.relu) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
                            *reinterpret_cast<float4*>(orow + j) = o;
                        }
                    }
                }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
        else
            cudaGetLastError();
    }
    return fn;
}

// row-major [rows, K] fp32 matrix, boxes of 32 floats x box_rows, 128-byte swizzle, zero fill
bool make_map(CUtensorMap* map, const float* base, int64_t rows, int K, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int mg_gemm_tf32(mg_ctx* ctx, const float* x, const float* w_t, const float* bias, float* out, int64_t M, int N, int K,
                 bool relu) {
    if (M <= 0) return MG_OK;
    if (K % 4 != 0 || N % 4 != 0) return mg_fail(ctx, MG_ERR_ARG, "GEMM sizes must be multiples of 4");
    GemmParams p;
    p.out = out; p.bias = bias; p.M = M; p.N = N; p.K = K; p.relu = relu ? 1 : 0; p.error = ctx->d_flags;
    p.BN = std::min(256, (N + 15) / 16 * 16);
    p.tmem_cols = 32;
    while (p.tmem_cols < p.BN) p.tmem_cols <<= 1;
    const int stage_bytes = BM * BK * 4 + p.BN * BK * 4;
    const int kt = (K + BK - 1) / BK;
    p.stages = std::max(1, std::min({kt, 8, (96 * 1024) / stage_bytes}));
    const size_t smem = (size_t)p.stages * stage_bytes + 1024;
    CUtensorMap ma, mb;
    if (!make_map(&ma, x, M, K, BM) || !make_map(&mb, w_t, N, K, p.BN))
        return mg_fail(ctx, MG_ERR_CUDA, "cuTensorMapEncodeTiled failed (M %lld N %d K %d)", (long long)M, N, K);
    static bool attr_set = false;
    if (!attr_set) {
        MG_CUDA(ctx, cudaFuncSetAttribute(k_gemm_tf32, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
        attr_set = true;
    }
    dim3 grid((unsigned)((M + BM - 1) / BM), (unsigned)((N + p.BN - 1) / p.BN));
    k_gemm_tf32<<<grid, kGemmThreads, smem, ctx->stream>>>(ma, mb, p);
    ctx->launches++;
    MG_CUDA(ctx, cudaGetLastError());
    return MG_OK;
}

// After the stream has drained: MG_ERR_TIMEOUT if a GEMM gave up on a barrier (the word is cleared).
int mg_gemm_tf32_status(mg_ctx* ctx) {
    uint32_t flag = 0;
    MG_CUDA(ctx, cudaMemcpy(&flag, ctx->d_flags, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    if (!flag) return MG_OK;
    cudaMemset(ctx->d_flags, 0, sizeof(uint32_t));
    return mg_fail(ctx, MG_ERR_TIMEOUT, "tensor-core GEMM gave up waiting on a barrier (role %u)", flag);
}
