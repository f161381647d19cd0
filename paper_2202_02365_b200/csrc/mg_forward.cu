// GraphSage forward over DENSE (Section 4.2): per layer a segment-mean over the sampled
// neighbours (Algorithm 3 with mean instead of sum) and the self / neighbour linear maps.
//
// Rows are kept in sampling order (targets first), so layer l's output rows of a batch are the
// prefix [0, N_l) of its local rows and the "update" of Algorithm 2 is only a smaller row count.
// All batches are packed: H^l holds rowbase[l][b] .. rowbase[l][b+1] for batch b.
// Layer 1 reads base representations straight from the partition buffer (H^0 is never stored).

#include <cuda_fp16.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>

#include "mg_device.cuh"

#include "mg_internal.cuh"

int mg_gemm_tf32(mg_ctx* ctx, const float* x, const float* w_t, const float* bias, float* out, int64_t M, int N, int K,
                 bool relu);  // mg_gemm_tcgen05.cu
int mg_gemm_tf32_status(mg_ctx* ctx);
int mg_gemm_tf32_splitk_add_rows(mg_ctx* ctx, const float* x, const float* g, float* out, int M, int N, int64_t K, int kt_per_slice);
// mg_layer_fused.cu
int mg_pack_layer_weights(mg_ctx* ctx, const float* w_cat_dev, float* w_pad_t_dev, int d_in, int N);
int mg_pack_layer_weights_f16(mg_ctx* ctx, const float* w_cat_dev, void* w_pad_h_dev, int d_in, int N);
bool mg_layer_fused_supported(int d_in, int d_out);
int mg_layer_rows(mg_ctx* ctx, const mg_dense* d, int layer, int d_in, int d_out, int4* row_meta);
int mg_layer_fused(mg_ctx* ctx, const mg_dense* d, int layer, int d_in, int d_out, const float* w_pad_t, const float* bias,
                   const float* h_prev, float* h_out, int flags /* 1 = ReLU, 2 = sum instead of mean */, const int4* row_meta,
                   int64_t row_lo, int64_t row_hi, int64_t safe_src_row, const void* w_pad_h /* the layer's fp16 weights, nullable */,
                   int in_f16 /* layers >= 2: h_prev holds fp16 rows */, int out_f16 /* h_out receives fp16 rows */);

namespace {

constexpr int kThreads = 256;

struct AggArgs {
    int32_t B, k, layer;     // layer l = 1..k
    int32_t d_in;
    int32_t row_lo, row_hi;  // packed output rows handled by this launch
    const int32_t* rowbase_out;  // [B+1] of layer l
    const int32_t* rowbase_in;   // [B+1] of layer l-1
    const int32_t* cum;          // [B][k+2]
    const int32_t* node_off;     // [k+1][B+1]
    const int32_t* nodes;
    const int32_t* ent_off;
    const int32_t* ent_nbrs;
    const int32_t* ent_repr;
    const float* h_prev;         // layers >= 2
    // layer 1: the partition buffer
    const char* slots;
    FeatGeom feat;
    int64_t row_bytes;
    float* x;                    // [rows, 2 * d_in], row r of this launch at x + (r - row_lo) * 2 * d_in
    int round_tf32;
    int sum_aggr;                // neighbour term = sum of the sampled neighbours instead of their mean
};

__device__ __forceinline__ float to_tf32(float v) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
    return __uint_as_float(u);
}

__device__ __forceinline__ const char* feature_row(const AggArgs& a, int32_t node) {
    return a.slots + feat_row(a.feat, node) * a.row_bytes;
}

// one 16-byte chunk -> 4 (fp32) or 8 (fp16) floats
template <bool HALF>
struct Chunk {
    static constexpr int kVals = HALF ? 8 : 4;
    float v[kVals];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int i = 0; i < kVals; ++i) v[i] = 0.f;
    }
    __device__ __forceinline__ void load(const char* row, int chunk) {
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(row) + chunk);
        if (HALF) {
            const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h[i]);
                v[2 * i] = f.x;
                v[2 * i + 1] = f.y;
            }
        } else {
            v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y);
            v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
        }
    }
    __device__ __forceinline__ void add(const Chunk& o) {
#pragma unroll
        for (int i = 0; i < kVals; ++i) v[i] += o.v[i];
    }
    __device__ __forceinline__ void store(float* dst, float scale, bool round) const {
#pragma unroll
        for (int i = 0; i < kVals; i += 4) {
            float4 o = make_float4(v[i] * scale, v[i + 1] * scale, v[i + 2] * scale, v[i + 3] * scale);
            if (round) { o.x = to_tf32(o.x); o.y = to_tf32(o.y); o.z = to_tf32(o.z); o.w = to_tf32(o.w); }
            *reinterpret_cast<float4*>(dst + i) = o;
        }
    }
};

// G lanes per output row; each lane owns NCH 16-byte chunks of the row (chunk = gl + j * G).
template <int G, int NCH, bool FIRST, bool HALF>
__global__ void __launch_bounds__(kThreads) k_aggregate(AggArgs a) {
    using C = Chunk<HALF>;
    constexpr int kRowsPerBlock = kThreads / G;
    const int gl = threadIdx.x % G;
    const int n_chunks = a.d_in / C::kVals;
    const int kk = a.k;
    for (int32_t r = a.row_lo + blockIdx.x * kRowsPerBlock + threadIdx.x / G; r < a.row_hi; r += gridDim.x * kRowsPerBlock) {
        const int b = upper_segment(a.rowbase_out, a.B + 1, r);
        const int32_t l = r - a.rowbase_out[b];
        const int32_t* cum = a.cum + b * (kk + 2);
        int h = 0;
        while (h < kk - a.layer && l >= cum[h + 1]) ++h;
        const int32_t idx = a.node_off[h * (a.B + 1) + b] + (l - cum[h]);
        const int32_t e0 = a.ent_off[idx], e1 = a.ent_off[idx + 1];
        const int64_t in_base = FIRST ? 0 : (int64_t)a.rowbase_in[b];
        float* xrow = a.x + (int64_t)(r - a.row_lo) * 2 * a.d_in;

        // self row
        const char* self_row = FIRST ? feature_row(a, a.nodes[idx])
                                     : reinterpret_cast<const char*>(a.h_prev + (in_base + l) * a.d_in);
        C acc[NCH];
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int c = gl + j * G;
            if (c < n_chunks) {
                C s;
                s.load(self_row, c);
                s.store(xrow + c * C::kVals, 1.f, a.round_tf32);
            }
            acc[j].zero();
        }
        // neighbours, in entry order, two rows in flight
        int32_t e = e0;
        for (; e + 1 < e1; e += 2) {
            const char* r0 = FIRST ? feature_row(a, a.ent_nbrs[e])
                                   : reinterpret_cast<const char*>(a.h_prev + (in_base + a.ent_repr[e]) * a.d_in);
            const char* r1 = FIRST ? feature_row(a, a.ent_nbrs[e + 1])
                                   : reinterpret_cast<const char*>(a.h_prev + (in_base + a.ent_repr[e + 1]) * a.d_in);
            C t0[NCH], t1[NCH];
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                const int c = gl + j * G;
                if (c < n_chunks) { t0[j].load(r0, c); t1[j].load(r1, c); }
            }
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                const int c = gl + j * G;
                if (c < n_chunks) { acc[j].add(t0[j]); acc[j].add(t1[j]); }
            }
        }
        if (e < e1) {
            const char* r0 = FIRST ? feature_row(a, a.ent_nbrs[e])
                                   : reinterpret_cast<const char*>(a.h_prev + (in_base + a.ent_repr[e]) * a.d_in);
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                const int c = gl + j * G;
                if (c < n_chunks) { C t; t.load(r0, c); acc[j].add(t); }
            }
        }
        const float inv = e1 > e0 ? (a.sum_aggr ? 1.f : 1.f / (float)(e1 - e0)) : 0.f;
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int c = gl + j * G;
            if (c < n_chunks) acc[j].store(xrow + a.d_in + c * C::kVals, inv, a.round_tf32);
        }
    }
}

// ---- CUDA-core fp32 GEMM with bias / ReLU epilogue (MG_GEMM_FP32) ---------------------------
// out[M, N] = act(x[M, K] . w[K, N] + bias)
template <bool RELU>
__global__ void __launch_bounds__(256) k_gemm_fp32(const float* __restrict__ x, const float* __restrict__ w,
                                                   const float* __restrict__ bias, float* __restrict__ out, int64_t M,
                                                   int N, int K) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int64_t m0 = (int64_t)blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        for (int i = threadIdx.x; i < BM * BK; i += 256) {
            const int mm = i / BK, kk = i % BK;
            As[kk][mm] = (m0 + mm < M && k0 + kk < K) ? x[(m0 + mm) * K + k0 + kk] : 0.f;
        }
        for (int i = threadIdx.x; i < BK * BN; i += 256) {
            const int kk = i / BN, nn = i % BN;
            Bs[kk][nn] = (k0 + kk < K && n0 + nn < N) ? w[(int64_t)(k0 + kk) * N + n0 + nn] : 0.f;
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
        if (m >= M) continue;
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc[i][j] + bias[n];
            if (RELU) v = fmaxf(v, 0.f);
            out[m * N + n] = v;
        }
    }
}

// ---- canonical-order exports ---------------------------------------------------------------
struct RowExportArgs {
    int32_t k, n_rows, first_delta;  // rows of Delta_{first_delta} .. Delta_k in the paper's order
    int32_t nio[MG_MAX_HOPS + 2];    // canonical offsets of the deltas of this batch
    int32_t cum[MG_MAX_HOPS + 2];
    int32_t dim;
    const int32_t* perm;             // local row of every canonical row of the mini-batch (mg_dense_batch_perm)
};

// out[c, :] = src[local(c), :] where c runs over the paper's row order
__global__ void __launch_bounds__(kThreads) k_export_rows(RowExportArgs a, const float* __restrict__ src, float* __restrict__ out) {
    const int vec = a.dim / 4;
    const int64_t total = (int64_t)a.n_rows * vec;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t c = (int32_t)(i / vec) + a.nio[a.first_delta];
        const int q = (int)(i % vec);
        const int32_t l = a.perm[c];
        reinterpret_cast<float4*>(out)[i] = reinterpret_cast<const float4*>(src + (int64_t)l * a.dim)[q];
    }
}

struct H0Args {
    RowExportArgs r;
    int32_t node_off[MG_MAX_HOPS + 1];
    const int32_t* nodes;
    const char* slots;
    FeatGeom feat;
    int64_t row_bytes;
};

template <bool HALF>
__global__ void __launch_bounds__(kThreads) k_gather_h0(H0Args a, float* __restrict__ out) {
    using C = Chunk<HALF>;
    const int n_chunks = a.r.dim / C::kVals;
    const int64_t total = (int64_t)a.r.n_rows * n_chunks;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t c = (int32_t)(i / n_chunks);
        const int q = (int)(i % n_chunks);
        const int32_t l = a.r.perm[c];
        int h = 0;
        while (h < a.r.k && l >= a.r.cum[h + 1]) ++h;
        const int32_t node = a.nodes[a.node_off[h] + (l - a.r.cum[h])];
        const char* row = a.slots + feat_row(a.feat, node) * a.row_bytes;
        C v;
        v.load(row, q);
        v.store(out + (int64_t)c * a.r.dim + q * C::kVals, 1.f, false);
    }
}

__global__ void k_transpose(const float* __restrict__ in, float* __restrict__ out, int rows, int cols, int round_tf32) {
    const int64_t n = (int64_t)rows * cols;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int r = (int)(i / cols), c = (int)(i % cols);
        const float v = in[i];
        out[(int64_t)c * rows + r] = round_tf32 ? to_tf32(v) : v;
    }
}

template <bool FIRST, bool HALF>
void launch_aggregate(const AggArgs& a, int grid, cudaStream_t st) {
    const int vals = HALF ? 8 : 4;
    const int n_chunks = a.d_in / vals;
    int G = 4;
    while (G < 32 && G < n_chunks) G <<= 1;
    const int nch = (n_chunks + G - 1) / G;
#define MG_AGG(GG, NN) k_aggregate<GG, NN, FIRST, HALF><<<grid, kThreads, 0, st>>>(a)
    if (G == 4) MG_AGG(4, 1);
    else if (G == 8) MG_AGG(8, 1);
    else if (G == 16) MG_AGG(16, 1);
    else if (nch == 1) MG_AGG(32, 1);
    else if (nch == 2) MG_AGG(32, 2);
    else if (nch == 3) MG_AGG(32, 3);
    else if (nch == 4) MG_AGG(32, 4);
    else if (nch <= 6) MG_AGG(32, 6);
    else MG_AGG(32, 8);
#undef MG_AGG
}

void fill_row_export(const mg_dense* d, int batch, int first_delta, int dim, RowExportArgs* r) {
    const int k = d->k;
    memset(r, 0, sizeof(*r));
    r->k = k;
    r->dim = dim;
    r->first_delta = first_delta;
    for (int h = 0; h <= k + 1; ++h) r->cum[h] = d->h_cum[(size_t)batch * (k + 2) + h];
    r->nio[0] = 0;
    for (int j = 0; j <= k; ++j) r->nio[j + 1] = r->nio[j] + (r->cum[k - j + 1] - r->cum[k - j]);
    r->n_rows = r->nio[k + 1] - r->nio[first_delta];
}

}  // namespace

// ---------------------------------------------------------------------------------------
extern "C" int mg_model_create(mg_ctx* ctx, int32_t k, const int32_t* dims, const float* const* w_self,
                               const float* const* w_nbr, const float* const* bias, int gemm_precision, mg_model** out) {
    if (!ctx) return MG_ERR_ARG;
    if (!out || !dims || !w_self || !w_nbr || !bias) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (k <= 0 || k > MG_MAX_HOPS) return mg_fail(ctx, MG_ERR_ARG, "k must be in [1, %d]", MG_MAX_HOPS);
    if (gemm_precision != MG_GEMM_TF32 && gemm_precision != MG_GEMM_FP32) return mg_fail(ctx, MG_ERR_ARG, "unknown gemm precision");
    for (int l = 0; l <= k; ++l)
        if (dims[l] <= 0 || dims[l] % 4 != 0 || dims[l] > 1024) return mg_fail(ctx, MG_ERR_ARG, "layer widths must be multiples of 4 in [4, 1024]");
    for (int l = 0; l < k; ++l)
        if (!w_self[l] || !w_nbr[l] || !bias[l]) return mg_fail(ctx, MG_ERR_ARG, "null weight pointer");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    mg_model* m = new mg_model();
    m->ctx = ctx;
    m->device = ctx->device;
    m->k = k;
    m->precision = gemm_precision;
    for (int l = 0; l <= k; ++l) m->dims[l] = dims[l];
    for (int l = 0; l < k; ++l) {
        const size_t di = dims[l], dn = dims[l + 1];
        if (cudaMalloc((void**)&m->w_cat[l], sizeof(float) * 2 * di * dn) != cudaSuccess ||
            cudaMalloc((void**)&m->w_cat_t[l], sizeof(float) * 2 * di * dn) != cudaSuccess ||
            cudaMalloc((void**)&m->w_pad_t[l], sizeof(float) * 2 * ((di + 31) / 32 * 32) * dn) != cudaSuccess ||
            cudaMalloc((void**)&m->bias[l], sizeof(float) * dn) != cudaSuccess) {
            cudaGetLastError();
            mg_model_free(m);
            return mg_fail(ctx, MG_ERR_OOM, "weight allocation failed");
        }
        cudaMemcpyAsync(m->w_cat[l], w_self[l], sizeof(float) * di * dn, cudaMemcpyHostToDevice, ctx->stream);
        cudaMemcpyAsync(m->w_cat[l] + di * dn, w_nbr[l], sizeof(float) * di * dn, cudaMemcpyHostToDevice, ctx->stream);
        cudaMemcpyAsync(m->bias[l], bias[l], sizeof(float) * dn, cudaMemcpyHostToDevice, ctx->stream);
        // K-major copy [d_out, 2 d_in], rounded to nearest TF32 once, for the tensor-core path
        k_transpose<<<mg_grid(ctx, 2), kThreads, 0, ctx->stream>>>(m->w_cat[l], m->w_cat_t[l], (int)(2 * di), (int)dn,
                                                                  gemm_precision == MG_GEMM_TF32);
        ctx->launches++;
        mg_pack_layer_weights(ctx, m->w_cat[l], m->w_pad_t[l], (int)di, (int)dn);
    }
    // Every layer's weights in fp16 form too, for layers whose input rows are fp16 (layer 1 over fp16 base
    // representations; later layers when the model stores its intermediate outputs as fp16).  fp16 keeps the 10-bit
    // mantissa TF32 keeps but has a 5-bit exponent: the copy is made only when the weights sit well inside its range
    // (largest magnitude below 2^15, root mean square above 2^-10); otherwise that layer stays on TF32 operands.
    for (int l = 0; l < k && gemm_precision == MG_GEMM_TF32; ++l) {
        const size_t di = dims[l], dn = dims[l + 1];
        if (di % 8 != 0) continue;
        double sq = 0.0, mx = 0.0;
        for (size_t i = 0; i < di * dn; ++i) {
            const double a = std::fabs((double)w_self[l][i]), b = std::fabs((double)w_nbr[l][i]);
            sq += a * a + b * b;
            mx = std::max(mx, std::max(a, b));
        }
        const double rms = std::sqrt(sq / (double)(2 * di * dn));
        if (!(mx < 32768.0 && rms > 1.0 / 1024.0)) continue;
        if (cudaMalloc(&m->w_pad_h[l], sizeof(uint16_t) * 2 * ((di + 63) / 64 * 64) * dn) != cudaSuccess) {
            cudaGetLastError();
            mg_model_free(m);
            return mg_fail(ctx, MG_ERR_OOM, "weight allocation failed");
        }
        mg_pack_layer_weights_f16(ctx, m->w_cat[l], m->w_pad_h[l], (int)di, (int)dn);
    }
    cudaError_t e = cudaStreamSynchronize(ctx->stream);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { mg_model_free(m); return mg_cuda_fail(ctx, e, "weight upload"); }
    *out = m;
    return MG_OK;
}

extern "C" int mg_model_set_aggregator(mg_model* m, int aggregator) {
    if (!m) return MG_ERR_ARG;
    if (aggregator != MG_AGGR_MEAN && aggregator != MG_AGGR_SUM) return mg_fail(m->ctx, MG_ERR_ARG, "unknown aggregator");
    m->sum_aggr = aggregator == MG_AGGR_SUM;
    return MG_OK;
}

extern "C" int mg_model_set_intermediates(mg_model* m, int dtype) {
    if (!m) return MG_ERR_ARG;
    if (dtype != MG_DTYPE_F32 && dtype != MG_DTYPE_F16) return mg_fail(m->ctx, MG_ERR_ARG, "unknown dtype");
    m->f16_intermediates = dtype == MG_DTYPE_F16;
    return MG_OK;
}

extern "C" int mg_model_free(mg_model* m) {
    if (!m) return MG_OK;
    cudaSetDevice(m->device);
    for (int l = 0; l < MG_MAX_HOPS; ++l) {
        cudaFree(m->w_cat[l]); cudaFree(m->w_cat_t[l]); cudaFree(m->w_pad_t[l]); cudaFree(m->bias[l]);
        cudaFree(m->g_w_cat[l]); cudaFree(m->g_bias[l]); cudaFree(m->s_w_cat[l]); cudaFree(m->s_bias[l]);
    }
    cudaFree(m->zeros);
    for (int l = 0; l < MG_MAX_HOPS; ++l) cudaFree(m->w_pad_h[l]);
    if (m->ctx && m->ctx->last_fwd_model == m) m->ctx->last_fwd_model = nullptr;
    delete m;
    return MG_OK;
}

static int forward_checks(mg_ctx* ctx, const mg_model* m, const mg_dense* d) {
    if (!m || !d) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (d->pending) return mg_fail(ctx, MG_ERR_STATE, "a sample is in flight on this mg_dense: call mg_sample_many_end first");
    if (!d->valid) return mg_fail(ctx, MG_ERR_STATE, "mg_dense holds no completed sample");
    if (d->ctx != ctx || m->ctx != ctx) return mg_fail(ctx, MG_ERR_ARG, "handle belongs to another context");
    if (!ctx->slots || ctx->feat_dim <= 0) return mg_fail(ctx, MG_ERR_STATE, "no feature table loaded");
    if (m->k != d->k) return mg_fail(ctx, MG_ERR_STATE, "model has %d layers, sample has %d hops", m->k, d->k);
    if (m->dims[0] != ctx->feat_dim) return mg_fail(ctx, MG_ERR_STATE, "model input width %d != feature dim %d", m->dims[0], ctx->feat_dim);
    return mg_check_sample_residency(ctx, d);
}

// rows of a layer are processed in chunks small enough for the [self | mean] staging matrix to
// stay in L2 between the aggregation kernel that writes it and the GEMM that reads it
static int64_t chunk_rows_for(int d_in) {
    const int64_t bytes_per_row = (int64_t)2 * d_in * 4;
    int64_t rows = (48ll << 20) / bytes_per_row;
    rows = std::max<int64_t>(rows / 128 * 128, 128);
    return rows;
}

enum { OUT_DEVICE = 0, OUT_HOST = 1, OUT_HOST_ASYNC = 2 };

// hands H^k (device, packed) to the caller: device or host copy, blocking or on the side stream
static int finish_forward(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out, int out_mode, const float* hk) {
    cudaStream_t st = ctx->stream;
    if (!d->ev_read_done) MG_CUDA(ctx, cudaEventCreateWithFlags(&d->ev_read_done, cudaEventDisableTiming));
    MG_CUDA(ctx, cudaEventRecord(d->ev_read_done, st));   // the next sample into d waits for this
    const int k = d->k;
    const size_t out_bytes = (size_t)d->h_hdr.rows_total[k] * m->dims[k] * sizeof(float);
    if (out_mode == OUT_HOST_ASYNC) {
        // the copy to the host runs on the side stream behind the last layer kernel; the caller's next
        // calls (sampling the next group) overlap it
        MG_CUDA(ctx, cudaEventRecord(ctx->ev_fwd_done, st));
        MG_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fwd_done, 0));
        MG_CUDA(ctx, cudaMemcpyAsync(out, hk, out_bytes, cudaMemcpyDeviceToHost, ctx->side));
        MG_CUDA(ctx, cudaEventRecord(ctx->ev_out_done, ctx->side));
        MG_CUDA(ctx, cudaEventRecord(ctx->ev_hk_done[ctx->hk_cur], ctx->side));   // this H^k buffer is free again after the copy
        ctx->hk_pending[ctx->hk_cur] = true;
        ctx->out_check_gemm = m->precision == MG_GEMM_TF32;
        return MG_OK;
    }
    MG_CUDA(ctx, cudaMemcpyAsync(out, hk, out_bytes, out_mode == OUT_DEVICE ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, st));
    MG_CUDA(ctx, cudaStreamSynchronize(st));
    if (m->precision == MG_GEMM_TF32) return mg_gemm_tf32_status(ctx);
    return MG_OK;
}

static int forward_impl(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out, int out_mode) {
    if (!ctx) return MG_ERR_ARG;
    int rc = forward_checks(ctx, m, d);
    if (rc) return rc;
    if (!out) return mg_fail(ctx, MG_ERR_ARG, "null output");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    const int k = d->k, B = d->n_batches;
    cudaStream_t st = ctx->stream;
    ctx->last_fwd_model = m; ctx->last_fwd_dense = d;
    // H^k of this pass goes to the buffer the pass before last used; an output copy of that pass to the host (side
    // stream) may still read it.  The copy of the previous pass reads the other buffer and is not waited for.
    float* hk = nullptr;
    {
        const int hi = ctx->hk_cur ^= 1;
        if (!ctx->ev_hk_done[hi]) MG_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_hk_done[hi], cudaEventDisableTiming));
        if (ctx->hk_pending[hi]) {
            MG_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_hk_done[hi], 0));
            ctx->hk_pending[hi] = false;
        }
        const size_t need = (size_t)d->h_hdr.rows_total[k] * m->dims[k];
        if (ctx->hk_elems[hi] < need && (rc = mg_ensure(ctx, &ctx->hk_buf[hi], &ctx->hk_elems[hi], need + need / 4 + 4))) return rc;
        hk = ctx->hk_buf[hi];
        ctx->last_hk = hk;
    }

    // Windowed schedule: when every layer runs in the fused kernel and the intermediate layer outputs need not
    // be kept, the layers are run over sub-groups of a few mini-batches at a time through small reused
    // buffers.  H^l of a sub-group is then still in L2 when layer l+1 reads it, and is overwritten in L2 by the
    // next sub-group before most of it is written back to DRAM.
    bool all_fused = m->precision == MG_GEMM_TF32;
    for (int l = 1; l <= k; ++l) all_fused = all_fused && mg_layer_fused_supported(m->dims[l - 1], m->dims[l]);
    const int sub = ctx->layer_window_batches;
    ctx->layers_kept = !(all_fused && sub > 0 && !ctx->keep_layers && k > 1);
    if (!ctx->layers_kept) {
        const int32_t* rb = d->h_rowbase.data();      // [(k+1)][B+1]
        size_t ring_off[MG_MAX_HOPS + 1] = {0}, ring_total = 0, meta_off[MG_MAX_HOPS + 1] = {0}, meta_total = 0;
        for (int l = 1; l <= k; ++l) {
            meta_off[l] = meta_total;
            meta_total += (size_t)d->h_hdr.rows_total[l];
            ring_off[l] = ring_total;
            if (l == k) break;
            int64_t widest = 0;
            for (int b0 = 0; b0 < B; b0 += sub) {
                const int b1 = std::min(B, b0 + sub);
                widest = std::max<int64_t>(widest, rb[(size_t)l * (B + 1) + b1] - rb[(size_t)l * (B + 1) + b0]);
            }
            ring_total += (size_t)widest * m->dims[l];
        }
        {
            size_t have = ctx->ws_h_bytes[0] / sizeof(float);
            if (have < ring_total && (rc = mg_ensure(ctx, &ctx->ws_h[0], &have, ring_total + ring_total / 4))) return rc;
            ctx->ws_h_bytes[0] = have * sizeof(float);
        }
        int4* meta = reinterpret_cast<int4*>(ctx->ws_x);
        {
            size_t have = ctx->ws_x_bytes / sizeof(int4);
            if (have < meta_total) {
                rc = mg_ensure(ctx, &meta, &have, meta_total + meta_total / 4);
                ctx->ws_x = reinterpret_cast<float*>(meta);
                ctx->ws_x_bytes = have * sizeof(int4);
                if (rc) return rc;
            }
        }
        {
            ProfScope ps(ctx, PH_OTHER, k);
            for (int l = 1; l <= k; ++l)
                if ((rc = mg_layer_rows(ctx, d, l, m->dims[l - 1], m->dims[l], meta + meta_off[l]))) return rc;
        }
        float* base = ctx->ws_h[0];
        for (int b0 = 0; b0 < B; b0 += sub) {
            const int b1 = std::min(B, b0 + sub);
            for (int l = 1; l <= k; ++l) {
                const int64_t lo = rb[(size_t)l * (B + 1) + b0], hi = rb[(size_t)l * (B + 1) + b1];
                const int64_t lo_in = rb[(size_t)(l - 1) * (B + 1) + b0];
                // pointers shifted so that the kernel's global packed row indices land inside the windows
                const float* h_prev = l > 1 ? base + ring_off[l - 1] - lo_in * m->dims[l - 1] : nullptr;
                float* h_out = l == k ? hk : base + ring_off[l] - lo * m->dims[l];
                ProfScope ps(ctx, l == 1 ? PH_AGG_L1 : PH_AGG_REST, 1);
                rc = mg_layer_fused(ctx, d, l, m->dims[l - 1], m->dims[l], m->w_pad_t[l - 1], m->bias[l - 1], h_prev, h_out,
                                    (l < k ? 1 : 0) | (m->sum_aggr ? 2 : 0), meta + meta_off[l], lo, hi, l > 1 ? lo_in : 0, l == 1 ? m->w_pad_h[0] : nullptr, 0, 0);
                if (rc) return rc;
            }
        }
        MG_CUDA(ctx, cudaGetLastError());
        return finish_forward(ctx, m, d, out, out_mode, hk);
    }

    // per-layer outputs H^1..H^k live in one workspace (kept for mg_layer_output).  A model may ask for fp16
    // intermediates (mg_model_set_intermediates): used when every layer runs in the fused kernel with fp16 weights
    // at hand, the widths allow 64-column output boxes, and nobody needs the fp32 layer outputs afterwards.
    bool f16_inter = m->f16_intermediates && all_fused && !ctx->keep_layers && !m->sum_aggr && k > 1;
    for (int l = 1; l < k && f16_inter; ++l) f16_inter = m->dims[l] % 128 == 0 && m->w_pad_h[l] != nullptr;
    ctx->layers_kept = !f16_inter;
    size_t total = 0;           // bytes
    size_t off[MG_MAX_HOPS + 1];
    for (int l = 1; l < k; ++l) {
        off[l] = total;
        total += (size_t)d->h_hdr.rows_total[l] * m->dims[l] * (f16_inter ? 2 : 4);   // (widths are multiples of 4: 16-byte aligned starts)
    }
    off[k] = 0;   // H^k has buffers of its own
    {
        size_t have = ctx->ws_h_bytes[0] / sizeof(float);
        // a quarter of headroom: the row counts of consecutive calls differ slightly, and growing means a
        // device-wide synchronising free + malloc
        const size_t need = (total + 3) / 4;
        if (have < need && (rc = mg_ensure(ctx, &ctx->ws_h[0], &have, need + need / 4))) return rc;
        ctx->ws_h_bytes[0] = have * sizeof(float);
    }
    char* ws_bytes = reinterpret_cast<char*>(ctx->ws_h[0]);
    int64_t max_x = 0;
    for (int l = 1; l <= k; ++l) {
        const int64_t rows = std::min<int64_t>(chunk_rows_for(m->dims[l - 1]), d->h_hdr.rows_total[l]);
        max_x = std::max<int64_t>(max_x, rows * 2 * m->dims[l - 1]);
    }
    {
        size_t have = ctx->ws_x_bytes / sizeof(float);
        if ((rc = mg_ensure(ctx, &ctx->ws_x, &have, (size_t)max_x))) return rc;
        ctx->ws_x_bytes = have * sizeof(float);
    }

    const bool half = ctx->feat_dtype == MG_DTYPE_F16;
    for (int l = 1; l <= k; ++l) {
        const int d_in = m->dims[l - 1], d_out = m->dims[l];
        const int64_t M = d->h_hdr.rows_total[l];
        float* h_out = l == k ? hk : reinterpret_cast<float*>(ws_bytes + off[l]);
        const float* h_prev = l > 1 ? reinterpret_cast<const float*>(ws_bytes + off[l - 1]) : nullptr;
        if (m->precision == MG_GEMM_TF32 && mg_layer_fused_supported(d_in, d_out)) {
            // gather + segment mean + both linear maps in one persistent tensor-core kernel (after a small
            // pre-pass that resolves every output row's sources)
            size_t have = ctx->ws_x_bytes / sizeof(int4);
            int4* meta = reinterpret_cast<int4*>(ctx->ws_x);
            if (have < (size_t)M) {
                rc = mg_ensure(ctx, &meta, &have, (size_t)M + (size_t)M / 4);
                ctx->ws_x = reinterpret_cast<float*>(meta);
                ctx->ws_x_bytes = have * sizeof(int4);
                if (rc) return rc;
            }
            {
                ProfScope ps(ctx, PH_OTHER, 1);
                if ((rc = mg_layer_rows(ctx, d, l, d_in, d_out, meta))) return rc;
            }
            {
                ProfScope ps(ctx, l == 1 ? PH_AGG_L1 : PH_AGG_REST, 1);
                rc = mg_layer_fused(ctx, d, l, d_in, d_out, m->w_pad_t[l - 1], m->bias[l - 1], h_prev, h_out,
                                    (l < k ? 1 : 0) | (m->sum_aggr ? 2 : 0), meta, 0, M, 0,
                                    (l == 1 || f16_inter) ? m->w_pad_h[l - 1] : nullptr, f16_inter && l > 1, f16_inter && l < k);
            }
            if (rc) return rc;
            continue;
        }
        const int64_t chunk = chunk_rows_for(d_in);
        for (int64_t r0 = 0; r0 < M; r0 += chunk) {
            const int64_t r1 = std::min(M, r0 + chunk);
            AggArgs a;
            a.B = B; a.k = k; a.layer = l; a.d_in = d_in;
            a.row_lo = (int32_t)r0; a.row_hi = (int32_t)r1;
            a.rowbase_out = d->rowbase + (size_t)l * (B + 1);
            a.rowbase_in = d->rowbase + (size_t)(l - 1) * (B + 1);
            a.cum = d->cum; a.node_off = d->node_off; a.nodes = d->nodes;
            a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
            a.h_prev = h_prev;
            a.slots = ctx->slots; a.feat = mg_feat_geom(ctx); a.row_bytes = ctx->row_bytes;
            a.x = ctx->ws_x;
            a.round_tf32 = m->precision == MG_GEMM_TF32;
            a.sum_aggr = m->sum_aggr ? 1 : 0;
            {
                ProfScope ps(ctx, l == 1 ? PH_AGG_L1 : PH_AGG_REST, 1);
                const int grid = mg_grid(ctx, 8);
                if (l == 1) { if (half) launch_aggregate<true, true>(a, grid, st); else launch_aggregate<true, false>(a, grid, st); }
                else launch_aggregate<false, false>(a, grid, st);
                ctx->launches++;
            }
            {
                ProfScope ps(ctx, PH_GEMM, 1);
                const int64_t rows = r1 - r0;
                const bool relu = l < k;
                if (m->precision == MG_GEMM_FP32) {
                    dim3 grid((unsigned)((rows + 63) / 64), (unsigned)((d_out + 63) / 64));
                    if (relu) k_gemm_fp32<true><<<grid, 256, 0, st>>>(ctx->ws_x, m->w_cat[l - 1], m->bias[l - 1], h_out + r0 * d_out, rows, d_out, 2 * d_in);
                    else k_gemm_fp32<false><<<grid, 256, 0, st>>>(ctx->ws_x, m->w_cat[l - 1], m->bias[l - 1], h_out + r0 * d_out, rows, d_out, 2 * d_in);
                    ctx->launches++;
                } else {
                    rc = mg_gemm_tf32(ctx, ctx->ws_x, m->w_cat_t[l - 1], m->bias[l - 1], h_out + r0 * d_out, rows, d_out, 2 * d_in, relu);
                    if (rc) return rc;
                }
            }
        }
    }
    MG_CUDA(ctx, cudaGetLastError());
    return finish_forward(ctx, m, d, out, out_mode, hk);
}

extern "C" int mg_forward(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out, int out_on_device) {
    return forward_impl(ctx, m, d, out, out_on_device ? OUT_DEVICE : OUT_HOST);
}

extern "C" int mg_forward_host_async(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out_host) {
    return forward_impl(ctx, m, d, out_host, OUT_HOST_ASYNC);
}

extern "C" int mg_wait_output(mg_ctx* ctx) {
    if (!ctx) return MG_ERR_ARG;
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    MG_CUDA(ctx, cudaEventSynchronize(ctx->ev_out_done));   // completes at once when nothing was recorded
    if (ctx->out_check_gemm) { ctx->out_check_gemm = false; return mg_gemm_tf32_status(ctx); }
    return MG_OK;
}

extern "C" int mg_gather_h0(mg_ctx* ctx, mg_dense* d, int32_t batch, float* out_dev) {
    if (!ctx) return MG_ERR_ARG;
    if (!d || !out_dev) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (!d->valid) return mg_fail(ctx, MG_ERR_STATE, "mg_dense holds no completed sample");
    if (!ctx->slots || ctx->feat_dim <= 0) return mg_fail(ctx, MG_ERR_STATE, "no feature table loaded");
    if (batch < 0 || batch >= d->n_batches) return mg_fail(ctx, MG_ERR_ARG, "batch out of range");
    if (int rs = mg_check_sample_residency(ctx, d)) return rs;
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    H0Args a;
    fill_row_export(d, batch, 0, ctx->feat_dim, &a.r);
    {
        const int32_t* inv_unused;
        const int rc0 = mg_dense_batch_perm(ctx, d, batch, &a.r.perm, &inv_unused);   // rows come in the paper's order
        if (rc0) return rc0;
    }
    for (int h = 0; h <= d->k; ++h) a.node_off[h] = d->h_node_off[(size_t)h * (d->n_batches + 1) + batch];
    a.nodes = d->nodes; a.slots = ctx->slots; a.feat = mg_feat_geom(ctx); a.row_bytes = ctx->row_bytes;
    if (a.r.n_rows > 0) {
        if (ctx->feat_dtype == MG_DTYPE_F16) k_gather_h0<true><<<mg_grid(ctx, 4), kThreads, 0, ctx->stream>>>(a, out_dev);
        else k_gather_h0<false><<<mg_grid(ctx, 4), kThreads, 0, ctx->stream>>>(a, out_dev);
        ctx->launches++;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return MG_OK;
}

extern "C" int mg_layer_output(mg_ctx* ctx, const mg_model* m, mg_dense* d, int32_t layer, int32_t batch, float* out_dev) {
    if (!ctx) return MG_ERR_ARG;
    int rc = forward_checks(ctx, m, d);
    if (rc) return rc;
    if (!out_dev) return mg_fail(ctx, MG_ERR_ARG, "null output");
    if (layer < 1 || layer > d->k) return mg_fail(ctx, MG_ERR_ARG, "layer must be in [1, k]");
    if (batch < 0 || batch >= d->n_batches) return mg_fail(ctx, MG_ERR_ARG, "batch out of range");
    if (!ctx->last_hk) return mg_fail(ctx, MG_ERR_STATE, "mg_forward has not run");
    if (!ctx->layers_kept) return mg_fail(ctx, MG_ERR_STATE, "the last forward did not keep its intermediate layers: call mg_keep_layer_outputs(ctx, 1) first");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    size_t off = 0;   // bytes; the layers were kept as fp32 (layers_kept)
    for (int l = 1; l < layer; ++l) off += (size_t)d->h_hdr.rows_total[l] * m->dims[l] * 4;
    const int B = d->n_batches;
    const float* layer_base = layer == d->k ? ctx->last_hk : reinterpret_cast<const float*>(reinterpret_cast<const char*>(ctx->ws_h[0]) + off);
    if (!layer_base) return mg_fail(ctx, MG_ERR_STATE, "mg_forward has not run");
    const float* src = layer_base + (size_t)d->h_rowbase[(size_t)layer * (B + 1) + batch] * m->dims[layer];
    RowExportArgs r;
    fill_row_export(d, batch, layer, m->dims[layer], &r);
    {
        const int32_t* inv_unused;
        if ((rc = mg_dense_batch_perm(ctx, d, batch, &r.perm, &inv_unused))) return rc;
    }
    if (r.n_rows > 0) {
        k_export_rows<<<mg_grid(ctx, 4), kThreads, 0, ctx->stream>>>(r, src, out_dev);
        ctx->launches++;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return MG_OK;
}

// ---------------------------------------------------------------------------------------
// Backward pass through the GraphSage layers (Section 3: the gradients of a mini-batch update the model and the
// base representations).  Chain rule through Algorithm 3 and Algorithm 2, layer k down to layer 1, over the same
// row chunks as the unfused forward path:
//   X = [self | aggregate] of the chunk is recomputed from H^{l-1} (kept by the forward pass),
//   dPre = dH^l (masked by H^l > 0 below the last layer),
//   dW += X^T dPre, dbias += column sums of dPre, dX = dPre W^T,
//   dH^{l-1}[self row] += dX[:, :d_in];  dH^{l-1}[source row of entry e] += dX[:, d_in:] / count (or x 1 for a sum).
// All arithmetic is fp32 on CUDA cores; sums over rows use atomic adds, so low-order bits vary from run to run.
// ---------------------------------------------------------------------------------------
namespace {

struct RowGeom {
    int32_t B, k;
    const int32_t* rowbase;   // [(k + 1)][B + 1]
    const int32_t* cum;       // [B][k + 2]
    const int32_t* node_off;  // [(k + 1)][B + 1]
};

// packed row of layer `layer` -> its mini-batch, its local row, its place in the hop-major node list
__device__ __forceinline__ void locate_row(const RowGeom& g, int layer, int64_t row, int32_t* b_out, int32_t* local_out, int32_t* node_out) {
    const int32_t* rb = g.rowbase + (int64_t)layer * (g.B + 1);
    int lo = 0, hi = g.B;   // rb[lo] <= row < rb[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)rb[mid] <= row) lo = mid; else hi = mid;
    }
    const int32_t local = (int32_t)(row - rb[lo]);
    const int32_t* cum = g.cum + (int64_t)lo * (g.k + 2);
    int j = 0;
    while (j + 1 <= g.k && cum[j + 1] <= local) ++j;
    *b_out = lo; *local_out = local;
    *node_out = g.node_off[(int64_t)j * (g.B + 1) + lo] + (local - cum[j]);
}

// The gradient of a layer's pre-activations and of its bias in one pass: g *= (y > 0) where the layer has a ReLU
// (MASK; y = the layer's kept outputs), db += column sums of g.  A thread keeps four columns and walks down the rows
// (16-byte accesses, a block covers whole rows); column sums meet in shared memory, one atomic add per column and block.
template <bool MASK>
__global__ void __launch_bounds__(kThreads) k_grad_pre_bias(float* g, const float* __restrict__ y, float* db, int64_t rows, int N) {
    __shared__ float sums[1024];
    const int n4 = N / 4;                       // (widths are multiples of 4, at most 1024)
    const int rows_per_pass = kThreads / n4;    // >= 1
    for (int c = threadIdx.x; c < N; c += kThreads) sums[c] = 0.f;
    __syncthreads();
    const int c4 = threadIdx.x % n4, rr = threadIdx.x / n4;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (rr < rows_per_pass) {
        float4* g4 = reinterpret_cast<float4*>(g);
        const float4* y4 = reinterpret_cast<const float4*>(y);
        const int64_t step = (int64_t)gridDim.x * rows_per_pass;
        for (int64_t r = (int64_t)blockIdx.x * rows_per_pass + rr; r < rows; r += 2 * step) {
            const int64_t i0 = r * n4 + c4, i1 = (r + step) * n4 + c4;
            const bool two = r + step < rows;
            float4 v0 = g4[i0], v1 = two ? g4[i1] : make_float4(0.f, 0.f, 0.f, 0.f);
            if (MASK) {
                const float4 a0 = y4[i0], a1 = two ? y4[i1] : make_float4(1.f, 1.f, 1.f, 1.f);
                const float4 m0 = make_float4(a0.x > 0.f ? v0.x : 0.f, a0.y > 0.f ? v0.y : 0.f, a0.z > 0.f ? v0.z : 0.f, a0.w > 0.f ? v0.w : 0.f);
                const float4 m1 = make_float4(a1.x > 0.f ? v1.x : 0.f, a1.y > 0.f ? v1.y : 0.f, a1.z > 0.f ? v1.z : 0.f, a1.w > 0.f ? v1.w : 0.f);
                g4[i0] = m0;
                if (two) g4[i1] = m1;
                v0 = m0; v1 = m1;
            }
            s.x += v0.x + v1.x; s.y += v0.y + v1.y; s.z += v0.z + v1.z; s.w += v0.w + v1.w;
        }
        atomicAdd(&sums[4 * c4], s.x); atomicAdd(&sums[4 * c4 + 1], s.y); atomicAdd(&sums[4 * c4 + 2], s.z); atomicAdd(&sums[4 * c4 + 3], s.w);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < N; c += kThreads) atomicAdd(&db[c], sums[c]);
}

// dW[Kx, N] += X[rows, Kx]^T dPre[rows, N]; a block owns a 64 x 64 tile of dW and a slice of the rows
constexpr int kGradRowsPerBlock = 1024;
__global__ void __launch_bounds__(256) k_grad_weights(const float* __restrict__ x, const float* __restrict__ dpre, float* dw,
                                                      int64_t rows, int Kx, int N) {
    constexpr int T = 64, BR = 16;
    __shared__ float xs[BR][T + 4];
    __shared__ float gs[BR][T + 4];
    const int k0 = blockIdx.x * T, n0 = blockIdx.y * T;
    const int64_t r_lo = (int64_t)blockIdx.z * kGradRowsPerBlock, r_hi = min(rows, r_lo + kGradRowsPerBlock);
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int64_t r0 = r_lo; r0 < r_hi; r0 += BR) {
        for (int i = threadIdx.x; i < BR * T; i += 256) {
            const int rr = i / T, c = i % T;
            const bool on = r0 + rr < r_hi;
            xs[rr][c] = (on && k0 + c < Kx) ? x[(r0 + rr) * Kx + k0 + c] : 0.f;
            gs[rr][c] = (on && n0 + c < N) ? dpre[(r0 + rr) * N + n0 + c] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int rr = 0; rr < BR; ++rr) {
            float xv[4], gv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { xv[i] = xs[rr][ty * 4 + i]; gv[i] = gs[rr][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xv[i], gv[j], acc[i][j]);
        }
        __syncthreads();
    }
    for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j) {
            const int kk = k0 + ty * 4 + i, n = n0 + tx * 4 + j;
            if (kk < Kx && n < N) atomicAdd(&dw[(int64_t)kk * N + n], acc[i][j]);
        }
}

// ---- dX of a layer -> the gradient of the layer's input rows ----
// A source row receives the self part of its own output row and a share of the neighbour part of every output row that
// aggregates it.  Instead of adding row by row with atomics (a read-modify-write of the target for every sampled
// entry), the entries are first turned round -- for every source row the list of (output row, weight) that name it: a
// count per source row, an exclusive scan, a fill -- and a warp then sums a source row's contributions in registers and
// stores the row once, through the ReLU of the layer below and into that layer's bias gradient on the way.
struct RevArgs {
    RowGeom g;
    int32_t layer;             // the layer whose entries are turned round (1 .. k)
    int64_t rows_out;          // its packed output rows
    const int32_t* ent_off;
    const int32_t* ent_repr;
    uint32_t* cnt;             // [rows of layer - 1]: counts (FILL = false) / fill cursors (FILL = true)
    const uint32_t* off;       // [rows of layer - 1 + 1] exclusive prefix of the counts
    int2* rev;                 // (output row, weight as float bits)
    int32_t sum_aggr;
};

template <bool FILL>
__global__ void __launch_bounds__(kThreads) k_rev_entries(RevArgs a) {
    const int32_t* rb_in = a.g.rowbase + (int64_t)(a.layer - 1) * (a.g.B + 1);
    for (int64_t row = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; row < a.rows_out; row += (int64_t)gridDim.x * blockDim.x) {
        int32_t b, local, node;
        locate_row(a.g, a.layer, row, &b, &local, &node);
        const int32_t e0 = a.ent_off[node], e1 = a.ent_off[node + 1];
        if (e1 <= e0) continue;
        const int64_t in0 = rb_in[b];
        const float w = a.sum_aggr ? 1.f : 1.f / (float)(e1 - e0);
        for (int32_t e = e0; e < e1; ++e) {
            const int64_t src = in0 + a.ent_repr[e];
            const uint32_t pos = atomicAdd(&a.cnt[src], 1u);
            if (FILL) a.rev[a.off[src] + pos] = make_int2((int32_t)row, __float_as_int(w));
        }
    }
}

// exclusive scan of data[0 .. n) in place, the total to data[n]: tile sums, their scan by one block, the tiles again
constexpr int kRevTile = kThreads * 16;
__global__ void __launch_bounds__(kThreads) k_rev_tile_sums(const uint32_t* __restrict__ data, int64_t n, uint32_t* sums) {
    __shared__ uint32_t part[kThreads / 32];
    const int64_t t0 = (int64_t)blockIdx.x * kRevTile;
    uint32_t s = 0;
    for (int i = threadIdx.x; i < kRevTile; i += kThreads) s += t0 + i < n ? data[t0 + i] : 0u;
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (int w = 0; w < kThreads / 32; ++w) t += part[w];
        sums[blockIdx.x] = t;
    }
}
__global__ void __launch_bounds__(1024) k_rev_scan_sums(uint32_t* sums, int n_tiles) {
    __shared__ uint32_t part[32];
    __shared__ uint32_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int i0 = 0; i0 < n_tiles; i0 += 1024) {
        const int i = i0 + threadIdx.x;
        const uint32_t v = i < n_tiles ? sums[i] : 0u;
        const uint32_t inc = warp_incl_scan(v);
        if ((threadIdx.x & 31) == 31) part[threadIdx.x >> 5] = inc;
        __syncthreads();
        if (threadIdx.x < 32) { const uint32_t w = part[threadIdx.x]; part[threadIdx.x] = warp_incl_scan(w) - w; }
        __syncthreads();
        const uint32_t excl = carry + part[threadIdx.x >> 5] + inc - v;
        if (i < n_tiles) sums[i] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
}
__global__ void __launch_bounds__(kThreads) k_rev_scan_tiles(uint32_t* data, int64_t n, const uint32_t* __restrict__ sums) {
    __shared__ uint32_t part[kThreads / 32];
    const int64_t t0 = (int64_t)blockIdx.x * kRevTile + (int64_t)threadIdx.x * 16;   // 16 consecutive elements per thread
    uint32_t v[16], s = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) { v[i] = t0 + i < n ? data[t0 + i] : 0u; s += v[i]; }
    const uint32_t inc = warp_incl_scan(s);
    if ((threadIdx.x & 31) == 31) part[threadIdx.x >> 5] = inc;
    __syncthreads();
    if (threadIdx.x < 32) {
        const uint32_t w = threadIdx.x < kThreads / 32 ? part[threadIdx.x] : 0u;
        const uint32_t wi = warp_incl_scan(w);
        if (threadIdx.x < kThreads / 32) part[threadIdx.x] = wi - w;
    }
    __syncthreads();
    uint32_t run = sums[blockIdx.x] + part[threadIdx.x >> 5] + inc - s;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        if (t0 + i < n) data[t0 + i] = run;
        run += v[i];
        if (t0 + i == n - 1) data[n] = run;
    }
}

struct GatherArgs {
    RowGeom g;
    int32_t layer;             // the layer whose dX is handed down (1 .. k); its inputs are the rows of layer - 1
    int64_t rows_in;
    const uint32_t* off;       // [rows_in + 1]
    const int2* rev;
    const float* dx;           // [rows of layer, 2 d_in]
    int32_t d_in;
    const float* y;            // [rows_in, d_in] kept outputs of layer - 1 (MASK), else null
    float* g_in;               // [rows_in, d_in]
    float* db;                 // [d_in] bias gradient of layer - 1 (MASK)
};

// A warp takes 32 consecutive source rows.  Lane = row first: where the row lies, its list bounds and its first
// contribution, one coalesced round of loads for all 32 rows instead of a chain of dependent look-ups per row.  Then
// row after row, lane = four columns (NCH groups of them: d_in <= 128 NCH), with the loads of the next row issued
// before the current one is summed.
template <bool MASK, int NCH>
__global__ void __launch_bounds__(kThreads) k_grad_gather(GatherArgs a) {
    __shared__ float sums[MASK ? 128 * NCH : 1];
    const int lane = threadIdx.x & 31;
    const int n4 = a.d_in / 4;
    const int32_t* rb_out = a.g.rowbase + (int64_t)a.layer * (a.g.B + 1);
    const float* __restrict__ dx = a.dx;
    const int64_t ld = 2 * (int64_t)a.d_in;
    if (MASK) {
        for (int c = threadIdx.x; c < 128 * NCH; c += kThreads) sums[c] = 0.f;
        __syncthreads();
    }
    float4 bias[NCH];
#pragma unroll
    for (int q = 0; q < NCH; ++q) bias[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    // the self part and the first contribution of row r of the warp's 32 (both optional), as loads in flight
    auto fetch = [&](int64_t self_row, int32_t first_row, float4* vs, float4* vf) {
#pragma unroll
        for (int q = 0; q < NCH; ++q) {
            const int c = lane + 32 * q;
            vs[q] = (self_row >= 0 && c < n4) ? reinterpret_cast<const float4*>(dx + self_row * ld)[c] : zero4;
            vf[q] = (first_row >= 0 && c < n4) ? reinterpret_cast<const float4*>(dx + (int64_t)first_row * ld + a.d_in)[c] : zero4;
        }
    };
    const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
    for (int64_t s0 = (blockIdx.x * (int64_t)(kThreads / 32) + (threadIdx.x >> 5)) * 32; s0 < a.rows_in; s0 += warps * 32) {
        // lane = row
        const int64_t sl = s0 + lane;
        uint32_t i0 = 0, i1 = 0;
        int64_t self_l = -1;
        int2 first_l = make_int2(-1, 0);
        if (sl < a.rows_in) {
            int32_t b, local, node;
            locate_row(a.g, a.layer - 1, sl, &b, &local, &node);
            i0 = a.off[sl]; i1 = a.off[sl + 1];
            if (local < rb_out[b + 1] - rb_out[b]) self_l = (int64_t)rb_out[b] + local;
            if (i1 > i0) first_l = a.rev[i0];
        }
        const int n_here = (int)min((int64_t)32, a.rows_in - s0);
        float4 vs[NCH], vf[NCH];
        fetch(__shfl_sync(0xFFFFFFFFu, self_l, 0), __shfl_sync(0xFFFFFFFFu, first_l.x, 0), vs, vf);
        for (int r = 0; r < n_here; ++r) {
            const float w_first = __int_as_float(__shfl_sync(0xFFFFFFFFu, first_l.y, r));
            const uint32_t j0 = __shfl_sync(0xFFFFFFFFu, i0, r), j1 = __shfl_sync(0xFFFFFFFFu, i1, r);
            float4 acc[NCH];
#pragma unroll
            for (int q = 0; q < NCH; ++q)
                acc[q] = make_float4(vs[q].x + w_first * vf[q].x, vs[q].y + w_first * vf[q].y, vs[q].z + w_first * vf[q].z,
                                     vs[q].w + w_first * vf[q].w);
            // the next row's loads go out before this row's remaining contributions and its store
            const int rn = min(r + 1, 31);
            fetch(r + 1 < n_here ? __shfl_sync(0xFFFFFFFFu, self_l, rn) : (int64_t)-1,
                  r + 1 < n_here ? __shfl_sync(0xFFFFFFFFu, first_l.x, rn) : -1, vs, vf);
            for (uint32_t i = j0 + 1; i < j1; ++i) {   // (most rows are named by one entry: this loop is the exception)
                const int2 rr = a.rev[i];
                const float w = __int_as_float(rr.y);
                const float4* pp = reinterpret_cast<const float4*>(dx + (int64_t)rr.x * ld + a.d_in);
#pragma unroll
                for (int q = 0; q < NCH; ++q) {
                    const int c = lane + 32 * q;
                    if (c >= n4) continue;
                    const float4 v = pp[c];
                    acc[q].x += w * v.x; acc[q].y += w * v.y; acc[q].z += w * v.z; acc[q].w += w * v.w;
                }
            }
            const int64_t s = s0 + r;
#pragma unroll
            for (int q = 0; q < NCH; ++q) {
                const int c = lane + 32 * q;
                if (c >= n4) continue;
                float4 v = acc[q];
                if (MASK) {
                    const float4 yy = reinterpret_cast<const float4*>(a.y + s * a.d_in)[c];
                    v = make_float4(yy.x > 0.f ? v.x : 0.f, yy.y > 0.f ? v.y : 0.f, yy.z > 0.f ? v.z : 0.f, yy.w > 0.f ? v.w : 0.f);
                    bias[q].x += v.x; bias[q].y += v.y; bias[q].z += v.z; bias[q].w += v.w;
                }
                reinterpret_cast<float4*>(a.g_in + s * a.d_in)[c] = v;
            }
        }
    }
    if (MASK) {
#pragma unroll
        for (int q = 0; q < NCH; ++q) {
            const int c = lane + 32 * q;
            if (c >= n4) continue;
            atomicAdd(&sums[4 * c], bias[q].x); atomicAdd(&sums[4 * c + 1], bias[q].y);
            atomicAdd(&sums[4 * c + 2], bias[q].z); atomicAdd(&sums[4 * c + 3], bias[q].w);
        }
        __syncthreads();
        for (int c = threadIdx.x; c < a.d_in; c += kThreads) atomicAdd(&a.db[c], sums[c]);
    }
}

template <bool MASK>
static void launch_grad_gather(const GatherArgs& a, int grid, cudaStream_t st) {
    const int nch = (a.d_in + 127) / 128;
    if (nch <= 1) k_grad_gather<MASK, 1><<<grid, kThreads, 0, st>>>(a);
    else if (nch <= 2) k_grad_gather<MASK, 2><<<grid, kThreads, 0, st>>>(a);
    else if (nch <= 4) k_grad_gather<MASK, 4><<<grid, kThreads, 0, st>>>(a);
    else k_grad_gather<MASK, 8><<<grid, kThreads, 0, st>>>(a);
}

__global__ void __launch_bounds__(kThreads) k_sgd(float* w, const float* __restrict__ g, float lr, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) w[i] -= lr * g[i];
}

struct PackedIdArgs {
    RowGeom g;
    const int32_t* nodes;
    int64_t n_rows;
    int32_t* ids;
};

__global__ void __launch_bounds__(kThreads) k_packed_ids(PackedIdArgs a) {
    for (int64_t row = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; row < a.n_rows; row += (int64_t)gridDim.x * blockDim.x) {
        int32_t b, local, node;
        locate_row(a.g, 0, row, &b, &local, &node);
        a.ids[row] = a.nodes[node];
    }
}

}  // namespace

extern "C" int mg_backward(mg_ctx* ctx, mg_model* m, mg_dense* d, const float* d_out_dev, float* d_h0_dev) {
    if (!ctx) return MG_ERR_ARG;
    int rc = forward_checks(ctx, m, d);
    if (rc) return rc;
    if (!d_out_dev) return mg_fail(ctx, MG_ERR_ARG, "null output gradient");
    if (!ctx->last_hk || ctx->last_fwd_model != m || ctx->last_fwd_dense != d)
        return mg_fail(ctx, MG_ERR_STATE, "mg_backward follows mg_forward of the same model and sample");
    if (!ctx->layers_kept) return mg_fail(ctx, MG_ERR_STATE, "the forward pass did not keep its intermediate layers: call mg_keep_layer_outputs(ctx, 1) first");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    const int k = d->k, B = d->n_batches;
    cudaStream_t st = ctx->stream;
    // gradient buffers of the model (allocated once), cleared for this pass
    int widest2 = 8;
    for (int l = 1; l <= k; ++l) widest2 = std::max(widest2, 2 * m->dims[l - 1]);
    for (int l = 0; l < k; ++l) {
        const size_t n_w = (size_t)2 * m->dims[l] * m->dims[l + 1], n_b = (size_t)m->dims[l + 1];
        if (!m->g_w_cat[l] && cudaMalloc((void**)&m->g_w_cat[l], n_w * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return mg_fail(ctx, MG_ERR_OOM, "gradient allocation failed"); }
        if (!m->g_bias[l] && cudaMalloc((void**)&m->g_bias[l], n_b * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return mg_fail(ctx, MG_ERR_OOM, "gradient allocation failed"); }
        MG_CUDA(ctx, cudaMemsetAsync(m->g_w_cat[l], 0, n_w * sizeof(float), st));
        MG_CUDA(ctx, cudaMemsetAsync(m->g_bias[l], 0, n_b * sizeof(float), st));
    }
    if (!m->zeros) {
        if (cudaMalloc((void**)&m->zeros, sizeof(float) * 2 * 1024) != cudaSuccess) { cudaGetLastError(); return mg_fail(ctx, MG_ERR_OOM, "gradient allocation failed"); }
        MG_CUDA(ctx, cudaMemsetAsync(m->zeros, 0, sizeof(float) * 2 * 1024, st));
    }
    // scratch: dH^1 .. dH^{k-1}, the X and dX rows of a chunk
    size_t g_off[MG_MAX_HOPS + 1] = {0}, g_total = 0, h_off[MG_MAX_HOPS + 1] = {0}, h_total = 0;
    for (int l = 1; l < k; ++l) {
        g_off[l] = g_total; g_total += ((size_t)d->h_hdr.rows_total[l] * m->dims[l] + 7) / 8 * 8;   // (32-byte aligned starts)
        h_off[l] = h_total; h_total += (size_t)d->h_hdr.rows_total[l] * m->dims[l];
    }
    // (chunks 16 times the forward pass's: nothing here gains from a chunk that stays in L2, and fewer, longer launches
    // mean fewer atomic adds into the weight gradients: 18.2 -> 14.6 ms at 128 mini-batches of the 1M-node workload)
    const int64_t bw_mult = 16;
    int64_t max_x = 0, max_dx = 0, max_in = 0, max_ent = 0;
    for (int l = 1; l <= k; ++l) {
        max_x = std::max<int64_t>(max_x, std::min<int64_t>(bw_mult * chunk_rows_for(m->dims[l - 1]), d->h_hdr.rows_total[l]) * 2 * m->dims[l - 1]);
        if (l > 1 || d_h0_dev) {   // layers whose dX is handed down: dX of the whole layer, the turned-round entries
            max_dx = std::max<int64_t>(max_dx, (int64_t)d->h_hdr.rows_total[l] * 2 * m->dims[l - 1]);
            max_in = std::max<int64_t>(max_in, d->h_hdr.rows_total[l - 1]);
            max_ent = std::max<int64_t>(max_ent, d->h_hdr.ent_base[k]);   // (entries of all hops bound any layer's)
        }
    }
    const int64_t n_sum_tiles = (max_in + kRevTile - 1) / kRevTile + 1;
    if (ctx->bw_g_elems < g_total && (rc = mg_ensure(ctx, &ctx->bw_g, &ctx->bw_g_elems, g_total + g_total / 4 + 16))) return rc;
    if (ctx->bw_x_elems < (size_t)max_x && (rc = mg_ensure(ctx, &ctx->bw_x, &ctx->bw_x_elems, (size_t)max_x + 16))) return rc;
    if (ctx->bw_dx_elems < (size_t)max_dx && (rc = mg_ensure(ctx, &ctx->bw_dx, &ctx->bw_dx_elems, (size_t)max_dx + 16))) return rc;
    if (ctx->bw_off_elems < (size_t)(2 * max_in + n_sum_tiles + 2) &&
        (rc = mg_ensure(ctx, &ctx->bw_off, &ctx->bw_off_elems, (size_t)(2 * max_in + n_sum_tiles + 2) + 16))) return rc;
    if (ctx->bw_rev_elems < (size_t)max_ent && (rc = mg_ensure(ctx, &ctx->bw_rev, &ctx->bw_rev_elems, (size_t)max_ent + 16))) return rc;
    const RowGeom geom{B, k, d->rowbase, d->cum, d->node_off};
    const bool half = ctx->feat_dtype == MG_DTYPE_F16;
    const int grid = mg_grid(ctx, 8);
    for (int l = k; l >= 1; --l) {
        const int d_in = m->dims[l - 1], d_out = m->dims[l];
        const int64_t M = d->h_hdr.rows_total[l];
        // dPre of the last layer is the caller's gradient; below it, the gather of the layer above has already gone through
        // the ReLU and summed the bias gradient
        const float* dpre_all = l == k ? d_out_dev : ctx->bw_g + g_off[l];
        if (l == k && M > 0) {
            const int blocks = (int)std::min<int64_t>(grid, (M + kThreads / (d_out / 4) - 1) / (kThreads / (d_out / 4)));
            k_grad_pre_bias<false><<<blocks, kThreads, 0, st>>>(const_cast<float*>(d_out_dev), nullptr, m->g_bias[l - 1], M, d_out);
            ctx->launches++;
        }
        const float* h_prev = l > 1 ? ctx->ws_h[0] + h_off[l - 1] : nullptr;
        float* g_in = l > 1 ? ctx->bw_g + g_off[l - 1] : d_h0_dev;
        const int64_t chunk = bw_mult * chunk_rows_for(d_in);
        for (int64_t r0 = 0; r0 < M; r0 += chunk) {
            const int64_t r1 = std::min(M, r0 + chunk), rows = r1 - r0;
            AggArgs a;
            a.B = B; a.k = k; a.layer = l; a.d_in = d_in;
            a.row_lo = (int32_t)r0; a.row_hi = (int32_t)r1;
            a.rowbase_out = d->rowbase + (size_t)l * (B + 1);
            a.rowbase_in = d->rowbase + (size_t)(l - 1) * (B + 1);
            a.cum = d->cum; a.node_off = d->node_off; a.nodes = d->nodes;
            a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
            a.h_prev = h_prev;
            a.slots = ctx->slots; a.feat = mg_feat_geom(ctx); a.row_bytes = ctx->row_bytes;
            a.x = ctx->bw_x;
            a.round_tf32 = 0;
            a.sum_aggr = m->sum_aggr ? 1 : 0;
            if (l == 1) { if (half) launch_aggregate<true, true>(a, grid, st); else launch_aggregate<true, false>(a, grid, st); }
            else launch_aggregate<false, false>(a, grid, st);
            const float* dpre = dpre_all + r0 * d_out;
            if (m->precision == MG_GEMM_TF32) {
                // dW += X^T dPre as a tcgen05 GEMM whose contraction runs over the chunk's rows: both operands are read
                // as they lie (rows x columns, the columns contiguous), the contraction is split over CTAs
                const int m_tiles = (2 * d_in + 127) / 128, n_tiles = (d_out + 255) / 256;
                const int64_t steps = (rows + 31) / 32;
                const int per_slice = (int)std::max<int64_t>(16, (steps * m_tiles * n_tiles + 4 * ctx->n_sms - 1) / (4 * ctx->n_sms));
                if ((rc = mg_gemm_tf32_splitk_add_rows(ctx, ctx->bw_x, dpre, m->g_w_cat[l - 1], 2 * d_in, d_out, rows, per_slice))) return rc;
            } else {
                const unsigned slices = (unsigned)((rows + kGradRowsPerBlock - 1) / kGradRowsPerBlock);
                dim3 gw((unsigned)((2 * d_in + 63) / 64), (unsigned)((d_out + 63) / 64), slices);
                k_grad_weights<<<gw, 256, 0, st>>>(ctx->bw_x, dpre, m->g_w_cat[l - 1], rows, 2 * d_in, d_out);
                ctx->launches++;
            }
            ctx->launches++;   // (the aggregation above)
            if (!g_in) continue;   // layer 1 without a gradient of the base representations
            float* dx = ctx->bw_dx + r0 * 2 * d_in;
            if (m->precision == MG_GEMM_TF32) {
                // dX = dPre W^T on the tensor cores: the K-major operand the kernel wants is W itself ([2 d_in, d_out])
                if ((rc = mg_gemm_tf32(ctx, dpre, m->w_cat[l - 1], m->zeros, dx, rows, 2 * d_in, d_out, false))) return rc;
            } else {
                dim3 gx((unsigned)((rows + 63) / 64), (unsigned)((2 * d_in + 63) / 64));
                k_gemm_fp32<false><<<gx, 256, 0, st>>>(dpre, m->w_cat_t[l - 1], m->zeros, dx, rows, 2 * d_in, d_out);
                ctx->launches++;
            }
        }
        if (!g_in) continue;
        // dX -> the gradient of the layer's input rows (see k_grad_gather)
        const int64_t rows_in = d->h_hdr.rows_total[l - 1];
        if (rows_in == 0) continue;
        uint32_t* off = ctx->bw_off;
        uint32_t* cur = ctx->bw_off + (rows_in + 1);
        uint32_t* tile_sums = cur + rows_in;
        const int n_tiles = (int)((rows_in + kRevTile - 1) / kRevTile);
        MG_CUDA(ctx, cudaMemsetAsync(off, 0, sizeof(uint32_t) * (size_t)(2 * rows_in + 1), st));
        RevArgs ra{geom, l, M, d->ent_off, d->ent_repr, off, off, ctx->bw_rev, m->sum_aggr ? 1 : 0};
        const int rgrid = (int)std::max<int64_t>(1, std::min<int64_t>(grid, (M + kThreads - 1) / kThreads));
        if (M > 0) k_rev_entries<false><<<rgrid, kThreads, 0, st>>>(ra);
        k_rev_tile_sums<<<n_tiles, kThreads, 0, st>>>(off, rows_in, tile_sums);
        k_rev_scan_sums<<<1, 1024, 0, st>>>(tile_sums, n_tiles);
        k_rev_scan_tiles<<<n_tiles, kThreads, 0, st>>>(off, rows_in, tile_sums);
        ra.cnt = cur;
        if (M > 0) k_rev_entries<true><<<rgrid, kThreads, 0, st>>>(ra);
        GatherArgs ga{geom, l, rows_in, off, ctx->bw_rev, ctx->bw_dx, d_in, l > 1 ? ctx->ws_h[0] + h_off[l - 1] : nullptr, g_in,
                      l > 1 ? m->g_bias[l - 2] : nullptr};
        const int ggrid = (int)std::max<int64_t>(1, std::min<int64_t>(grid, (rows_in + kThreads - 1) / kThreads));   // 32 rows per warp
        if (l > 1) launch_grad_gather<true>(ga, ggrid, st); else launch_grad_gather<false>(ga, ggrid, st);
        ctx->launches += 6;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(st));
    return m->precision == MG_GEMM_TF32 ? mg_gemm_tf32_status(ctx) : MG_OK;
}

extern "C" int mg_model_grads(const mg_model* m, int32_t layer, const float** d_w_self, const float** d_w_nbr, const float** d_bias) {
    if (!m) return MG_ERR_ARG;
    if (layer < 1 || layer > m->k) return mg_fail(m->ctx, MG_ERR_ARG, "layer must be in [1, k]");
    if (!m->g_w_cat[layer - 1]) return mg_fail(m->ctx, MG_ERR_STATE, "mg_backward has not run");
    const size_t half_elems = (size_t)m->dims[layer - 1] * m->dims[layer];
    if (d_w_self) *d_w_self = m->g_w_cat[layer - 1];
    if (d_w_nbr) *d_w_nbr = m->g_w_cat[layer - 1] + half_elems;
    if (d_bias) *d_bias = m->g_bias[layer - 1];
    return MG_OK;
}

namespace {
// Adagrad: state += g^2; w -= lr * g / (sqrt(state) + eps)
__global__ void __launch_bounds__(kThreads) k_adagrad(float* w, const float* __restrict__ g, float* state, float lr, float eps, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const float gi = g[i];
        const float s = state[i] + gi * gi;
        state[i] = s;
        w[i] -= lr * gi / (sqrtf(s) + eps);
    }
}
}  // namespace

// the copies of a layer's weights that the forward kernels read
static int refresh_weight_copies(mg_ctx* ctx, mg_model* m, int l) {
    const size_t di = m->dims[l], dn = m->dims[l + 1];
    k_transpose<<<mg_grid(ctx, 2), kThreads, 0, ctx->stream>>>(m->w_cat[l], m->w_cat_t[l], (int)(2 * di), (int)dn, m->precision == MG_GEMM_TF32);
    ctx->launches++;
    if (m->w_pad_h[l]) mg_pack_layer_weights_f16(ctx, m->w_cat[l], m->w_pad_h[l], (int)di, (int)dn);
    return mg_pack_layer_weights(ctx, m->w_cat[l], m->w_pad_t[l], (int)di, (int)dn);
}

extern "C" int mg_model_adagrad_step(mg_ctx* ctx, mg_model* m, float lr, float eps) {
    if (!ctx) return MG_ERR_ARG;
    if (!m || m->ctx != ctx) return mg_fail(ctx, MG_ERR_ARG, "bad model handle");
    if (!m->g_w_cat[0]) return mg_fail(ctx, MG_ERR_STATE, "mg_backward has not run");
    if (!(eps > 0.f)) return mg_fail(ctx, MG_ERR_ARG, "eps must be positive");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->stream;
    for (int l = 0; l < m->k; ++l) {
        const size_t n_w = (size_t)2 * m->dims[l] * m->dims[l + 1], n_b = (size_t)m->dims[l + 1];
        if (!m->s_w_cat[l]) {   // accumulated squared gradients start at zero
            if (cudaMalloc((void**)&m->s_w_cat[l], n_w * sizeof(float)) != cudaSuccess || cudaMalloc((void**)&m->s_bias[l], n_b * sizeof(float)) != cudaSuccess) {
                cudaGetLastError();
                return mg_fail(ctx, MG_ERR_OOM, "optimizer state allocation failed");
            }
            MG_CUDA(ctx, cudaMemsetAsync(m->s_w_cat[l], 0, n_w * sizeof(float), st));
            MG_CUDA(ctx, cudaMemsetAsync(m->s_bias[l], 0, n_b * sizeof(float), st));
        }
        k_adagrad<<<mg_grid(ctx, 2), kThreads, 0, st>>>(m->w_cat[l], m->g_w_cat[l], m->s_w_cat[l], lr, eps, (int64_t)n_w);
        k_adagrad<<<1, kThreads, 0, st>>>(m->bias[l], m->g_bias[l], m->s_bias[l], lr, eps, (int64_t)n_b);
        ctx->launches += 2;
        const int rc = refresh_weight_copies(ctx, m, l);
        if (rc) return rc;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(st));
    return MG_OK;
}

extern "C" int mg_model_sgd_step(mg_ctx* ctx, mg_model* m, float lr) {
    if (!ctx) return MG_ERR_ARG;
    if (!m || m->ctx != ctx) return mg_fail(ctx, MG_ERR_ARG, "bad model handle");
    if (!m->g_w_cat[0]) return mg_fail(ctx, MG_ERR_STATE, "mg_backward has not run");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    cudaStream_t st = ctx->stream;
    for (int l = 0; l < m->k; ++l) {
        const size_t di = m->dims[l], dn = m->dims[l + 1];
        k_sgd<<<mg_grid(ctx, 2), kThreads, 0, st>>>(m->w_cat[l], m->g_w_cat[l], lr, (int64_t)(2 * di * dn));
        k_sgd<<<1, kThreads, 0, st>>>(m->bias[l], m->g_bias[l], lr, (int64_t)dn);
        ctx->launches += 2;
        const int rc = refresh_weight_copies(ctx, m, l);
        if (rc) return rc;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(st));
    return MG_OK;
}

namespace {

struct EmbSgdArgs {
    RowGeom g;
    const int32_t* nodes;
    const float* grad;          // [n_rows, dim] packed like H^0
    int64_t n_rows;
    char* slots;
    FeatGeom feat;
    int64_t row_bytes;
    int32_t dim;
    float lr;
};

// base representation of node(row) -= lr * grad[row]; a node of several mini-batches receives several updates
__global__ void __launch_bounds__(kThreads) k_embedding_sgd(EmbSgdArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
    for (int64_t row = blockIdx.x * (int64_t)(kThreads / 32) + (threadIdx.x >> 5); row < a.n_rows; row += warps) {
        int32_t b, local, node;
        locate_row(a.g, 0, row, &b, &local, &node);
        float* dst = reinterpret_cast<float*>(a.slots + feat_row(a.feat, a.nodes[node]) * a.row_bytes);
        const float* g = a.grad + row * a.dim;
        for (int c = lane; c < a.dim; c += 32) {
            const float v = g[c];
            if (v != 0.f) atomicAdd(&dst[c], -a.lr * v);
        }
    }
}

}  // namespace

extern "C" int mg_apply_embedding_sgd(mg_ctx* ctx, mg_dense* d, const float* d_h0_dev, float lr) {
    if (!ctx) return MG_ERR_ARG;
    if (!d || !d_h0_dev) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (d->pending) return mg_fail(ctx, MG_ERR_STATE, "a sample is in flight on this mg_dense: call mg_sample_many_end first");
    if (!d->valid) return mg_fail(ctx, MG_ERR_STATE, "mg_dense holds no completed sample");
    if (d->ctx != ctx) return mg_fail(ctx, MG_ERR_ARG, "handle belongs to another context");
    if (!ctx->slots || ctx->feat_dim <= 0) return mg_fail(ctx, MG_ERR_STATE, "no feature table loaded");
    if (ctx->feat_dtype != MG_DTYPE_F32) return mg_fail(ctx, MG_ERR_ARG, "base representations are updated in fp32 tables only");
    if (int rs = mg_check_sample_residency(ctx, d)) return rs;
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    EmbSgdArgs a{{d->n_batches, d->k, d->rowbase, d->cum, d->node_off}, d->nodes, d_h0_dev, d->h_hdr.rows_total[0], ctx->slots,
                 mg_feat_geom(ctx), ctx->row_bytes, ctx->feat_dim, lr};
    if (a.n_rows > 0) {
        k_embedding_sgd<<<mg_grid(ctx, 8), kThreads, 0, ctx->stream>>>(a);
        ctx->launches++;
    }
    // with host backing the updated slots go back to the host table when their partitions are evicted
    ctx->dirty_part.assign(ctx->n_parts, 0);
    for (int p = 0; p < ctx->n_parts; ++p) ctx->dirty_part[p] = ctx->slot_of_part[p] >= 0 ? 1 : 0;
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return MG_OK;
}

extern "C" int mg_dense_packed_ids(mg_ctx* ctx, mg_dense* d, int32_t* ids_dev) {
    if (!ctx) return MG_ERR_ARG;
    if (!d || !ids_dev) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (d->pending) return mg_fail(ctx, MG_ERR_STATE, "a sample is in flight on this mg_dense: call mg_sample_many_end first");
    if (!d->valid) return mg_fail(ctx, MG_ERR_STATE, "mg_dense holds no completed sample");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    PackedIdArgs a{{d->n_batches, d->k, d->rowbase, d->cum, d->node_off}, d->nodes, d->h_hdr.rows_total[0], ids_dev};
    if (a.n_rows > 0) {
        k_packed_ids<<<mg_grid(ctx, 4), kThreads, 0, ctx->stream>>>(a);
        ctx->launches++;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return MG_OK;
}

// ---------------------------------------------------------------------------------------
// Forward pass that allocates nothing (the paper has no counterpart).
//
// All temporaries live in one file-scope device array that every GPU loading this library
// holds until the process exits:
//   [0, kNoAllocStagingBytes)                     the [self | mean] staging rows of one chunk
//   [kNoAllocStagingBytes, MG_NOALLOC_SCRATCH_BYTES)  the intermediate layer outputs H^1 .. H^{k-1}
// Nothing in it has to start at zero: every element a kernel reads was written earlier in the
// same call (rows past the end of a tile are zero-filled by the TMA load, not read from here).
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[MG_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr size_t kNoAllocStagingBytes = 4u << 20;
constexpr int kNoAllocMaxDevices = 64;
unsigned char* g_noalloc_ptr[kNoAllocMaxDevices] = {nullptr};
}  // namespace

extern "C" int mg_forward_noalloc(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out_dev) {
    if (!ctx) return MG_ERR_ARG;
    int rc = forward_checks(ctx, m, d);
    if (rc) return rc;
    if (!out_dev) return mg_fail(ctx, MG_ERR_ARG, "null output");
    if (ctx->device < 0 || ctx->device >= kNoAllocMaxDevices) return mg_fail(ctx, MG_ERR_ARG, "device ordinal above %d", kNoAllocMaxDevices - 1);
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    // once per device, with that device current: the array's name is only a host-side handle, the
    // kernels need its device address
    if (!g_noalloc_ptr[ctx->device]) {
        unsigned char* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) return mg_cuda_fail(ctx, e, "cudaGetSymbolAddress(g_noalloc_scratch)");
        g_noalloc_ptr[ctx->device] = p;
    }
    unsigned char* scratch = g_noalloc_ptr[ctx->device];
    const int k = d->k, B = d->n_batches;
    cudaStream_t st = ctx->stream;

    // intermediates H^1 .. H^{k-1} must fit behind the staging area
    size_t off[MG_MAX_HOPS + 1] = {0};
    size_t inter_floats = 0;
    for (int l = 1; l < k; ++l) {
        off[l] = inter_floats;
        inter_floats += (size_t)d->h_hdr.rows_total[l] * m->dims[l];
    }
    const size_t inter_cap = (MG_NOALLOC_SCRATCH_BYTES - kNoAllocStagingBytes) / sizeof(float);
    if (inter_floats > inter_cap)
        return mg_fail(ctx, MG_ERR_CAPACITY,
                       "mg_forward_noalloc: intermediate layer outputs need %zu bytes, the built-in scratch holds %zu "
                       "(MG_NOALLOC_SCRATCH_BYTES = %u in total); use mg_forward or fewer mini-batches per call",
                       inter_floats * sizeof(float), inter_cap * sizeof(float), (unsigned)MG_NOALLOC_SCRATCH_BYTES);
    float* staging = reinterpret_cast<float*>(scratch);
    float* inter = reinterpret_cast<float*>(scratch + kNoAllocStagingBytes);

    const bool half = ctx->feat_dtype == MG_DTYPE_F16;
    for (int l = 1; l <= k; ++l) {
        const int d_in = m->dims[l - 1], d_out = m->dims[l];
        const int64_t M = d->h_hdr.rows_total[l];
        float* h_out = l == k ? out_dev : inter + off[l];
        const float* h_prev = l > 1 ? inter + off[l - 1] : nullptr;
        int64_t chunk = (int64_t)(kNoAllocStagingBytes / sizeof(float)) / (2 * d_in);
        chunk = chunk / 128 * 128;
        if (chunk < 128) return mg_fail(ctx, MG_ERR_CAPACITY, "mg_forward_noalloc: layer width %d too large for the staging area", d_in);
        for (int64_t r0 = 0; r0 < M; r0 += chunk) {
            const int64_t r1 = std::min(M, r0 + chunk);
            AggArgs a;
            a.B = B; a.k = k; a.layer = l; a.d_in = d_in;
            a.row_lo = (int32_t)r0; a.row_hi = (int32_t)r1;
            a.rowbase_out = d->rowbase + (size_t)l * (B + 1);
            a.rowbase_in = d->rowbase + (size_t)(l - 1) * (B + 1);
            a.cum = d->cum; a.node_off = d->node_off; a.nodes = d->nodes;
            a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
            a.h_prev = h_prev;
            a.slots = ctx->slots; a.feat = mg_feat_geom(ctx); a.row_bytes = ctx->row_bytes;
            a.x = staging;
            a.round_tf32 = m->precision == MG_GEMM_TF32;
            a.sum_aggr = m->sum_aggr ? 1 : 0;
            const int grid = mg_grid(ctx, 8);
            if (l == 1) { if (half) launch_aggregate<true, true>(a, grid, st); else launch_aggregate<true, false>(a, grid, st); }
            else launch_aggregate<false, false>(a, grid, st);
            ctx->launches++;
            const int64_t rows = r1 - r0;
            const bool relu = l < k;
            if (m->precision == MG_GEMM_FP32) {
                dim3 g2((unsigned)((rows + 63) / 64), (unsigned)((d_out + 63) / 64));
                if (relu) k_gemm_fp32<true><<<g2, 256, 0, st>>>(staging, m->w_cat[l - 1], m->bias[l - 1], h_out + r0 * d_out, rows, d_out, 2 * d_in);
                else k_gemm_fp32<false><<<g2, 256, 0, st>>>(staging, m->w_cat[l - 1], m->bias[l - 1], h_out + r0 * d_out, rows, d_out, 2 * d_in);
                ctx->launches++;
            } else {
                rc = mg_gemm_tf32(ctx, staging, m->w_cat_t[l - 1], m->bias[l - 1], h_out + r0 * d_out, rows, d_out, 2 * d_in, relu);
                if (rc) return rc;
            }
        }
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(st));
    if (m->precision == MG_GEMM_TF32) return mg_gemm_tf32_status(ctx);
    return MG_OK;
}

extern "C" int mg_keep_layer_outputs(mg_ctx* ctx, int enable) {
    if (!ctx) return MG_ERR_ARG;
    ctx->keep_layers = enable != 0;
    return MG_OK;
}

extern "C" int mg_set_layer_window(mg_ctx* ctx, int32_t mini_batches) {
    if (!ctx) return MG_ERR_ARG;
    if (mini_batches < 0) return mg_fail(ctx, MG_ERR_ARG, "negative window");
    ctx->layer_window_batches = mini_batches;
    return MG_OK;
}
