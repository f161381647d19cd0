// Graph attention over DENSE: the second model family of Section 7.1 (GAT, named there by citation), single head.
//
// Layer l (rows are kept targets-first, so layer l's output rows are a prefix of layer l-1's rows, Algorithm 2):
//   Z = H^{l-1} W                       every input row is transformed BEFORE it is aggregated: one dense GEMM
//   s_src = Z a_src, s_dst = Z a_dst    two numbers per input row
//   for output row i with entries j (sampled neighbours, repeats count) and itself:
//     e_ij = LeakyReLU(s_dst[i] + s_src[j]),  alpha = softmax over {i} + entries,  H^l[i] = sum alpha_ij Z[j] + bias
//   ReLU on all but the last layer.
// The GEMM is the library's tcgen05 TF32 kernel (inputs rounded to TF32 where they are produced) or an fp32 CUDA-core
// kernel; attention is one warp per output row: scores by lane, softmax by warp reductions, then the weighted sum with
// every lane owning a slice of the row's width.  A layer moves N_{l-1} (d_{l-1} + 2 d_l) + (E_l + N_l) d_l floats:
// HBM-bound like the GraphSage layers, with the intermediate Z on top.
#include <cuda_fp16.h>
#include <stdint.h>

#include <algorithm>

#include "mg_internal.cuh"
#include "mgdense.h"

int mg_gemm_tf32(mg_ctx* ctx, const float* x, const float* w_t, const float* bias, float* out, int64_t M, int N, int K,
                 bool relu);
int mg_gemm_tf32_status(mg_ctx* ctx);

struct mg_gat_model {
    mg_ctx* ctx = nullptr;
    int device = 0;
    int32_t k = 0;
    int32_t dims[MG_MAX_HOPS + 1] = {0};
    int precision = MG_GEMM_TF32;
    float slope = 0.2f;
    int32_t heads = 1;                       // attention heads per layer: equal column blocks of Z, a_src, a_dst
    float* w[MG_MAX_HOPS] = {nullptr};       // device [d_in, d_out]
    float* w_t[MG_MAX_HOPS] = {nullptr};     // device [d_out, d_in], rounded to TF32 for the tensor-core path
    float* a_src[MG_MAX_HOPS] = {nullptr};   // device [d_out]
    float* a_dst[MG_MAX_HOPS] = {nullptr};
    float* bias[MG_MAX_HOPS] = {nullptr};
    float* u_src[MG_MAX_HOPS] = {nullptr};   // device [d_in]: W a_src and W a_dst -- the score terms taken on the layer's
    float* u_dst[MG_MAX_HOPS] = {nullptr};   // INPUT rows (single head: Z a = (H W) a = H (W a))
    float* zeros = nullptr;                  // device [max d_out]: the GEMM's bias
};

namespace {

constexpr int kThreads = 256;
constexpr int kMaxWidthPerLane = 16;   // attention rows up to 512 wide

__device__ __forceinline__ float round_tf32(float v) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(v));
    return __uint_as_float(u);
}

__global__ void __launch_bounds__(kThreads) k_gat_transpose(const float* __restrict__ w, float* w_t, int rows, int cols, int round) {
    const int64_t n = (int64_t)rows * cols;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int r = (int)(i / cols), c = (int)(i % cols);
        const float v = w[i];
        w_t[(int64_t)c * rows + r] = round ? round_tf32(v) : v;
    }
}

struct GatGeom {
    int32_t B, k;
    const int32_t* rowbase;   // [(k + 1)][B + 1] packed first row of every mini-batch per layer
    const int32_t* cum;       // [B][k + 2] rows of a mini-batch before hop j
    const int32_t* node_off;  // [(k + 1)][B + 1]
};

// packed row of layer `layer` -> its mini-batch, its local row, its place in the hop-major node list
__device__ __forceinline__ void locate(const GatGeom& g, int layer, int64_t row, int32_t* b_out, int32_t* local_out, int32_t* node_out) {
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

struct GatherArgs {
    GatGeom g;
    const int32_t* nodes;
    const char* slots;
    FeatGeom feat;
    int64_t row_bytes, n_rows;
    int32_t dim, half, round;
    float* x;   // [n_rows, dim]
};

// H^0: the base representation of every node of every mini-batch, packed targets-first (one warp per row)
__global__ void __launch_bounds__(kThreads) k_gat_gather0(GatherArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
    for (int64_t row = blockIdx.x * (int64_t)(kThreads / 32) + (threadIdx.x >> 5); row < a.n_rows; row += warps) {
        int32_t b, local, node;
        locate(a.g, 0, row, &b, &local, &node);
        const char* src = a.slots + feat_row(a.feat, a.nodes[node]) * a.row_bytes;
        float4* dst = reinterpret_cast<float4*>(a.x + row * a.dim);   // (rows are multiples of 16 bytes on both sides)
        for (int c = lane; c < a.dim / 4; c += 32) {
            float4 v;
            if (a.half) {
                const uint2 raw = reinterpret_cast<const uint2*>(src)[c];
                const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
                const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
                v = make_float4(lo.x, lo.y, hi.x, hi.y);
            } else {
                v = reinterpret_cast<const float4*>(src)[c];
            }
            if (a.round) v = make_float4(round_tf32(v.x), round_tf32(v.y), round_tf32(v.z), round_tf32(v.w));
            dst[c] = v;
        }
    }
}

// fp32 GEMM on CUDA cores (the precision option): out[M, N] = act(x[M, K] w[K, N] + bias) (bias may be null)
__global__ void __launch_bounds__(256) k_gat_gemm_fp32(const float* __restrict__ x, const float* __restrict__ w, float* out,
                                                       int64_t M, int N, int K, const float* __restrict__ bias = nullptr, int relu = 0) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float xs[BK][BM + 4];
    __shared__ float ws[BK][BN + 4];
    const int64_t m0 = (int64_t)blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        for (int i = threadIdx.x; i < BM * BK; i += 256) {
            const int mm = i / BK, kk = i % BK;
            xs[kk][mm] = (m0 + mm < M && k0 + kk < K) ? x[(m0 + mm) * K + k0 + kk] : 0.f;
        }
        for (int i = threadIdx.x; i < BN * BK; i += 256) {
            const int kk = i / BN, nn = i % BN;
            ws[kk][nn] = (n0 + nn < N && k0 + kk < K) ? w[(int64_t)(k0 + kk) * N + n0 + nn] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float xv[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { xv[i] = xs[kk][ty * 4 + i]; wv[i] = ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xv[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= M) continue;
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < N) {
                float v = acc[i][j] + (bias ? bias[n] : 0.f);
                if (relu) v = fmaxf(v, 0.f);
                out[m * N + n] = v;
            }
        }
    }
}

// per head: s_src[row * heads + h] = Z[row] . a_src, s_dst likewise, over the head's columns [h * dh, (h + 1) * dh) (one warp per row)
__global__ void __launch_bounds__(kThreads) k_gat_scores_heads(const float* __restrict__ z, const float* __restrict__ a_src,
                                                               const float* __restrict__ a_dst, int64_t n_rows, int dim, int heads,
                                                               float* s_src, float* s_dst) {
    const int lane = threadIdx.x & 31;
    const int dh = dim / heads;
    const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
    for (int64_t row = blockIdx.x * (int64_t)(kThreads / 32) + (threadIdx.x >> 5); row < n_rows; row += warps) {
        const float* zr = z + row * dim;
        for (int h = 0; h < heads; ++h) {
            float ps = 0.f, pd = 0.f;
            for (int c = h * dh + lane; c < (h + 1) * dh; c += 32) { const float v = zr[c]; ps = fmaf(v, a_src[c], ps); pd = fmaf(v, a_dst[c], pd); }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) { ps += __shfl_xor_sync(0xFFFFFFFFu, ps, o); pd += __shfl_xor_sync(0xFFFFFFFFu, pd, o); }
            if (lane == 0) { s_src[row * heads + h] = ps; s_dst[row * heads + h] = pd; }
        }
    }
}

struct AttendArgs {
    GatGeom g;
    int32_t layer;              // 1 .. k
    const int32_t* ent_off;
    const int32_t* ent_repr;
    const float* z;             // [rows of layer - 1, dim]
    const float* s_src;
    const float* s_dst;
    const float* bias;
    int64_t n_rows;             // rows of this layer
    int32_t dim, relu, round;
    float slope;
    float* out;                 // [n_rows, dim]
    int32_t heads;              // > 1: s_src / s_dst hold `heads` values per row (k_gat_attend_heads)
};

__device__ __forceinline__ float leaky(float v, float slope) { return v > 0.f ? v : slope * v; }

// Single head, attention taken in the layer's input space.  Z a = (H W) a = H (W a): the two score terms of a row are
// dot products of its INPUT row with u_src = W a_src and u_dst = W a_dst, and sum_j alpha_ij Z_j = (sum_j alpha_ij H_j) W:
// one warp per OUTPUT row reads the row's own input row and its entries' input rows once each (layer 1: straight from
// the partition buffer), keeps a running softmax (maximum, denominator, weighted sum, rescaled when the maximum
// grows) and stores the attention-weighted input row; the linear map then runs over the output rows only.  Nothing of
// the width of Z exists for the input rows, and no H^0 copy.
struct InAttendArgs {
    GatGeom g;
    int32_t layer;              // 1 .. k
    const int32_t* nodes;
    const int32_t* ent_off;
    const int32_t* ent_nbrs;    // layer 1: the entries' node ids
    const int32_t* ent_repr;    // later layers: the entries' local rows of layer - 1
    const char* slots; FeatGeom feat; int64_t row_bytes;   // layer 1
    const float* h_prev;        // later layers: [rows of layer - 1, dim]
    const float* u_src; const float* u_dst;   // [dim]
    int64_t n_rows;             // rows of this layer
    int32_t dim, round;
    float slope;
    float* x;                   // [n_rows, dim]
};

template <bool FIRST, bool HALF, int NCH>   // a lane owns NCH groups of four columns: rows up to 128 NCH wide
__global__ void __launch_bounds__(kThreads) k_gat_attend_inputs(InAttendArgs a) {
    constexpr int U = NCH == 1 ? 4 : (NCH == 2 ? 2 : 1);   // entries whose rows are in flight together
    const int lane = threadIdx.x & 31;
    const int n4 = a.dim / 4;
    const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
    const int32_t* rb_in = a.g.rowbase + (int64_t)(a.layer - 1) * (a.g.B + 1);
    float4 us[NCH], ud[NCH];
#pragma unroll
    for (int q = 0; q < NCH; ++q) {
        const int c = lane + 32 * q;
        us[q] = c < n4 ? reinterpret_cast<const float4*>(a.u_src)[c] : make_float4(0.f, 0.f, 0.f, 0.f);
        ud[q] = c < n4 ? reinterpret_cast<const float4*>(a.u_dst)[c] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    auto load_row = [&](const char* p, float4* v) {
#pragma unroll
        for (int q = 0; q < NCH; ++q) {
            const int c = lane + 32 * q;
            if (c >= n4) { v[q] = make_float4(0.f, 0.f, 0.f, 0.f); continue; }
            if (HALF) {
                const uint2 raw = reinterpret_cast<const uint2*>(p)[c];
                const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
                const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
                v[q] = make_float4(lo.x, lo.y, hi.x, hi.y);
            } else {
                v[q] = reinterpret_cast<const float4*>(p)[c];
            }
        }
    };
    auto dot = [&](const float4* v, const float4* u) {
        float s = 0.f;
#pragma unroll
        for (int q = 0; q < NCH; ++q) s += v[q].x * u[q].x + v[q].y * u[q].y + v[q].z * u[q].z + v[q].w * u[q].w;
        return s;
    };
    for (int64_t row = blockIdx.x * (int64_t)(kThreads / 32) + (threadIdx.x >> 5); row < a.n_rows; row += warps) {
        int32_t b, local, node;
        locate(a.g, a.layer, row, &b, &local, &node);
        const int64_t in0 = rb_in[b];
        auto row_of = [&](bool self, int32_t e) -> const char* {
            if (FIRST) return a.slots + feat_row(a.feat, self ? a.nodes[node] : a.ent_nbrs[e]) * a.row_bytes;
            return reinterpret_cast<const char*>(a.h_prev + (in0 + (self ? local : a.ent_repr[e])) * a.dim);
        };
        const int32_t e0 = a.ent_off[node], e1 = a.ent_off[node + 1];
        float4 acc[NCH];
        load_row(row_of(true, 0), acc);
        float ss = dot(acc, us), sd = dot(acc, ud);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o); sd += __shfl_xor_sync(0xFFFFFFFFu, sd, o); }
        float mx = leaky(sd + ss, a.slope), den = 1.f;   // the row itself: weight exp(0) so far
        for (int32_t e = e0; e < e1; e += U) {
            float4 v[U][NCH];
            float s[U];
#pragma unroll
            for (int u = 0; u < U; ++u) load_row(row_of(false, min(e + u, e1 - 1)), v[u]);
#pragma unroll
            for (int u = 0; u < U; ++u) s[u] = dot(v[u], us);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int u = 0; u < U; ++u) s[u] += __shfl_xor_sync(0xFFFFFFFFu, s[u], o);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (e + u >= e1) continue;
                const float logit = leaky(sd + s[u], a.slope);
                const float m_new = fmaxf(mx, logit);
                const float keep = __expf(mx - m_new), w = __expf(logit - m_new);
                den = den * keep + w;
#pragma unroll
                for (int q = 0; q < NCH; ++q) {
                    acc[q].x = acc[q].x * keep + w * v[u][q].x; acc[q].y = acc[q].y * keep + w * v[u][q].y;
                    acc[q].z = acc[q].z * keep + w * v[u][q].z; acc[q].w = acc[q].w * keep + w * v[u][q].w;
                }
                mx = m_new;
            }
        }
        const float inv = 1.f / den;
#pragma unroll
        for (int q = 0; q < NCH; ++q) {
            const int c = lane + 32 * q;
            if (c >= n4) continue;
            float4 o = make_float4(acc[q].x * inv, acc[q].y * inv, acc[q].z * inv, acc[q].w * inv);
            if (a.round) o = make_float4(round_tf32(o.x), round_tf32(o.y), round_tf32(o.z), round_tf32(o.w));
            reinterpret_cast<float4*>(a.x + row * a.dim)[c] = o;
        }
    }
}

template <bool FIRST, bool HALF>
void launch_attend_inputs(const InAttendArgs& a, int grid, cudaStream_t st) {
    const int nch = (a.dim + 127) / 128;
    if (nch <= 1) k_gat_attend_inputs<FIRST, HALF, 1><<<grid, kThreads, 0, st>>>(a);
    else if (nch <= 2) k_gat_attend_inputs<FIRST, HALF, 2><<<grid, kThreads, 0, st>>>(a);
    else if (nch <= 4) k_gat_attend_inputs<FIRST, HALF, 4><<<grid, kThreads, 0, st>>>(a);
    else k_gat_attend_inputs<FIRST, HALF, 8><<<grid, kThreads, 0, st>>>(a);
}

constexpr int kMaxHeads = 8;

// several heads: one warp per output row; per head a softmax over {self} + entries with that head's scores, then the
// weighted sums of the Z rows, every column with the weights of the head it belongs to
template <int W>
__global__ void __launch_bounds__(kThreads) k_gat_attend_heads(AttendArgs a) {
    const int lane = threadIdx.x & 31;
    const int H = a.heads, dh = a.dim / a.heads;
    const int64_t warps = (int64_t)gridDim.x * (kThreads / 32);
    const int32_t* rb_in = a.g.rowbase + (int64_t)(a.layer - 1) * (a.g.B + 1);
    int head_of[W];
#pragma unroll
    for (int q = 0; q < W; ++q) head_of[q] = min((lane + 32 * q) / dh, H - 1);
    for (int64_t row = blockIdx.x * (int64_t)(kThreads / 32) + (threadIdx.x >> 5); row < a.n_rows; row += warps) {
        int32_t b, local, node;
        locate(a.g, a.layer, row, &b, &local, &node);
        const int64_t in0 = rb_in[b];
        const int64_t me = in0 + local;
        const int32_t e0 = a.ent_off[node], e1 = a.ent_off[node + 1];
        float sd[kMaxHeads], mx[kMaxHeads], inv[kMaxHeads];
        for (int h = 0; h < H; ++h) {
            sd[h] = a.s_dst[me * H + h];
            const float self_score = leaky(sd[h] + a.s_src[me * H + h], a.slope);
            float m = self_score;
            for (int32_t e = e0 + lane; e < e1; e += 32) m = fmaxf(m, leaky(sd[h] + a.s_src[(in0 + a.ent_repr[e]) * H + h], a.slope));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            float den = lane == 0 ? __expf(self_score - m) : 0.f;
            for (int32_t e = e0 + lane; e < e1; e += 32) den += __expf(leaky(sd[h] + a.s_src[(in0 + a.ent_repr[e]) * H + h], a.slope) - m);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xFFFFFFFFu, den, o);
            mx[h] = m;
            inv[h] = 1.f / den;
        }
        float acc[W];
        {
            const float* zr = a.z + me * a.dim;
#pragma unroll
            for (int q = 0; q < W; ++q) {
                const int c = lane + 32 * q, h = head_of[q];
                acc[q] = c < a.dim ? __expf(leaky(sd[h] + a.s_src[me * H + h], a.slope) - mx[h]) * inv[h] * zr[c] : 0.f;
            }
        }
        for (int32_t e = e0; e < e1; ++e) {
            const int64_t src = in0 + a.ent_repr[e];
            const float* zr = a.z + src * a.dim;
#pragma unroll
            for (int q = 0; q < W; ++q) {
                const int c = lane + 32 * q, h = head_of[q];
                if (c < a.dim) acc[q] = fmaf(__expf(leaky(sd[h] + a.s_src[src * H + h], a.slope) - mx[h]) * inv[h], zr[c], acc[q]);
            }
        }
        float* dst = a.out + row * a.dim;
#pragma unroll
        for (int q = 0; q < W; ++q) {
            const int c = lane + 32 * q;
            if (c >= a.dim) continue;
            float v = acc[q] + a.bias[c];
            if (a.relu) v = fmaxf(v, 0.f);
            dst[c] = a.round ? round_tf32(v) : v;
        }
    }
}

}  // namespace

extern "C" int mg_gat_model_set_heads(mg_gat_model* m, int32_t heads) {
    if (!m) return MG_ERR_ARG;
    if (heads < 1 || heads > kMaxHeads) return mg_fail(m->ctx, MG_ERR_ARG, "heads must be in [1, %d]", kMaxHeads);
    for (int l = 1; l <= m->k; ++l)
        if (m->dims[l] % heads) return mg_fail(m->ctx, MG_ERR_ARG, "layer width %d is not a multiple of %d heads", m->dims[l], heads);
    m->heads = heads;
    return MG_OK;
}

extern "C" int mg_gat_model_free(mg_gat_model* m) {
    if (!m) return MG_OK;
    cudaSetDevice(m->device);
    for (int l = 0; l < MG_MAX_HOPS; ++l) {
        cudaFree(m->w[l]); cudaFree(m->w_t[l]); cudaFree(m->a_src[l]); cudaFree(m->a_dst[l]); cudaFree(m->bias[l]);
        cudaFree(m->u_src[l]); cudaFree(m->u_dst[l]);
    }
    cudaFree(m->zeros);
    delete m;
    return MG_OK;
}

extern "C" int mg_gat_model_create(mg_ctx* ctx, int32_t k, const int32_t* dims, const float* const* w, const float* const* a_src,
                                   const float* const* a_dst, const float* const* bias, float negative_slope, int gemm_precision,
                                   mg_gat_model** out) {
    if (!ctx) return MG_ERR_ARG;
    if (!out || !dims || !w || !a_src || !a_dst || !bias) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (k <= 0 || k > MG_MAX_HOPS) return mg_fail(ctx, MG_ERR_ARG, "k must be in [1, %d]", MG_MAX_HOPS);
    if (gemm_precision != MG_GEMM_TF32 && gemm_precision != MG_GEMM_FP32) return mg_fail(ctx, MG_ERR_ARG, "unknown gemm precision");
    if (!(negative_slope >= 0.f && negative_slope <= 1.f)) return mg_fail(ctx, MG_ERR_ARG, "negative_slope must be in [0, 1]");
    for (int l = 0; l <= k; ++l)
        if (dims[l] <= 0 || dims[l] % 4 != 0 || dims[l] > 1024) return mg_fail(ctx, MG_ERR_ARG, "layer widths must be multiples of 4 in [4, 1024]");
    for (int l = 1; l <= k; ++l)
        if (dims[l] > 32 * kMaxWidthPerLane) return mg_fail(ctx, MG_ERR_ARG, "attention layers are at most %d wide", 32 * kMaxWidthPerLane);
    for (int l = 0; l < k; ++l)
        if (!w[l] || !a_src[l] || !a_dst[l] || !bias[l]) return mg_fail(ctx, MG_ERR_ARG, "null weight pointer");
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    mg_gat_model* m = new mg_gat_model();
    m->ctx = ctx; m->device = ctx->device; m->k = k; m->precision = gemm_precision; m->slope = negative_slope;
    for (int l = 0; l <= k; ++l) m->dims[l] = dims[l];
    int widest = 4;
    for (int l = 1; l <= k; ++l) widest = std::max(widest, dims[l]);
    bool ok = cudaMalloc((void**)&m->zeros, sizeof(float) * widest) == cudaSuccess &&
              cudaMemsetAsync(m->zeros, 0, sizeof(float) * widest, ctx->stream) == cudaSuccess;
    for (int l = 0; l < k && ok; ++l) {
        const size_t di = dims[l], dn = dims[l + 1];
        ok = cudaMalloc((void**)&m->w[l], sizeof(float) * di * dn) == cudaSuccess &&
             cudaMalloc((void**)&m->w_t[l], sizeof(float) * di * dn) == cudaSuccess &&
             cudaMalloc((void**)&m->a_src[l], sizeof(float) * dn) == cudaSuccess &&
             cudaMalloc((void**)&m->a_dst[l], sizeof(float) * dn) == cudaSuccess &&
             cudaMalloc((void**)&m->bias[l], sizeof(float) * dn) == cudaSuccess;
        if (!ok) break;
        cudaMemcpyAsync(m->w[l], w[l], sizeof(float) * di * dn, cudaMemcpyHostToDevice, ctx->stream);
        cudaMemcpyAsync(m->a_src[l], a_src[l], sizeof(float) * dn, cudaMemcpyHostToDevice, ctx->stream);
        cudaMemcpyAsync(m->a_dst[l], a_dst[l], sizeof(float) * dn, cudaMemcpyHostToDevice, ctx->stream);
        cudaMemcpyAsync(m->bias[l], bias[l], sizeof(float) * dn, cudaMemcpyHostToDevice, ctx->stream);
        k_gat_transpose<<<mg_grid(ctx, 2), kThreads, 0, ctx->stream>>>(m->w[l], m->w_t[l], (int)di, (int)dn, gemm_precision == MG_GEMM_TF32);
        ctx->launches++;
        // W a_src and W a_dst (double sums, rounded once): the score terms on the layer's input rows
        std::vector<float> us(di), ud(di);
        for (size_t r = 0; r < di; ++r) {
            double s1 = 0.0, s2 = 0.0;
            for (size_t c = 0; c < dn; ++c) { s1 += (double)w[l][r * dn + c] * a_src[l][c]; s2 += (double)w[l][r * dn + c] * a_dst[l][c]; }
            us[r] = (float)s1; ud[r] = (float)s2;
        }
        ok = cudaMalloc((void**)&m->u_src[l], sizeof(float) * di) == cudaSuccess &&
             cudaMalloc((void**)&m->u_dst[l], sizeof(float) * di) == cudaSuccess &&
             cudaMemcpy(m->u_src[l], us.data(), sizeof(float) * di, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(m->u_dst[l], ud.data(), sizeof(float) * di, cudaMemcpyHostToDevice) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        mg_gat_model_free(m);
        return mg_fail(ctx, MG_ERR_OOM, "weight allocation failed");
    }
    cudaError_t e = cudaStreamSynchronize(ctx->stream);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) { mg_gat_model_free(m); return mg_cuda_fail(ctx, e, "weight upload"); }
    *out = m;
    return MG_OK;
}

extern "C" int mg_gat_forward(mg_ctx* ctx, const mg_gat_model* m, mg_dense* d, float* out_dev) {
    if (!ctx) return MG_ERR_ARG;
    if (!m || !d || !out_dev) return mg_fail(ctx, MG_ERR_ARG, "null argument");
    if (d->pending) return mg_fail(ctx, MG_ERR_STATE, "a sample is in flight on this mg_dense: call mg_sample_many_end first");
    if (!d->valid) return mg_fail(ctx, MG_ERR_STATE, "mg_dense holds no completed sample");
    if (d->ctx != ctx || m->ctx != ctx) return mg_fail(ctx, MG_ERR_ARG, "handle belongs to another context");
    if (!ctx->slots || ctx->feat_dim <= 0) return mg_fail(ctx, MG_ERR_STATE, "no feature table loaded");
    if (m->k != d->k) return mg_fail(ctx, MG_ERR_STATE, "model has %d layers, sample has %d hops", m->k, d->k);
    if (m->dims[0] != ctx->feat_dim) return mg_fail(ctx, MG_ERR_STATE, "model input width %d != feature dim %d", m->dims[0], ctx->feat_dim);
    if (int rs = mg_check_sample_residency(ctx, d)) return rs;
    MG_CUDA(ctx, cudaSetDevice(ctx->device));
    const int k = d->k, B = d->n_batches;
    cudaStream_t st = ctx->stream;
    const bool tf32 = m->precision == MG_GEMM_TF32;
    int rc;
    // (a quarter of headroom when a buffer grows: calls of slightly different sizes then share it)
    auto grow = [&](float** p, size_t* have, size_t need) { return *have >= need && *p ? MG_OK : mg_ensure(ctx, p, have, need + need / 4 + 16); };
    const GatGeom geom{B, k, d->rowbase, d->cum, d->node_off};
    const int grid = mg_grid(ctx, 8);
    if (m->heads == 1) {
        // single head: attention on the input rows, then the linear map over the output rows (k_gat_attend_inputs)
        size_t need_x = 0, need_h = 0;
        for (int l = 1; l <= k; ++l) {
            need_x = std::max(need_x, (size_t)d->h_hdr.rows_total[l] * m->dims[l - 1]);
            if (l < k) need_h = std::max(need_h, (size_t)d->h_hdr.rows_total[l] * m->dims[l]);
        }
        if ((rc = grow(&ctx->gat_x, &ctx->gat_x_elems, need_x))) return rc;
        for (int i = 0; i < 2; ++i)
            if ((rc = grow(&ctx->gat_h[i], &ctx->gat_h_elems[i], need_h))) return rc;
        if (d->h_hdr.rows_total[k] == 0) return MG_OK;
        const float* h_in = nullptr;
        for (int l = 1; l <= k; ++l) {
            const int d_in = m->dims[l - 1], d_out = m->dims[l];
            const int64_t rows_out = d->h_hdr.rows_total[l];
            {
                ProfScope ps(ctx, l == 1 ? PH_AGG_L1 : PH_AGG_REST, 1);
                InAttendArgs a;
                a.g = geom; a.layer = l; a.nodes = d->nodes; a.ent_off = d->ent_off; a.ent_nbrs = d->ent_nbrs; a.ent_repr = d->ent_repr;
                a.slots = ctx->slots; a.feat = mg_feat_geom(ctx); a.row_bytes = ctx->row_bytes; a.h_prev = h_in;
                a.u_src = m->u_src[l - 1]; a.u_dst = m->u_dst[l - 1]; a.n_rows = rows_out; a.dim = d_in; a.round = tf32 ? 1 : 0;
                a.slope = m->slope; a.x = ctx->gat_x;
                if (l == 1) {
                    if (ctx->feat_dtype == MG_DTYPE_F16) launch_attend_inputs<true, true>(a, grid, st);
                    else launch_attend_inputs<true, false>(a, grid, st);
                } else {
                    launch_attend_inputs<false, false>(a, grid, st);
                }
                ctx->launches++;
            }
            float* out_l = l == k ? out_dev : ctx->gat_h[l & 1];
            {
                ProfScope ps(ctx, PH_GEMM, 1);
                if (tf32) {
                    if ((rc = mg_gemm_tf32(ctx, ctx->gat_x, m->w_t[l - 1], m->bias[l - 1], out_l, rows_out, d_out, d_in, l < k))) return rc;
                } else {
                    dim3 g2((unsigned)((rows_out + 63) / 64), (unsigned)((d_out + 63) / 64));
                    k_gat_gemm_fp32<<<g2, 256, 0, st>>>(ctx->gat_x, m->w[l - 1], out_l, rows_out, d_out, d_in, m->bias[l - 1], l < k ? 1 : 0);
                    ctx->launches++;
                }
            }
            h_in = out_l;
        }
        MG_CUDA(ctx, cudaGetLastError());
        MG_CUDA(ctx, cudaStreamSynchronize(st));
        return tf32 ? mg_gemm_tf32_status(ctx) : MG_OK;
    }
    // several heads: Z = H W for the input rows, per-head scores, attention over Z
    // scratch: H^0, Z and the two score vectors of the widest layer, two buffers for the layer outputs
    size_t need_x = (size_t)d->h_hdr.rows_total[0] * m->dims[0], need_z = 0, need_s = 0, need_h = 0;
    for (int l = 1; l <= k; ++l) {
        need_z = std::max(need_z, (size_t)d->h_hdr.rows_total[l - 1] * m->dims[l]);
        need_s = std::max(need_s, (size_t)d->h_hdr.rows_total[l - 1] * 2 * m->heads);
        if (l < k) need_h = std::max(need_h, (size_t)d->h_hdr.rows_total[l] * m->dims[l]);
    }
    if ((rc = grow(&ctx->gat_x, &ctx->gat_x_elems, need_x))) return rc;
    if ((rc = grow(&ctx->gat_z, &ctx->gat_z_elems, need_z))) return rc;
    if ((rc = grow(&ctx->gat_s, &ctx->gat_s_elems, need_s))) return rc;
    for (int i = 0; i < 2; ++i)
        if ((rc = grow(&ctx->gat_h[i], &ctx->gat_h_elems[i], need_h))) return rc;
    if (d->h_hdr.rows_total[k] == 0) return MG_OK;
    {
        ProfScope ps(ctx, PH_AGG_L1, 1);
        GatherArgs a;
        a.g = geom; a.nodes = d->nodes; a.slots = ctx->slots; a.feat = mg_feat_geom(ctx);
        a.row_bytes = ctx->row_bytes; a.n_rows = d->h_hdr.rows_total[0];
        a.dim = m->dims[0]; a.half = ctx->feat_dtype == MG_DTYPE_F16; a.round = tf32;
        a.x = ctx->gat_x;
        k_gat_gather0<<<grid, kThreads, 0, st>>>(a);
        ctx->launches++;
    }
    const float* h_prev = ctx->gat_x;
    for (int l = 1; l <= k; ++l) {
        const int d_in = m->dims[l - 1], d_out = m->dims[l];
        const int64_t rows_in = d->h_hdr.rows_total[l - 1], rows_out = d->h_hdr.rows_total[l];
        float* s_src = ctx->gat_s;
        const int H = m->heads;
        float* s_dst = ctx->gat_s + rows_in * H;
        {
            ProfScope ps(ctx, PH_GEMM, 1);
            if (tf32) {
                if ((rc = mg_gemm_tf32(ctx, h_prev, m->w_t[l - 1], m->zeros, ctx->gat_z, rows_in, d_out, d_in, false))) return rc;
            } else {
                dim3 g2((unsigned)((rows_in + 63) / 64), (unsigned)((d_out + 63) / 64));
                k_gat_gemm_fp32<<<g2, 256, 0, st>>>(h_prev, m->w[l - 1], ctx->gat_z, rows_in, d_out, d_in);
                ctx->launches++;
            }
        }
        ProfScope ps(ctx, PH_AGG_REST, 2);
        k_gat_scores_heads<<<grid, kThreads, 0, st>>>(ctx->gat_z, m->a_src[l - 1], m->a_dst[l - 1], rows_in, d_out, H, s_src, s_dst);
        AttendArgs a;
        a.g = geom; a.layer = l; a.ent_off = d->ent_off; a.ent_repr = d->ent_repr; a.z = ctx->gat_z; a.s_src = s_src; a.s_dst = s_dst;
        a.bias = m->bias[l - 1]; a.n_rows = rows_out; a.dim = d_out; a.relu = l < k; a.round = (tf32 && l < k) ? 1 : 0;
        a.slope = m->slope;
        a.heads = H;
        a.out = l == k ? out_dev : ctx->gat_h[l & 1];
        const int slices = (d_out + 31) / 32;   // instantiations for rows of up to 32, 64, 128, 256, 512 floats
        if (slices <= 1) k_gat_attend_heads<1><<<grid, kThreads, 0, st>>>(a);
        else if (slices <= 2) k_gat_attend_heads<2><<<grid, kThreads, 0, st>>>(a);
        else if (slices <= 4) k_gat_attend_heads<4><<<grid, kThreads, 0, st>>>(a);
        else if (slices <= 8) k_gat_attend_heads<8><<<grid, kThreads, 0, st>>>(a);
        else k_gat_attend_heads<kMaxWidthPerLane><<<grid, kThreads, 0, st>>>(a);
        ctx->launches += 2;
        h_prev = a.out;
    }
    MG_CUDA(ctx, cudaGetLastError());
    MG_CUDA(ctx, cudaStreamSynchronize(st));
    return tf32 ? mg_gemm_tf32_status(ctx) : MG_OK;
}
