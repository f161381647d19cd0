// Context, graph store and partition buffer (Section 3): CSR in device memory, the resident
// set with its partition -> slot map, host-backed feature slots filled on a side stream, and
// the in-buffer view of the graph that sampling reads.

#include <stdarg.h>

#include <algorithm>
#include <chrono>
#include <thread>

#include "mg_device.cuh"
#include "mg_internal.cuh"

static const char* kPhaseNames[PH_COUNT] = {
    "sample_init", "sample_count", "sample_scan", "sample_pick", "sample_sort", "sample_place",
    "sample_relabel", "sample_final", "aggregate_l1", "aggregate_rest", "gemm", "distmult", "other"};

int mg_fail(mg_ctx* ctx, int code, const char* fmt, ...) {
    if (ctx) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof(buf), fmt, ap);
        va_end(ap);
        ctx->err = buf;
    }
    return code;
}

int mg_cuda_fail(mg_ctx* ctx, cudaError_t e, const char* what) {
    cudaGetLastError();
    const int code = (e == cudaErrorMemoryAllocation) ? MG_ERR_OOM : MG_ERR_CUDA;
    return mg_fail(ctx, code, "%s: %s", what, cudaGetErrorString(e));
}

int mg_check_sample_residency(mg_ctx* ctx, const mg_dense* d) {
    if (d->resident_serial == ctx->resident_serial) return MG_OK;
    const std::vector<int32_t>& then = d->slot_of_part_at_sample;
    bool ok = then.size() == ctx->slot_of_part.size();
    for (size_t p = 0; ok && p < then.size(); ++p) ok = then[p] < 0 || then[p] == ctx->slot_of_part[p];
    if (ok) return MG_OK;
    return mg_fail(ctx, MG_ERR_STATE, "the resident set changed since this sample was drawn: a partition it uses was evicted or moved; sample again");
}

void mg_prof_begin(mg_ctx* ctx, int phase) {
    if (!ctx->prof_on) return;
    cudaEvent_t a, b;
    cudaEventCreate(&a);
    cudaEventCreate(&b);
    cudaEventRecord(a, ctx->stream);
    ctx->prof_pending.push_back({phase, {a, b}});
}

void mg_prof_end(mg_ctx* ctx, int phase, int n_launches) {
    if (!ctx->prof_on) return;
    for (size_t i = ctx->prof_pending.size(); i-- > 0;) {
        if (ctx->prof_pending[i].first == phase) {
            cudaEventRecord(ctx->prof_pending[i].second.second, ctx->stream);
            break;
        }
    }
    ctx->prof[phase].launches += n_launches;
}

namespace {

constexpr int kThreads = 256;

__global__ void k_widen_offsets(const int32_t* in, int64_t* out, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = in[i];
}

// checks that offsets are non-decreasing and neighbour ids are in range; flags[0] |= 1 / 2
__global__ void k_check_graph(const int64_t* off, int64_t n_nodes, const int32_t* nbrs, int64_t n_edges, uint32_t* flags) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    for (int64_t i = tid; i < n_nodes; i += stride)
        if (off[i + 1] < off[i]) atomicOr(flags, 1u);
    for (int64_t e = tid; e < n_edges; e += stride)
        if (nbrs[e] < 0 || (int64_t)nbrs[e] >= n_nodes) atomicOr(flags, 2u);
}

// ---- in-buffer view: rows of resident nodes restricted to resident neighbours -------------
// Edge-parallel, so that a hub's million-entry row costs what a million short rows cost.  Partitions are contiguous id
// ranges and rows are stored in id order, so the rows of a partition are one contiguous range of edges: an edge stays
// when its position lies in a resident partition's range and its neighbour's partition is resident.
//   k_view_mask     per tile of 2048 edges: a keep bit per edge (32 per word), the number of kept edges before each
//                   word inside the tile, the tile's count
//   (64-bit scan of the tile counts)
//   k_view_compact  kept edges to their places, in order
//   k_view_offsets  a row's new offset = the number of kept edges before its first edge (tile base + word prefix +
//                   population count of the word's lower bits)
constexpr int kViewTile = 2048;   // edges per tile: 256 threads x 8

struct ViewArgs {
    const int64_t* off;
    const int32_t* nbrs;
    int64_t n_nodes, n_edges;
    uint32_t part_size;
    int32_t n_parts;
    const int32_t* slot_of_part;
    const uint8_t* part_of_node;   // null: partitions are contiguous id ranges
    uint32_t* mask;        // [ceil(E / 32)]
    uint16_t* word_before; // [ceil(E / 32)] kept edges of the tile before the word
    int32_t* tile_cnt;     // [tiles]
    const int64_t* tile_base;  // [tiles + 1]
};

// first edge of partition p's rows
__device__ __forceinline__ int64_t part_edge_lo(const ViewArgs& a, int p) {
    const int64_t v = (int64_t)p * a.part_size;
    return a.off[v < a.n_nodes ? v : a.n_nodes];
}
// With a partition-id array the rows of a partition are not one range of edges.  The view then keeps every edge whose
// NEIGHBOUR is resident, whatever its row: sampling only ever reads the rows of resident nodes (targets are checked,
// neighbours were filtered), so the rows of the others are dead weight in the view, not an error.

__global__ void __launch_bounds__(kThreads) k_view_mask(ViewArgs a) {
    __shared__ int64_t bound[MG_MAX_PARTS + 1];
    __shared__ int32_t res[MG_MAX_PARTS];
    __shared__ uint32_t warp_tot[kThreads / 32];
    const bool ranges = a.part_of_node == nullptr;
    for (int p = threadIdx.x; p <= a.n_parts; p += kThreads) bound[p] = ranges ? part_edge_lo(a, p) : (p == 0 ? 0 : a.n_edges);
    for (int p = threadIdx.x; p < a.n_parts; p += kThreads) res[p] = a.slot_of_part[p] >= 0 ? 1 : 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t n_tiles = (a.n_edges + kViewTile - 1) / kViewTile;
    for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int64_t e0 = t * kViewTile + (int64_t)threadIdx.x * 8;
        // partition whose edge range holds e0 (ranges of empty partitions are empty and skipped)
        int p = 0;
        {
            int lo = 0, hi = a.n_parts;   // bound[lo] <= e0 < bound[hi] (bound[n_parts] = E)
            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (bound[mid] <= e0) lo = mid; else hi = mid; }
            p = lo;
        }
        uint32_t bits = 0;
        const bool any_row = e0 < a.n_edges && (!ranges || res[p] || bound[p + 1] < e0 + 8);   // (a thread's 8 edges may cross into a resident range)
        if (any_row) {
            int32_t u[8];
            if (e0 + 8 <= a.n_edges) {
                const int4 x = __ldg(reinterpret_cast<const int4*>(a.nbrs + e0)), y = __ldg(reinterpret_cast<const int4*>(a.nbrs + e0 + 4));
                u[0] = x.x; u[1] = x.y; u[2] = x.z; u[3] = x.w; u[4] = y.x; u[5] = y.y; u[6] = y.z; u[7] = y.w;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] = e0 + j < a.n_edges ? a.nbrs[e0 + j] : 0;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t e = e0 + j;
                if (ranges) {
                    while (p + 1 < a.n_parts && e >= bound[p + 1]) ++p;
                    if (e < a.n_edges && res[p] && res[(uint32_t)u[j] / a.part_size]) bits |= 1u << j;
                } else if (e < a.n_edges && res[a.part_of_node[u[j]]]) {
                    bits |= 1u << j;
                }
            }
        }
        // four lanes make a word; counts: exclusive scan over the block's 256 threads
        uint32_t word = bits << (8 * (lane & 3));
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
        const uint32_t mine = __popc(bits);
        const uint32_t inc = warp_incl_scan(mine);
        if (lane == 31) warp_tot[warp] = inc;
        __syncthreads();
        uint32_t before = inc - mine;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if ((lane & 3) == 0 && e0 < a.n_edges) {
            a.mask[e0 >> 5] = word;
            a.word_before[e0 >> 5] = (uint16_t)before;
        }
        if (threadIdx.x == kThreads - 1) a.tile_cnt[t] = (int32_t)(before + mine);
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kThreads) k_view_compact(ViewArgs a, int32_t* view_nbrs) {
    const int lane = threadIdx.x & 31;
    const int64_t n_tiles = (a.n_edges + kViewTile - 1) / kViewTile;
    for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const int64_t base = a.tile_base[t];
        if (a.tile_base[t + 1] == base) continue;             // nothing of this tile stays: its edges are not even read
        const int64_t e0 = t * kViewTile + (int64_t)threadIdx.x * 8;
        if (e0 >= a.n_edges) continue;
        const uint32_t word = a.mask[e0 >> 5];
        const uint32_t bits = (word >> (8 * (lane & 3))) & 0xFFu;
        if (!bits) continue;
        int64_t out = base + a.word_before[e0 >> 5] + __popc(word & ((1u << (8 * (lane & 3))) - 1u));
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (bits & (1u << j)) view_nbrs[out++] = a.nbrs[e0 + j];
    }
}

__global__ void __launch_bounds__(kThreads) k_view_offsets(ViewArgs a, int64_t* view_off) {
    const int64_t n_tiles = (a.n_edges + kViewTile - 1) / kViewTile;
    for (int64_t v = blockIdx.x * (int64_t)kThreads + threadIdx.x; v <= a.n_nodes; v += (int64_t)gridDim.x * kThreads) {
        const int64_t e = a.off[v];
        int64_t r;
        if (e >= a.n_edges) r = a.tile_base[n_tiles];
        else r = a.tile_base[e / kViewTile] + a.word_before[e >> 5] + __popc(a.mask[e >> 5] & ((1u << (e & 31)) - 1u));
        view_off[v] = r;
    }
}

// ---- 64-bit exclusive scan of int32 counts: out[i] = sum_{j<i} in[j], i in [0, n] ----------
constexpr int kTile = 2048;

__device__ __forceinline__ uint64_t block_scan64(uint64_t v, uint64_t* sm /*9*/, uint64_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint64_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint64_t t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) sm[warp] = inc;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint64_t run = 0;
        for (int w = 0; w < 8; ++w) { const uint64_t t = sm[w]; sm[w] = run; run += t; }
        sm[8] = run;
    }
    __syncthreads();
    const uint64_t res = inc - v + sm[warp];
    *total = sm[8];
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(kThreads) k_scan64_reduce(const int32_t* in, int64_t n, uint64_t* tile_sums) {
    __shared__ uint64_t sm[9];
    const int64_t ntiles = (n + kTile - 1) / kTile;
    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        uint64_t s = 0;
        const int64_t start = t * kTile + threadIdx.x * 8;
        for (int j = 0; j < 8; ++j)
            if (start + j < n) s += (uint64_t)in[start + j];
        uint64_t total;
        block_scan64(s, sm, &total);
        if (threadIdx.x == 0) tile_sums[t] = total;
    }
}

__global__ void k_scan64_tiles(uint64_t* tile_sums, int64_t ntiles, int64_t* total_out) {
    // one thread block, sequential over chunks; ntiles is at most a few 10^4
    __shared__ uint64_t sm[9];
    __shared__ uint64_t carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int64_t start = 0; start < ntiles; start += kThreads) {
        const int64_t i = start + threadIdx.x;
        const uint64_t v = i < ntiles ? tile_sums[i] : 0ull;
        uint64_t total;
        const uint64_t ex = block_scan64(v, sm, &total);
        if (i < ntiles) tile_sums[i] = carry_s + ex;
        __syncthreads();
        if (threadIdx.x == 0) carry_s += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) *total_out = (int64_t)carry_s;
}

__global__ void __launch_bounds__(kThreads)
k_scan64_down(const int32_t* in, int64_t n, const uint64_t* tile_sums, int64_t* out) {
    __shared__ uint64_t sm[9];
    const int64_t ntiles = (n + kTile - 1) / kTile;
    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        uint32_t v[8];
        uint64_t s = 0;
        const int64_t start = t * kTile + threadIdx.x * 8;
        for (int j = 0; j < 8; ++j) { v[j] = (start + j < n) ? (uint32_t)in[start + j] : 0u; s += v[j]; }
        uint64_t total;
        uint64_t run = block_scan64(s, sm, &total) + tile_sums[t];
        for (int j = 0; j < 8; ++j) {
            if (start + j < n) out[start + j] = (int64_t)run;
            run += v[j];
        }
        if (t == ntiles - 1 && threadIdx.x == kThreads - 1) out[n] = (int64_t)(tile_sums[t] + total);
    }
}

}  // namespace

// ---------------------------------------------------------------------------------------
extern "C" int mg_create(mg_ctx** out, int device, void* stream) {
    if (!out) return MG_ERR_ARG;
    *out = nullptr;
    int n_dev = 0;
    cudaError_t e = cudaGetDeviceCount(&n_dev);
    if (e != cudaSuccess || device < 0 || device >= n_dev) { cudaGetLastError(); return MG_ERR_CUDA; }
    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return MG_ERR_CUDA; }
    mg_ctx* c = new mg_ctx();
    c->device = device;
    c->stream = (cudaStream_t)stream;
    cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, device);
    if (c->n_sms <= 0) c->n_sms = 148;
    for (int i = 0; i < PH_COUNT; ++i) c->prof[i] = ProfPhase{kPhaseNames[i], 0.0, 0};
    // the sampling stream has the lowest priority: when a layer kernel and sampler kernels are both ready, the layer
    // kernel's blocks are placed first and the sampler's short blocks fill what is left of every SM
    int prio_least = 0, prio_greatest = 0;
    cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest);
    if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithPriority(&c->sample_stream, cudaStreamNonBlocking, prio_least) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_user, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_fwd_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_out_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaMalloc((void**)&c->d_slot_of_part, sizeof(int32_t) * MG_MAX_PARTS) != cudaSuccess ||
        cudaMalloc((void**)&c->d_res_prefix, sizeof(int64_t) * (MG_MAX_PARTS + 1)) != cudaSuccess ||
        cudaMalloc((void**)&c->d_part_start, sizeof(int64_t) * (MG_MAX_PARTS + 1)) != cudaSuccess ||
        cudaMalloc((void**)&c->d_flags, sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(c->d_flags, 0, sizeof(uint32_t)) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return MG_ERR_CUDA;
    }
    *out = c;
    return MG_OK;
}

static void free_view(mg_ctx* c) {
    if (c->view_owned) { cudaFree(c->view_off); cudaFree(c->view_nbrs); }
    c->view_off = nullptr; c->view_nbrs = nullptr; c->view_owned = false; c->view_edges = 0;
    if (c->view_out_owned) { cudaFree(c->view_off_out); cudaFree(c->view_nbrs_out); }
    c->view_off_out = nullptr; c->view_nbrs_out = nullptr; c->view_out_owned = false; c->view_edges_out = 0;
}

static void free_out_graph(mg_ctx* c) {
    if (c->view_out_owned) { cudaFree(c->view_off_out); cudaFree(c->view_nbrs_out); }
    c->view_off_out = nullptr; c->view_nbrs_out = nullptr; c->view_out_owned = false; c->view_edges_out = 0;
    cudaFree(c->row_off_out); cudaFree(c->nbrs_out);
    c->row_off_out = nullptr; c->nbrs_out = nullptr; c->n_edges_out = 0;
    c->sample_inout = false;
}

static void free_features(mg_ctx* c) {
    if (c->slots_owned) cudaFree(c->slots);
    c->slots = nullptr; c->slots_owned = false; c->host_table = nullptr; c->feat_dim = 0; c->n_slots = 0;
    c->part_source.clear();
}

extern "C" int mg_destroy(mg_ctx* c) {
    if (!c) return MG_OK;
    cudaSetDevice(c->device);
    cudaStreamSynchronize(c->stream);
    cudaStreamSynchronize(c->side);
    cudaStreamSynchronize(c->sample_stream);
    for (auto ev : c->pending_events) cudaEventDestroy(ev);
    for (auto& p : c->prof_pending) { cudaEventDestroy(p.second.first); cudaEventDestroy(p.second.second); }
    free_view(c);
    free_features(c);
    free_out_graph(c);
    cudaFree(c->row_off); cudaFree(c->nbrs); cudaFree(c->d_slot_of_part); cudaFree(c->d_res_prefix); cudaFree(c->d_flags);
    cudaFree(c->view_ws); cudaFree(c->d_part_start); cudaFree(c->d_part_of_node); cudaFree(c->d_local_of_node); cudaFree(c->d_nodes_by_part);
    cudaFree(c->ws_x); cudaFree(c->ws_h[0]); cudaFree(c->ws_h[1]);
    cudaEventDestroy(c->ev_fwd_done); cudaEventDestroy(c->ev_out_done); cudaEventDestroy(c->ev_user);
    for (int i = 0; i < 2; ++i) { if (c->ev_hk_done[i]) cudaEventDestroy(c->ev_hk_done[i]); cudaFree(c->hk_buf[i]); }
    cudaFree(c->lp_ws); cudaFree(c->lp_spare); cudaFree(c->dm_images); cudaFree(c->lp_range);
    if (c->lp_words) cudaFreeHost(c->lp_words);
    cudaFree(c->bw_g); cudaFree(c->bw_x); cudaFree(c->bw_dx); cudaFree(c->bw_off); cudaFree(c->bw_rev);
    cudaFree(c->gat_x); cudaFree(c->gat_z); cudaFree(c->gat_s); cudaFree(c->gat_h[0]); cudaFree(c->gat_h[1]);
    cudaStreamDestroy(c->sample_stream);
    cudaStreamDestroy(c->side);
    delete c;
    return MG_OK;
}

extern "C" const char* mg_last_error(const mg_ctx* c) { return c ? c->err.c_str() : "null context"; }
extern "C" int64_t mg_kernel_launches(const mg_ctx* c) { return c ? c->launches : 0; }

extern "C" int mg_profile(mg_ctx* c, int enable) {
    if (!c) return MG_ERR_ARG;
    c->prof_on = enable != 0;
    return MG_OK;
}

extern "C" int mg_profile_read(mg_ctx* c, int32_t* n_phases, const char** names, double* ms, int64_t* launches, int reset) {
    if (!c) return MG_ERR_ARG;
    cudaSetDevice(c->device);
    cudaStreamSynchronize(c->stream);
    cudaStreamSynchronize(c->sample_stream);
    for (auto& p : c->prof_pending) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, p.second.first, p.second.second) == cudaSuccess) c->prof[p.first].ms += t;
        else cudaGetLastError();
        cudaEventDestroy(p.second.first);
        cudaEventDestroy(p.second.second);
    }
    c->prof_pending.clear();
    if (n_phases) *n_phases = PH_COUNT;
    for (int i = 0; i < PH_COUNT; ++i) {
        if (names) names[i] = c->prof[i].name;
        if (ms) ms[i] = c->prof[i].ms;
        if (launches) launches[i] = c->prof[i].launches;
        if (reset) { c->prof[i].ms = 0; c->prof[i].launches = 0; }
    }
    return MG_OK;
}

// upload the committed slot map and the resident-node prefix counts
static int upload_slot_map(mg_ctx* c) {
    ++c->resident_serial;   // every change of the committed slot map (or of the slots behind it) comes through here
    int32_t slots[MG_MAX_PARTS];
    int64_t prefix[MG_MAX_PARTS + 1];
    prefix[0] = 0;
    for (int p = 0; p < MG_MAX_PARTS; ++p) {
        slots[p] = p < c->n_parts ? c->slot_of_part[p] : -1;
        const int64_t sz = (p < c->n_parts && slots[p] >= 0) ? c->part_count[p] : 0;
        prefix[p + 1] = prefix[p] + sz;
    }
    c->n_resident_nodes = prefix[MG_MAX_PARTS];
    int64_t starts[MG_MAX_PARTS + 1];
    for (int p = 0; p <= MG_MAX_PARTS; ++p) starts[p] = p < c->n_parts ? c->part_start[p] : c->n_nodes;
    MG_CUDA(c, cudaMemcpyAsync(c->d_part_start, starts, sizeof(starts), cudaMemcpyHostToDevice, c->stream));
    MG_CUDA(c, cudaMemcpyAsync(c->d_slot_of_part, slots, sizeof(slots), cudaMemcpyHostToDevice, c->stream));
    MG_CUDA(c, cudaMemcpyAsync(c->d_res_prefix, prefix, sizeof(prefix), cudaMemcpyHostToDevice, c->stream));
    MG_CUDA(c, cudaStreamSynchronize(c->stream));
    return MG_OK;
}

// One edge list's in-buffer view: the rows of resident nodes restricted to resident neighbours (the list itself when
// every partition is resident).
static int rebuild_one_view(mg_ctx* c, bool all, const int64_t* row_off, const int32_t* nbrs, int64_t n_edges,
                            int64_t** view_off, int32_t** view_nbrs, bool* owned, int64_t* view_edges) {
    if (all) {
        if (*owned) { cudaFree(*view_off); cudaFree(*view_nbrs); }
        *view_off = const_cast<int64_t*>(row_off); *view_nbrs = const_cast<int32_t*>(nbrs); *view_edges = n_edges; *owned = false;
        return MG_OK;
    }
    if (!*owned) {
        *view_off = nullptr; *view_nbrs = nullptr;
        if (cudaMalloc((void**)view_off, sizeof(int64_t) * (c->n_nodes + 1)) != cudaSuccess ||
            cudaMalloc((void**)view_nbrs, sizeof(int32_t) * std::max<int64_t>(n_edges, 1)) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(*view_off);
            *view_off = nullptr; *view_nbrs = nullptr;
            return mg_fail(c, MG_ERR_OOM, "allocation of the in-buffer graph view failed");
        }
        *owned = true;
    }
    // scratch (kept by the context, grown on demand): keep bits, per-word prefixes, tile counts and bases, scan scratch
    const int64_t n_words = (n_edges + 31) / 32 + 1;
    const int64_t n_tiles = (n_edges + kViewTile - 1) / kViewTile;
    const int64_t n_scan_tiles = (n_tiles + kTile - 1) / kTile;
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t o_mask = 0, o_before = o_mask + up(sizeof(uint32_t) * n_words), o_cnt = o_before + up(sizeof(uint16_t) * n_words),
                 o_base = o_cnt + up(sizeof(int32_t) * (n_tiles + 1)), o_scan = o_base + up(sizeof(int64_t) * (n_tiles + 2)),
                 o_total = o_scan + up(sizeof(uint64_t) * (n_scan_tiles + 1)), need = o_total + 256;
    if (c->view_ws_bytes < need) {
        cudaFree(c->view_ws);
        c->view_ws = nullptr; c->view_ws_bytes = 0;
        if (cudaMalloc((void**)&c->view_ws, need) != cudaSuccess) { cudaGetLastError(); return mg_fail(c, MG_ERR_OOM, "scratch allocation for the in-buffer graph view failed"); }
        c->view_ws_bytes = need;
    }
    ViewArgs a;
    a.off = row_off; a.nbrs = nbrs; a.n_nodes = c->n_nodes; a.n_edges = n_edges;
    a.part_size = (uint32_t)c->part_size; a.n_parts = c->n_parts; a.slot_of_part = c->d_slot_of_part;
    a.part_of_node = c->d_part_of_node;
    a.mask = reinterpret_cast<uint32_t*>(c->view_ws + o_mask);
    a.word_before = reinterpret_cast<uint16_t*>(c->view_ws + o_before);
    a.tile_cnt = reinterpret_cast<int32_t*>(c->view_ws + o_cnt);
    int64_t* tile_base = reinterpret_cast<int64_t*>(c->view_ws + o_base);
    a.tile_base = tile_base;
    uint64_t* scan_tiles = reinterpret_cast<uint64_t*>(c->view_ws + o_scan);
    int64_t* d_total = reinterpret_cast<int64_t*>(c->view_ws + o_total);
    const int grid = mg_grid(c, 8);
    cudaStream_t st = c->stream;
    int64_t total = 0;
    cudaError_t e = cudaSuccess;
    if (n_edges > 0) {
        k_view_mask<<<grid, kThreads, 0, st>>>(a);
        k_scan64_reduce<<<grid, kThreads, 0, st>>>(a.tile_cnt, n_tiles, scan_tiles);
        k_scan64_tiles<<<1, kThreads, 0, st>>>(scan_tiles, n_scan_tiles, d_total);
        k_scan64_down<<<grid, kThreads, 0, st>>>(a.tile_cnt, n_tiles, scan_tiles, tile_base);
        k_view_compact<<<grid, kThreads, 0, st>>>(a, *view_nbrs);
        k_view_offsets<<<grid, kThreads, 0, st>>>(a, *view_off);
        c->launches += 6;
        e = cudaMemcpyAsync(&total, d_total, sizeof(int64_t), cudaMemcpyDeviceToHost, st);
    } else {
        e = cudaMemsetAsync(*view_off, 0, sizeof(int64_t) * (c->n_nodes + 1), st);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return mg_cuda_fail(c, e, "rebuild of the in-buffer graph view");
    *view_edges = total;
    return MG_OK;
}

static int rebuild_view(mg_ctx* c) {
    bool all = true, any = false;
    for (int p = 0; p < c->n_parts; ++p) { all = all && c->slot_of_part[p] >= 0; any = any || c->slot_of_part[p] >= 0; }
    if (!any) {   // nothing in the buffer: there is no view, and sampling refuses to run
        free_view(c);
        return MG_OK;
    }
    int rc = rebuild_one_view(c, all, c->row_off, c->nbrs, c->n_edges, &c->view_off, &c->view_nbrs, &c->view_owned, &c->view_edges);
    if (rc == MG_OK && c->row_off_out)
        rc = rebuild_one_view(c, all, c->row_off_out, c->nbrs_out, c->n_edges_out, &c->view_off_out, &c->view_nbrs_out,
                              &c->view_out_owned, &c->view_edges_out);
    return rc;
}

// Copy one CSR to the device and validate it there; *row_off_out / *nbrs_out own the copies.
static int upload_csr(mg_ctx* c, int64_t n_nodes, int64_t n_edges, const void* row_offsets, int offsets_are_i64,
                      const int32_t* nbrs, int ptrs_are_device, int64_t** d_row_off, int32_t** d_nbrs) {
    const cudaMemcpyKind kind = ptrs_are_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    *d_row_off = nullptr; *d_nbrs = nullptr;
    if (cudaMalloc((void**)d_row_off, sizeof(int64_t) * (n_nodes + 1)) != cudaSuccess ||
        cudaMalloc((void**)d_nbrs, sizeof(int32_t) * std::max<int64_t>(n_edges, 1)) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(*d_row_off); *d_row_off = nullptr; *d_nbrs = nullptr;
        return mg_fail(c, MG_ERR_OOM, "allocation of the graph store failed");
    }
    auto drop = [&]() { cudaFree(*d_row_off); cudaFree(*d_nbrs); *d_row_off = nullptr; *d_nbrs = nullptr; };
    cudaStream_t st = c->stream;
    cudaError_t e = cudaSuccess;
    if (offsets_are_i64) {
        e = cudaMemcpyAsync(*d_row_off, row_offsets, sizeof(int64_t) * (n_nodes + 1), kind, st);
    } else {
        int32_t* tmp = nullptr;
        e = cudaMalloc((void**)&tmp, sizeof(int32_t) * (n_nodes + 1));
        if (e == cudaSuccess) e = cudaMemcpyAsync(tmp, row_offsets, sizeof(int32_t) * (n_nodes + 1), kind, st);
        if (e == cudaSuccess) {
            k_widen_offsets<<<mg_grid(c, 4), kThreads, 0, st>>>(tmp, *d_row_off, n_nodes + 1);
            c->launches++;
            e = cudaStreamSynchronize(st);
        }
        cudaFree(tmp);
    }
    if (e == cudaSuccess && n_edges > 0) e = cudaMemcpyAsync(*d_nbrs, nbrs, sizeof(int32_t) * n_edges, kind, st);
    // validate on the device; only the two end offsets come back
    uint32_t* flags = nullptr;
    if (e == cudaSuccess) e = cudaMalloc((void**)&flags, sizeof(uint32_t));
    if (e != cudaSuccess) { cudaGetLastError(); drop(); return mg_cuda_fail(c, e, "graph upload"); }
    cudaMemsetAsync(flags, 0, sizeof(uint32_t), st);
    k_check_graph<<<mg_grid(c, 8), kThreads, 0, st>>>(*d_row_off, n_nodes, *d_nbrs, n_edges, flags);
    c->launches++;
    uint32_t h_flags = 0;
    int64_t ends[2] = {0, 0};
    cudaMemcpyAsync(&h_flags, flags, sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(&ends[0], *d_row_off, sizeof(int64_t), cudaMemcpyDeviceToHost, st);
    cudaMemcpyAsync(&ends[1], *d_row_off + n_nodes, sizeof(int64_t), cudaMemcpyDeviceToHost, st);
    e = cudaStreamSynchronize(st);
    cudaFree(flags);
    if (e != cudaSuccess) { drop(); return mg_cuda_fail(c, e, "graph upload"); }
    if (h_flags || ends[0] != 0 || ends[1] != n_edges) {
        drop();
        return mg_fail(c, MG_ERR_ARG, "malformed CSR: %s", (h_flags & 2) ? "neighbour id out of range"
                                                            : (h_flags & 1) ? "row offsets decrease"
                                                                            : "row_offsets[0] != 0 or row_offsets[n_nodes] != n_edges");
    }
    return MG_OK;
}

extern "C" int mg_load_graph(mg_ctx* c, int64_t n_nodes, int64_t n_edges, const void* row_offsets, int offsets_are_i64,
                             const int32_t* nbrs, int ptrs_are_device) {
    if (!c) return MG_ERR_ARG;
    if (!row_offsets || (n_edges > 0 && !nbrs)) return mg_fail(c, MG_ERR_ARG, "null argument");
    if (n_nodes <= 0 || n_nodes >= (1ll << 31) - 1 || n_edges < 0) return mg_fail(c, MG_ERR_ARG, "n_nodes must be in [1, 2^31 - 2], n_edges >= 0");
    MG_CUDA(c, cudaSetDevice(c->device));
    MG_CUDA(c, cudaStreamSynchronize(c->stream));
    free_view(c);
    free_features(c);
    free_out_graph(c);
    cudaFree(c->row_off); cudaFree(c->nbrs);
    c->row_off = nullptr; c->nbrs = nullptr; c->n_nodes = 0; c->n_edges = 0;
    const int rc = upload_csr(c, n_nodes, n_edges, row_offsets, offsets_are_i64, nbrs, ptrs_are_device, &c->row_off, &c->nbrs);
    if (rc) return rc;
    c->n_nodes = n_nodes;
    c->n_edges = n_edges;
    return mg_set_partitioning(c, 1, nullptr);
}

extern "C" int mg_load_out_graph(mg_ctx* c, int64_t n_edges, const void* row_offsets, int offsets_are_i64, const int32_t* nbrs,
                                 int ptrs_are_device) {
    if (!c) return MG_ERR_ARG;
    if (!row_offsets || (n_edges > 0 && !nbrs)) return mg_fail(c, MG_ERR_ARG, "null argument");
    if (n_edges < 0) return mg_fail(c, MG_ERR_ARG, "n_edges must not be negative");
    if (!c->row_off) return mg_fail(c, MG_ERR_STATE, "no graph loaded");
    MG_CUDA(c, cudaSetDevice(c->device));
    MG_CUDA(c, cudaStreamSynchronize(c->stream));
    free_out_graph(c);
    const int rc = upload_csr(c, c->n_nodes, n_edges, row_offsets, offsets_are_i64, nbrs, ptrs_are_device, &c->row_off_out, &c->nbrs_out);
    if (rc) return rc;
    c->n_edges_out = n_edges;
    return rebuild_view(c);   // the in-buffer filter of the current resident set
}

extern "C" int mg_set_sample_direction(mg_ctx* c, int direction) {
    if (!c) return MG_ERR_ARG;
    if (direction != MG_SAMPLE_IN && direction != MG_SAMPLE_INOUT) return mg_fail(c, MG_ERR_ARG, "unknown sampling direction");
    if (direction == MG_SAMPLE_INOUT && !c->row_off_out) return mg_fail(c, MG_ERR_STATE, "no outgoing edge list loaded");
    c->sample_inout = direction == MG_SAMPLE_INOUT;
    return MG_OK;
}

extern "C" int mg_set_partitioning(mg_ctx* c, int32_t n_parts, const uint8_t* part_of_node) {
    if (!c) return MG_ERR_ARG;
    if (!c->row_off) return mg_fail(c, MG_ERR_STATE, "no graph loaded");
    if (n_parts <= 0 || n_parts > MG_MAX_PARTS) return mg_fail(c, MG_ERR_ARG, "n_parts must be in [1, %d]", MG_MAX_PARTS);
    MG_CUDA(c, cudaSetDevice(c->device));
    MG_CUDA(c, cudaStreamSynchronize(c->stream));
    MG_CUDA(c, cudaStreamSynchronize(c->sample_stream));
    free_features(c);
    cudaFree(c->d_part_of_node); cudaFree(c->d_local_of_node); cudaFree(c->d_nodes_by_part);
    c->d_part_of_node = nullptr; c->d_local_of_node = nullptr; c->d_nodes_by_part = nullptr;
    c->part_count.assign(n_parts, 0);
    c->part_start.assign(n_parts + 1, 0);
    const int64_t N = c->n_nodes;
    if (!part_of_node) {
        // contiguous equal id ranges (the sequential lookup table of Section 3 cut into n_parts pieces)
        c->part_size = (N + n_parts - 1) / n_parts;
        for (int p = 0; p < n_parts; ++p) {
            c->part_start[p] = std::min<int64_t>((int64_t)p * c->part_size, N);
            c->part_count[p] = std::max<int64_t>(0, std::min<int64_t>(c->part_size, N - (int64_t)p * c->part_size));
        }
        c->part_start[n_parts] = N;
    } else {
        // a partition id per node: populations, each node's rank inside its partition and the partitions' node lists
        for (int64_t v = 0; v < N; ++v) {
            if (part_of_node[v] >= n_parts) return mg_fail(c, MG_ERR_ARG, "part_of_node[%lld] = %d is not below n_parts", (long long)v, (int)part_of_node[v]);
            ++c->part_count[part_of_node[v]];
        }
        int64_t largest = 1;
        for (int p = 0; p < n_parts; ++p) { c->part_start[p + 1] = c->part_start[p] + c->part_count[p]; largest = std::max(largest, c->part_count[p]); }
        c->part_size = largest;
        std::vector<int32_t> local((size_t)N), by_part((size_t)N);
        std::vector<int64_t> next(c->part_start.begin(), c->part_start.end() - 1);
        for (int64_t v = 0; v < N; ++v) {
            const int p = part_of_node[v];
            local[(size_t)v] = (int32_t)(next[p] - c->part_start[p]);
            by_part[(size_t)next[p]++] = (int32_t)v;
        }
        if (cudaMalloc((void**)&c->d_part_of_node, (size_t)N) != cudaSuccess ||
            cudaMalloc((void**)&c->d_local_of_node, sizeof(int32_t) * (size_t)N) != cudaSuccess ||
            cudaMalloc((void**)&c->d_nodes_by_part, sizeof(int32_t) * (size_t)N) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(c->d_part_of_node); cudaFree(c->d_local_of_node); cudaFree(c->d_nodes_by_part);
            c->d_part_of_node = nullptr; c->d_local_of_node = nullptr; c->d_nodes_by_part = nullptr;
            return mg_fail(c, MG_ERR_OOM, "allocation of the partition tables failed");
        }
        MG_CUDA(c, cudaMemcpy(c->d_part_of_node, part_of_node, (size_t)N, cudaMemcpyHostToDevice));
        MG_CUDA(c, cudaMemcpy(c->d_local_of_node, local.data(), sizeof(int32_t) * (size_t)N, cudaMemcpyHostToDevice));
        MG_CUDA(c, cudaMemcpy(c->d_nodes_by_part, by_part.data(), sizeof(int32_t) * (size_t)N, cudaMemcpyHostToDevice));
    }
    c->n_parts = n_parts;
    c->capacity = n_parts;
    c->slot_of_part.assign(n_parts, n_parts == 1 ? 0 : -1);
    c->dirty_part.clear();
    c->pending_slot.clear();
    c->has_pending = false;
    int rc = upload_slot_map(c);
    if (rc) return rc;
    return rebuild_view(c);
}

extern "C" int mg_load_features(mg_ctx* c, const void* table, int table_is_device, int dtype, int32_t dim,
                                int32_t buffer_capacity_parts, int backing) {
    if (!c) return MG_ERR_ARG;
    if (!c->row_off) return mg_fail(c, MG_ERR_STATE, "no graph loaded");
    if (!table && backing != MG_BACKING_HOST) return mg_fail(c, MG_ERR_ARG, "null table");
    if (dtype != MG_DTYPE_F32 && dtype != MG_DTYPE_F16) return mg_fail(c, MG_ERR_ARG, "unknown dtype");
    const int64_t esz = dtype == MG_DTYPE_F32 ? 4 : 2;
    if (dim <= 0 || (dim * esz) % 16 != 0) return mg_fail(c, MG_ERR_ARG, "dim * sizeof(dtype) must be a positive multiple of 16 bytes");
    if (buffer_capacity_parts <= 0 || buffer_capacity_parts > c->n_parts) return mg_fail(c, MG_ERR_ARG, "buffer capacity must be in [1, n_parts]");
    if (backing != MG_BACKING_HBM && backing != MG_BACKING_HOST) return mg_fail(c, MG_ERR_ARG, "unknown backing");
    if (backing == MG_BACKING_HOST && table_is_device) return mg_fail(c, MG_ERR_ARG, "host backing needs a host table");
    MG_CUDA(c, cudaSetDevice(c->device));
    MG_CUDA(c, cudaStreamSynchronize(c->stream));
    free_features(c);
    c->feat_dtype = dtype;
    c->row_bytes = dim * esz;
    c->slot_bytes = c->part_size * c->row_bytes;
    c->capacity = buffer_capacity_parts;
    c->backing = backing;
    int n_res = 0;
    for (int p = 0; p < c->n_parts; ++p) n_res += c->slot_of_part[p] >= 0;
    if (backing == MG_BACKING_HBM) {
        if (table_is_device) {
            c->slots = (char*)const_cast<void*>(table);
            c->slots_owned = false;
        } else {
            const size_t bytes = (size_t)c->n_nodes * c->row_bytes;
            if (cudaMalloc((void**)&c->slots, bytes) != cudaSuccess) { cudaGetLastError(); c->slots = nullptr; return mg_fail(c, MG_ERR_OOM, "feature table allocation failed"); }
            c->slots_owned = true;
            MG_CUDA(c, cudaMemcpyAsync(c->slots, table, bytes, cudaMemcpyHostToDevice, c->stream));
            MG_CUDA(c, cudaStreamSynchronize(c->stream));
        }
        c->n_slots = c->n_parts;
        // resident partitions keep slot == partition id
        for (int p = 0; p < c->n_parts; ++p)
            if (c->slot_of_part[p] >= 0) c->slot_of_part[p] = p;
    } else {
        c->n_slots = buffer_capacity_parts + 1;
        const size_t bytes = (size_t)c->n_slots * c->slot_bytes;
        if (cudaMalloc((void**)&c->slots, bytes) != cudaSuccess) { cudaGetLastError(); c->slots = nullptr; return mg_fail(c, MG_ERR_OOM, "buffer slot allocation failed"); }
        c->slots_owned = true;
        c->host_table = (const char*)table;
        // whatever was resident for sampling only is reloaded into slots
        std::vector<int32_t> keep;
        for (int p = 0; p < c->n_parts; ++p)
            if (c->slot_of_part[p] >= 0) keep.push_back(p);
        c->slot_of_part.assign(c->n_parts, -1);
        c->dirty_part.clear();
        c->feat_dim = dim;
        if ((int)keep.size() > c->capacity) keep.resize(c->capacity);
        if (!table) keep.clear();   // no whole table: partitions come in once their host blocks have been named
        if (!keep.empty()) {
            int rc = mg_set_resident(c, keep.data(), (int32_t)keep.size(), 0);
            if (rc) return rc;
        } else {
            int rc = upload_slot_map(c);
            if (rc) return rc;
            rc = rebuild_view(c);
            if (rc) return rc;
        }
    }
    if (n_res > c->capacity && backing == MG_BACKING_HBM) {
        // more partitions resident than the new capacity allows: keep the lowest ids
        int kept = 0;
        for (int p = 0; p < c->n_parts; ++p)
            if (c->slot_of_part[p] >= 0 && ++kept > c->capacity) c->slot_of_part[p] = -1;
    }
    c->feat_dim = dim;
    int rc = upload_slot_map(c);
    if (rc) return rc;
    return rebuild_view(c);
}

// where partition p's rows live in host memory (MG_BACKING_HOST), or null when nobody said
static const char* host_block_of(const mg_ctx* c, int p) {
    if (p < (int)c->part_source.size() && c->part_source[p]) return c->part_source[p];
    return c->host_table ? c->host_table + (size_t)c->part_start[p] * c->row_bytes : nullptr;   // partition-major table
}

extern "C" int mg_set_partition_source(mg_ctx* c, int32_t part, const void* host_block) {
    if (!c) return MG_ERR_ARG;
    if (!c->slots || c->backing != MG_BACKING_HOST) return mg_fail(c, MG_ERR_STATE, "partition sources belong to a host-backed feature buffer");
    if (part < 0 || part >= c->n_parts) return mg_fail(c, MG_ERR_ARG, "partition id out of range");
    if (c->has_pending) return mg_fail(c, MG_ERR_STATE, "a resident set is pending (its copies may still read the old block); commit it first");
    if ((int)c->part_source.size() < c->n_parts) c->part_source.resize(c->n_parts, nullptr);
    c->part_source[part] = (const char*)host_block;
    return MG_OK;
}

extern "C" int mg_set_resident(mg_ctx* c, const int32_t* part_ids, int32_t n, int async) {
    if (!c) return MG_ERR_ARG;
    if (!c->row_off) return mg_fail(c, MG_ERR_STATE, "no graph loaded");
    if (n < 0 || (n > 0 && !part_ids)) return mg_fail(c, MG_ERR_ARG, "bad partition list");
    if (n > c->capacity) return mg_fail(c, MG_ERR_CAPACITY, "%d partitions asked, buffer holds %d", n, c->capacity);
    if (c->has_pending) return mg_fail(c, MG_ERR_STATE, "a resident set is already pending; commit it first");
    std::vector<char> want(c->n_parts, 0);
    for (int i = 0; i < n; ++i) {
        if (part_ids[i] < 0 || part_ids[i] >= c->n_parts) return mg_fail(c, MG_ERR_ARG, "partition id out of range");
        if (want[part_ids[i]]) return mg_fail(c, MG_ERR_ARG, "partition listed twice");
        want[part_ids[i]] = 1;
    }
    MG_CUDA(c, cudaSetDevice(c->device));
    std::vector<int32_t> next(c->n_parts, -1);
    const bool host_backed = c->slots && c->backing == MG_BACKING_HOST;
    if (host_backed)
        for (int p = 0; p < c->n_parts; ++p)
            if (want[p] && c->slot_of_part[p] < 0 && !host_block_of(c, p))
                return mg_fail(c, MG_ERR_STATE, "partition %d has no host block: no table was given and mg_set_partition_source was not called for it", p);
    if (!host_backed) {
        for (int p = 0; p < c->n_parts; ++p) next[p] = want[p] ? p : -1;
    } else {
        // slots free right now can be filled at once; slots of evicted partitions only after the
        // work already queued on the main stream has finished with them
        std::vector<char> used(c->n_slots, 0), evicted_slot(c->n_slots, 0);
        for (int p = 0; p < c->n_parts; ++p) {
            const int s = c->slot_of_part[p];
            if (s < 0) continue;
            if (want[p]) { next[p] = s; used[s] = 1; }
            else evicted_slot[s] = 1;
        }
        std::vector<int> free_now, free_later;
        for (int s = 0; s < c->n_slots; ++s) {
            if (used[s]) continue;
            (evicted_slot[s] ? free_later : free_now).push_back(s);
        }
        cudaEvent_t main_done = nullptr;
        // evicted partitions whose rows were updated in the buffer go back to the host table first (side stream, after
        // the work queued on the main stream; the copies into reused slots below are queued behind them)
        for (int p = 0; p < c->n_parts; ++p) {
            const int s = c->slot_of_part[p];
            if (s < 0 || want[p] || p >= (int)c->dirty_part.size() || !c->dirty_part[p]) continue;
            if (!main_done) {
                MG_CUDA(c, cudaEventCreateWithFlags(&main_done, cudaEventDisableTiming));
                MG_CUDA(c, cudaEventRecord(main_done, c->stream));
                MG_CUDA(c, cudaStreamWaitEvent(c->side, main_done, 0));
            }
            const int64_t rows = c->part_count[p];
            char* back = const_cast<char*>(host_block_of(c, p));
            if (rows > 0 && back)
                MG_CUDA(c, cudaMemcpyAsync(back, c->slots + (size_t)s * c->slot_bytes, (size_t)rows * c->row_bytes,
                                           cudaMemcpyDeviceToHost, c->side));
            c->dirty_part[p] = 0;
        }
        for (int p = 0; p < c->n_parts; ++p) {
            if (!want[p] || next[p] >= 0) continue;
            int s;
            if (!free_now.empty()) { s = free_now.back(); free_now.pop_back(); }
            else if (!free_later.empty()) {
                s = free_later.back(); free_later.pop_back();
                if (!main_done) {
                    MG_CUDA(c, cudaEventCreateWithFlags(&main_done, cudaEventDisableTiming));
                    MG_CUDA(c, cudaEventRecord(main_done, c->stream));
                    MG_CUDA(c, cudaStreamWaitEvent(c->side, main_done, 0));
                }
            } else return mg_fail(c, MG_ERR_CAPACITY, "no free buffer slot");
            next[p] = s;
            const int64_t rows = c->part_count[p];
            // in pieces: a copy engine finishes what it has started, and one 5 GB copy would hold up every small
            // host-to-device copy another stream issues meanwhile (targets of a sample, say) for a tenth of a second
            const size_t bytes = (size_t)std::max<int64_t>(rows, 0) * c->row_bytes, piece = (size_t)8 << 20;
            for (size_t at = 0; at < bytes; at += piece)
                MG_CUDA(c, cudaMemcpyAsync(c->slots + (size_t)s * c->slot_bytes + at, host_block_of(c, p) + at,
                                           std::min(piece, bytes - at), cudaMemcpyHostToDevice, c->side));
        }
        if (main_done) cudaEventDestroy(main_done);
        cudaEvent_t done;
        MG_CUDA(c, cudaEventCreateWithFlags(&done, cudaEventDisableTiming));
        MG_CUDA(c, cudaEventRecord(done, c->side));
        c->pending_events.push_back(done);
    }
    c->pending_slot = next;
    c->has_pending = true;
    if (!async) return mg_commit_resident(c, 600000);
    return MG_OK;
}

extern "C" int mg_commit_resident(mg_ctx* c, int32_t timeout_ms) {
    if (!c) return MG_ERR_ARG;
    if (!c->has_pending) return mg_fail(c, MG_ERR_STATE, "no pending resident set");
    MG_CUDA(c, cudaSetDevice(c->device));
    const auto t0 = std::chrono::steady_clock::now();
    for (auto ev : c->pending_events) {
        for (;;) {
            const cudaError_t q = cudaEventQuery(ev);
            if (q == cudaSuccess) break;
            if (q != cudaErrorNotReady) return mg_cuda_fail(c, q, "waiting for a partition copy");
            const auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(std::chrono::steady_clock::now() - t0).count();
            if (ms >= timeout_ms) return mg_fail(c, MG_ERR_TIMEOUT, "partition copies still running after %d ms", timeout_ms);
            std::this_thread::sleep_for(std::chrono::microseconds(200));
        }
    }
    for (auto ev : c->pending_events) cudaEventDestroy(ev);
    c->pending_events.clear();
    MG_CUDA(c, cudaStreamSynchronize(c->sample_stream));   // samples in flight were drawn under the old set
    c->slot_of_part = c->pending_slot;
    c->has_pending = false;
    int rc = upload_slot_map(c);
    if (rc) return rc;
    return rebuild_view(c);
}
