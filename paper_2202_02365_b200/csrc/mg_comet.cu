// COMET: the partition-replacement policy for link prediction out of core (Section 5.1) and the rules that set its
// parameters (Section 6).  Host code only: the plan of an epoch is a few KB of integers that drive mg_set_resident and
// tell which edge buckets a resident set trains; nothing here touches the device.
//
// Readings of what the paper leaves open (the same as the CPU oracle's, stated in include/mgdense.h):
//  * grouping: physical partitions ordered by a Philox word keyed by (seed, partition), cut into l groups of p / l;
//  * one-swap greedy order over logical partitions: the first set holds 0 .. c_l - 1; every later set replaces one
//    member e by one outside partition a, maximising the number of pairs {a, x} (x a remaining member) that have not
//    shared a set yet; ties: smallest a, then the member with the fewest such pairs left with outside partitions, then
//    the smallest member; when no swap sees a new pair, the outside partition that misses the most pairs comes in;
//  * edge bucket (i, j): one of the sets that hold both logical partitions, chosen by a Philox word keyed by
//    (seed, i, j) mapped to the number of such sets by multiply-high.
#include <math.h>
#include <stdint.h>

#include <algorithm>
#include <utility>
#include <vector>

#include "mgdense.h"

namespace {

void philox_host(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1, uint32_t out[4]) {
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

constexpr uint32_t kGroupTag = 0xC0E7u, kBucketTag = 0xB0C4E7u;

}  // namespace

extern "C" int mg_comet_plan(int32_t p, int32_t l, int32_t c_l, uint64_t seed, int32_t cap_sets, int32_t* logical_of_physical,
                             int32_t* n_sets_out, int32_t* sets, int32_t* bucket_set) {
    if (!logical_of_physical || !n_sets_out || !sets || !bucket_set) return MG_ERR_ARG;
    if (p <= 0 || l <= 0 || p % l != 0 || c_l < 2 || c_l > l || cap_sets < 1) return MG_ERR_ARG;
    const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    // random grouping of the physical partitions
    {
        std::vector<std::pair<uint32_t, int32_t>> order(p);
        for (int32_t q = 0; q < p; ++q) {
            uint32_t w[4];
            philox_host((uint32_t)q, 0u, kGroupTag, 0u, k0, k1, w);
            order[q] = {w[0], q};
        }
        std::sort(order.begin(), order.end());
        const int32_t per = p / l;
        for (int32_t rank = 0; rank < p; ++rank) logical_of_physical[order[rank].second] = rank / per;
    }
    // greedy one-swap sequence over the logical partitions
    std::vector<uint8_t> unseen((size_t)l * l, 0);   // symmetric
    int64_t n_unseen = 0;
    for (int a = 0; a < l; ++a)
        for (int b = a + 1; b < l; ++b) { unseen[(size_t)a * l + b] = unseen[(size_t)b * l + a] = 1; ++n_unseen; }
    auto see = [&](int a, int b) {
        if (unseen[(size_t)a * l + b]) { unseen[(size_t)a * l + b] = unseen[(size_t)b * l + a] = 0; --n_unseen; }
    };
    std::vector<int32_t> cur(c_l);
    std::vector<uint8_t> inside(l, 0);
    for (int i = 0; i < c_l; ++i) { cur[i] = i; inside[i] = 1; }
    for (int i = 0; i < c_l; ++i)
        for (int j = i + 1; j < c_l; ++j) see(i, j);
    int32_t n_sets = 0;
    auto emit = [&]() -> bool {
        if (n_sets >= cap_sets) return false;
        for (int i = 0; i < c_l; ++i) sets[(size_t)n_sets * c_l + i] = cur[i];
        ++n_sets;
        return true;
    };
    if (!emit()) return MG_ERR_CAPACITY;
    std::vector<int32_t> left(l);
    while (n_unseen > 0) {
        for (int i = 0; i < c_l; ++i) {   // pairs a member still misses with outside partitions
            int32_t n = 0;
            for (int a = 0; a < l; ++a) n += (!inside[a] && unseen[(size_t)a * l + cur[i]]) ? 1 : 0;
            left[cur[i]] = n;
        }
        int best_gain = -1, best_a = -1, best_e = -1;
        for (int a = 0; a < l; ++a) {
            if (inside[a]) continue;
            int with_all = 0;
            for (int i = 0; i < c_l; ++i) with_all += unseen[(size_t)a * l + cur[i]];
            for (int i = 0; i < c_l; ++i) {
                const int e = cur[i];
                const int gain = with_all - unseen[(size_t)a * l + e];
                bool better = gain > best_gain;
                if (!better && gain == best_gain && a == best_a)
                    better = left[e] < left[best_e] || (left[e] == left[best_e] && e < best_e);
                if (better) { best_gain = gain; best_a = a; best_e = e; }
            }
        }
        if (best_gain == 0) {
            int most = -1;
            for (int a = 0; a < l; ++a) {
                if (inside[a]) continue;
                int n = 0;
                for (int z = 0; z < l; ++z) n += unseen[(size_t)a * l + z];
                if (n > most) { most = n; best_a = a; }
            }
            best_e = -1;
            for (int i = 0; i < c_l; ++i) {
                const int e = cur[i];
                if (best_e < 0 || left[e] < left[best_e] || (left[e] == left[best_e] && e < best_e)) best_e = e;
            }
        }
        for (int i = 0; i < c_l; ++i)
            if (cur[i] == best_e) cur[i] = best_a;
        inside[best_e] = 0; inside[best_a] = 1;
        for (int i = 0; i < c_l; ++i)
            if (cur[i] != best_a) see(best_a, cur[i]);
        if (!emit()) return MG_ERR_CAPACITY;
    }
    *n_sets_out = n_sets;
    // edge buckets: a random set among those that hold both logical partitions
    std::vector<uint8_t> member((size_t)n_sets * l, 0);
    for (int32_t k = 0; k < n_sets; ++k)
        for (int i = 0; i < c_l; ++i) member[(size_t)k * l + sets[(size_t)k * c_l + i]] = 1;
    std::vector<int32_t> cands;
    for (int32_t i = 0; i < p; ++i)
        for (int32_t j = 0; j < p; ++j) {
            const int32_t li = logical_of_physical[i], lj = logical_of_physical[j];
            cands.clear();
            for (int32_t k = 0; k < n_sets; ++k)
                if (member[(size_t)k * l + li] && member[(size_t)k * l + lj]) cands.push_back(k);
            uint32_t w[4];
            philox_host((uint32_t)i, (uint32_t)j, kBucketTag, 0u, k0, k1, w);
            bucket_set[(size_t)i * p + j] = cands[(size_t)(((uint64_t)w[0] * (uint64_t)cands.size()) >> 32)];
        }
    return MG_OK;
}

extern "C" int mg_comet_bias(int32_t p, int32_t n_sets, const int32_t* bucket_set, double* bias_out) {
    if (!bucket_set || !bias_out || p <= 0 || n_sets <= 0) return MG_ERR_ARG;
    std::vector<int64_t> total(p, 0), tally(p, 0);
    std::vector<int64_t> per_set((size_t)n_sets * p, 0);
    for (int32_t i = 0; i < p; ++i)
        for (int32_t j = 0; j < p; ++j) {
            const int32_t k = bucket_set[(size_t)i * p + j];
            if (k < 0 || k >= n_sets) return MG_ERR_ARG;
            per_set[(size_t)k * p + i]++; per_set[(size_t)k * p + j]++;
            total[i]++; total[j]++;
        }
    double bias = 0.0;
    for (int32_t k = 0; k < n_sets; ++k) {
        double lo = 2.0, hi = -1.0;
        for (int32_t q = 0; q < p; ++q) {
            tally[q] += per_set[(size_t)k * p + q];
            const double t = (double)tally[q] / (double)total[q];
            lo = std::min(lo, t); hi = std::max(hi, t);
        }
        bias = std::max(bias, hi - lo);
    }
    *bias_out = bias;
    return MG_OK;
}

extern "C" int mg_comet_autotune(int64_t n_nodes, int32_t dim, int64_t n_edges, int32_t bytes_per_edge, int64_t cpu_bytes,
                                 int64_t block_bytes, int64_t fudge_bytes, int32_t max_parts, int32_t* p_out, int32_t* l_out,
                                 int32_t* c_out) {
    if (!p_out || !l_out || !c_out) return MG_ERR_ARG;
    if (n_nodes <= 0 || dim <= 0 || n_edges < 0 || bytes_per_edge <= 0 || cpu_bytes <= 0 || block_bytes <= 0 || fudge_bytes < 0 ||
        max_parts < 2)
        return MG_ERR_ARG;
    const double node_overhead = (double)n_nodes * (double)dim * 4.0;
    const double edge_overhead = (double)n_edges * (double)bytes_per_edge;
    const double alpha4 = std::min(node_overhead / (double)block_bytes, sqrt(edge_overhead / (double)block_bytes));
    const int32_t p = (int32_t)std::max<double>(2.0, std::min<double>(floor(alpha4), (double)max_parts));
    const double part_overhead = node_overhead / p, bucket_overhead = edge_overhead / ((double)p * p);
    int32_t best = 0;
    for (int32_t c = 2; c <= p; c += 2)
        if (c * part_overhead + 2.0 * c * c * bucket_overhead + (double)fudge_bytes < (double)cpu_bytes && p % (c / 2) == 0) best = c;
    if (!best) return MG_ERR_CAPACITY;
    *p_out = p; *l_out = 2 * p / best; *c_out = best;
    return MG_OK;
}
