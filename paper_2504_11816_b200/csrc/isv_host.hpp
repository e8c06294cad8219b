// Host-side bookkeeping of the split KV cache: geometry, block allocation by
// the residency rule, block tables, lengths, and the plan that tells the
// staging engine which host blocks a layer's decode needs.  No CUDA here, so
// the same code serves plan-only handles on machines without a GPU.
#pragma once

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <utility>
#include <vector>

#include "../../include/isv.h"
#include "isv_kernels.cuh"

namespace isv {

struct Geometry {
    int layers = 0, phys_layers = 0;
    int Hq = 0, Hkv = 0, D = 0, BT = 0, dtype = 0;
    float f = 0.f;                 // offload fraction C_off
    int max_seqs = 0, max_tokens = 0;
    int NB = 0;                    // max blocks per sequence = table row stride
    int G = 0;                     // query heads per KV head
    int GT = 0;                    // query heads handled together by one warp
    int P = 0;                     // passes over a KV head = G / GT
    int HP = 1;                    // KV heads per head group (2: two adjacent heads of a multi-head shape per visit)
    int groups() const { return Hkv * P / HP; }   // head groups per sequence
    int max_ctas = 0;              // cap on the decode kernel's grid (0 = one CTA per SM)
    uint32_t tile_bytes = 0;       // one (block, K|V, head) tile
    uint64_t block_bytes = 0;      // 2 * Hkv * tile_bytes
    uint64_t kappa = 0;            // KV bytes per token per layer
    int hbm_cap = 0, host_cap = 0; // pool capacities per physical layer, in blocks
    uint64_t chunk_bytes = 0;
    int chunk_blocks = 0;          // host blocks per staging chunk
    int ring = 0;
};

// splitmix64 (Steele, Lea, Flood 2014): the stream behind the block-id permutation.
struct SplitMix64 {
    uint64_t x;
    explicit SplitMix64(uint64_t seed) : x(seed) {}
    uint64_t next() {
        uint64_t z = (x += 0x9E3779B97F4A7C15ull);
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        return z ^ (z >> 31);
    }
    // uniform in [0, n) by rejection of the biased tail
    uint64_t below(uint64_t n) {
        const uint64_t lim = UINT64_MAX - (UINT64_MAX % n);
        uint64_t r;
        do { r = next(); } while (r >= lim);
        return r % n;
    }
};

struct TableUpdate { int32_t index; int32_t value; };   // table[index] = value

// One staging chunk: a contiguous run of host block ids and the (sequence,
// blocks) units whose attention it feeds.
struct Chunk {
    int32_t first_id = 0;      // first host block id copied
    int32_t n_ids = 0;         // blocks copied (contiguous)
    int32_t unit_begin = 0;    // range in OffPlan::cu_*
    int32_t unit_end = 0;
};

struct OffPlan {
    bool valid = false;
    int n_seqs = 0;
    int chunk_blocks = 0;           // host blocks per chunk this plan was cut with
    std::vector<int32_t> key;       // per sequence: index of its newest block (-1 if empty)
    std::vector<Chunk> chunks;
    std::vector<int32_t> cu_seq;    // unit -> sequence
    std::vector<int32_t> cu_beg;    // unit -> range in cblk
    std::vector<int32_t> cu_end;
    std::vector<int32_t> cblk;      // block slot inside the chunk's staging buffer
    uint64_t bytes_resident = 0;    // algorithmic bytes read from GPU memory
    uint64_t bytes_offloaded = 0;   // algorithmic bytes fetched over the host link
    uint64_t bytes_staged = 0;      // bytes the copy engine moves
    uint64_t version = 0;
};

class BlockManager {
public:
    Geometry g;
    std::vector<int32_t> table;        // [max_seqs][NB]
    std::vector<int32_t> len;          // [layers][max_seqs]
    std::vector<int32_t> host_owner_s; // host block id -> sequence
    std::vector<int32_t> host_owner_j; // host block id -> logical block
    int hbm_used = 0, host_used = 0;

    void init(const Geometry &geo, uint64_t perm_seed) {
        g = geo;
        seed_ = perm_seed;
        reset();
    }

    void reset() {
        table.assign((size_t)g.max_seqs * g.NB, ISV_BLOCK_NONE);
        len.assign((size_t)g.layers * g.max_seqs, 0);
        host_owner_s.assign(g.host_cap, -1);
        host_owner_j.assign(g.host_cap, -1);
        hbm_used = host_used = 0;
        hbm_order_.resize(g.hbm_cap);
        for (int i = 0; i < g.hbm_cap; ++i) hbm_order_[i] = i;
        rng_ = SplitMix64(seed_);
        if (seed_ != 0) shuffle(hbm_order_.data(), g.hbm_cap);
        plan_.valid = false;
    }

    // Residency rule: logical block j is host-resident iff
    // floor((j+1) f) > floor(j f), evaluated in double (exact for float f, j < 2^28).
    bool is_host(int j) const {
        const double f = (double)g.f;
        return std::floor((double)(j + 1) * f) > std::floor((double)j * f);
    }

    int32_t &entry(int s, int j) { return table[(size_t)s * g.NB + j]; }
    int32_t entry(int s, int j) const { return table[(size_t)s * g.NB + j]; }
    int32_t &length(int layer, int s) { return len[(size_t)layer * g.max_seqs + s]; }
    int32_t length(int layer, int s) const { return len[(size_t)layer * g.max_seqs + s]; }

    // Allocates every listed (sequence, block) that has no block yet.  Host
    // ids stay compact ([0, host_used)); with a seed the ids of one call are
    // assigned in shuffled order.  Returns ISV_ECAPACITY if a pool is full
    // (nothing is changed then).
    int allocate(const std::vector<std::pair<int, int>> &need, std::vector<TableUpdate> *updates) {
        std::vector<std::pair<int, int>> hbm, host;
        for (auto &sj : need) {
            if (entry(sj.first, sj.second) != ISV_BLOCK_NONE) continue;
            (is_host(sj.second) ? host : hbm).push_back(sj);
        }
        if (hbm_used + (int)hbm.size() > g.hbm_cap || host_used + (int)host.size() > g.host_cap)
            return ISV_ECAPACITY;
        for (auto &sj : hbm) {
            const int32_t id = hbm_order_[hbm_used++];
            entry(sj.first, sj.second) = id;
            if (updates) updates->push_back({(int32_t)((size_t)sj.first * g.NB + sj.second), id});
        }
        if (!host.empty()) {
            std::vector<int32_t> ids(host.size());
            for (size_t i = 0; i < ids.size(); ++i) ids[i] = host_used + (int32_t)i;
            if (seed_ != 0) shuffle(ids.data(), (int)ids.size());
            for (size_t i = 0; i < host.size(); ++i) {
                const int32_t id = ids[i];
                host_owner_s[id] = host[i].first;
                host_owner_j[id] = host[i].second;
                const int32_t e = id | ISV_BLOCK_HOST_BIT;
                entry(host[i].first, host[i].second) = e;
                if (updates)
                    updates->push_back({(int32_t)((size_t)host[i].first * g.NB + host[i].second), e});
            }
            host_used += (int)host.size();
            plan_.valid = false;
        }
        return ISV_OK;
    }

    // Index of the block holding the newest token of (layer, s); -1 if empty.
    int newest_block(int layer, int s) const {
        const int n = length(layer, s);
        return n > 0 ? (n - 1) / g.BT : -1;
    }

    // The offloaded part of a decode of `layer` over sequences [0, n_seqs):
    // every host block that is complete and older than its sequence's newest
    // block, grouped by staging chunk and, inside a chunk, by sequence.
    // Cached while the newest-block indices stay the same.
    const OffPlan &plan(int layer, int n_seqs, int chunk_blocks = 0) {
        if (chunk_blocks <= 0) chunk_blocks = g.chunk_blocks;
        std::vector<int32_t> key(n_seqs);
        for (int s = 0; s < n_seqs; ++s) key[s] = newest_block(layer, s);
        bool same = plan_.valid && plan_.n_seqs == n_seqs && plan_.chunk_blocks == chunk_blocks && plan_.key == key;
        if (same) {
            // byte counters depend on exact lengths, not only on block counts
            account(layer, n_seqs);
            return plan_;
        }
        const uint64_t ver = plan_.version + 1;
        plan_ = OffPlan();
        plan_.version = ver;
        plan_.valid = true;
        plan_.n_seqs = n_seqs;
        plan_.chunk_blocks = chunk_blocks;
        plan_.key = key;
        const int Bc = chunk_blocks;
        std::vector<std::pair<int32_t, int32_t>> items;   // (sequence, slot) of one chunk
        for (long long c0 = 0; c0 < host_used; c0 += Bc) {
            const int c1 = (int)std::min<long long>(host_used, c0 + Bc);
            int first = -1, last = -1;
            for (int id = (int)c0; id < c1; ++id) {
                const int s = host_owner_s[id], j = host_owner_j[id];
                if (s < 0 || s >= n_seqs || j >= key[s]) continue;
                if (first < 0) first = id;
                last = id;
            }
            if (first < 0) continue;
            items.clear();
            for (int id = first; id <= last; ++id) {
                const int s = host_owner_s[id], j = host_owner_j[id];
                if (s < 0 || s >= n_seqs || j >= key[s]) continue;
                items.push_back({s, id - first});
            }
            std::stable_sort(items.begin(), items.end(),
                             [](const std::pair<int32_t, int32_t> &a, const std::pair<int32_t, int32_t> &b) {
                                 return a.first < b.first;
                             });
            Chunk ch;
            ch.first_id = first;
            ch.n_ids = last - first + 1;
            ch.unit_begin = (int32_t)plan_.cu_seq.size();
            for (size_t i = 0; i < items.size();) {
                size_t k = i;
                plan_.cu_seq.push_back(items[i].first);
                plan_.cu_beg.push_back((int32_t)plan_.cblk.size());
                while (k < items.size() && items[k].first == items[i].first)
                    plan_.cblk.push_back(items[k++].second);
                plan_.cu_end.push_back((int32_t)plan_.cblk.size());
                i = k;
            }
            ch.unit_end = (int32_t)plan_.cu_seq.size();
            plan_.chunks.push_back(ch);
            plan_.bytes_staged += (uint64_t)ch.n_ids * g.block_bytes;
        }
        account(layer, n_seqs);
        return plan_;
    }

private:
    uint64_t seed_ = 0;
    SplitMix64 rng_{0};
    std::vector<int32_t> hbm_order_;
    OffPlan plan_;

    void shuffle(int32_t *a, int n) {   // Fisher-Yates
        for (int i = n - 1; i > 0; --i) {
            const int k = (int)rng_.below((uint64_t)i + 1);
            std::swap(a[i], a[k]);
        }
    }

    void account(int layer, int n_seqs) {
        uint64_t res = 0, off = 0;
        for (int s = 0; s < n_seqs; ++s) {
            const int n = length(layer, s);
            if (n <= 0) continue;
            const int jn = (n - 1) / g.BT;
            uint64_t host_tokens = 0;
            for (int j = 0; j < jn; ++j) {
                const int32_t e = entry(s, j);
                if (e != ISV_BLOCK_NONE && (e & ISV_BLOCK_HOST_BIT)) host_tokens += g.BT;
            }
            off += host_tokens * g.kappa;
            res += ((uint64_t)n - host_tokens) * g.kappa;
        }
        plan_.bytes_resident = res;
        plan_.bytes_offloaded = off;
    }
};

// Fills the derived fields of a geometry from a description; returns an error
// text or nullptr.
inline const char *make_geometry(const isv_kv_desc &d, Geometry *out) {
    Geometry g;
    if (d.layers < 1) return "layers must be >= 1";
    g.layers = d.layers;
    g.phys_layers = d.phys_layers == 0 ? d.layers : d.phys_layers;
    if (g.phys_layers < 1 || g.phys_layers > g.layers) return "phys_layers must be in [1, layers]";
    if (d.kv_heads < 1 || d.q_heads < 1 || d.q_heads % d.kv_heads != 0)
        return "q_heads must be a positive multiple of kv_heads";
    g.Hq = d.q_heads;
    g.Hkv = d.kv_heads;
    g.G = g.Hq / g.Hkv;
    g.HP = pair_heads(g.G, d.head_dim, g.Hkv);
    g.GT = g.HP == 2 ? 2 : group_heads(g.G);
    g.P = g.HP == 2 ? 1 : g.G / g.GT;
    if (d.head_dim != 64 && d.head_dim != 80 && d.head_dim != 128) return "head_dim must be 64, 80 or 128";
    g.D = d.head_dim;
    if (d.block_tokens != 16) return "block_tokens must be 16";
    g.BT = d.block_tokens;
    if (d.dtype != ISV_F16 && d.dtype != ISV_BF16) return "dtype must be ISV_F16 or ISV_BF16";
    g.dtype = d.dtype;
    if (!(d.offload_frac >= 0.f && d.offload_frac <= 1.f)) return "offload_frac must be in [0, 1]";
    g.f = d.offload_frac;
    if (d.max_seqs < 1 || d.max_seqs > 4096) return "max_seqs must be in [1, 4096]";
    if (d.max_tokens_per_seq < 1 || d.max_tokens_per_seq > (1 << 24))
        return "max_tokens_per_seq must be in [1, 2^24]";
    g.max_seqs = d.max_seqs;
    g.max_tokens = d.max_tokens_per_seq;
    g.NB = (g.max_tokens + g.BT - 1) / g.BT;
    g.tile_bytes = (uint32_t)g.BT * g.D * 2u;
    g.block_bytes = 2ull * g.Hkv * g.tile_bytes;
    g.kappa = 2ull * g.Hkv * g.D * 2ull;
    const int host_per_seq = (int)std::floor((double)g.NB * (double)g.f);
    const long long hbm_cap = (long long)g.max_seqs * (g.NB - host_per_seq);
    const long long host_cap = (long long)g.max_seqs * host_per_seq;
    if (hbm_cap >= ISV_BLOCK_HOST_BIT || host_cap >= ISV_BLOCK_HOST_BIT) return "too many blocks";
    g.hbm_cap = (int)hbm_cap;
    g.host_cap = (int)host_cap;
    if (d.max_ctas < 0) return "max_ctas must be >= 0";
    g.max_ctas = d.max_ctas;
    if ((long long)g.max_seqs * g.NB * g.Hkv * g.P >= (1ll << 31)) return "max_seqs * blocks * heads too large";
    // default chunk: 128 MiB, or a layer's whole host pool where that is smaller (measured on B200: every copy
    // costs a few us of link idle time; 128 MiB chunks reach 0.994-0.996 of the probed link rate at the 13B and
    // OPT-2.7B shapes where 32 MiB chunks reach 0.988-0.992; copies of the next layer run ahead, so even one chunk
    // per layer keeps the link busy)
    const uint64_t pool_bytes = std::max<uint64_t>(g.block_bytes, (uint64_t)g.host_cap * g.block_bytes);
    g.chunk_bytes = d.chunk_bytes != 0 ? d.chunk_bytes : std::min<uint64_t>(128ull << 20, pool_bytes);
    g.chunk_blocks = (int)std::max<uint64_t>(1, g.chunk_bytes / g.block_bytes);
    g.chunk_bytes = (uint64_t)g.chunk_blocks * g.block_bytes;
    g.ring = d.ring_depth == 0 ? 3 : d.ring_depth;
    if (g.ring < 2 || g.ring > 16) return "ring_depth must be in [2, 16]";
    *out = g;
    return nullptr;
}

}  // namespace isv
