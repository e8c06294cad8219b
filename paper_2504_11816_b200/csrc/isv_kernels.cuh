// Kernel parameter blocks and launchers (sm_100a).  Host code fills the
// structs with plain pointers and sizes; nothing here owns memory.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

namespace isv {

constexpr int kMaxTableUpdates = 480;    // entries one update launch carries by value

enum DecodeMode : int { MODE_RESIDENT = 0, MODE_STAGED = 1 };

// One launch of the split decode kernel.
//   MODE_RESIDENT: the KV blocks of all (sequence, kv head x pass) pairs form
//     one flat list that is cut into equal contiguous ranges, one per warp; a
//     warp walks the block table for its range, reads HBM-pool blocks and a
//     host-flagged newest block from its tail slot, skips other host blocks.
//     A (sequence, head group) that spans several warps is finished by
//     whichever of them arrives last (ticket), which merges their partials.
//   A head group is the GT query heads one block visit serves: GT = 2..16 query heads that share a KV head,
//     on the tensor cores (group_heads picks GT); or, for multi-head attention, on the CUDA cores, one query
//     head with its KV head (GT = 1) or two adjacent ones, each with its own KV head (GT = 2, pair_heads).
//   MODE_STAGED: units are (chunk unit, kv head x pass) from the plan lists;
//     blocks are read from the staging buffer; results are merged into the
//     running state acc_o / acc_ml, which one unit per launch owns.
struct DecodeParams {
    const uint8_t *pool;        // resident: layer slab of the HBM pool; staged: staging buffer
    const uint8_t *tail;        // resident: layer slab of tail slots (NULL when nothing is offloaded)
    const int32_t *table;       // [n_seqs][table_stride]
    const int32_t *lens;        // [n_seqs] tokens to attend
    int32_t table_stride;
    int32_t max_blocks;         // resident: table entries of a row that may be read; lengths beyond
                                // max_blocks * BT tokens (or negative) are clamped and flagged
    int32_t n_pool_blocks;      // bound for block ids (pool blocks, or slots in the staging buffer)
    // staged mode lists
    const int32_t *cu_seq;
    const int32_t *cu_beg;
    const int32_t *cu_end;
    const int32_t *cblk;
    int32_t cu_first;
    int32_t cu_count;
    // fused append (resident mode, optional): when k_new is set, `lens` holds the lengths BEFORE
    // this step's token; the kernel stores the token's K/V rows into the cache, writes lens + 1 to
    // lens_out, and attends to the new token straight from k_new / v_new
    const void *k_new, *v_new;  // [n_seqs][Hkv][D] 16-bit, or NULL
    int32_t *lens_out;          // [lens_count]
    int32_t lens_count;         // entries of `lens` / `lens_out` per layer (>= n_seqs): those beyond n_seqs are
                                // copied over unchanged
    uint8_t *pool_w, *tail_w;   // writable aliases of pool / tail
    // several layers in one launch (resident mode with fused append only): n_layers > 1 makes the launch
    // cover logical layers layer0 .. layer0 + n_layers - 1 of one decode step.  The work list is then the
    // flat space of KV blocks ordered by (layer, sequence, head group, block), cut evenly over the grid's
    // warps as before, so the start-up and the tail of a launch are paid once per step instead of once per
    // layer.  q, k_new, v_new, out and out_f32 hold the layers back to back ([layer][n_seqs][heads][D]), so a
    // (layer, sequence) pair indexes them like a sequence number layer * n_seqs + s; `pool` / `tail` point at
    // physical slab 0 and layer l uses slab l % phys_layers; `lens` points at the first of two copies of
    // [layers][lens_layer_stride] lengths, bit l of lens_cur_mask says which copy is current for layer l, and
    // the advanced lengths go to the other one.  The host puts at most phys_layers layers into a launch, so
    // no two layers of a launch share a slab (were they to, only the last of them would store its token: the
    // earlier rows would be overwritten anyway and nothing in the launch reads them).
    int32_t n_layers;           // 0 or 1: one layer, the fields below are unused
    int32_t layer0, phys_layers;
    int32_t lens_layer_stride, lens_copy_stride;   // in elements
    uint64_t lens_cur_mask;
    uint64_t pool_layer_stride, tail_layer_stride; // bytes between physical slabs
    // inputs / outputs
    const void *q;              // [n_seqs][Hq][D] 16-bit
    void *out;                  // [n_seqs][Hq][D] 16-bit or NULL
    float *out_f32;             // [n_seqs][Hq][D] or NULL
    // scratch
    float *part_o;              // [2 * warps in grid][GT][D]   (a warp leaves at most two partials)
    float *part_ml;             // [2 * warps in grid][GT][2]
    int32_t *tickets;           // [n_seqs][Hkv*P], zero between launches
    float *acc_o;               // [n_seqs][Hq][D]  unnormalised result (resident, !finalize) / running state (staged)
    float *acc_ml;              // [n_seqs][Hq][2]
    uint32_t *status;
    int32_t n_seqs, Hq, Hkv, P;
    int32_t GT;                 // query heads of one head group (Hq = Hkv * P * GT / HP, HP = KV heads per group:
                                // fixed by the kernel variant, see pair_heads)
    int32_t finalize;           // resident: 1 = normalise and write out; 0 = leave (m, l, o) in acc_*
    int32_t early_reads;        // 1 = lengths, table and KV may be read before the dependency wait
    uint32_t spin_limit;        // polls after which a wait on a copy gives up (0 = default)
    int32_t drop_first_copy;    // failure injection: warp 0 of CTA 0 arms its first K slot without issuing
                                // the copy, as if the transfer had been lost (its wait then runs out)
    float scale_log2;           // log2(e) / sqrt(D)
    uint64_t block_bytes;
};

struct TableUpdateBatch {
    int32_t n;
    int32_t index[kMaxTableUpdates];
    int32_t value[kMaxTableUpdates];
};

struct AppendParams {
    const void *k, *v;          // [n_seqs][Hkv][D]
    uint8_t *pool;              // layer slab, HBM pool
    uint8_t *tail;              // layer slab, tail slots (may be NULL)
    const int32_t *table;
    int32_t *lens;              // [n_seqs], incremented by the kernel
    uint32_t *status;
    int32_t table_stride, n_pool_blocks;
    int32_t max_blocks;         // table entries of a row that may be read (a full sequence is flagged)
    int32_t n_seqs, Hkv, D, BT;
    uint64_t block_bytes;
};

struct FillParams {
    const void *k, *v;          // [n_seqs][T][Hkv][D]
    uint8_t *pool, *tail, *host; // layer slabs: HBM pool, tail slots, host pool (mapped; NULL = complete
                                 // host blocks are stored by the caller through PackParams instead)
    const int32_t *table;
    const int32_t *lens;        // [n_seqs] device
    uint32_t *status;
    int32_t table_stride, n_pool_blocks, n_host_blocks;
    int32_t n_seqs, T, Hkv, D, BT, max_blocks;
    uint64_t block_bytes;
};

// Packs complete host-resident blocks of a prompt into a staging buffer in host-id order, so that
// one device-to-host copy stores the whole run.
struct PackParams {
    const void *k, *v;          // [n_seqs][T][Hkv][D]
    const int32_t *owner;       // [host blocks][2]: (sequence, logical block) of each host block id
    uint8_t *dst;               // staging buffer; block b of the run goes to dst + b * block_bytes
    int32_t first_id, n_ids;    // the run of host block ids
    int32_t T, Hkv, D, BT;
    uint64_t block_bytes;
};

struct GatherParams {
    void *k_out, *v_out;        // [len][Hkv][D] device
    const uint8_t *pool, *tail, *host;
    const int32_t *table;       // row of the sequence
    uint32_t *status;
    int32_t seq, len, n_pool_blocks, n_host_blocks;
    int32_t Hkv, D, BT;
    uint64_t block_bytes;
};

struct MergeParams {
    const float *res_o, *res_ml;    // resident result (m, l, o)
    const float *run_o, *run_ml;    // offloaded running state; l == 0 means empty
    void *out;
    float *out_f32;
    int32_t rows, D, bf16;
};

// Query heads handled together on one KV tile, for G query heads per KV head: the largest divisor of G
// that is at most 16 (the row count of the tensor-core tile), so up to 16 heads read their KV once.
inline int group_heads(int G) {
    for (int gt = G < 16 ? G : 16; gt > 1; --gt)
        if (G % gt == 0) return gt;
    return 1;
}

// KV heads whose tiles one block visit carries, for G query heads per KV head: 2 for multi-head attention
// (G = 1) at head_dim 64 and 80 with an even head count - adjacent heads' tiles are contiguous in a block, one
// copy brings both, and each is attended by its own query head, which halves the per-visit bookkeeping per
// byte where tiles are small - else 1.  With 2, a head group is those two query heads (GT = 2).
inline int pair_heads(int G, int D, int Hkv) {
    if (const char *e = getenv("ISV_PAIR_HEADS"))   // tuning knob: 0 = one KV head per visit everywhere
        if (atoi(e) == 0) return 1;
    return (G == 1 && D < 128 && Hkv % 2 == 0) ? 2 : 1;
}

// Warps per CTA of the decode kernel that handles GT query heads per visit at head_dim D (HP: pair_heads).
int decode_warps(int GT, int D, int HP);

// Ring depth per warp (tile slots, an even number: a block visit takes a K and a V slot) that keeps about
// 128 KiB of copies in flight per SM (measured on B200: deeper rings lower the achieved HBM rate).
int decode_default_stages(int D, int BT, int GT, int HP);

// Bytes of dynamic shared memory the decode kernel needs for `stages` ring
// stages (one K or V tile each) per warp.
size_t decode_smem_bytes(int D, int BT, int GT, int HP, int stages, int max_seqs, int mode);   // max_seqs: sequences x layers of a launch

// Launchers return the CUDA error of the launch.
cudaError_t decode_configure(int D, int GT, int HP, int BT, bool bf16, int mode, size_t smem);
cudaError_t launch_decode(const DecodeParams &p, int D, int GT, int HP, int BT, bool bf16, int mode,
                          int grid, int stages, size_t smem, cudaStream_t st);
cudaError_t launch_table_update(int32_t *table, const TableUpdateBatch &b, cudaStream_t st);
cudaError_t launch_append(const AppendParams &p, cudaStream_t st);
cudaError_t launch_fill(const FillParams &p, cudaStream_t st);
cudaError_t launch_gather(const GatherParams &p, cudaStream_t st);
cudaError_t launch_pack(const PackParams &p, cudaStream_t st);
cudaError_t launch_merge(const MergeParams &p, cudaStream_t st);

}  // namespace isv
