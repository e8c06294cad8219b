/*
 * isv.h - decode attention over a paged KV cache that is split between GPU HBM
 * and pinned host memory (KV cache offloading), for NVIDIA B200 (sm_100a).
 *
 * The library executes the computation whose time the InferSave cost model
 * predicts per layer and decode step (paper Section IV-C, Eq. 6):
 *     T_dec = CTCF(T_compute^d) + T_trans^d
 * i.e. the self-attention part of T_compute^d (4 * BS * ctx * h1 flops) over a
 * KV cache of which the fraction C_off (Section IV-B) lives in CPU memory and
 * must cross the host link (T_trans^d) every step.
 *
 * Conventions
 *   - All entry points return 0 (ISV_OK) or a negative ISV_E* code; the text of
 *     the last error of the calling thread is available from isv_last_error().
 *     Nothing aborts, throws across the boundary or traps on the device.
 *   - "device" pointers are CUDA device addresses on the GPU that was current
 *     when the handle was created; "host" pointers are ordinary CPU addresses.
 *   - Work is enqueued on the handle's compute stream (and on internal copy
 *     streams) and is asynchronous unless a function says it synchronises.
 *     Caller-owned buffers must stay valid until that work has completed.
 *   - K/V/q/out elements are 16-bit (fp16 or bf16, chosen at allocation);
 *     arithmetic is fp32.
 *   - KV pool layout, per physical layer and pool (HBM pool, host pool):
 *         [block][K|V][kv_head][block_tokens][head_dim]
 *     so one (block, K-or-V, head) tile is contiguous.  Inside a tile the row
 *     of token t (head_dim elements) is stored as 16-byte chunks, and chunk c
 *     sits at chunk position c XOR (t mod 8) of that row (head_dim 80: chunks
 *     0..7 only; chunks 8 and 9 stay in place): the arrangement
 *     that lets the tensor-core path load eight tokens at once without
 *     shared-memory bank conflicts.  isv_kv_fill / isv_kv_append / isv_kv_gather
 *     apply it; only a caller that builds a pool itself
 *     (isv_attn_decode_static) has to.
 *   - Block table entry (int32): ISV_BLOCK_NONE = not allocated; otherwise the
 *     physical block id, with ISV_BLOCK_HOST_BIT set when the block belongs to
 *     the host pool.  The block that holds a sequence's newest token is kept in
 *     GPU memory even when it is host-flagged (it is still being written); it
 *     is copied to the host pool when it becomes full.
 */
#ifndef ISV_H
#define ISV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ISV_OK               0
#define ISV_EINVAL          (-1)   /* bad argument                                   */
#define ISV_ENOMEM_DEVICE   (-2)   /* cudaMalloc refused                             */
#define ISV_ENOMEM_PINNED   (-3)   /* pinned host allocation refused (by the system, or because it  */
                                   /* exceeds the environment variable ISV_PINNED_LIMIT_BYTES)      */
#define ISV_ECAPACITY       (-4)   /* sequence or pool would exceed its capacity     */
#define ISV_ECUDA           (-5)   /* a CUDA runtime call failed                     */
#define ISV_ETIMEOUT        (-6)   /* a host-side wait exceeded isv_set_host_timeout */
#define ISV_EDEVICE_STATUS  (-7)   /* a kernel reported a problem (see status bits)  */
#define ISV_ENODEVICE       (-8)   /* compute requested on a plan-only handle        */

#define ISV_F16   0
#define ISV_BF16  1

#define ISV_BLOCK_NONE      (-1)
#define ISV_BLOCK_HOST_BIT  (1 << 30)

/* bits of the device status word (isv_step_times.status, isv_sync, isv_linear_status) */
#define ISV_STATUS_BAD_BLOCK_ID  1u   /* a table entry pointed outside its pool; block skipped */
#define ISV_STATUS_WAIT_EXPIRED  2u   /* a bounded wait inside a kernel gave up                */
#define ISV_STATUS_BAD_LENGTH    4u   /* a device-side sequence length was negative or exceeded */
                                      /* the table row; it was clamped to what the row covers  */

typedef struct isv_kv isv_kv;   /* opaque; created by isv_kv_alloc, destroyed by isv_kv_free */

/*
 * Problem statement of one cache (paper Table II: model shape, batch size,
 * input/output lengths, precision; Section IV-B: offload ratio).
 */
typedef struct {
    int32_t  layers;             /* logical layers (n)                                          */
    int32_t  phys_layers;        /* physical KV slabs; 0 = layers.  Logical layer l uses slab   */
                                 /* l % phys_layers (lets a benchmark hold fewer slabs than     */
                                 /* layers; layers sharing a slab overwrite each other's data)  */
    int32_t  q_heads;            /* query heads; multiple of kv_heads                           */
    int32_t  kv_heads;
    int32_t  head_dim;           /* 64, 80 (OPT-2.7B, the paper's main model: h1 2560 / 32) or 128 */
    int32_t  block_tokens;       /* tokens per KV block; 16                                     */
    int32_t  dtype;              /* ISV_F16 or ISV_BF16                                         */
    float    offload_frac;       /* C_off in [0, 1]: of every prefix of j blocks of a sequence, */
                                 /* floor(j * C_off) are host-resident                          */
    int32_t  max_seqs;           /* capacity in sequences (BS), <= 4096                         */
    int32_t  max_tokens_per_seq; /* capacity per sequence (L_in + L_out)                        */
    uint64_t perm_seed;          /* 0 = physical block ids handed out in order; otherwise they  */
                                 /* follow a seeded permutation (host pool ids stay compact)    */
    uint64_t chunk_bytes;        /* staging chunk size; 0 = 128 MiB or a layer's host pool if smaller */
    int32_t  ring_depth;         /* staging ring buffers; 0 = 3                                 */
    int32_t  max_ctas;           /* cap on the resident kernel's grid; 0 = one CTA per SM.      */
                                 /* The KV blocks are cut evenly over the grid's warps, so this */
                                 /* also sets into how many splits a sequence falls             */
    int32_t  plan_only;          /* 1 = host bookkeeping only: no CUDA call is made, no memory  */
                                 /* is allocated, compute entry points return ISV_ENODEVICE     */
    void    *compute_stream;     /* cudaStream_t to enqueue on, or NULL = library creates one   */
                                 /* (the legacy default stream, handle 0, cannot be passed)     */
} isv_kv_desc;

/* Sizes the library derived from a description (filled by isv_kv_info). */
typedef struct {
    uint64_t block_bytes;        /* one block: 2 * kv_heads * block_tokens * head_dim * 2 B     */
    uint64_t kv_bytes_per_token; /* K and V of one token in one layer                           */
    int32_t  max_blocks_per_seq;
    int32_t  hbm_blocks;         /* HBM pool capacity per physical layer, in blocks             */
    int32_t  host_blocks;        /* host pool capacity per physical layer, in blocks            */
    int32_t  hbm_blocks_used;
    int32_t  host_blocks_used;
    uint64_t hbm_pool_bytes;     /* all physical layers, tail slots included                    */
    uint64_t host_pool_bytes;    /* all physical layers                                         */
    uint64_t scratch_bytes;      /* split partials, running state, staging ring                 */
    int32_t  phys_layers;
    int32_t  max_ctas;
    int32_t  ring_depth;
    int32_t  sm_count;
    uint64_t chunk_bytes;
    uint64_t kernel_launches;    /* kernels this handle has launched since it was created       */
} isv_kv_info_t;

/*
 * Per-layer timing of the most recent decode of that layer, and what the
 * paper's terms are for it: h2d_ms is T_trans^d, attn_resident_ms +
 * attn_offloaded_ms + merge_ms is the self-attention part of T_compute^d,
 * total_ms is T_dec without the linear layers.  Byte counters: bytes_resident
 * and bytes_offloaded are the KV bytes the attention had to read from HBM and
 * to fetch over the host link; bytes_offloaded equals the first term of the
 * T_trans^d numerator, C_off * 2 * L * h1 * Precision * BS, counted per block.
 * bytes_staged is what the copy engine actually moved (whole chunks).
 */
typedef struct {
    float    append_ms;           /* 0 when the append was fused into the attention kernel */
    float    h2d_ms;
    float    attn_resident_ms;
    float    attn_offloaded_ms;
    float    merge_ms;
    float    total_ms;
    uint64_t bytes_resident;
    uint64_t bytes_offloaded;
    uint64_t bytes_staged;
    uint64_t bytes_appended;
    int32_t  n_chunks;
    uint32_t status;
} isv_step_times;

/* ---- lifetime ---------------------------------------------------------- */

/* Allocates pools (HBM, pinned host), block tables, scratch, staging ring,
 * streams and events on the current device.  Synchronous.  *out is NULL on
 * failure.  The handle must be used from one host thread at a time. */
int isv_kv_alloc(isv_kv **out, const isv_kv_desc *desc);

/* Waits for all work of the handle, then frees everything it owns. */
int isv_kv_free(isv_kv *h);

/* Forgets all sequences (lengths 0, all blocks free).  Synchronises. */
int isv_kv_reset(isv_kv *h);

int isv_kv_info(isv_kv *h, isv_kv_info_t *out);

/* ---- loading and appending (the KV cache of Section II-A) --------------- */

/* Prompt load for one layer (prefill's KV, not timed): k, v are device arrays
 * [n_seqs][T][kv_heads][head_dim]; lens_host[s] <= T tokens of sequence s are
 * kept and replace what the layer held for s.  Blocks are allocated by the
 * residency rule on first use and shared by all layers.  Synchronises. */
int isv_kv_fill(isv_kv *h, int32_t layer, const void *k_dev, const void *v_dev,
                const int32_t *lens_host, int32_t n_seqs, int32_t T);

/* The same load without the final wait: returns once the work is enqueued (k_dev and v_dev must stay valid
 * until isv_sync or isv_fill_timing).  Resident blocks are written by a kernel; the complete host-resident
 * blocks - the share C_off of the prompt's KV that the paper's prefill stage stores to CPU memory,
 * T_trans^p = C_off * 2 * (L_in + 1) * h1 * Precision * BS / BW_gpu->cpu (Section IV-C) - are packed into
 * the staging ring in host-block order and stored by device-to-host copies on the write-back stream, so
 * that the store overlaps whatever the caller computes next (the paper's Eq. 5 takes the max of both). */
int isv_kv_fill_async(isv_kv *h, int32_t layer, const void *k_dev, const void *v_dev,
                      const int32_t *lens_host, int32_t n_seqs, int32_t T);

/* Timing of the latest isv_kv_fill / isv_kv_fill_async: store_ms is the measured T_trans^p of that layer
 * (first to last device-to-host copy), bytes_stored its numerator counted per block.  Synchronises. */
typedef struct {
    float    pack_ms;          /* kernels: resident blocks, tails, packing of host blocks */
    float    store_ms;         /* device-to-host copies, first start to last end          */
    float    total_ms;         /* start of the load to the end of its last copy           */
    uint64_t bytes_stored;     /* KV bytes written to the host pool                       */
    uint64_t bytes_resident;   /* KV bytes written to GPU memory                          */
    int32_t  n_copies;
} isv_fill_times;
int isv_fill_timing(isv_kv *h, isv_fill_times *out);

/* Appends one token to sequences 0..n_seqs-1 of one layer at that layer's
 * current lengths (the cache growth of one decode step): k, v are device
 * arrays [n_seqs][kv_heads][head_dim].  K and V are written by one kernel; the
 * copy is bit-exact.  ISV_ECAPACITY if a sequence is full. */
int isv_kv_append(isv_kv *h, int32_t layer, const void *k_dev, const void *v_dev,
                  int32_t n_seqs);

/* ---- decode attention (self-attention term of T_compute^d; T_trans^d) ---- */

/* out[s][h][:] = softmax(q[s][h] . K_s^T / sqrt(head_dim)) V_s over the
 * layer's current tokens of sequence s (the newest token included), for
 * s < n_seqs.  q_dev: [n_seqs][q_heads][head_dim] 16-bit; out_dev (same shape
 * and dtype) and out_f32_dev (fp32) may each be NULL but not both.  Query head
 * h reads KV head h / (q_heads / kv_heads).  A sequence of length 0 yields
 * zeros.  Host-resident blocks are streamed through the staging ring on the
 * copy stream while the resident blocks are processed; partial results are
 * combined by a log-sum-exp merge.
 * block_table_dev / seq_lens_dev: NULL = the library's own (normal use).  If
 * given, they replace the library's device arrays for the resident kernel
 * (same format, row stride as isv_block_table_dev reports) and must agree with
 * the library's bookkeeping on lengths and on host-resident entries. */
int isv_attn_decode(isv_kv *h, int32_t layer, const void *q_dev, void *out_dev,
                    float *out_f32_dev, const int32_t *block_table_dev,
                    const int32_t *seq_lens_dev, int32_t n_seqs);

/* isv_kv_append followed by isv_attn_decode for one layer, as one kernel: the
 * resident attention kernel also stores the new token's K/V rows and advances
 * the lengths, and attends to the new token straight from k_dev / v_dev, so
 * the step needs one launch per layer instead of two.  Same arguments and
 * result as the two calls (up to fp32 summation order). */
int isv_decode_layer(isv_kv *h, int32_t layer, const void *q_dev, const void *k_dev, const void *v_dev,
                     void *out_dev, float *out_f32_dev, int32_t n_seqs);

/* Second design point for the offloaded part: with on = 1 the host-resident blocks are not staged
 * through the ring by the copy engine; the attention kernel's bulk copies read them in place from the
 * mapped pinned pool, over the host link.  No HBM staging traffic and no copy-engine work, but the link
 * is driven by SM-issued reads.  Results are the same; isv_step_timing then reports h2d_ms = 0 and the
 * link time inside attn_offloaded_ms.  Off by default. */
int isv_set_zero_copy(isv_kv *h, int32_t on);

/* One decode step of all layers: the result of isv_decode_layer for l in 0..layers-1.
 * Device arrays: q, out (16-bit) and out_f32 (fp32) [layers][n_seqs][q_heads][head_dim];
 * k, v [layers][n_seqs][kv_heads][head_dim].  out_dev and out_f32_dev may each be NULL, not both.
 * Because all layers' inputs are handed over at once, the resident attention (and the appends) of up to
 * phys_layers consecutive layers run as ONE launch whose work list spans those layers: the start-up and
 * the tail of a launch are then paid once per step instead of once per layer, which matters when a
 * layer's KV is read in under 100 microseconds.  With offloaded blocks each layer's staged launches and
 * merge follow that launch, and the copy engine's queue is filled for all of them at once.  (Layers that
 * share a physical slab are never put into one launch.  With offload_frac = 0 and per-layer timing on it
 * is one launch per layer.)  A caller whose layers depend on one another (a real model) uses
 * isv_decode_layer per layer. */
int isv_decode_step(isv_kv *h, const void *q_dev, const void *k_dev, const void *v_dev,
                    void *out_dev, float *out_f32_dev, int32_t n_seqs);

/* The same step with HOST buffers of the same shapes (pinned memory gives
 * asynchronous copies): inputs are copied to library-owned device buffers a
 * few layers at a time on a copy stream while earlier layers compute, and
 * each group's result is copied back as soon as it is ready.  Returns after
 * the whole result is in out_host (synchronises).  The first call on a handle
 * allocates the device buffers for one step's q, k, v and out (cudaMalloc,
 * counted in isv_kv_info's scratch_bytes) and a copy stream; make it outside
 * any region that must not allocate. */
int isv_decode_step_host(isv_kv *h, const void *q_host, const void *k_host,
                         const void *v_host, void *out_host, int32_t n_seqs);

/* ---- inspection --------------------------------------------------------- */

/* Logical-order copy of one sequence's K and V of one layer to host arrays
 * [len][kv_heads][head_dim] (capacity max_tokens_per_seq rows each).
 * Bit-exact; synchronises. */
int isv_kv_gather(isv_kv *h, int32_t layer, int32_t seq, void *k_host, void *v_host,
                  int32_t *len_out);

/* Library-maintained device arrays: table [max_seqs][*row_stride] int32 and
 * one layer's lengths [max_seqs] int32.  NULL on a plan-only handle. */
const int32_t *isv_block_table_dev(isv_kv *h, int32_t *row_stride);
const int32_t *isv_seq_lens_dev(isv_kv *h, int32_t layer);

/* Host copies of the same (work on plan-only handles too). */
int isv_block_table_host(isv_kv *h, int32_t *out, int32_t n_seqs, int32_t row_stride);
int isv_seq_lens_host(isv_kv *h, int32_t layer, int32_t *out, int32_t n_seqs);

/* KV bytes a decode of this layer over n_seqs sequences would read now:
 * resident (HBM) and offloaded (host link) algorithmic bytes, the bytes the
 * staging engine would copy, and its chunk count.  Any pointer may be NULL. */
int isv_plan_bytes(isv_kv *h, int32_t layer, int32_t n_seqs, uint64_t *bytes_resident,
                   uint64_t *bytes_offloaded, uint64_t *bytes_staged, int32_t *n_chunks);

/* ---- timing (feeds the terms of Eq. 6) ----------------------------------- */

/* Turns event recording per layer on or off (off by default: events cost a
 * little on short steps). */
int isv_set_timing(isv_kv *h, int32_t on);

/* Times of the latest decode of `layer`, or with layer = -1 the sums over all
 * layers (total_ms then spans first layer start to last layer end).
 * Synchronises.  Times are 0 where timing was off. */
int isv_step_timing(isv_kv *h, int32_t layer, isv_step_times *out);

/* Waits for everything enqueued by the handle; returns ISV_EDEVICE_STATUS if
 * a kernel flagged a problem since the last call (bits in *status_out). */
int isv_sync(isv_kv *h, uint32_t *status_out);

/* ---- failure handling ----------------------------------------------------- */

/* (The paper treats only predicted out-of-memory, Algorithm 1's "Unsuitable" case, which isv_kv_alloc's
 * ISV_ENOMEM_* codes mirror; it has no counterpart for what follows.  These calls keep a lost transfer or
 * a stuck stream from turning into a hang: every wait of the library, on the device and on the host, can
 * be given a limit, and running into it is reported as a status or an error code with the handle intact.) */

/* Limit, in seconds, of every host-side wait of this handle (isv_sync, isv_step_timing, isv_kv_fill,
 * isv_fill_timing, isv_kv_gather, isv_decode_step_host): a wait that exceeds it returns ISV_ETIMEOUT
 * and leaves the work enqueued, so the caller can wait again, report, or tear down.  0 (the default)
 * waits without limit.  The wait polls the stream instead of blocking in the driver. */
int isv_set_host_timeout(isv_kv *h, double seconds);

/* Limit of a device-side wait for a K/V copy, in polls of its barrier (0 = the built-in default, about
 * 4 million polls, i.e. seconds).  A warp whose wait runs out sets ISV_STATUS_WAIT_EXPIRED, gives its
 * other copies one more bounded chance to land and leaves the kernel; the handle stays usable and the
 * next isv_sync / isv_step_timing returns ISV_EDEVICE_STATUS once and clears the state.  The outputs of
 * that launch are incomplete. */
int isv_set_wait_limit(isv_kv *h, uint32_t polls);

/* Failure injection for tests of the path above: in each of the next `launches` resident attention
 * launches one warp arms the barrier of its first K tile without issuing the copy, as if the transfer
 * had been lost; its wait then runs out after the limit set by isv_set_wait_limit.  Nothing faults
 * and nothing hangs. */
int isv_inject_lost_copy(isv_kv *h, int32_t launches);

/* Measures pinned host<->device copy bandwidth on the current device: `bytes`
 * per copy, best of `reps`, CUDA events.  This is the measured host-link rate
 * that T_trans^d's BW_cpu->gpu stands for.  Allocates and frees its buffers. */
int isv_link_probe(uint64_t bytes, int32_t reps, double *h2d_gbs, double *d2h_gbs);

/* ---- decode linear layers (linear-layer term of T_compute^d) -------------- */

/* y = x . w^T for a batch of M <= max_M <= 256 tokens: the QKV / output / MLP projections whose
 * flops the paper counts as BS * (8 h1^2 + 4 h1 h2) per layer (Section IV-C, T_compute^d).  At
 * decode batch sizes the product is bound by reading w once from HBM; it runs on the tensor cores
 * (tcgen05, fp32 accumulation in tensor memory) so that the arithmetic keeps up with that read.
 *   w_dev  [N][K] 16-bit row-major (the usual weight layout), N and K multiples of 128;
 *          must stay valid and unchanged while the handle lives
 *   x_dev  [M][K] 16-bit;  y_dev [M][N] 16-bit and / or y_f32_dev [M][N] fp32 (one may be NULL)
 * isv_linear_create allocates split-K scratch and encodes the weight's tensor map (synchronous);
 * isv_linear_forward enqueues the streaming kernel and, where tiles of the output are shared by
 * several CTAs, a small kernel that adds their partial sums, on `stream` (asynchronous, no host
 * wait); isv_linear_status waits for the stream and returns ISV_EDEVICE_STATUS if a bounded wait
 * inside the kernel expired. */
typedef struct isv_linear isv_linear;
int isv_linear_create(isv_linear **out, const void *w_dev, int32_t N, int32_t K, int32_t dtype,
                      int32_t max_M, void *stream);
int isv_linear_forward(isv_linear *l, const void *x_dev, void *y_dev, float *y_f32_dev, int32_t M);
int isv_linear_status(isv_linear *l, uint32_t *status_out);
int isv_linear_free(isv_linear *l);

/* ---- decode attention for callers that cannot allocate ------------------- */

/* Size of the fixed device array that holds this entry point's scratch.  Every
 * GPU on which the library is loaded keeps this much memory until the process
 * exits, whether or not the entry point is ever called. */
#define ISV_STATIC_SCRATCH_BYTES (8u << 20)

/* (The paper has no counterpart for this call: it is a packaging variant of
 * isv_attn_decode's resident kernel, added for deployment reasons.)
 *
 * Some callers may not call cudaMalloc: a serving process that has handed all
 * of its GPU memory to a framework's caching allocator, a latency-critical
 * loop in which an allocation would stall the device, a plugin that is given
 * pointers and a stream and nothing else.  This call is for them.  It makes no
 * cudaMalloc / cudaFree / cudaHostAlloc and uses no allocating library call;
 * it needs no handle.  The caller owns and passes every buffer:
 *   kv_pool_dev      KV pool in the library's layout,
 *                    [n_pool_blocks][K|V][kv_heads][block_tokens][head_dim], 16-bit,
 *                    with the 16-byte chunks of each token row permuted as
 *                    described under "KV pool layout" above
 *   block_table_dev  int32 [n_seqs][table_stride]: pool block ids in logical
 *                    order (ISV_BLOCK_NONE or host-flagged entries are skipped;
 *                    ids outside the pool are skipped and flagged)
 *   seq_lens_dev     int32 [n_seqs]: tokens to attend; at most
 *                    max_blocks_per_seq * block_tokens each (the table rows must
 *                    cover them)
 *   q_dev            [n_seqs][q_heads][head_dim] 16-bit
 *   out_dev / out_f32_dev   same shape, 16-bit / fp32; either may be NULL, not both
 *   status_dev       optional uint32 the kernel ORs ISV_STATUS_* bits into
 *                    (the caller clears it); NULL = not reported
 *   stream           cudaStream_t the work is enqueued on (asynchronous)
 * max_ctas: cap on the kernel's grid, 0 = one CTA per SM.
 * The split kernel's partial results and arrival counters live in one fixed
 * device array of ISV_STATIC_SCRATCH_BYTES:
 *   n_seqs * (q_heads / heads per warp) * 4 B of counters
 *   + 2 * warps in the grid * heads per warp * (head_dim + 2) * 4 B of partials.
 * When the partials of a full grid do not fit, the grid is cut down to the
 * CTAs whose partials do (the kernel divides the work among the CTAs it
 * gets).  A shape that leaves no room for a single CTA is refused with
 * ISV_ECAPACITY and a message; nothing runs then.
 * All calls on a GPU share that array and it keeps the previous call's
 * contents; each call zeroes the counters it needs on `stream` first.  Two
 * calls whose GPU work overlaps (different streams, or different threads
 * without ordering) race on it: order them on one stream or with events.
 * The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress) and the device limits; make that first call with the
 * device current and before starting any stream capture. */
int isv_attn_decode_static(const void *kv_pool_dev, int32_t n_pool_blocks,
                           const int32_t *block_table_dev, int32_t table_stride,
                           const int32_t *seq_lens_dev, int32_t n_seqs, int32_t max_blocks_per_seq,
                           int32_t q_heads, int32_t kv_heads, int32_t head_dim, int32_t block_tokens,
                           int32_t dtype, int32_t max_ctas, const void *q_dev, void *out_dev,
                           float *out_f32_dev, uint32_t *status_dev, void *stream);

/* Text of the calling thread's last error; valid until its next call. */
const char *isv_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ISV_H */
