// C ABI of the library (include/isv.h): handle, pools, staging engine,
// stream/event plumbing.  All arithmetic runs in the kernels of
// isv_kernels.cu; there is no CPU path for attention.
#include <cuda_runtime.h>

#include <chrono>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "../../include/isv.h"
#include "isv_host.hpp"
#include "isv_kernels.cuh"

using namespace isv;

namespace {

thread_local std::string g_err;

int fail(int code, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

#define CU(call)                                                                          \
    do {                                                                                  \
        cudaError_t e_ = (call);                                                          \
        if (e_ != cudaSuccess) return fail(ISV_ECUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
    } while (0)

constexpr int kPlanSlots = 4;

struct PlanSlot {
    int32_t *host = nullptr;     // pinned staging of the plan lists
    int32_t *dev = nullptr;
    size_t cap = 0;              // int32 capacity
    cudaEvent_t used = nullptr;  // recorded after the last kernel that reads `dev`
    bool used_recorded = false;
    uint64_t version = 0;        // plan version held (0 = none)
    int32_t off_seq = 0, off_beg = 0, off_end = 0, off_blk = 0;
};

struct LayerEvents {
    cudaEvent_t a0, a1, d0, d1, r0, r1, c0, c1, o0, o1, m0, m1;
    bool have_append = false, have_decode = false, have_off = false, fused_append = false;
    uint64_t bytes_res = 0, bytes_off = 0, bytes_staged = 0, bytes_app = 0;
    int n_chunks = 0;
};

}  // namespace

struct isv_kv {
    Geometry g;
    BlockManager bm;
    bool plan_only = false;
    int device = 0, sm_count = 0;
    // device memory
    uint8_t *pool_hbm = nullptr, *tail = nullptr;
    uint8_t *pool_host = nullptr, *pool_host_dev = nullptr;   // pinned host pool and its device alias
    int32_t *table_dev = nullptr, *lens_dev = nullptr;   // lens_dev: two copies of [layers][max_seqs]
    std::vector<char> lens_cur;            // per layer: which copy is current
    uint32_t *status_dev = nullptr;
    float *part_o = nullptr, *part_ml = nullptr, *res_o = nullptr, *res_ml = nullptr, *run_o = nullptr,
          *run_ml = nullptr;
    int32_t *tickets = nullptr;
    uint8_t *stage = nullptr;              // ring * chunk_bytes
    uint8_t *step_buf = nullptr;           // device copies of one step's q, k, v, out (host-buffer entry point)
    uint64_t hbm_pool_bytes = 0, host_pool_bytes = 0, scratch_bytes = 0;
    // streams and events
    cudaStream_t s_compute = nullptr, s_copy = nullptr, s_off = nullptr, s_d2h = nullptr, s_in = nullptr;
    std::vector<cudaEvent_t> ev_step_in, ev_step_out;   // host-buffer step: per group of layers
    bool own_compute = false;
    std::vector<cudaEvent_t> ev_ready, ev_freed;
    std::vector<char> freed_recorded;
    cudaEvent_t ev_q = nullptr, ev_off_done = nullptr, ev_app = nullptr;
    std::vector<cudaEvent_t> ev_flush;     // per physical layer
    std::vector<char> flush_recorded;
    uint64_t chunk_counter = 0;
    bool zero_copy = false;                // offloaded blocks are read in place over the host link, no staging
    // prompt write-back (device -> host) through the same ring
    std::vector<cudaEvent_t> ev_packed, ev_stored;
    std::vector<char> stored_recorded;
    int32_t *owner_dev = nullptr;          // [host_cap][2]: (sequence, block) of each host block id
    int owner_uploaded = -1;               // host blocks in use when owner_dev was last uploaded
    uint64_t store_counter = 0;
    cudaEvent_t ev_f0 = nullptr, ev_f1 = nullptr, ev_s0 = nullptr, ev_s1 = nullptr;   // timing of the latest fill
    bool fill_timed = false, fill_stored = false;
    uint64_t fill_bytes_stored = 0, fill_bytes_resident = 0;
    int fill_copies = 0;
    PlanSlot plan_slot[kPlanSlots];
    int plan_cur = -1;
    // kernel configuration
    int stages_res = 0, stages_stg = 0;
    size_t smem_res = 0, smem_stg = 0;
    int smem_limit = 0;                    // opt-in shared memory per block of the device
    int res_layers = 1;                    // layers the resident-result and running-state buffers hold
    uint64_t launches = 0;                 // kernels launched so far
    int last_fused_layer = -1;             // layer of the latest fused decode launch if nothing else of ours
                                           // was launched on the compute stream since, else -1
    // failure handling
    double host_timeout_s = 0.0;           // limit of a host-side wait; 0 = none
    uint32_t spin_limit = 0;               // device-side wait limit in polls; 0 = the kernels' default
    int lost_copies = 0;                   // failure injection: resident launches still to lose a copy
    // timing
    bool timing = false;
    std::vector<LayerEvents> lev;
    bool lev_created = false;
};

namespace {

// Device lengths of one layer: the current copy (which = 0) or the other one (which = 1).  The fused
// append + attention kernel reads the current copy and writes the other, then they swap.
int32_t *lens_ptr(const isv_kv *h, int layer, int which) {
    const int copy = (h->lens_cur[layer] ^ which) & 1;
    return h->lens_dev + ((size_t)copy * h->g.layers + layer) * h->g.max_seqs;
}

size_t tickets_bytes(const Geometry &g) { return (size_t)g.layers * g.max_seqs * g.Hkv * g.P * 4; }

size_t slab_hbm(const isv_kv *h, int layer) {
    return (size_t)(layer % h->g.phys_layers) * h->g.hbm_cap * h->g.block_bytes;
}
size_t slab_tail(const isv_kv *h, int layer) {
    return (size_t)(layer % h->g.phys_layers) * h->g.max_seqs * h->g.block_bytes;
}
size_t slab_host(const isv_kv *h, int layer) {
    return (size_t)(layer % h->g.phys_layers) * h->g.host_cap * h->g.block_bytes;
}

void destroy(isv_kv *h) {
    if (!h) return;
    if (!h->plan_only) {
        if (h->s_compute) cudaStreamSynchronize(h->s_compute);
        if (h->s_copy) cudaStreamSynchronize(h->s_copy);
        if (h->s_off) cudaStreamSynchronize(h->s_off);
        if (h->s_d2h) cudaStreamSynchronize(h->s_d2h);
        if (h->s_in) cudaStreamSynchronize(h->s_in);
        cudaFree(h->pool_hbm); cudaFree(h->tail); cudaFree(h->table_dev); cudaFree(h->lens_dev);
        cudaFree(h->status_dev); cudaFree(h->part_o); cudaFree(h->part_ml); cudaFree(h->res_o);
        cudaFree(h->res_ml); cudaFree(h->run_o); cudaFree(h->run_ml); cudaFree(h->tickets);
        cudaFree(h->stage); cudaFree(h->step_buf); cudaFree(h->owner_dev);
        for (auto e : h->ev_packed) cudaEventDestroy(e);
        for (auto e : h->ev_stored) cudaEventDestroy(e);
        for (cudaEvent_t e : {h->ev_f0, h->ev_f1, h->ev_s0, h->ev_s1}) if (e) cudaEventDestroy(e);
        if (h->pool_host) cudaFreeHost(h->pool_host);
        for (auto &ps : h->plan_slot) {
            if (ps.host) cudaFreeHost(ps.host);
            cudaFree(ps.dev);
            if (ps.used) cudaEventDestroy(ps.used);
        }
        for (auto e : h->ev_ready) cudaEventDestroy(e);
        for (auto e : h->ev_freed) cudaEventDestroy(e);
        for (auto e : h->ev_flush) cudaEventDestroy(e);
        for (auto e : h->ev_step_in) cudaEventDestroy(e);
        for (auto e : h->ev_step_out) cudaEventDestroy(e);
        if (h->s_in) cudaStreamDestroy(h->s_in);
        if (h->ev_q) cudaEventDestroy(h->ev_q);
        if (h->ev_off_done) cudaEventDestroy(h->ev_off_done);
        if (h->ev_app) cudaEventDestroy(h->ev_app);
        if (h->lev_created)
            for (auto &le : h->lev)
                for (cudaEvent_t e : {le.a0, le.a1, le.d0, le.d1, le.r0, le.r1, le.c0, le.c1, le.o0, le.o1, le.m0, le.m1})
                    cudaEventDestroy(e);
        if (h->s_copy) cudaStreamDestroy(h->s_copy);
        if (h->s_off) cudaStreamDestroy(h->s_off);
        if (h->s_d2h) cudaStreamDestroy(h->s_d2h);
        if (h->own_compute && h->s_compute) cudaStreamDestroy(h->s_compute);
    }
    delete h;
}

int dev_alloc(void **p, size_t bytes, uint64_t *tally, const char *what) {
    if (bytes == 0) bytes = 256;
    cudaError_t e = cudaMalloc(p, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        *p = nullptr;
        return fail(ISV_ENOMEM_DEVICE, "cudaMalloc of %zu bytes for %s failed: %s", bytes, what,
                    cudaGetErrorString(e));
    }
    if (tally) *tally += bytes;
    return ISV_OK;
}

// Ring depth per warp: the default depth (or ISV_DECODE_STAGES, a tuning knob), reduced until it fits.
int pick_stages(const Geometry &g, int mode, int smem_limit, size_t *smem_out) {
    int best = 0;
    int cap = decode_default_stages(g.D, g.BT, g.GT, g.HP);
    if (const char *e = getenv("ISV_DECODE_STAGES")) cap = std::max(2, std::min(12, atoi(e)));
    for (int st = 2; st <= cap; ++st) {
        const size_t b = decode_smem_bytes(g.D, g.BT, g.GT, g.HP, st, g.max_seqs, mode);
        if (b <= (size_t)smem_limit) { best = st; *smem_out = b; }
    }
    return best;
}

// ISV_PINNED_LIMIT_BYTES caps the host KV pool the way a locked-memory limit of the system would: a
// pool beyond it is refused before anything is allocated.
int check_pinned_limit(uint64_t bytes) {
    const char *e = getenv("ISV_PINNED_LIMIT_BYTES");
    if (!e || !*e) return ISV_OK;
    const unsigned long long lim = strtoull(e, nullptr, 10);
    if (bytes > lim)
        return fail(ISV_ENOMEM_PINNED,
                    "pinned allocation of %llu bytes for the host KV pool refused: ISV_PINNED_LIMIT_BYTES is %llu "
                    "(fewer phys_layers or a smaller offload_frac need less)",
                    (unsigned long long)bytes, lim);
    return ISV_OK;
}

int check_handle(isv_kv *h, int layer, bool need_device) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    if (layer < 0 || layer >= h->g.layers) return fail(ISV_EINVAL, "layer %d out of range [0, %d)", layer, h->g.layers);
    if (need_device && h->plan_only) return fail(ISV_ENODEVICE, "plan-only handle: no device work possible");
    return ISV_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Host-side wait for a stream.  Without a limit it blocks in the driver; with one (isv_set_host_timeout)
// it polls and returns ISV_ETIMEOUT when the deadline passes, leaving the work enqueued.
int wait_stream(isv_kv *h, cudaStream_t st, const char *what) {
    if (!st) return ISV_OK;
    if (h->host_timeout_s <= 0.0) {
        CU(cudaStreamSynchronize(st));
        return ISV_OK;
    }
    const auto deadline = std::chrono::steady_clock::now() + std::chrono::duration<double>(h->host_timeout_s);
    for (;;) {
        const cudaError_t e = cudaStreamQuery(st);
        if (e == cudaSuccess) return ISV_OK;
        if (e != cudaErrorNotReady) return fail(ISV_ECUDA, "cudaStreamQuery(%s): %s", what, cudaGetErrorString(e));
        if (std::chrono::steady_clock::now() >= deadline)
            return fail(ISV_ETIMEOUT, "the %s stream did not finish within %.3f s (work is still enqueued)", what,
                        h->host_timeout_s);
        std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
}
#define WAIT(stream, what)                                   \
    do {                                                     \
        const int rc_ = wait_stream(h, (stream), (what));    \
        if (rc_) return rc_;                                 \
    } while (0)

// Pushes table updates to the device copy, kMaxTableUpdates per launch (by value).
int push_updates(isv_kv *h, const std::vector<TableUpdate> &upd) {
    size_t i = 0;
    while (i < upd.size()) {
        TableUpdateBatch b;
        b.n = 0;
        while (i < upd.size() && b.n < kMaxTableUpdates) {
            b.index[b.n] = upd[i].index;
            b.value[b.n] = upd[i].value;
            ++b.n; ++i;
        }
        CU(launch_table_update(h->table_dev, b, h->s_compute));
        ++h->launches;
        h->last_fused_layer = -1;
    }
    return ISV_OK;
}

// Copies the full tail slots of the listed sequences to their host blocks
// (device -> pinned host, on the write-back stream, after the compute stream's
// work so far).
int flush_tails(isv_kv *h, int layer, const std::vector<int> &seqs) {
    if (seqs.empty()) return ISV_OK;
    const int pl = layer % h->g.phys_layers;
    CU(cudaEventRecord(h->ev_app, h->s_compute));
    CU(cudaStreamWaitEvent(h->s_d2h, h->ev_app, 0));
    for (int s : seqs) {
        const int j = h->bm.newest_block(layer, s);
        const int32_t e = h->bm.entry(s, j);
        const int id = e & (ISV_BLOCK_HOST_BIT - 1);
        CU(cudaMemcpyAsync(h->pool_host + slab_host(h, layer) + (size_t)id * h->g.block_bytes,
                           h->tail + slab_tail(h, layer) + (size_t)s * h->g.block_bytes, h->g.block_bytes,
                           cudaMemcpyDeviceToHost, h->s_d2h));
    }
    CU(cudaEventRecord(h->ev_flush[pl], h->s_d2h));
    h->flush_recorded[pl] = 1;
    return ISV_OK;
}

int ensure_timing_events(isv_kv *h) {
    if (h->lev_created) return ISV_OK;
    h->lev.resize(h->g.layers);
    for (auto &le : h->lev)
        for (cudaEvent_t *e : {&le.a0, &le.a1, &le.d0, &le.d1, &le.r0, &le.r1, &le.c0, &le.c1, &le.o0, &le.o1, &le.m0, &le.m1})
            CU(cudaEventCreate(e));
    h->lev_created = true;
    return ISV_OK;
}

// Makes the current plan's lists available on the device; returns its slot.
int upload_plan(isv_kv *h, const OffPlan &pl, PlanSlot **out) {
    if (h->plan_cur >= 0 && h->plan_slot[h->plan_cur].version == pl.version) {
        *out = &h->plan_slot[h->plan_cur];
        return ISV_OK;
    }
    const int slot = (h->plan_cur + 1) % kPlanSlots;
    PlanSlot &ps = h->plan_slot[slot];
    if (ps.used_recorded) CU(cudaEventSynchronize(ps.used));   // kernels that read this slot have finished
    const size_t nu = pl.cu_seq.size(), nb = pl.cblk.size();
    const size_t need = 3 * nu + nb + 16;
    if (need > ps.cap) {
        if (ps.host) cudaFreeHost(ps.host);
        cudaFree(ps.dev);
        ps.host = nullptr; ps.dev = nullptr; ps.cap = 0;
        const size_t cap = need + need / 2;
        if (cudaHostAlloc((void **)&ps.host, cap * 4, cudaHostAllocDefault) != cudaSuccess) {
            cudaGetLastError();
            return fail(ISV_ENOMEM_PINNED, "pinned allocation of %zu bytes for the plan failed", cap * 4);
        }
        int rc = dev_alloc((void **)&ps.dev, cap * 4, nullptr, "plan lists");
        if (rc) return rc;
        ps.cap = cap;
    }
    ps.off_seq = 0;
    ps.off_beg = (int32_t)nu;
    ps.off_end = (int32_t)(2 * nu);
    ps.off_blk = (int32_t)(3 * nu);
    if (nu) {
        memcpy(ps.host + ps.off_seq, pl.cu_seq.data(), nu * 4);
        memcpy(ps.host + ps.off_beg, pl.cu_beg.data(), nu * 4);
        memcpy(ps.host + ps.off_end, pl.cu_end.data(), nu * 4);
    }
    if (nb) memcpy(ps.host + ps.off_blk, pl.cblk.data(), nb * 4);
    CU(cudaMemcpyAsync(ps.dev, ps.host, (3 * nu + nb) * 4, cudaMemcpyHostToDevice, h->s_off));
    ps.version = pl.version;
    h->plan_cur = slot;
    *out = &ps;
    return ISV_OK;
}

// One layer of a step whose resident part has already been enqueued for all layers by a single launch:
// where that launch left the layer's unnormalised result, the layer's own running state of the offloaded
// part, and how many CTAs a staged launch may take (the resident launch leaves that many SMs free).
struct FusedLayer {
    float *res_o, *res_ml, *run_o, *run_ml;
    int staged_grid_cap;
};

struct AppendPlan {
    std::vector<TableUpdate> upd;   // table entries of blocks allocated for this step
    std::vector<int> flush;         // sequences whose host-flagged newest block becomes full
    bool new_host_block = false;    // some sequence starts a host-flagged block (needs its tail slot free)
};

// Host side of appending one token to sequences [0, n_seqs) of a layer: capacity checks, block
// allocation by the residency rule, length mirror.  Nothing is changed when an error is returned.
int append_bookkeeping(isv_kv *h, int layer, int n_seqs, AppendPlan *ap) {
    const Geometry &g = h->g;
    if (n_seqs < 0 || n_seqs > g.max_seqs) return fail(ISV_EINVAL, "n_seqs %d outside [0, %d]", n_seqs, g.max_seqs);
    std::vector<std::pair<int, int>> need;
    for (int s = 0; s < n_seqs; ++s) {
        const int pos = h->bm.length(layer, s);
        if (pos >= g.max_tokens) return fail(ISV_ECAPACITY, "sequence %d is full (%d tokens)", s, pos);
        if (pos % g.BT == 0) {
            const int j = pos / g.BT;
            if (h->bm.entry(s, j) == ISV_BLOCK_NONE) need.push_back({s, j});
            if (h->bm.is_host(j)) ap->new_host_block = true;
        }
    }
    int rc = h->bm.allocate(need, &ap->upd);
    if (rc) return fail(rc, "KV pool full");
    for (int s = 0; s < n_seqs; ++s) {
        const int n = ++h->bm.length(layer, s);
        if (n % g.BT == 0 && h->bm.is_host((n - 1) / g.BT)) ap->flush.push_back(s);
    }
    return ISV_OK;
}

}  // namespace

// Lets the library's other translation units record the calling thread's last error.
namespace isv {
int set_error(int code, const char *msg) { return fail(code, "%s", msg); }
}  // namespace isv

// =========================================================================== C ABI

extern "C" {

const char *isv_last_error(void) { return g_err.c_str(); }

int isv_kv_alloc(isv_kv **out, const isv_kv_desc *desc) {
    if (!out) return fail(ISV_EINVAL, "out is null");
    *out = nullptr;
    if (!desc) return fail(ISV_EINVAL, "desc is null");
    Geometry g;
    if (const char *msg = make_geometry(*desc, &g)) return fail(ISV_EINVAL, "%s", msg);
    isv_kv *h = new (std::nothrow) isv_kv();
    if (!h) return fail(ISV_EINVAL, "out of host memory");
    h->g = g;
    h->plan_only = desc->plan_only != 0;
    h->bm.init(g, desc->perm_seed);
    if (h->plan_only) {   // a plan tells whether the host pool would be accepted, without allocating it
        const int rc_lim = check_pinned_limit((uint64_t)g.phys_layers * g.host_cap * g.block_bytes);
        if (rc_lim) { delete h; return rc_lim; }
        *out = h;
        return ISV_OK;
    }

    int rc = ISV_OK;
    auto bail = [&](int code) { destroy(h); return code; };
#define CUB(call)                                                                                   \
    do {                                                                                            \
        cudaError_t e_ = (call);                                                                    \
        if (e_ != cudaSuccess) return bail(fail(ISV_ECUDA, "%s: %s", #call, cudaGetErrorString(e_))); \
    } while (0)

    CUB(cudaGetDevice(&h->device));
    cudaDeviceProp prop;
    CUB(cudaGetDeviceProperties(&prop, h->device));
    h->sm_count = prop.multiProcessorCount;
    if (prop.major < 9)
        return bail(fail(ISV_ECUDA, "device compute capability %d.%d lacks bulk async copies", prop.major, prop.minor));
    const int smem_limit = (int)prop.sharedMemPerBlockOptin;
    h->smem_limit = smem_limit;
    h->stages_res = pick_stages(g, MODE_RESIDENT, smem_limit, &h->smem_res);
    h->stages_stg = pick_stages(g, MODE_STAGED, smem_limit, &h->smem_stg);
    if (h->stages_res < 2 || h->stages_stg < 2)
        return bail(fail(ISV_EINVAL, "shared memory (%d bytes) too small for this shape", smem_limit));
    const bool bf16 = g.dtype == ISV_BF16;
    // the per-function limit is shared by all handles: always raise it to the device maximum
    CUB(decode_configure(g.D, g.GT, g.HP, g.BT, bf16, MODE_RESIDENT, (size_t)smem_limit));
    CUB(decode_configure(g.D, g.GT, g.HP, g.BT, bf16, MODE_STAGED, (size_t)smem_limit));

    if (desc->compute_stream) {
        h->s_compute = (cudaStream_t)desc->compute_stream;
    } else {
        CUB(cudaStreamCreateWithFlags(&h->s_compute, cudaStreamNonBlocking));
        h->own_compute = true;
    }
    CUB(cudaStreamCreateWithFlags(&h->s_copy, cudaStreamNonBlocking));
    CUB(cudaStreamCreateWithFlags(&h->s_off, cudaStreamNonBlocking));
    CUB(cudaStreamCreateWithFlags(&h->s_d2h, cudaStreamNonBlocking));

    // pools
    const size_t hbm_bytes = (size_t)g.phys_layers * g.hbm_cap * g.block_bytes;
    if ((rc = dev_alloc((void **)&h->pool_hbm, hbm_bytes, &h->hbm_pool_bytes, "HBM KV pool"))) return bail(rc);
    if (g.host_cap > 0) {
        const size_t tail_bytes = (size_t)g.phys_layers * g.max_seqs * g.block_bytes;
        if ((rc = dev_alloc((void **)&h->tail, tail_bytes, &h->hbm_pool_bytes, "tail slots"))) return bail(rc);
        h->host_pool_bytes = (uint64_t)g.phys_layers * g.host_cap * g.block_bytes;
        if ((rc = check_pinned_limit(h->host_pool_bytes))) return bail(rc);
        cudaError_t e = cudaHostAlloc((void **)&h->pool_host, h->host_pool_bytes,
                                      cudaHostAllocMapped | cudaHostAllocPortable);
        if (e != cudaSuccess) {
            cudaGetLastError();
            h->pool_host = nullptr;
            return bail(fail(ISV_ENOMEM_PINNED, "pinned allocation of %llu bytes for the host KV pool failed: %s",
                             (unsigned long long)h->host_pool_bytes, cudaGetErrorString(e)));
        }
        CUB(cudaHostGetDevicePointer((void **)&h->pool_host_dev, h->pool_host, 0));
        if ((rc = dev_alloc((void **)&h->stage, (size_t)g.ring * g.chunk_bytes, &h->scratch_bytes, "staging ring")))
            return bail(rc);
    }
    // tables
    if ((rc = dev_alloc((void **)&h->table_dev, (size_t)g.max_seqs * g.NB * 4, nullptr, "block table"))) return bail(rc);
    if ((rc = dev_alloc((void **)&h->lens_dev, 2 * (size_t)g.layers * g.max_seqs * 4, nullptr, "lengths"))) return bail(rc);
    h->lens_cur.assign(g.layers, 0);
    if ((rc = dev_alloc((void **)&h->status_dev, 4, nullptr, "status"))) return bail(rc);
    CUB(cudaMemset(h->table_dev, 0xff, (size_t)g.max_seqs * g.NB * 4));
    CUB(cudaMemset(h->lens_dev, 0, 2 * (size_t)g.layers * g.max_seqs * 4));
    CUB(cudaMemset(h->status_dev, 0, 4));
    // scratch
    const size_t rows = (size_t)g.max_seqs * g.Hq;
    const int max_grid = g.max_ctas > 0 ? std::min(g.max_ctas, h->sm_count) : h->sm_count;
    const size_t slots = 2ull * max_grid * decode_warps(g.GT, g.D, g.HP) * g.GT;   // two partials per warp and query head
    if ((rc = dev_alloc((void **)&h->part_o, slots * g.D * 4, &h->scratch_bytes, "split partials"))) return bail(rc);
    if ((rc = dev_alloc((void **)&h->part_ml, slots * 2 * 4, &h->scratch_bytes, "split partials"))) return bail(rc);
    // one arrival counter per (layer, sequence, head group): a launch that covers several layers uses them all
    if ((rc = dev_alloc((void **)&h->tickets, tickets_bytes(g), &h->scratch_bytes, "tickets"))) return bail(rc);
    CUB(cudaMemset(h->tickets, 0, tickets_bytes(g)));
    if (g.host_cap > 0) {
        // one copy per layer of a launch where the resident part of several layers can be a single launch (its
        // per-layer results then wait for the layers' offloaded parts), else one; a launch covers at most
        // phys_layers layers
        if (g.phys_layers > 1 && g.layers <= 64 &&
            decode_smem_bytes(g.D, g.BT, g.GT, g.HP, h->stages_res, 2 * g.max_seqs, MODE_RESIDENT) <= (size_t)smem_limit)
            h->res_layers = g.phys_layers;
        const size_t nl = (size_t)h->res_layers;
        if ((rc = dev_alloc((void **)&h->res_o, nl * rows * g.D * 4, &h->scratch_bytes, "resident result"))) return bail(rc);
        if ((rc = dev_alloc((void **)&h->res_ml, nl * rows * 2 * 4, &h->scratch_bytes, "resident result"))) return bail(rc);
        if ((rc = dev_alloc((void **)&h->run_o, nl * rows * g.D * 4, &h->scratch_bytes, "running state"))) return bail(rc);
        if ((rc = dev_alloc((void **)&h->run_ml, nl * rows * 2 * 4, &h->scratch_bytes, "running state"))) return bail(rc);
    }
    // events
    h->ev_ready.resize(g.ring);
    h->ev_freed.resize(g.ring);
    h->freed_recorded.assign(g.ring, 0);
    for (int r = 0; r < g.ring; ++r) {
        CUB(cudaEventCreateWithFlags(&h->ev_ready[r], cudaEventDisableTiming));
        CUB(cudaEventCreateWithFlags(&h->ev_freed[r], cudaEventDisableTiming));
    }
    h->ev_packed.resize(g.ring);
    h->ev_stored.resize(g.ring);
    h->stored_recorded.assign(g.ring, 0);
    for (int r = 0; r < g.ring; ++r) {
        CUB(cudaEventCreateWithFlags(&h->ev_packed[r], cudaEventDisableTiming));
        CUB(cudaEventCreateWithFlags(&h->ev_stored[r], cudaEventDisableTiming));
    }
    CUB(cudaEventCreate(&h->ev_f0)); CUB(cudaEventCreate(&h->ev_f1));
    CUB(cudaEventCreate(&h->ev_s0)); CUB(cudaEventCreate(&h->ev_s1));
    if (g.host_cap > 0 && (rc = dev_alloc((void **)&h->owner_dev, (size_t)g.host_cap * 8, nullptr, "host block owners")))
        return bail(rc);
    h->ev_flush.resize(g.phys_layers);
    h->flush_recorded.assign(g.phys_layers, 0);
    for (int l = 0; l < g.phys_layers; ++l) CUB(cudaEventCreateWithFlags(&h->ev_flush[l], cudaEventDisableTiming));
    CUB(cudaEventCreateWithFlags(&h->ev_q, cudaEventDisableTiming));
    CUB(cudaEventCreateWithFlags(&h->ev_off_done, cudaEventDisableTiming));
    CUB(cudaEventCreateWithFlags(&h->ev_app, cudaEventDisableTiming));
    for (auto &ps : h->plan_slot) CUB(cudaEventCreateWithFlags(&ps.used, cudaEventDisableTiming));
    CUB(cudaDeviceSynchronize());
#undef CUB
    *out = h;
    return ISV_OK;
}

int isv_kv_free(isv_kv *h) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    destroy(h);
    return ISV_OK;
}

int isv_sync(isv_kv *h, uint32_t *status_out) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    if (status_out) *status_out = 0;
    if (h->plan_only) return ISV_OK;
    WAIT(h->s_compute, "compute");
    WAIT(h->s_copy, "copy");
    WAIT(h->s_off, "offloaded-attention");
    WAIT(h->s_d2h, "write-back");
    WAIT(h->s_in, "step-input");
    uint32_t st = 0;
    CU(cudaMemcpy(&st, h->status_dev, 4, cudaMemcpyDeviceToHost));
    if (status_out) *status_out = st;
    if (st != 0) {
        CU(cudaMemset(h->status_dev, 0, 4));
        // a kernel that gave up may have left its arrival counters half way
        CU(cudaMemset(h->tickets, 0, tickets_bytes(h->g)));
        return fail(ISV_EDEVICE_STATUS, "a kernel reported status 0x%x (%s%s%s)", st,
                    (st & ISV_STATUS_BAD_BLOCK_ID) ? "bad block id " : "",
                    (st & ISV_STATUS_WAIT_EXPIRED) ? "wait expired " : "",
                    (st & ISV_STATUS_BAD_LENGTH) ? "bad length" : "");
    }
    return ISV_OK;
}

int isv_kv_reset(isv_kv *h) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    if (!h->plan_only) {
        int rc = isv_sync(h, nullptr);
        if (rc && rc != ISV_EDEVICE_STATUS) return rc;
        CU(cudaMemset(h->table_dev, 0xff, (size_t)h->g.max_seqs * h->g.NB * 4));
        CU(cudaMemset(h->lens_dev, 0, 2 * (size_t)h->g.layers * h->g.max_seqs * 4));
        CU(cudaMemset(h->tickets, 0, tickets_bytes(h->g)));
        std::fill(h->flush_recorded.begin(), h->flush_recorded.end(), 0);
        h->owner_uploaded = -1;
        h->last_fused_layer = -1;
    }
    h->bm.reset();
    return ISV_OK;
}

int isv_kv_info(isv_kv *h, isv_kv_info_t *o) {
    if (!h || !o) return fail(ISV_EINVAL, "null argument");
    memset(o, 0, sizeof *o);
    o->block_bytes = h->g.block_bytes;
    o->kv_bytes_per_token = h->g.kappa;
    o->max_blocks_per_seq = h->g.NB;
    o->hbm_blocks = h->g.hbm_cap;
    o->host_blocks = h->g.host_cap;
    o->hbm_blocks_used = h->bm.hbm_used;
    o->host_blocks_used = h->bm.host_used;
    o->hbm_pool_bytes = h->plan_only ? (uint64_t)h->g.phys_layers * (h->g.hbm_cap + (h->g.host_cap ? h->g.max_seqs : 0)) * h->g.block_bytes
                                     : h->hbm_pool_bytes;
    o->host_pool_bytes = (uint64_t)h->g.phys_layers * h->g.host_cap * h->g.block_bytes;
    o->scratch_bytes = h->scratch_bytes;
    o->phys_layers = h->g.phys_layers;
    o->max_ctas = h->g.max_ctas;
    o->ring_depth = h->g.ring;
    o->sm_count = h->sm_count;
    o->chunk_bytes = h->g.chunk_bytes;
    o->kernel_launches = h->launches;
    return ISV_OK;
}

int isv_kv_fill_async(isv_kv *h, int32_t layer, const void *k, const void *v, const int32_t *lens_host,
                      int32_t n_seqs, int32_t T) {
    int rc = check_handle(h, layer, false);
    if (rc) return rc;
    const Geometry &g = h->g;
    if (!lens_host || n_seqs < 0 || n_seqs > g.max_seqs || T < 0)
        return fail(ISV_EINVAL, "bad lens/n_seqs/T (n_seqs %d, max %d)", n_seqs, g.max_seqs);
    if (!h->plan_only && (!k || !v || !aligned16(k) || !aligned16(v)))
        return fail(ISV_EINVAL, "k and v must be non-null and 16-byte aligned");
    std::vector<std::pair<int, int>> need;
    for (int s = 0; s < n_seqs; ++s) {
        const int n = lens_host[s];
        if (n < 0 || n > T) return fail(ISV_EINVAL, "lens[%d] = %d outside [0, T=%d]", s, n, T);
        if (n > g.max_tokens) return fail(ISV_ECAPACITY, "lens[%d] = %d exceeds max_tokens_per_seq %d", s, n, g.max_tokens);
        for (int j = 0; j < (n + g.BT - 1) / g.BT; ++j) need.push_back({s, j});
    }
    if ((rc = h->bm.allocate(need, nullptr))) return fail(rc, "KV pool full while loading the prompt");
    for (int s = 0; s < n_seqs; ++s) h->bm.length(layer, s) = lens_host[s];
    if (h->plan_only) return ISV_OK;

    // the table and lengths are replaced wholesale: earlier kernels must be done with them
    WAIT(h->s_compute, "compute");
    CU(cudaMemcpy(h->table_dev, h->bm.table.data(), h->bm.table.size() * 4, cudaMemcpyHostToDevice));
    CU(cudaMemcpy(lens_ptr(h, layer, 0), &h->bm.len[(size_t)layer * g.max_seqs],
                  (size_t)g.max_seqs * 4, cudaMemcpyHostToDevice));
    if (h->owner_dev && h->owner_uploaded != h->bm.host_used) {
        std::vector<int32_t> own(2 * (size_t)h->bm.host_used);
        for (int id = 0; id < h->bm.host_used; ++id) {
            own[2 * id] = h->bm.host_owner_s[id];
            own[2 * id + 1] = h->bm.host_owner_j[id];
        }
        if (!own.empty()) CU(cudaMemcpy(h->owner_dev, own.data(), own.size() * 4, cudaMemcpyHostToDevice));
        h->owner_uploaded = h->bm.host_used;
    }
    const int pl = layer % g.phys_layers;
    if (h->flush_recorded[pl]) CU(cudaStreamWaitEvent(h->s_compute, h->ev_flush[pl], 0));
    h->fill_timed = true;
    h->last_fused_layer = -1;
    h->fill_stored = false;
    h->fill_bytes_stored = h->fill_bytes_resident = 0;
    h->fill_copies = 0;
    CU(cudaEventRecord(h->ev_f0, h->s_compute));
    int max_blocks = 0;
    uint64_t tokens = 0;
    for (int s = 0; s < n_seqs; ++s) {
        max_blocks = std::max(max_blocks, (lens_host[s] + g.BT - 1) / g.BT);
        tokens += lens_host[s];
    }
    // resident blocks and newest blocks: straight into the HBM pool / tail slots
    if (n_seqs > 0 && max_blocks > 0) {
        FillParams p{};
        p.k = k; p.v = v;
        p.pool = h->pool_hbm + slab_hbm(h, layer);
        p.tail = h->tail ? h->tail + slab_tail(h, layer) : nullptr;
        p.host = nullptr;   // complete host-resident blocks take the packed path below
        p.table = h->table_dev;
        p.lens = lens_ptr(h, layer, 0);
        p.status = h->status_dev;
        p.table_stride = g.NB; p.n_pool_blocks = g.hbm_cap; p.n_host_blocks = g.host_cap;
        p.n_seqs = n_seqs; p.T = T; p.Hkv = g.Hkv; p.D = g.D; p.BT = g.BT; p.max_blocks = max_blocks;
        p.block_bytes = g.block_bytes;
        CU(launch_fill(p, h->s_compute));
        ++h->launches;
    }
    // complete host-resident blocks: packed into the ring in host-id order by a kernel, then stored with one
    // device-to-host copy per run of consecutive ids, on the write-back stream, ring slot by ring slot
    if (h->owner_dev) {
        int id = 0;
        bool first = true;
        auto final_block = [&](int i) {
            const int s = h->bm.host_owner_s[i], j = h->bm.host_owner_j[i];
            return s >= 0 && s < n_seqs && j < h->bm.newest_block(layer, s);
        };
        while (id < h->bm.host_used) {
            if (!final_block(id)) { ++id; continue; }
            int n = 1;
            while (id + n < h->bm.host_used && n < g.chunk_blocks && final_block(id + n)) ++n;
            const int r = (int)(h->store_counter++ % (uint64_t)g.ring);
            uint8_t *buf = h->stage + (size_t)r * g.chunk_bytes;
            if (h->stored_recorded[r]) CU(cudaStreamWaitEvent(h->s_compute, h->ev_stored[r], 0));   // slot free again
            if (h->freed_recorded[r]) CU(cudaStreamWaitEvent(h->s_compute, h->ev_freed[r], 0));
            PackParams pp{};
            pp.k = k; pp.v = v;
            pp.owner = h->owner_dev;
            pp.dst = buf;
            pp.first_id = id; pp.n_ids = n;
            pp.T = T; pp.Hkv = g.Hkv; pp.D = g.D; pp.BT = g.BT;
            pp.block_bytes = g.block_bytes;
            CU(launch_pack(pp, h->s_compute));
            ++h->launches;
            CU(cudaEventRecord(h->ev_packed[r], h->s_compute));
            CU(cudaStreamWaitEvent(h->s_d2h, h->ev_packed[r], 0));
            if (first) {
                CU(cudaEventRecord(h->ev_s0, h->s_d2h));
                first = false;
            }
            CU(cudaMemcpyAsync(h->pool_host + slab_host(h, layer) + (size_t)id * g.block_bytes, buf,
                               (size_t)n * g.block_bytes, cudaMemcpyDeviceToHost, h->s_d2h));
            CU(cudaEventRecord(h->ev_stored[r], h->s_d2h));
            h->stored_recorded[r] = 1;
            h->fill_bytes_stored += (uint64_t)n * g.block_bytes;
            ++h->fill_copies;
            id += n;
        }
        if (!first) {
            CU(cudaEventRecord(h->ev_s1, h->s_d2h));
            h->fill_stored = true;
            // the layer's next staging must see the stored blocks
            CU(cudaEventRecord(h->ev_flush[pl], h->s_d2h));
            h->flush_recorded[pl] = 1;
        }
    }
    h->fill_bytes_resident = tokens * g.kappa - h->fill_bytes_stored;
    CU(cudaEventRecord(h->ev_f1, h->s_compute));
    // a full, host-flagged newest block goes to the host pool right away
    std::vector<int> flush;
    for (int s = 0; s < n_seqs; ++s) {
        const int n = lens_host[s];
        if (n > 0 && n % g.BT == 0 && h->bm.is_host((n - 1) / g.BT)) flush.push_back(s);
    }
    return flush_tails(h, layer, flush);
}

int isv_kv_fill(isv_kv *h, int32_t layer, const void *k, const void *v, const int32_t *lens_host,
                int32_t n_seqs, int32_t T) {
    int rc = isv_kv_fill_async(h, layer, k, v, lens_host, n_seqs, T);
    if (rc || h->plan_only) return rc;
    WAIT(h->s_compute, "compute");
    WAIT(h->s_d2h, "write-back");
    return ISV_OK;
}

int isv_fill_timing(isv_kv *h, isv_fill_times *out) {
    if (!h || !out) return fail(ISV_EINVAL, "null argument");
    if (h->plan_only) return fail(ISV_ENODEVICE, "plan-only handle");
    memset(out, 0, sizeof *out);
    if (!h->fill_timed) return ISV_OK;
    WAIT(h->s_compute, "compute");
    WAIT(h->s_d2h, "write-back");
    float t = 0.f;
    if (cudaEventElapsedTime(&t, h->ev_f0, h->ev_f1) == cudaSuccess) out->pack_ms = t;
    out->total_ms = out->pack_ms;
    if (h->fill_stored) {
        if (cudaEventElapsedTime(&t, h->ev_s0, h->ev_s1) == cudaSuccess) out->store_ms = t;
        if (cudaEventElapsedTime(&t, h->ev_f0, h->ev_s1) == cudaSuccess) out->total_ms = std::max(out->total_ms, t);
    }
    out->bytes_stored = h->fill_bytes_stored;
    out->bytes_resident = h->fill_bytes_resident;
    out->n_copies = h->fill_copies;
    cudaGetLastError();
    return ISV_OK;
}

int isv_kv_append(isv_kv *h, int32_t layer, const void *k, const void *v, int32_t n_seqs) {
    int rc = check_handle(h, layer, false);
    if (rc) return rc;
    const Geometry &g = h->g;
    if (!h->plan_only && (!k || !v || !aligned16(k) || !aligned16(v)))
        return fail(ISV_EINVAL, "k and v must be non-null and 16-byte aligned");
    AppendPlan ap;
    if ((rc = append_bookkeeping(h, layer, n_seqs, &ap))) return rc;
    if (h->plan_only || n_seqs == 0) return ISV_OK;

    LayerEvents *le = nullptr;
    if (h->timing) {
        le = &h->lev[layer];
        CU(cudaEventRecord(le->a0, h->s_compute));
    }
    if ((rc = push_updates(h, ap.upd))) return rc;
    const int pl = layer % g.phys_layers;
    // a tail slot about to take a new block must have finished its write-back
    if (ap.new_host_block && h->flush_recorded[pl]) CU(cudaStreamWaitEvent(h->s_compute, h->ev_flush[pl], 0));
    AppendParams p{};
    p.k = k; p.v = v;
    p.pool = h->pool_hbm + slab_hbm(h, layer);
    p.tail = h->tail ? h->tail + slab_tail(h, layer) : nullptr;
    p.table = h->table_dev;
    p.lens = lens_ptr(h, layer, 0);
    p.status = h->status_dev;
    p.table_stride = g.NB; p.n_pool_blocks = g.hbm_cap; p.max_blocks = g.NB;
    p.n_seqs = n_seqs; p.Hkv = g.Hkv; p.D = g.D; p.BT = g.BT;
    p.block_bytes = g.block_bytes;
    CU(launch_append(p, h->s_compute));
    ++h->launches;
    h->last_fused_layer = -1;
    if (le) {
        CU(cudaEventRecord(le->a1, h->s_compute));
        le->have_append = true;
        le->fused_append = false;
        le->bytes_app = (uint64_t)n_seqs * g.kappa;
    }
    return flush_tails(h, layer, ap.flush);
}

// Attention of one layer; with k_new / v_new also this step's append, fused into the resident kernel
// (the device lengths then still hold the values before the append and the kernel advances them).
static int decode_impl(isv_kv *h, int32_t layer, const void *q, void *out, float *out_f32,
                       const int32_t *block_table_dev, const int32_t *seq_lens_dev, int32_t n_seqs,
                       const void *k_new, const void *v_new, bool tables_settled, const FusedLayer *fc = nullptr) {
    int rc = ISV_OK;
    const Geometry &g = h->g;
    if (n_seqs < 0 || n_seqs > g.max_seqs) return fail(ISV_EINVAL, "n_seqs %d outside [0, %d]", n_seqs, g.max_seqs);
    if (!q || (!out && !out_f32)) return fail(ISV_EINVAL, "q and one of out / out_f32 must be given");
    if (!aligned16(q) || !aligned16(out) || !aligned16(out_f32))
        return fail(ISV_EINVAL, "q, out and out_f32 must be 16-byte aligned");
    if (n_seqs == 0) return ISV_OK;
    const bool bf16 = g.dtype == ISV_BF16;
    const int Hg = g.groups();
    const int nw = decode_warps(g.GT, g.D, g.HP);
    const OffPlan &pl = h->bm.plan(layer, n_seqs, h->zero_copy ? (1 << 30) : g.chunk_blocks);
    const bool offloaded = !pl.chunks.empty();
    const int phys = layer % g.phys_layers;

    LayerEvents *le = nullptr;
    if (h->timing) {
        le = &h->lev[layer];
        le->have_decode = true;
        le->have_off = offloaded;
        le->bytes_res = pl.bytes_resident;
        le->bytes_off = pl.bytes_offloaded;
        le->bytes_staged = (offloaded && !h->zero_copy) ? pl.bytes_staged : 0;
        le->n_chunks = (int)pl.chunks.size();
        if (!fc) CU(cudaEventRecord(le->d0, h->s_compute));   // (a step-wide resident launch recorded it already)
    }
    float *run_o = fc ? fc->run_o : h->run_o, *run_ml = fc ? fc->run_ml : h->run_ml;

    DecodeParams base{};
    base.table = block_table_dev ? block_table_dev : h->table_dev;
    base.lens = seq_lens_dev ? seq_lens_dev : lens_ptr(h, layer, 0);
    base.table_stride = g.NB;
    base.max_blocks = g.NB;
    base.spin_limit = h->spin_limit;
    base.q = q;
    base.status = h->status_dev;
    base.n_seqs = n_seqs; base.Hq = g.Hq; base.Hkv = g.Hkv; base.P = g.P; base.GT = g.GT;
    base.block_bytes = g.block_bytes;
    base.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)g.D));

    if (offloaded) {
        // ---- staging engine: host blocks stream through the ring while the resident kernel runs
        PlanSlot *ps = nullptr;
        if (!fc) {   // (with a step-wide resident launch the offload stream was released before that launch)
            CU(cudaEventRecord(h->ev_q, h->s_compute));          // q (and everything before) is ready
            CU(cudaStreamWaitEvent(h->s_off, h->ev_q, 0));
        }
        if ((rc = upload_plan(h, pl, &ps))) return rc;
        CU(cudaMemsetAsync(run_ml, 0, (size_t)n_seqs * g.Hq * 2 * 4, h->s_off));
        if (h->flush_recorded[phys]) CU(cudaStreamWaitEvent(h->zero_copy ? h->s_off : h->s_copy, h->ev_flush[phys], 0));
        if (le) {
            CU(cudaEventRecord(le->c0, h->s_copy));
            CU(cudaEventRecord(le->o0, h->s_off));
        }
        const uint8_t *host_slab = h->pool_host + slab_host(h, layer);
        for (const Chunk &ch : pl.chunks) {
            const uint8_t *buf;
            int r = -1;
            if (h->zero_copy) {
                // the kernel's bulk copies pull the blocks straight out of mapped pinned memory
                buf = h->pool_host_dev + slab_host(h, layer) + (size_t)ch.first_id * g.block_bytes;
            } else {
                r = (int)(h->chunk_counter++ % (uint64_t)g.ring);
                uint8_t *ring_buf = h->stage + (size_t)r * g.chunk_bytes;
                if (h->freed_recorded[r]) CU(cudaStreamWaitEvent(h->s_copy, h->ev_freed[r], 0));
                if (h->stored_recorded[r]) {   // a prompt write-back may still be reading this slot
                    CU(cudaStreamWaitEvent(h->s_copy, h->ev_stored[r], 0));
                    h->stored_recorded[r] = 0;
                }
                CU(cudaMemcpyAsync(ring_buf, host_slab + (size_t)ch.first_id * g.block_bytes, (size_t)ch.n_ids * g.block_bytes,
                                   cudaMemcpyHostToDevice, h->s_copy));
                CU(cudaEventRecord(h->ev_ready[r], h->s_copy));
                CU(cudaStreamWaitEvent(h->s_off, h->ev_ready[r], 0));
                buf = ring_buf;
            }
            DecodeParams p = base;
            p.pool = buf;
            p.n_pool_blocks = ch.n_ids;
            p.cu_seq = ps->dev + ps->off_seq;
            p.cu_beg = ps->dev + ps->off_beg;
            p.cu_end = ps->dev + ps->off_end;
            p.cblk = ps->dev + ps->off_blk;
            p.cu_first = ch.unit_begin;
            p.cu_count = ch.unit_end - ch.unit_begin;
            p.acc_o = run_o;
            p.acc_ml = run_ml;
            const long long nu2 = (long long)p.cu_count * Hg;
            // reading in place needs few CTAs to saturate the link and leaves the other SMs to the resident kernel
            const long long cap2 = h->zero_copy ? std::max(1, h->sm_count / 4) : (fc ? fc->staged_grid_cap : h->sm_count);
            const int grid = (int)std::max<long long>(1, std::min<long long>(cap2, (nu2 + nw - 1) / nw));
            CU(launch_decode(p, g.D, g.GT, g.HP, g.BT, bf16, MODE_STAGED, grid, h->stages_stg, h->smem_stg, h->s_off));
            ++h->launches;
            if (r >= 0) {
                CU(cudaEventRecord(h->ev_freed[r], h->s_off));
                h->freed_recorded[r] = 1;
            }
        }
        if (le) {
            CU(cudaEventRecord(le->c1, h->s_copy));
            CU(cudaEventRecord(le->o1, h->s_off));
        }
        CU(cudaEventRecord(h->ev_off_done, h->s_off));
        CU(cudaEventRecord(ps->used, h->s_off));
        ps->used_recorded = true;
    }

    // ---- resident part
    if (!fc) {
        DecodeParams p = base;
        p.pool = h->pool_hbm + slab_hbm(h, layer);
        p.tail = h->tail ? h->tail + slab_tail(h, layer) : nullptr;
        p.n_pool_blocks = g.hbm_cap;
        p.out = out; p.out_f32 = out_f32;
        p.part_o = h->part_o; p.part_ml = h->part_ml; p.tickets = h->tickets;
        p.acc_o = h->res_o; p.acc_ml = h->res_ml;
        p.finalize = offloaded ? 0 : 1;
        if (k_new) {
            p.k_new = k_new; p.v_new = v_new;
            p.lens_out = lens_ptr(h, layer, 1);
            p.lens_count = g.max_seqs;
            p.pool_w = h->pool_hbm + slab_hbm(h, layer);
            p.tail_w = h->tail ? h->tail + slab_tail(h, layer) : nullptr;
            // the kernel launched just before this one (the previous layer's, or a caller's) writes neither
            // the table, nor these lengths, nor this layer's slab: their reads need not wait for it
            // (it is the previous fused launch, of another layer on another slab, possibly followed by the
            // caller's own kernels, which do not write library memory)
            p.early_reads = (tables_settled && h->last_fused_layer >= 0 && h->last_fused_layer != layer &&
                             h->last_fused_layer % g.phys_layers != layer % g.phys_layers) ? 1 : 0;
        }
        long long nu = 0;   // KV blocks in the flat work list
        for (int s = 0; s < n_seqs; ++s)
            nu += (long long)std::max(1, (h->bm.length(layer, s) + g.BT - 1) / g.BT) * Hg;
        const int cap = g.max_ctas > 0 ? std::min(g.max_ctas, h->sm_count) : h->sm_count;
        const int grid = (int)std::max<long long>(1, std::min<long long>(cap, (nu + nw - 1) / nw));
        if (h->lost_copies > 0) {
            --h->lost_copies;
            p.drop_first_copy = 1;
        }
        if (le) CU(cudaEventRecord(le->r0, h->s_compute));
        CU(launch_decode(p, g.D, g.GT, g.HP, g.BT, bf16, MODE_RESIDENT, grid, h->stages_res, h->smem_res, h->s_compute));
        ++h->launches;
        if (le) CU(cudaEventRecord(le->r1, h->s_compute));
        if (k_new) h->lens_cur[layer] ^= 1;   // the kernel wrote the advanced lengths to the other copy
        h->last_fused_layer = k_new ? layer : -1;
    }

    if (offloaded || fc) {
        if (offloaded) CU(cudaStreamWaitEvent(h->s_compute, h->ev_off_done, 0));
        else CU(cudaMemsetAsync(run_ml, 0, (size_t)n_seqs * g.Hq * 2 * 4, h->s_compute));   // nothing offloaded here: an empty running state
        MergeParams mp{};
        mp.res_o = fc ? fc->res_o : h->res_o; mp.res_ml = fc ? fc->res_ml : h->res_ml;
        mp.run_o = run_o; mp.run_ml = run_ml;
        mp.out = out; mp.out_f32 = out_f32;
        mp.rows = n_seqs * g.Hq; mp.D = g.D; mp.bf16 = bf16 ? 1 : 0;
        if (le) CU(cudaEventRecord(le->m0, h->s_compute));
        CU(launch_merge(mp, h->s_compute));
        ++h->launches;
        if (le) CU(cudaEventRecord(le->m1, h->s_compute));
    }
    if (le) CU(cudaEventRecord(le->d1, h->s_compute));
    return ISV_OK;
}

int isv_attn_decode(isv_kv *h, int32_t layer, const void *q, void *out, float *out_f32,
                    const int32_t *block_table_dev, const int32_t *seq_lens_dev, int32_t n_seqs) {
    int rc = check_handle(h, layer, true);
    if (rc) return rc;
    return decode_impl(h, layer, q, out, out_f32, block_table_dev, seq_lens_dev, n_seqs, nullptr, nullptr, false);
}

int isv_decode_layer(isv_kv *h, int32_t layer, const void *q, const void *k, const void *v, void *out,
                     float *out_f32, int32_t n_seqs) {
    int rc = check_handle(h, layer, true);
    if (rc) return rc;
    const Geometry &g = h->g;
    if (!k || !v || !aligned16(k) || !aligned16(v)) return fail(ISV_EINVAL, "k and v must be non-null and 16-byte aligned");
    if (!q || (!out && !out_f32) || !aligned16(q) || !aligned16(out) || !aligned16(out_f32))
        return fail(ISV_EINVAL, "q and one of out / out_f32 must be given, 16-byte aligned");
    AppendPlan ap;
    if ((rc = append_bookkeeping(h, layer, n_seqs, &ap))) return rc;
    if (n_seqs == 0) return ISV_OK;
    if (h->timing) {
        h->lev[layer].have_append = false;
        h->lev[layer].fused_append = true;
    }
    if ((rc = push_updates(h, ap.upd))) return rc;
    const int pl = layer % g.phys_layers;
    if (ap.new_host_block && h->flush_recorded[pl]) CU(cudaStreamWaitEvent(h->s_compute, h->ev_flush[pl], 0));
    if ((rc = decode_impl(h, layer, q, out, out_f32, nullptr, nullptr, n_seqs, k, v, ap.upd.empty()))) return rc;
    if (h->timing) h->lev[layer].bytes_app = (uint64_t)n_seqs * g.kappa;
    return flush_tails(h, layer, ap.flush);
}

// How many of the layers l0, l0 + 1, ... (at most nl) can have their resident attention (and appends) in one
// launch; 1 = none beyond the first, i.e. the per-layer path.  A launch never covers two layers that share a
// physical slab, so at most phys_layers layers: layers sharing a slab then keep the order of separate
// launches (the later one's token stays), and a benchmark that holds fewer slabs than layers cannot have two
// layers of a launch stream the same bytes at the same time and find them in L2.  With nothing offloaded
// per-layer timing must be off (there is no per-layer launch to time); with part of the cache on the host
// the blocks must be staged through the ring and the per-layer result buffers exist.  The kernel's
// per-(layer, sequence) tables must fit in shared memory beside the full ring.
static int fusable_layers(const isv_kv *h, int nl, int n_seqs, size_t *smem) {
    const Geometry &g = h->g;
    nl = std::min(nl, g.phys_layers);
    if (nl < 2 || n_seqs < 1 || g.layers > 64) return 1;
    if (const char *e = getenv("ISV_LAYERS_PER_LAUNCH"))   // tuning knob: 1 = one launch per layer
        if (atoi(e) == 1) return 1;
    if (g.host_cap == 0) {
        if (h->timing) return 1;
    } else {
        if (h->zero_copy || h->res_layers < 2) return 1;
        nl = std::min(nl, h->res_layers);
    }
    while (nl >= 2 && decode_smem_bytes(g.D, g.BT, g.GT, g.HP, h->stages_res, nl * n_seqs, MODE_RESIDENT) > (size_t)h->smem_limit)
        --nl;
    if (nl < 2) return 1;
    *smem = decode_smem_bytes(g.D, g.BT, g.GT, g.HP, h->stages_res, nl * n_seqs, MODE_RESIDENT);
    return nl;
}

// Layers [l0, l0 + nl) of one decode step with ONE launch of the resident kernel for all of them (appends
// fused).  q, out, out_f32: [nl][n_seqs][q_heads][head_dim]; k, v: [nl][n_seqs][kv_heads][head_dim], device.
// With host-resident blocks the launch leaves every layer's unnormalised result, a few SMs stay free for the
// staged launches, and the layers' offloaded parts and merges are enqueued behind it: the copy engine's queue
// is filled for the whole step at once and never waits for a resident launch.
static int decode_layers_fused(isv_kv *h, int l0, int nl, const void *q, const void *k, const void *v, void *out,
                               float *out_f32, int n_seqs, size_t smem) {
    const Geometry &g = h->g;
    int rc = ISV_OK;
    const bool split = g.host_cap > 0;
    // host side of the appends; nothing stays changed when a layer cannot take its token
    for (int l = l0; l < l0 + nl; ++l)
        for (int s = 0; s < n_seqs; ++s)
            if (h->bm.length(l, s) >= g.max_tokens)
                return fail(ISV_ECAPACITY, "sequence %d is full (%d tokens)", s, h->bm.length(l, s));
    std::vector<AppendPlan> aps(nl);
    std::vector<TableUpdate> upd;
    for (int l = l0; l < l0 + nl; ++l) {
        AppendPlan &ap = aps[l - l0];
        rc = append_bookkeeping(h, l, n_seqs, &ap);
        upd.insert(upd.end(), ap.upd.begin(), ap.upd.end());
        if (rc) {
            for (int lb = l0; lb < l; ++lb)
                for (int s = 0; s < n_seqs; ++s) --h->bm.length(lb, s);
            push_updates(h, upd);   // blocks handed out so far stay allocated
            return rc;
        }
    }
    if ((rc = push_updates(h, upd))) return rc;
    if (split)   // a tail slot about to take a new block must have finished its write-back
        for (int l = l0; l < l0 + nl; ++l) {
            const int pl = l % g.phys_layers;
            if (aps[l - l0].new_host_block && h->flush_recorded[pl]) CU(cudaStreamWaitEvent(h->s_compute, h->ev_flush[pl], 0));
        }
    if (h->timing) {
        for (int l = l0; l < l0 + nl; ++l) {
            h->lev[l].have_append = false;
            h->lev[l].fused_append = true;
            h->lev[l].bytes_app = (uint64_t)n_seqs * g.kappa;
            CU(cudaEventRecord(h->lev[l].d0, h->s_compute));
        }
    }
    if (split) {   // the offload stream may start on the step's staged launches now: they do not depend on the resident launch
        CU(cudaEventRecord(h->ev_q, h->s_compute));
        CU(cudaStreamWaitEvent(h->s_off, h->ev_q, 0));
    }

    const bool bf16 = g.dtype == ISV_BF16;
    const int Hg = g.groups();
    const int nw = decode_warps(g.GT, g.D, g.HP);
    DecodeParams p{};
    p.table = h->table_dev;
    p.table_stride = g.NB;
    p.max_blocks = g.NB;
    p.spin_limit = h->spin_limit;
    p.status = h->status_dev;
    p.n_seqs = n_seqs; p.Hq = g.Hq; p.Hkv = g.Hkv; p.P = g.P; p.GT = g.GT;
    p.block_bytes = g.block_bytes;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)g.D));
    p.pool = h->pool_hbm; p.pool_w = h->pool_hbm;
    p.tail = h->tail; p.tail_w = h->tail;
    p.n_pool_blocks = g.hbm_cap;
    p.q = q; p.k_new = k; p.v_new = v; p.out = out; p.out_f32 = out_f32;
    p.part_o = h->part_o; p.part_ml = h->part_ml; p.tickets = h->tickets;
    p.acc_o = h->res_o; p.acc_ml = h->res_ml;
    p.finalize = split ? 0 : 1;
    p.n_layers = nl; p.layer0 = l0; p.phys_layers = g.phys_layers;
    p.lens = h->lens_dev; p.lens_out = h->lens_dev;
    p.lens_count = g.max_seqs;
    p.lens_layer_stride = g.max_seqs;
    p.lens_copy_stride = g.layers * g.max_seqs;
    for (int l = 0; l < g.layers; ++l)
        if (h->lens_cur[l]) p.lens_cur_mask |= 1ull << l;
    p.pool_layer_stride = (uint64_t)g.hbm_cap * g.block_bytes;
    p.tail_layer_stride = (uint64_t)g.max_seqs * g.block_bytes;
    if (h->lost_copies > 0) {
        --h->lost_copies;
        p.drop_first_copy = 1;
    }
    long long nu = 0;   // KV blocks in the flat work list (host lengths already include this step's token)
    for (int l = l0; l < l0 + nl; ++l)
        for (int s = 0; s < n_seqs; ++s)
            nu += (long long)std::max(1, (h->bm.length(l, s) + g.BT - 1) / g.BT) * Hg;
    int cap = g.max_ctas > 0 ? std::min(g.max_ctas, h->sm_count) : h->sm_count;
    const int reserve = std::max(1, std::min(12, h->sm_count / 8));   // SMs left to the staged launches
    if (split && cap == h->sm_count) cap = std::max(1, cap - reserve);
    const int grid = (int)std::max<long long>(1, std::min<long long>(cap, (nu + nw - 1) / nw));
    if (h->timing) CU(cudaEventRecord(h->lev[l0].r0, h->s_compute));
    CU(launch_decode(p, g.D, g.GT, g.HP, g.BT, bf16, MODE_RESIDENT, grid, h->stages_res, smem, h->s_compute));
    ++h->launches;
    if (h->timing) {   // the launch is booked on the first layer; the others show no resident time of their own
        CU(cudaEventRecord(h->lev[l0].r1, h->s_compute));
        for (int l = l0 + 1; l < l0 + nl; ++l) {
            CU(cudaEventRecord(h->lev[l].r0, h->s_compute));
            CU(cudaEventRecord(h->lev[l].r1, h->s_compute));
        }
    }
    for (int l = l0; l < l0 + nl; ++l) h->lens_cur[l] ^= 1;   // the kernel wrote the advanced lengths to the other copies
    h->last_fused_layer = -1;
    if (!split) return ISV_OK;

    // ---- per layer: staged launches over the host-resident blocks, then the merge with the resident result
    const size_t rows = (size_t)n_seqs * g.Hq;
    const size_t qs = rows * g.D * 2;
    for (int l = l0; l < l0 + nl; ++l) {
        const size_t i = (size_t)(l - l0);
        FusedLayer fc;
        fc.res_o = h->res_o + i * rows * g.D;
        fc.res_ml = h->res_ml + i * rows * 2;
        fc.run_o = h->run_o + i * rows * g.D;
        fc.run_ml = h->run_ml + i * rows * 2;
        fc.staged_grid_cap = reserve;
        if ((rc = decode_impl(h, l, (const uint8_t *)q + i * qs, out ? (uint8_t *)out + i * qs : nullptr,
                              out_f32 ? out_f32 + i * rows * g.D : nullptr, nullptr, nullptr, n_seqs, nullptr, nullptr,
                              false, &fc)))
            return rc;
        if ((rc = flush_tails(h, l, aps[i].flush))) return rc;
    }
    return ISV_OK;
}

// Layers [l0, l0 + nl) of a step from buffers that hold them back to back: as few launches of the resident
// kernel as fusable_layers allows.
static int decode_layer_range(isv_kv *h, int l0, int nl, const void *q, const void *k, const void *v, void *out,
                              float *out_f32, int n_seqs) {
    const Geometry &g = h->g;
    const size_t rows = (size_t)n_seqs * g.Hq * g.D;
    const size_t qs = rows * 2, ks = (size_t)n_seqs * g.Hkv * g.D * 2;
    int rc = ISV_OK;
    for (int l = l0; l < l0 + nl;) {
        const size_t i = (size_t)(l - l0);
        const void *ql = (const uint8_t *)q + i * qs, *kl = (const uint8_t *)k + i * ks, *vl = (const uint8_t *)v + i * ks;
        void *ol = out ? (uint8_t *)out + i * qs : nullptr;
        float *fl = out_f32 ? out_f32 + i * rows : nullptr;
        size_t smem = 0;
        const int n = fusable_layers(h, l0 + nl - l, n_seqs, &smem);
        if (n >= 2) rc = decode_layers_fused(h, l, n, ql, kl, vl, ol, fl, n_seqs, smem);
        else rc = isv_decode_layer(h, l, ql, kl, vl, ol, fl, n_seqs);
        if (rc) return rc;
        l += n;
    }
    return ISV_OK;
}

int isv_decode_step(isv_kv *h, const void *q, const void *k, const void *v, void *out, float *out_f32,
                    int32_t n_seqs) {
    int rc = check_handle(h, 0, true);
    if (rc) return rc;
    const Geometry &g = h->g;
    if (!q || !k || !v || (!out && !out_f32)) return fail(ISV_EINVAL, "q, k, v and one of out / out_f32 must be given");
    if (n_seqs < 0 || n_seqs > g.max_seqs) return fail(ISV_EINVAL, "n_seqs %d outside [0, %d]", n_seqs, g.max_seqs);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(out_f32))
        return fail(ISV_EINVAL, "q, k, v, out and out_f32 must be 16-byte aligned");
    return decode_layer_range(h, 0, g.layers, q, k, v, out, out_f32, n_seqs);
}

int isv_decode_step_host(isv_kv *h, const void *q, const void *k, const void *v, void *out, int32_t n_seqs) {
    int rc = check_handle(h, 0, true);
    if (rc) return rc;
    const Geometry &g = h->g;
    if (!q || !k || !v || !out) return fail(ISV_EINVAL, "q, k, v and out must be given");
    if (n_seqs < 0 || n_seqs > g.max_seqs) return fail(ISV_EINVAL, "n_seqs %d outside [0, %d]", n_seqs, g.max_seqs);
    const size_t qs_max = (size_t)g.layers * g.max_seqs * g.Hq * g.D * 2;
    const size_t ks_max = (size_t)g.layers * g.max_seqs * g.Hkv * g.D * 2;
    if (!h->step_buf) {
        if ((rc = dev_alloc((void **)&h->step_buf, 2 * qs_max + 2 * ks_max, &h->scratch_bytes, "step buffers"))) return rc;
    }
    uint8_t *dq = h->step_buf, *dout = dq + qs_max, *dk = dout + qs_max, *dv = dk + ks_max;
    // Inputs travel in groups of layers on their own stream and results go back on the write-back stream,
    // so that only the first group's copy and the last group's read-back are not hidden behind the attention
    // of the other layers.  Those two groups are a single layer; in between the groups grow fourfold (a layer's
    // inputs cross the link several times faster than its attention runs, so the copies stay ahead), because
    // every group boundary is a cross-stream wait and ends a launch.
    std::vector<int> first;   // first layer of each group, and the end
    {
        int l = 0, n = 1;
        while (l < g.layers - 1) {
            first.push_back(l);
            l += std::min(n, g.layers - 1 - l);
            n *= 4;
        }
        first.push_back(l);           // the last layer on its own
        first.push_back(g.layers);
    }
    const int n_groups = (int)first.size() - 1;
    if (h->ev_step_in.empty()) {
        h->ev_step_in.resize(n_groups);
        h->ev_step_out.resize(n_groups);
        for (int i = 0; i < n_groups; ++i) {
            CU(cudaEventCreateWithFlags(&h->ev_step_in[i], cudaEventDisableTiming));
            CU(cudaEventCreateWithFlags(&h->ev_step_out[i], cudaEventDisableTiming));
        }
        CU(cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking));
    }
    const size_t ql = (size_t)n_seqs * g.Hq * g.D * 2, kl = (size_t)n_seqs * g.Hkv * g.D * 2;   // one layer
    // the device buffers are free once the compute stream has finished the previous call's work (it has:
    // the previous call synchronised), and caller data already on its way is ordered by the compute stream
    CU(cudaEventRecord(h->ev_app, h->s_compute));
    CU(cudaStreamWaitEvent(h->s_in, h->ev_app, 0));
    for (int gi = 0; gi < n_groups; ++gi) {
        const int l0 = first[gi], nl = first[gi + 1] - l0;
        CU(cudaMemcpyAsync(dk + l0 * kl, (const uint8_t *)k + l0 * kl, nl * kl, cudaMemcpyHostToDevice, h->s_in));
        CU(cudaMemcpyAsync(dv + l0 * kl, (const uint8_t *)v + l0 * kl, nl * kl, cudaMemcpyHostToDevice, h->s_in));
        CU(cudaMemcpyAsync(dq + l0 * ql, (const uint8_t *)q + l0 * ql, nl * ql, cudaMemcpyHostToDevice, h->s_in));
        CU(cudaEventRecord(h->ev_step_in[gi], h->s_in));
    }
    for (int gi = 0; gi < n_groups; ++gi) {
        const int l0 = first[gi], nl = first[gi + 1] - l0;
        CU(cudaStreamWaitEvent(h->s_compute, h->ev_step_in[gi], 0));
        // a group whose inputs have arrived runs as one launch where it can
        if ((rc = decode_layer_range(h, l0, nl, dq + l0 * ql, dk + l0 * kl, dv + l0 * kl, dout + l0 * ql, nullptr, n_seqs)))
            return rc;
        CU(cudaEventRecord(h->ev_step_out[gi], h->s_compute));
        CU(cudaStreamWaitEvent(h->s_d2h, h->ev_step_out[gi], 0));
        CU(cudaMemcpyAsync((uint8_t *)out + l0 * ql, dout + l0 * ql, nl * ql, cudaMemcpyDeviceToHost, h->s_d2h));
    }
    WAIT(h->s_compute, "compute");
    WAIT(h->s_d2h, "write-back");
    return ISV_OK;
}

int isv_kv_gather(isv_kv *h, int32_t layer, int32_t seq, void *k_host, void *v_host, int32_t *len_out) {
    int rc = check_handle(h, layer, true);
    if (rc) return rc;
    const Geometry &g = h->g;
    if (seq < 0 || seq >= g.max_seqs || !k_host || !v_host) return fail(ISV_EINVAL, "bad seq or null output");
    if ((rc = isv_sync(h, nullptr)) && rc != ISV_EDEVICE_STATUS) return rc;
    const int n = h->bm.length(layer, seq);
    if (len_out) *len_out = n;
    if (n == 0) return ISV_OK;
    const size_t bytes = (size_t)n * g.Hkv * g.D * 2;
    uint8_t *tmp = nullptr;
    if ((rc = dev_alloc((void **)&tmp, 2 * bytes, nullptr, "gather buffer"))) return rc;
    GatherParams p{};
    p.k_out = tmp; p.v_out = tmp + bytes;
    p.pool = h->pool_hbm + slab_hbm(h, layer);
    p.tail = h->tail ? h->tail + slab_tail(h, layer) : nullptr;
    p.host = h->pool_host_dev ? h->pool_host_dev + slab_host(h, layer) : nullptr;
    p.table = h->table_dev + (size_t)seq * g.NB;
    p.status = h->status_dev;
    p.seq = seq; p.len = n; p.n_pool_blocks = g.hbm_cap; p.n_host_blocks = g.host_cap;
    p.Hkv = g.Hkv; p.D = g.D; p.BT = g.BT; p.block_bytes = g.block_bytes;
    h->last_fused_layer = -1;
    cudaError_t e = launch_gather(p, h->s_compute);
    ++h->launches;
    if (e == cudaSuccess && (rc = wait_stream(h, h->s_compute, "compute"))) {
        cudaFree(tmp);
        return rc;
    }
    if (e == cudaSuccess) e = cudaMemcpy(k_host, tmp, bytes, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(v_host, tmp + bytes, bytes, cudaMemcpyDeviceToHost);
    cudaFree(tmp);
    if (e != cudaSuccess) return fail(ISV_ECUDA, "gather: %s", cudaGetErrorString(e));
    return isv_sync(h, nullptr);
}

const int32_t *isv_block_table_dev(isv_kv *h, int32_t *row_stride) {
    if (!h) return nullptr;
    if (row_stride) *row_stride = h->g.NB;
    return h->table_dev;
}

const int32_t *isv_seq_lens_dev(isv_kv *h, int32_t layer) {
    if (!h || layer < 0 || layer >= h->g.layers || !h->lens_dev) return nullptr;
    return lens_ptr(h, layer, 0);
}

int isv_block_table_host(isv_kv *h, int32_t *out, int32_t n_seqs, int32_t row_stride) {
    if (!h || !out) return fail(ISV_EINVAL, "null argument");
    if (n_seqs < 0 || n_seqs > h->g.max_seqs || row_stride < h->g.NB)
        return fail(ISV_EINVAL, "n_seqs %d or row_stride %d too small (need >= %d)", n_seqs, row_stride, h->g.NB);
    for (int s = 0; s < n_seqs; ++s) {
        for (int j = 0; j < row_stride; ++j)
            out[(size_t)s * row_stride + j] = j < h->g.NB ? h->bm.entry(s, j) : ISV_BLOCK_NONE;
    }
    return ISV_OK;
}

int isv_seq_lens_host(isv_kv *h, int32_t layer, int32_t *out, int32_t n_seqs) {
    int rc = check_handle(h, layer, false);
    if (rc) return rc;
    if (!out || n_seqs < 0 || n_seqs > h->g.max_seqs) return fail(ISV_EINVAL, "bad out / n_seqs");
    for (int s = 0; s < n_seqs; ++s) out[s] = h->bm.length(layer, s);
    return ISV_OK;
}

int isv_plan_bytes(isv_kv *h, int32_t layer, int32_t n_seqs, uint64_t *res, uint64_t *off, uint64_t *staged,
                   int32_t *n_chunks) {
    int rc = check_handle(h, layer, false);
    if (rc) return rc;
    if (n_seqs < 0 || n_seqs > h->g.max_seqs) return fail(ISV_EINVAL, "n_seqs %d outside [0, %d]", n_seqs, h->g.max_seqs);
    const OffPlan &pl = h->bm.plan(layer, n_seqs);
    if (res) *res = pl.bytes_resident;
    if (off) *off = pl.bytes_offloaded;
    if (staged) *staged = pl.bytes_staged;
    if (n_chunks) *n_chunks = (int32_t)pl.chunks.size();
    return ISV_OK;
}

int isv_set_zero_copy(isv_kv *h, int32_t on) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    h->zero_copy = on != 0;
    return ISV_OK;
}

int isv_set_host_timeout(isv_kv *h, double seconds) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    if (!(seconds >= 0.0)) return fail(ISV_EINVAL, "the timeout must be >= 0 seconds (0 = none)");
    h->host_timeout_s = seconds;
    return ISV_OK;
}

int isv_set_wait_limit(isv_kv *h, uint32_t polls) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    h->spin_limit = polls;
    return ISV_OK;
}

int isv_inject_lost_copy(isv_kv *h, int32_t launches) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    if (launches < 0) return fail(ISV_EINVAL, "launches must be >= 0");
    h->lost_copies = launches;
    return ISV_OK;
}

int isv_set_timing(isv_kv *h, int32_t on) {
    if (!h) return fail(ISV_EINVAL, "null handle");
    if (h->plan_only) return fail(ISV_ENODEVICE, "plan-only handle");
    if (on) {
        int rc = ensure_timing_events(h);
        if (rc) return rc;
    }
    h->timing = on != 0;
    if (h->lev_created)
        for (auto &le : h->lev) le.have_append = le.have_decode = le.have_off = le.fused_append = false;
    return ISV_OK;
}

int isv_step_timing(isv_kv *h, int32_t layer, isv_step_times *out) {
    if (!h || !out) return fail(ISV_EINVAL, "null argument");
    if (h->plan_only) return fail(ISV_ENODEVICE, "plan-only handle");
    if (layer < -1 || layer >= h->g.layers) return fail(ISV_EINVAL, "layer %d out of range", layer);
    memset(out, 0, sizeof *out);
    uint32_t st = 0;
    int rc = isv_sync(h, &st);
    if (rc && rc != ISV_EDEVICE_STATUS) return rc;
    out->status = st;
    if (!h->lev_created) return ISV_OK;
    auto ms = [](cudaEvent_t a, cudaEvent_t b) {
        float t = 0.f;
        return cudaEventElapsedTime(&t, a, b) == cudaSuccess ? t : 0.f;
    };
    const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? h->g.layers : layer + 1;
    const LayerEvents *first = nullptr, *last = nullptr;
    for (int l = l0; l < l1; ++l) {
        const LayerEvents &le = h->lev[l];
        if (le.have_append) out->append_ms += ms(le.a0, le.a1);
        if (le.have_append || le.fused_append) out->bytes_appended += le.bytes_app;
        if (!le.have_decode) continue;
        if (!first) first = &le;
        last = &le;
        out->attn_resident_ms += ms(le.r0, le.r1);
        if (le.have_off) {
            out->h2d_ms += ms(le.c0, le.c1);
            out->attn_offloaded_ms += ms(le.o0, le.o1);
            out->merge_ms += ms(le.m0, le.m1);
        }
        out->bytes_resident += le.bytes_res;
        out->bytes_offloaded += le.bytes_off;
        out->bytes_staged += le.bytes_staged;
        out->n_chunks += le.n_chunks;
    }
    if (first) out->total_ms = ms(first->have_append ? first->a0 : first->d0, last->d1);
    cudaGetLastError();
    return ISV_OK;
}

int isv_link_probe(uint64_t bytes, int32_t reps, double *h2d_gbs, double *d2h_gbs) {
    if (bytes == 0 || reps < 1) return fail(ISV_EINVAL, "bytes and reps must be positive");
    void *hbuf = nullptr, *dbuf = nullptr;
    cudaStream_t st = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaHostAlloc(&hbuf, bytes, cudaHostAllocDefault) != cudaSuccess) {
        cudaGetLastError();
        return fail(ISV_ENOMEM_PINNED, "pinned allocation of %llu bytes failed", (unsigned long long)bytes);
    }
    cudaError_t e = cudaMalloc(&dbuf, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        cudaFreeHost(hbuf);
        return fail(ISV_ENOMEM_DEVICE, "cudaMalloc of %llu bytes failed", (unsigned long long)bytes);
    }
    memset(hbuf, 1, bytes);
    double best[2] = {0.0, 0.0};
    e = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    for (int dir = 0; dir < 2 && e == cudaSuccess; ++dir) {
        for (int r = 0; r < reps + 1 && e == cudaSuccess; ++r) {   // first pass warms up
            cudaEventRecord(e0, st);
            if (dir == 0) e = cudaMemcpyAsync(dbuf, hbuf, bytes, cudaMemcpyHostToDevice, st);
            else e = cudaMemcpyAsync(hbuf, dbuf, bytes, cudaMemcpyDeviceToHost, st);
            cudaEventRecord(e1, st);
            if (e == cudaSuccess) e = cudaStreamSynchronize(st);
            float t = 0.f;
            if (e == cudaSuccess) e = cudaEventElapsedTime(&t, e0, e1);
            if (e == cudaSuccess && r > 0 && t > 0.f) best[dir] = std::max(best[dir], (double)bytes / (t * 1e-3) / 1e9);
        }
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (st) cudaStreamDestroy(st);
    cudaFree(dbuf);
    cudaFreeHost(hbuf);
    if (e != cudaSuccess) return fail(ISV_ECUDA, "link probe: %s", cudaGetErrorString(e));
    if (h2d_gbs) *h2d_gbs = best[0];
    if (d2h_gbs) *d2h_gbs = best[1];
    return ISV_OK;
}

}  // extern "C"
