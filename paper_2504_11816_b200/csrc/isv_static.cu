// isv_attn_decode_static: decode attention over an all-resident paged KV pool
// for callers that must not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits - inside a
// serving loop whose memory is fully handed to a framework's caching allocator
// (a raw cudaMalloc there can fail or fragment the pool), in latency-critical
// paths where an allocation would synchronise the device, or in plugins that
// are only given pointers and a stream.  The handle-based entry points
// allocate their pools and scratch in isv_kv_alloc; this one allocates nothing
// at all: the caller brings the KV pool, table, lengths, q and out, and the
// split kernel's scratch (per-split partial results and arrival tickets) lives
// in the fixed array below, which every GPU that loads the library holds until
// the process exits.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <mutex>

#include "../../include/isv.h"
#include "isv_kernels.cuh"

namespace isv {
int set_error(int code, const char *msg);   // isv_api.cu: records the calling thread's last error
}

using namespace isv;

namespace {

// Scratch of the static entry point.  In host code this name is only a
// stand-in for the symbol, not a device address: the address is looked up
// with cudaGetSymbolAddress below and that pointer is what kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[ISV_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
constexpr size_t kHeaderBytes = 256;   // status word, padded

struct DeviceSetup {
    bool ready = false;
    unsigned char *scratch = nullptr;   // device address of g_static_scratch on this device
    int sm_count = 0;
    int smem_optin = 0;
};
DeviceSetup g_dev[kMaxDevices];
std::mutex g_mu;

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

int err(int code, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    return set_error(code, buf);
}

}  // namespace

extern "C" int isv_attn_decode_static(const void *kv_pool_dev, int32_t n_pool_blocks,
                                      const int32_t *block_table_dev, int32_t table_stride,
                                      const int32_t *seq_lens_dev, int32_t n_seqs, int32_t max_blocks_per_seq,
                                      int32_t q_heads, int32_t kv_heads, int32_t head_dim, int32_t block_tokens,
                                      int32_t dtype, int32_t max_ctas, const void *q_dev, void *out_dev,
                                      float *out_f32_dev, uint32_t *status_dev, void *stream) {
    if (!kv_pool_dev || !block_table_dev || !seq_lens_dev || !q_dev || (!out_dev && !out_f32_dev))
        return err(ISV_EINVAL, "isv_attn_decode_static: pool, table, lengths, q and one output are required");
    auto mis = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (mis(kv_pool_dev) || mis(q_dev) || mis(out_dev) || mis(out_f32_dev))
        return err(ISV_EINVAL, "isv_attn_decode_static: pool, q and outputs must be 16-byte aligned");
    if (kv_heads < 1 || q_heads < 1 || q_heads % kv_heads != 0)
        return err(ISV_EINVAL, "isv_attn_decode_static: q_heads must be a positive multiple of kv_heads");
    if ((head_dim != 64 && head_dim != 80 && head_dim != 128) || block_tokens != 16 ||
        (dtype != ISV_F16 && dtype != ISV_BF16))
        return err(ISV_EINVAL, "isv_attn_decode_static: head_dim 64/80/128, block_tokens 16, dtype f16/bf16 only");
    if (n_seqs < 0 || n_seqs > 4096 || max_blocks_per_seq < 1 || table_stride < max_blocks_per_seq ||
        n_pool_blocks < 1 || max_ctas < 0)
        return err(ISV_EINVAL, "isv_attn_decode_static: bad n_seqs (%d) or block counts (%d)", n_seqs,
                   max_blocks_per_seq);
    if (n_seqs == 0) return ISV_OK;

    const int G = q_heads / kv_heads;
    const int HP = pair_heads(G, head_dim, kv_heads);   // KV heads per head group
    const int GT = HP == 2 ? 2 : group_heads(G);
    const int P = HP == 2 ? 1 : G / GT;
    if ((long long)n_seqs * max_blocks_per_seq * kv_heads * P >= (1ll << 31))
        return err(ISV_EINVAL, "isv_attn_decode_static: n_seqs * blocks * heads too large");

    // ---- once per device: address of the scratch symbol and device limits
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return err(ISV_ECUDA, "isv_attn_decode_static: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return err(ISV_EINVAL, "isv_attn_decode_static: device index %d not supported", dev);
    DeviceSetup ds;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_dev[dev].ready) {
            void *ptr = nullptr;
            e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            if (e != cudaSuccess || !ptr) {
                cudaGetLastError();
                return err(ISV_ECUDA, "isv_attn_decode_static: cudaGetSymbolAddress failed");
            }
            int sms = 0, optin = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
            if (e != cudaSuccess) return err(ISV_ECUDA, "isv_attn_decode_static: %s", cudaGetErrorString(e));
            g_dev[dev].scratch = static_cast<unsigned char *>(ptr);
            g_dev[dev].sm_count = sms;
            g_dev[dev].smem_optin = optin;
            g_dev[dev].ready = true;
        }
        ds = g_dev[dev];
    }

    // ---- scratch: counters per (sequence, head group) and two partials per warp of the grid.
    // A grid whose partials would not fit is cut down to the CTAs that do fit (the kernel is persistent
    // and divides the work among however many CTAs it gets); only a shape that leaves no room for one
    // CTA is refused.
    const int nw = decode_warps(GT, head_dim, HP);
    const long long blocks = (long long)n_seqs * max_blocks_per_seq * kv_heads * P / HP;   // visits of the flat work list
    const int cap = max_ctas > 0 ? std::min(max_ctas, ds.sm_count) : ds.sm_count;
    int grid = (int)std::max<long long>(1, std::min<long long>(cap, (blocks + nw - 1) / nw));
    const size_t tickets_bytes = align256((size_t)n_seqs * kv_heads * P * 4);
    const size_t per_cta = 2ull * nw * GT * (2 + head_dim) * 4;   // (m, l) and o of two partials per warp and head
    const size_t fixed = kHeaderBytes + tickets_bytes + 256;      // + alignment slack of the (m, l) array
    const long long fit =
        fixed < (size_t)ISV_STATIC_SCRATCH_BYTES ? (long long)(((size_t)ISV_STATIC_SCRATCH_BYTES - fixed) / per_cta) : 0;
    if (fit < 1)
        return err(ISV_ECAPACITY,
                   "isv_attn_decode_static: this shape needs %lld bytes of scratch (arrival counters for %d sequences "
                   "x %d head groups plus the split partials of one CTA) but the fixed array holds %lld; use fewer "
                   "sequences or heads per call, or the handle-based isv_attn_decode",
                   (long long)(fixed + per_cta), n_seqs, kv_heads * P, (long long)ISV_STATIC_SCRATCH_BYTES);
    grid = (int)std::min<long long>(grid, fit);
    const size_t slots = 2ull * grid * nw * GT;
    const size_t ml_bytes = align256(slots * 2 * 4);

    // ---- shared-memory ring depth that fits
    const bool bf16 = dtype == ISV_BF16;
    int stages = 0;
    size_t smem = 0;
    for (int st = 2; st <= decode_default_stages(head_dim, block_tokens, GT, HP); ++st) {
        const size_t b = decode_smem_bytes(head_dim, block_tokens, GT, HP, st, n_seqs, MODE_RESIDENT);
        if (b <= (size_t)ds.smem_optin) { stages = st; smem = b; }
    }
    if (stages < 2) return err(ISV_EINVAL, "isv_attn_decode_static: shared memory too small for this shape");
    // the limit is raised to the device maximum so that it never undercuts another user of the kernel
    e = decode_configure(head_dim, GT, HP, block_tokens, bf16, MODE_RESIDENT, (size_t)ds.smem_optin);
    if (e != cudaSuccess) return err(ISV_ECUDA, "isv_attn_decode_static: %s", cudaGetErrorString(e));

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char *base = ds.scratch;
    // status word and tickets must start at zero; the array keeps whatever the previous call left
    e = cudaMemsetAsync(base, 0, kHeaderBytes + tickets_bytes, st);
    if (e != cudaSuccess) return err(ISV_ECUDA, "isv_attn_decode_static: %s", cudaGetErrorString(e));

    DecodeParams p{};
    p.pool = static_cast<const uint8_t *>(kv_pool_dev);
    p.tail = nullptr;                       // host-flagged table entries are skipped
    p.table = block_table_dev;
    p.lens = seq_lens_dev;
    p.table_stride = table_stride;
    p.max_blocks = max_blocks_per_seq;      // longer (or negative) lengths are clamped and flagged
    p.n_pool_blocks = n_pool_blocks;
    p.q = q_dev;
    p.out = out_dev;
    p.out_f32 = out_f32_dev;
    p.status = status_dev ? status_dev : reinterpret_cast<uint32_t *>(base);
    p.tickets = reinterpret_cast<int32_t *>(base + kHeaderBytes);
    p.part_ml = reinterpret_cast<float *>(base + kHeaderBytes + tickets_bytes);
    p.part_o = reinterpret_cast<float *>(base + kHeaderBytes + tickets_bytes + ml_bytes);
    p.acc_o = nullptr;
    p.acc_ml = nullptr;
    p.n_seqs = n_seqs; p.Hq = q_heads; p.Hkv = kv_heads; p.P = P; p.GT = GT;
    p.finalize = 1;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)head_dim));
    p.block_bytes = 2ull * kv_heads * block_tokens * head_dim * 2ull;
    e = launch_decode(p, head_dim, GT, HP, block_tokens, bf16, MODE_RESIDENT, grid, stages, smem, st);
    if (e != cudaSuccess) return err(ISV_ECUDA, "isv_attn_decode_static: %s", cudaGetErrorString(e));
    return ISV_OK;
}
