// Decode linear layers (the "linear layer" term of the paper's T_compute^d, Section IV-C:
// BS * (8 h1^2 + 4 h1 h2) flops per layer): y = x . w^T for a small batch of tokens, i.e. a
// skinny GEMM that streams the weight matrix once.  With M <= 256 tokens it is bound by the HBM
// read of w, but needs 2 * M flops per weight element, which only the tensor cores deliver at
// that rate, so this is the one dense contraction of the decode step and it runs on tcgen05:
//
//   - the weight rows are the MMA's M dimension (128 rows per CTA), the tokens its N dimension
//     (the batch, padded to a multiple of 16), so one instruction covers the whole batch;
//   - operands are staged by 2-D TMA copies with the 128-byte swizzle into a shared-memory ring,
//     issued by one thread of a producer warp; one thread of a second warp issues tcgen05.mma
//     (kind::f16, fp32 accumulation in tensor memory) and releases ring stages with
//     tcgen05.commit; four epilogue warps read the accumulator with tcgen05.ld;
//   - the (column tile, K block) list is cut into equal ranges, one per persistent CTA, so every
//     SM streams the same number of weight bytes; a CTA leaves the fp32 partial of a tile it shares
//     with others in global memory and exits, and a second, small kernel adds a tile's partials in
//     fixed order.  The streaming CTAs thus all end together and free their shared memory at once,
//     so the next call's CTAs can fill their rings with weights while the sums are still being taken.
// Every wait is bounded; on expiry the kernel flags the status word, still frees its tensor
// memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "../../include/isv.h"

namespace isv {
int set_error(int code, const char *msg);
}

namespace {

constexpr int kTileN = 128;        // weight rows per CTA (MMA M)
constexpr int kSwzK = 64;          // elements of one 128-byte swizzle row
// A ring stage holds KS sub-tiles along K (KS swizzle rows of 64 elements per matrix row), fetched by one TMA
// copy per operand: KS = 4 (512 contiguous bytes of every weight row per copy) where two such stages fit beside
// the activation tiles, else KS = 2.  Measured on B200: 4 is 1-2 % faster than 2 up to 32 tokens, 1 is slower.
constexpr int kMinTileK = 2 * kSwzK;   // K must be a multiple of this
constexpr int kWideMaxTokens = 32;     // padded batch up to which KS = 4 is chosen
constexpr int kMmaK = 16;          // K of one tcgen05.mma for 16-bit operands
constexpr int kThreads = 192;      // warp 0: TMA, warp 1: MMA + tensor memory, warps 2-5: epilogue
constexpr uint32_t kSpin = 1u << 22;

int err(int code, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    return isv::set_error(code, buf);
}

// ---------------------------------------------------------------- device helpers

__device__ __forceinline__ uint32_t s32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kSpin; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if (i > 256) __nanosleep(64);
    }
    return false;
}
// 3-D tiled TMA load.  The matrices are described as [K / 64][rows][64 elements], so that one box of
// {64, rows, KS} lands as KS consecutive [rows][64] sub-tiles, each in the 128-byte swizzle.
// x = 0 always (a multiple of 8 elements, as the 16-byte rule for the innermost coordinate asks).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int row, int kchunk, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(map), "r"(0), "r"(row), "r"(kchunk), "r"(bar)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes with the
// 128-byte swizzle: 8-row groups are 1024 bytes apart (stride byte offset), the leading byte offset
// is not used by swizzled K-major layouts, descriptor version 1, layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);          // start address, bits [0,14)
    d |= (uint64_t)1 << 16;                           // leading byte offset (ignored), bits [16,30)
    d |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                           // version, bits [46,48)
    d |= (uint64_t)2 << 61;                           // layout type, bits [61,64)
    return d;
}

// Instruction descriptor of kind::f16: fp32 accumulator, A and B of the same 16-bit type, both K-major.
__host__ __device__ constexpr uint32_t instr_desc(bool bf16, int mma_m, int mma_n) {
    return (1u << 4)                                  // D format: F32
         | ((bf16 ? 1u : 0u) << 7)                    // A format
         | ((bf16 ? 1u : 0u) << 10)                   // B format
         | (0u << 15) | (0u << 16)                    // A, B K-major
         | ((uint32_t)(mma_n >> 3) << 17)             // N / 8
         | ((uint32_t)(mma_m >> 4) << 24);            // M / 16
}

__device__ __forceinline__ void mma_f16_ss(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives on the mbarrier once all tcgen05 operations issued so far by this thread have completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32b_x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

struct LinearParams {
    void *y;                 // [M][N] 16-bit or NULL
    float *y_f32;            // [M][N] or NULL
    float *partials;         // [2 * grid][M][128] fp32: a CTA leaves at most two partial tiles
    uint32_t *status;
    int32_t M, N, K;
    int32_t mma_n;           // batch padded to a multiple of 16
    int32_t stages, tmem_cols, bf16;
    int32_t tile_k;          // elements per ring stage along K (64 * KS)
    int32_t grid_main;       // CTAs of linear_kernel (the reduction needs the same cut)
};

// One epilogue thread's 16 accumulator values (tokens c0 .. c0 + 15 of one weight row) to memory: as fp32
// at f32[token * f32_stride] (F32), as 16-bit values at h16[token * h16_stride] (H16), tokens beyond M left out.
// The destinations are chosen once per segment, outside the loop over the tokens.
template <bool F32, bool H16, bool BF16>
__device__ __forceinline__ void put16(const uint32_t (&r)[16], int c0, int M, float *f32, size_t f32_stride,
                                      uint16_t *h16, size_t h16_stride) {
    const bool whole = c0 + 16 <= M;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        if (!whole && c0 + j >= M) break;
        const float v = __uint_as_float(r[j]);
        if (F32) f32[(size_t)(c0 + j) * f32_stride] = v;
        if (H16) {
            if (BF16) {
                const __nv_bfloat16 h = __float2bfloat16_rn(v);
                h16[(size_t)(c0 + j) * h16_stride] = *reinterpret_cast<const uint16_t *>(&h);
            } else {
                const __half h = __float2half_rn(v);
                h16[(size_t)(c0 + j) * h16_stride] = *reinterpret_cast<const uint16_t *>(&h);
            }
        }
    }
}

// Four adjacent outputs of one token (n a multiple of 4).
__device__ __forceinline__ void store_out4(const LinearParams &p, int m, int n, float4 v) {
    const size_t idx = (size_t)m * p.N + n;
    if (p.y_f32) *reinterpret_cast<float4 *>(p.y_f32 + idx) = v;
    if (p.y) {
        uint2 w;
        if (p.bf16) {
            const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
            w.x = *reinterpret_cast<const uint32_t *>(&a);
            w.y = *reinterpret_cast<const uint32_t *>(&b);
        } else {
            const __half2 a = __floats2half2_rn(v.x, v.y), b = __floats2half2_rn(v.z, v.w);
            w.x = *reinterpret_cast<const uint32_t *>(&a);
            w.y = *reinterpret_cast<const uint32_t *>(&b);
        }
        *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(p.y) + idx) = w;
    }
}

// The work is the flat list of (column tile, K block) pairs, tile-major; it is cut into equal
// contiguous ranges, one per CTA (persistent, one CTA per SM), so every SM streams the same number
// of weight bytes whatever the matrix shape.  A run of K blocks of one tile inside a range is a
// segment: a segment that covers its whole tile is stored directly, otherwise its fp32 partial goes
// to one of the CTA's two slots (slot 0 if the segment opens the CTA's range, else slot 1) and
// linear_reduce_kernel adds the partials in fixed order.  The ring of TMA stages runs across
// segments without draining, and two accumulators in tensor memory let the epilogue of one segment
// overlap the MMAs of the next.
struct Cut {
    long long total;
    int n;
    __device__ long long first(int c) const { return total * c / n; }
    __device__ int range_of(long long x) const { return (int)(((x + 1) * n - 1) / total); }
    __device__ static Cut of(const LinearParams &p, int grid) {
        Cut c;
        c.total = (long long)(p.N / kTileN) * (p.K / p.tile_k);
        c.n = (int)min((long long)grid, c.total);
        return c;
    }
};

template <int KS>
__global__ void __launch_bounds__(kThreads, 2)
linear_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const LinearParams p) {
    extern __shared__ uint8_t smem_raw[];
    // the 128-byte swizzle wants tile bases on 1024-byte boundaries of the shared address space
    uint8_t *smem = smem_raw + ((1024u - (s32(smem_raw) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kTileK = kSwzK * KS;
    const int kblocks = p.K / kTileK;
    const Cut cut = Cut::of(p, gridDim.x);
    const int cta = blockIdx.x;
    if (cta >= cut.n) return;
    const long long f0 = cut.first(cta), f1 = cut.first(cta + 1);

    const uint32_t a_bytes = kTileN * kTileK * 2;                 // weight tile of one stage
    const uint32_t b_bytes = (uint32_t)p.mma_n * kTileK * 2;      // activation tile of one stage
    const uint32_t stage_bytes = a_bytes + ((b_bytes + 1023u) & ~1023u);
    uint8_t *ring = smem;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)p.stages * stage_bytes);
    uint64_t *empty = full + p.stages;
    uint64_t *acc_full = empty + p.stages;      // [2]
    uint64_t *acc_empty = acc_full + 2;         // [2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile int *failed = reinterpret_cast<volatile int *>(tmem_slot + 1);
    volatile int *ep_fail = failed + 1;   // written and read by the epilogue warps only, around their barrier
    const int prefill = (int)min((long long)p.stages, f1 - f0);

    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(s32(&full[s]), 1);
            mbar_init(s32(&empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(s32(&acc_full[b]), 1);
            mbar_init(s32(&acc_empty[b]), 4);   // one arrival per epilogue warp
        }
        *failed = 0;
        *ep_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // The weights never change, so the ring is filled with weight tiles at once, before tensor memory
        // is allocated and before the kernels launched ahead of this one have finished (programmatic
        // dependent launch): the ramp-up overlaps the previous kernel's tail.  The matching activation
        // tiles follow once that kernel is complete.
        for (int it = 0; it < prefill; ++it) {
            const long long f = f0 + it;
            const uint32_t bar = s32(&full[it]);
            mbar_expect_tx(bar, a_bytes + b_bytes);
            tma_load_3d(s32(ring + (size_t)it * stage_bytes), &map_w, (int)(f / kblocks) * kTileN,
                        (int)(f % kblocks) * KS, bar);
        }
    }
    if (warp == 1) {   // tensor memory: two accumulators of mma_n columns, power-of-two total
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(tmem_slot)), "r"(p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ---- producer: one thread walks the CTA's range and issues the TMA copies
        if (lane == 0) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int it = 0; it < prefill; ++it)
                tma_load_3d(s32(ring + (size_t)it * stage_bytes + a_bytes), &map_x, 0,
                            (int)((f0 + it) % kblocks) * KS, s32(&full[it]));
            int it = prefill;
            for (long long f = f0 + prefill; f < f1; ++f, ++it) {
                const int t = (int)(f / kblocks), kb = (int)(f % kblocks);
                const int s = it % p.stages;
                if (!mbar_wait(s32(&empty[s]), ((it / p.stages) - 1) & 1)) { *failed = 1; break; }
                if (*failed) break;
                const uint32_t bar = s32(&full[s]);
                uint8_t *st = ring + (size_t)s * stage_bytes;
                mbar_expect_tx(bar, a_bytes + b_bytes);
                tma_load_3d(s32(st), &map_w, t * kTileN, kb * KS, bar);
                tma_load_3d(s32(st + a_bytes), &map_x, 0, kb * KS, bar);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: one thread; accumulators alternate between segments
        if (lane == 0) {
            const uint32_t idesc = instr_desc(p.bf16 != 0, kTileN, p.mma_n);
            int it = 0, g = 0;
            bool ok = true;
            for (long long f = f0; f < f1 && ok; ++g) {
                const int t = (int)(f / kblocks);
                const long long seg_end = min(f1, (long long)(t + 1) * kblocks);
                const int b = g & 1, u = g >> 1;
                if (u >= 1 && !mbar_wait(s32(&acc_empty[b]), (u - 1) & 1)) { ok = false; break; }   // epilogue drained it
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem_base + (uint32_t)(b * p.mma_n);
                for (int i = 0; f < seg_end; ++f, ++it, ++i) {
                    const int s = it % p.stages;
                    if (!mbar_wait(s32(&full[s]), (it / p.stages) & 1) || *failed) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = s32(ring + (size_t)s * stage_bytes);
#pragma unroll
                    for (int sub = 0; sub < KS; ++sub) {
                        const uint64_t da = smem_desc_sw128(a_addr + sub * (kTileN * kSwzK * 2));
                        const uint64_t db = smem_desc_sw128(a_addr + a_bytes + sub * (p.mma_n * kSwzK * 2));
#pragma unroll
                        for (int k = 0; k < kSwzK / kMmaK; ++k) {
                            // 16 elements = 32 bytes further along K inside the swizzled row: +2 in units of 16 bytes
                            mma_f16_ss(acc, da + 2 * k, db + 2 * k, idesc, (i > 0 || sub > 0 || k > 0) ? 1u : 0u);
                        }
                    }
                    mma_commit(s32(&empty[s]));       // the stage may be refilled once these MMAs have read it
                }
                if (!ok) break;
                mma_commit(s32(&acc_full[b]));        // this segment's accumulator is complete
            }
            if (!ok) {   // a wait expired: flag it; the epilogue warps run into their own bounded waits
                *failed = 1;
                atomicOr(p.status, ISV_STATUS_WAIT_EXPIRED);
            }
        }
    } else {
        // ---- epilogue: warp w reads tensor-memory lanes [32 * (w % 4), +32) = weight rows of the tile
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        asm volatile("griddepcontrol.wait;" ::: "memory");   // outputs and partials may still be in use
        int g = 0;
        for (long long f = f0; f < f1; ++g) {
            const int t = (int)(f / kblocks);
            const long long start = (long long)t * kblocks, seg_end = min(f1, start + kblocks);
            const bool complete = (f == start) && (seg_end == start + kblocks);
            const bool first_seg = (f == f0);
            f = seg_end;
            const int b = g & 1, u = g >> 1;
            if (!mbar_wait(s32(&acc_full[b]), u & 1)) *ep_fail = 1;
            asm volatile("bar.sync 1, 128;" ::: "memory");          // the four epilogue warps decide together
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (*ep_fail) {
                if (lane == 0) atomicOr(p.status, ISV_STATUS_WAIT_EXPIRED);
                break;
            }
            float *slot = p.partials + (size_t)(2 * cta + (first_seg ? 0 : 1)) * p.M * kTileN;
            const int n = t * kTileN + row;
            // a partial goes to the CTA's slot as fp32 rows of 128; a whole tile straight to the outputs
            float *f32 = complete ? (p.y_f32 ? p.y_f32 + n : nullptr) : slot + row;
            uint16_t *h16 = complete && p.y ? reinterpret_cast<uint16_t *>(p.y) + n : nullptr;
            const size_t f32_stride = complete ? (size_t)p.N : (size_t)kTileN;
            const int mode = (f32 ? 1 : 0) | (h16 ? (p.bf16 ? 4 : 2) : 0);
            for (int c0 = 0; c0 < p.mma_n; c0 += 16) {
                uint32_t r[16];
                tmem_ld_32x32b_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * p.mma_n + c0), r);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                switch (mode) {
                case 1: put16<true, false, false>(r, c0, p.M, f32, f32_stride, h16, (size_t)p.N); break;
                case 2: put16<false, true, false>(r, c0, p.M, f32, f32_stride, h16, (size_t)p.N); break;
                case 3: put16<true, true, false>(r, c0, p.M, f32, f32_stride, h16, (size_t)p.N); break;
                case 4: put16<false, true, true>(r, c0, p.M, f32, f32_stride, h16, (size_t)p.N); break;
                default: put16<true, true, true>(r, c0, p.M, f32, f32_stride, h16, (size_t)p.N); break;
                }
            }
            // the accumulator may be overwritten by the segment after next
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(&acc_empty[b])) : "memory");
        }
    }

    // ---- tear-down: everyone meets, tensor memory is returned
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
    }
}

// Adds the partials of every tile that several CTAs of linear_kernel shared: CTA (tile, group of
// kRedRows tokens), thread = 4 adjacent outputs of one token, contributors in their fixed order, kFly
// of them in flight at a time.  Its loads queue behind the weight tiles that the next call's CTAs are
// already fetching, so a round trip costs 1.5-2 us: a small grid takes up to eight contributors in
// one round; a large grid (many tokens) keeps four, because more registers per thread would leave too
// few of these CTAs beside the streaming ones (measured slower).  It runs as a programmatic dependent
// of linear_kernel; every CTA waits for that kernel, also one with nothing to add, so that this grid
// never completes first.
constexpr int kRedThreads = 256, kRedRows = 2 * (kRedThreads / 32);

// 16-byte load that bypasses L1, issued only if `pred`; the result is zero otherwise
__device__ __forceinline__ float4 ldcg_if(const float *src, bool pred) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    asm volatile(
        "{\n.reg .pred q;\nsetp.ne.b32 q, %5, 0;\n@q ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];\n}\n"
        : "+f"(v.x), "+f"(v.y), "+f"(v.z), "+f"(v.w)
        : "l"(src), "r"((int)pred)
        : "memory");
    return v;
}

template <int kFly>
__global__ void __launch_bounds__(kRedThreads, kFly == 4 ? 4 : 2) linear_reduce_kernel(const LinearParams p) {
    const int kblocks = p.K / p.tile_k;
    const Cut cut = Cut::of(p, p.grid_main);
    const int groups = (p.M + kRedRows - 1) / kRedRows;
    const int t = blockIdx.x / groups, m0 = (blockIdx.x % groups) * kRedRows;
    const long long start = (long long)t * kblocks;
    const int cf = cut.range_of(start), cl = cut.range_of(start + kblocks - 1);
    const int nc = cl - cf + 1;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (nc == 1) return;                              // the tile was stored whole by its one CTA
    if (m0 + (int)(threadIdx.x >> 5) >= p.M) return;  // this warp's tokens lie beyond the batch
    const int cf_slot = (cut.first(cf) == start) ? 0 : 1;
    const int cg = threadIdx.x & 31, mr = threadIdx.x >> 5;
    const int m[2] = {m0 + mr, m0 + mr + kRedThreads / 32};
    float4 acc[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
    for (int c0 = 0; c0 < nc; c0 += kFly) {
        float4 v[kFly][2];
#pragma unroll
        for (int j = 0; j < kFly; ++j) {
            // predicated loads, not branches, so that all of them are issued before the first is used
            const int c = min(c0 + j, nc - 1);
            const int sl = c == 0 ? 2 * cf + cf_slot : 2 * (cf + c);
            const float *src = p.partials + (size_t)sl * p.M * kTileN + 4 * cg;
#pragma unroll
            for (int r = 0; r < 2; ++r)
                v[j][r] = ldcg_if(src + (size_t)min(m[r], p.M - 1) * kTileN, c0 + j < nc && m[r] < p.M);
        }
#pragma unroll
        for (int j = 0; j < kFly; ++j)
#pragma unroll
            for (int r = 0; r < 2; ++r) {   // adding the zeros of a load that was not issued changes nothing
                acc[r].x += v[j][r].x; acc[r].y += v[j][r].y; acc[r].z += v[j][r].z; acc[r].w += v[j][r].w;
            }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r)
        if (m[r] < p.M) store_out4(p, m[r], t * kTileN + 4 * cg, acc[r]);
}

// ---------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Map of a row-major [rows][K] 16-bit matrix seen as [K / 64][rows][64], boxes of ks x box_rows x 64
// elements, 128-byte swizzle, zero fill outside the matrix.
int make_map(CUtensorMap *m, const void *base, int rows, int K, int box_rows, int ks, bool bf16) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return err(ISV_ECUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t dims[3] = {(cuuint64_t)kSwzK, (cuuint64_t)rows, (cuuint64_t)(K / kSwzK)};
    const cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)kSwzK * 2};   // bytes: next row, next 64-element chunk
    const cuuint32_t box[3] = {(cuuint32_t)kSwzK, (cuuint32_t)box_rows, (cuuint32_t)ks};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
                          const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return err(ISV_ECUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return ISV_OK;
}

}  // namespace

struct isv_linear {
    const void *w = nullptr;
    int N = 0, K = 0, max_M = 0;
    bool bf16 = false;
    cudaStream_t stream = nullptr;
    CUtensorMap map_w[2];   // stages of 2 and of 4 sub-tiles along K
    bool has_ks[2] = {false, false};
    int grid = 1;
    float *partials = nullptr;
    bool split[2] = {false, false};   // some tile is shared by several CTAs: the reduction kernel follows every launch
    uint32_t *status = nullptr;
    int smem_optin = 0;
};

extern "C" {

int isv_linear_free(isv_linear *l) {
    if (!l) return err(ISV_EINVAL, "null handle");
    if (l->stream) cudaStreamSynchronize(l->stream);
    cudaFree(l->partials);
    cudaFree(l->status);
    delete l;
    return ISV_OK;
}

int isv_linear_create(isv_linear **out, const void *w_dev, int32_t N, int32_t K, int32_t dtype, int32_t max_M,
                      void *stream) {
    if (!out) return err(ISV_EINVAL, "out is null");
    *out = nullptr;
    if (!w_dev || (reinterpret_cast<uintptr_t>(w_dev) & 15u)) return err(ISV_EINVAL, "w must be non-null, 16-byte aligned");
    if (N < kTileN || N % kTileN != 0) return err(ISV_EINVAL, "N (%d) must be a positive multiple of %d", N, kTileN);
    if (K < kMinTileK || K % kMinTileK != 0) return err(ISV_EINVAL, "K (%d) must be a positive multiple of %d", K, kMinTileK);
    if (max_M < 1 || max_M > 256) return err(ISV_EINVAL, "max_M (%d) must be in [1, 256]", max_M);
    if (dtype != ISV_F16 && dtype != ISV_BF16) return err(ISV_EINVAL, "dtype must be ISV_F16 or ISV_BF16");
    isv_linear *l = new (std::nothrow) isv_linear();
    if (!l) return err(ISV_EINVAL, "out of host memory");
    l->w = w_dev; l->N = N; l->K = K; l->max_M = max_M; l->bf16 = dtype == ISV_BF16;
    l->stream = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&l->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) { delete l; return err(ISV_ECUDA, "isv_linear_create: %s", cudaGetErrorString(e)); }
    const int n_tiles = N / kTileN;
    l->grid = sms;                      // persistent: one CTA per SM (two per SM with half the ring each measured no faster)
    for (int v = 0; v < 2; ++v) {       // variant v: stages of KS = 2 << v sub-tiles
        const int ks = 2 << v;
        if (K % (kSwzK * ks) != 0) continue;
        l->has_ks[v] = true;
        int rc = make_map(&l->map_w[v], w_dev, N, K, kTileN, ks, l->bf16);
        if (rc) { delete l; return rc; }
        // the kernel's cut of the (tile, K block) list: a range border inside a tile splits that tile
        const long long kblocks = K / (kSwzK * ks), total = (long long)n_tiles * kblocks;
        const long long n = std::min<long long>(l->grid, total);
        for (long long c = 1; c < n && !l->split[v]; ++c) l->split[v] = (total * c / n) % kblocks != 0;
    }
    e = cudaMalloc((void **)&l->status, 4);
    if (e == cudaSuccess) e = cudaMemset(l->status, 0, 4);
    if (e == cudaSuccess) e = cudaMalloc((void **)&l->partials, (size_t)2 * l->grid * max_M * kTileN * 4);
    // the kernel also has a few bytes of static shared memory: leave room for them under the limit
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(linear_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, l->smem_optin - 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(linear_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, l->smem_optin - 1024);
    if (e != cudaSuccess) {
        cudaGetLastError();
        isv_linear_free(l);
        return err(ISV_ENOMEM_DEVICE, "isv_linear_create: %s", cudaGetErrorString(e));
    }
    *out = l;
    return ISV_OK;
}

int isv_linear_forward(isv_linear *l, const void *x_dev, void *y_dev, float *y_f32_dev, int32_t M) {
    if (!l) return err(ISV_EINVAL, "null handle");
    if (!x_dev || (!y_dev && !y_f32_dev)) return err(ISV_EINVAL, "x and one of y / y_f32 must be given");
    if ((reinterpret_cast<uintptr_t>(x_dev) & 15u)) return err(ISV_EINVAL, "x must be 16-byte aligned");
    if (M < 1 || M > l->max_M) return err(ISV_EINVAL, "M (%d) must be in [1, %d]", M, l->max_M);
    LinearParams p{};
    p.y = y_dev; p.y_f32 = y_f32_dev; p.partials = l->partials; p.status = l->status;
    p.M = M; p.N = l->N; p.K = l->K;
    p.mma_n = std::max(16, (M + 15) / 16 * 16);
    p.bf16 = l->bf16 ? 1 : 0;
    p.grid_main = l->grid;
    int cols = 32;
    while (cols < 2 * p.mma_n) cols *= 2;        // two accumulators
    p.tmem_cols = cols;
    const size_t fixed = 1024 /* alignment slack */ + 1024 /* static */ + 512 /* barriers, slots */;
    // about 200 KB of ring (measured on B200: 100 -> 180 KB is 8-10 % faster on the large projections although
    // the next launch's CTA then no longer fits beside this one's to prefetch its weights early); 216 KB where
    // that is what two or three of the wider stages take
    size_t ring_budget = 200u << 10;
    if (const char *e = getenv("ISV_LINEAR_RING_KB")) ring_budget = (size_t)std::max(32, std::min(220, atoi(e))) << 10;   // tuning knob
    int v = 0, stages = 0;                        // stage variant: KS = 2 << v
    size_t stage_bytes = 0;
    // ISV_LINEAR_KS (tuning knob) = 2 or 4 asks for that stage width where the matrix and the batch allow it
    const int asked = getenv("ISV_LINEAR_KS") ? atoi(getenv("ISV_LINEAR_KS")) : 0;
    for (int pass = asked ? 0 : 1; pass < 2 && stages < 2; ++pass)
        for (int cand = 1; cand >= 0 && stages < 2; --cand) {
            if (!l->has_ks[cand]) continue;
            if (pass == 0 ? asked != (2 << cand) : (cand == 1 && p.mma_n > kWideMaxTokens)) continue;
            const size_t tile_k = (size_t)kSwzK * (2 << cand);
            const size_t sb = (size_t)kTileN * tile_k * 2 + (((size_t)p.mma_n * tile_k * 2 + 1023) & ~(size_t)1023);
            const size_t budget = (cand == 1 && !getenv("ISV_LINEAR_RING_KB")) ? (216u << 10) : ring_budget;
            const int st = (int)std::min<size_t>(std::max<size_t>(2, budget / sb), ((size_t)l->smem_optin - fixed) / sb);
            if (st >= 2) { v = cand; stage_bytes = sb; stages = st; }
        }
    if (stages < 2) return err(ISV_EINVAL, "shared memory too small for this batch");
    p.stages = stages;
    p.tile_k = kSwzK * (2 << v);
    const size_t smem = 1024 + (size_t)stages * stage_bytes + (2 * stages + 4) * 8 + 64;
    CUtensorMap map_x;
    int rc = make_map(&map_x, x_dev, M, l->K, p.mma_n, 2 << v, l->bf16);   // rows beyond M read as zeros
    if (rc) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(l->grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = l->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;   // see the kernel's griddepcontrol use
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = v == 1 ? cudaLaunchKernelEx(&cfg, linear_kernel<4>, l->map_w[1], map_x, p)
                           : cudaLaunchKernelEx(&cfg, linear_kernel<2>, l->map_w[0], map_x, p);
    if (e == cudaSuccess && l->split[v]) {
        const int red_grid = (l->N / kTileN) * ((M + kRedRows - 1) / kRedRows);
        cfg.gridDim = dim3((unsigned)red_grid);
        cfg.blockDim = dim3(kRedThreads);
        cfg.dynamicSmemBytes = 0;
        e = red_grid <= 2 * l->grid ? cudaLaunchKernelEx(&cfg, linear_reduce_kernel<8>, p)
                                    : cudaLaunchKernelEx(&cfg, linear_reduce_kernel<4>, p);
    }
    if (e != cudaSuccess) return err(ISV_ECUDA, "isv_linear_forward: %s", cudaGetErrorString(e));
    return ISV_OK;
}

int isv_linear_status(isv_linear *l, uint32_t *status_out) {
    if (!l || !status_out) return err(ISV_EINVAL, "null argument");
    cudaError_t e = cudaStreamSynchronize(l->stream);
    if (e == cudaSuccess) e = cudaMemcpy(status_out, l->status, 4, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return err(ISV_ECUDA, "isv_linear_status: %s", cudaGetErrorString(e));
    if (*status_out) {
        cudaMemset(l->status, 0, 4);
        return err(ISV_EDEVICE_STATUS, "the linear kernel reported status 0x%x", *status_out);
    }
    return ISV_OK;
}

}  // extern "C"
