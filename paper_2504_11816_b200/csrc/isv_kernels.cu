// CUDA kernels of the offloaded-KV decode path (sm_100a):
//   decode_kernel   split flash-decoding over paged K/V tiles, persistent CTAs,
//                   one autonomous TMA-fed pipeline per warp
//   merge_kernel    log-sum-exp merge of the resident result and the
//                   offloaded running state
//   append_kernel   K and V of one new token per sequence, one launch
//   fill / gather   prompt load and logical-order read-back
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/isv.h"
#include "isv_kernels.cuh"

namespace isv {

namespace {

constexpr float kNegBig = -1.0e30f;          // "no score yet": finite so differences never give NaN
constexpr uint32_t kFull = 0xffffffffu;
constexpr uint32_t kSpinLimit = 1u << 22;    // polls before a wait gives up (DecodeParams::spin_limit overrides it)

// ---------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false when the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit) {
    if (mbar_try_wait(bar, parity)) return true;   // the usual case: the copy landed while the warp computed
    for (uint32_t i = 1; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 256) __nanosleep(64);
    }
    return false;
}
// 1-D bulk copy global -> shared of this CTA, completion counted on an mbarrier.
// Addresses and size are multiples of 16 bytes by construction of the pool layout.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

template <bool BF16>
__device__ __forceinline__ void cvt8(const uint4 &r, float (&f)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (BF16) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        } else {
            const __half2 h = *reinterpret_cast<const __half2 *>(&w[i]);
            const float2 t = __half22float2(h);
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
    }
}

// Two independent fp32 FMAs in one instruction (sm_100 packed fp32): d0 += a0 * b0, d1 += a1 * b1,
// each rounded exactly like fmaf.  Halves the issue slots of the dot products and the weighted sums.
__device__ __forceinline__ void ffma2(float &d0, float &d1, float a0, float a1, float b0, float b1) {
#ifndef ISV_NO_FFMA2
    asm("{\n"
        ".reg .b64 ra, rb, rd;\n"
        "mov.b64 ra, {%2, %3};\n"
        "mov.b64 rb, {%4, %5};\n"
        "mov.b64 rd, {%0, %1};\n"
        "fma.rn.f32x2 rd, ra, rb, rd;\n"
        "mov.b64 {%0, %1}, rd;\n"
        "}\n"
        : "+f"(d0), "+f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
#else
    d0 = fmaf(a0, b0, d0);
    d1 = fmaf(a1, b1, d1);
#endif
}

// 2^x by the special-function unit alone (ex2.approx: relative error about 2^-22, 2^0 = 1 exactly, results
// below the normal range flush to zero).  exp2f adds a range-scaling sequence around the same instruction;
// softmax weights need neither the extra bits nor denormal results, and the tile loops run it per token.
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <bool BF16>
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    if (BF16) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<const uint32_t *>(&h);
    } else {
        const __half2 h = __floats2half2_rn(a, b);
        return *reinterpret_cast<const uint32_t *>(&h);
    }
}

// Inside a (block, K|V, head) tile the 16-byte chunk c of token t's row is stored at chunk position
// c ^ (t & 7) of that row, in HBM, host memory and shared memory alike (tiles are copied verbatim).
// Eight consecutive tokens then keep the same logical chunk in eight different bank groups, which makes
// the matrix loads of the tensor-core path conflict-free; readers that take a whole 128-byte span of
// one row per quarter-warp are unaffected.  A row of `nchunks` chunks is permuted in its complete groups
// of eight; a trailing incomplete group (head_dim 80: chunks 8 and 9) stays in place.
__device__ __forceinline__ int swz(int chunk, int t, int nchunks) {
    return chunk < (nchunks & ~7) ? chunk ^ (t & 7) : chunk;
}

// ---------------------------------------------------------------- one K tile, one V tile

// Lane layout inside a warp: grp = lane / 8 owns tokens grp, grp+4, ... of the
// tile; sub = lane % 8 owns head-dim elements [v*64 + sub*8, +8) of every complete
// 64-element span v.  Each group keeps its own running (m, l, o); groups are merged at unit end.
// head_dim 80 leaves a tail of 16 elements = 2 chunks per token.  Giving it to lanes sub 0 and 1 of every
// pass would cost a whole span's instructions for a quarter of the lanes, so the tails of a group's four
// tokens are handled in one extra step instead: lane sub takes the tail chunk (sub & 1) of one token of
// pass sub / 2 (for K: tail_token below; for V: the group's own token of that pass).  Its registers q[.][NVF*8 ..] / o[.][NVF*8 ..] then belong to elements
// NVF*64 + (sub & 1)*8 .., and the o tails of the lanes with equal sub & 1 are summed at unit end.

// Token whose 16-element K tail lane (grp, sub) handles: that of pass pi = sub / 2 of group (grp + pi) mod 4.
// The rotation by pi makes the four tokens one quarter-warp reads differ mod 4, so its eight 16-byte loads
// (rows are 160 bytes apart) fall into eight different bank groups instead of colliding four ways.  Scores
// are plain numbers and travel back to the owning group by a shuffle.
__device__ __forceinline__ int tail_token(int grp, int sub) {
    const int pi = sub >> 1;
    return 4 * pi + ((grp + pi) & 3);
}

// Scores of the tokens of GT K tiles, one per query head (head g's tile is sK + g * TSTRIDE), in the log2
// domain (q is pre-scaled), and the running maxima brought up to date (o and l rescaled).
template <int D, int GT, int BT, bool BF16, int TSTRIDE>
__device__ __forceinline__ void tile_scores(const uint8_t *sK, int ntok, int grp, int sub,
                                            const float (&q)[GT][(D + 63) / 64 * 8], float (&sc)[BT / 4][GT],
                                            float (&o)[GT][(D + 63) / 64 * 8], float (&m)[GT], float (&l)[GT]) {
    constexpr int NVF = D / 64, NV = (D + 63) / 64, NQ = BT / 4, ROW = D * 2;
    static_assert(D % 64 == 0 || D % 64 == 16, "head_dim: whole 64-element spans, plus at most a 16-element tail");
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        const uint8_t *tile = sK + g * TSTRIDE;
#pragma unroll
        for (int i = 0; i < NQ; ++i) {
            const int t = 4 * i + grp;
            const uint4 *krow = reinterpret_cast<const uint4 *>(tile + t * ROW);
            float a0 = 0.f, a1 = 0.f;   // two chains per dot product
#pragma unroll
            for (int v = 0; v < NVF; ++v) {
                float kf[8];
                cvt8<BF16>(krow[swz(v * 8 + sub, t, D / 8)], kf);
#pragma unroll
                for (int e = 0; e < 8; e += 2) ffma2(a0, a1, q[g][v * 8 + e], q[g][v * 8 + e + 1], kf[e], kf[e + 1]);
            }
            float a = a0 + a1;
            a += __shfl_xor_sync(kFull, a, 4);
            a += __shfl_xor_sync(kFull, a, 2);
            a += __shfl_xor_sync(kFull, a, 1);
            sc[i][g] = a;
        }
        if (NV > NVF) {   // the 16-element tails, one chunk per lane (token assignment: see tail_token)
            const int tt = tail_token(grp, sub);
            float kf[8];
            cvt8<BF16>(reinterpret_cast<const uint4 *>(tile + tt * ROW)[NVF * 8 + (sub & 1)], kf);
            float tp = 0.f, tp1 = 0.f;
#pragma unroll
            for (int e = 0; e < 8; e += 2) ffma2(tp, tp1, q[g][NVF * 8 + e], q[g][NVF * 8 + e + 1], kf[e], kf[e + 1]);
            tp += tp1;
            tp += __shfl_xor_sync(kFull, tp, 1);   // lanes 2i and 2i+1 of a group: the two tail chunks of one token
#pragma unroll
            for (int i = 0; i < NQ; ++i)   // the tail of this group's token of pass i was taken by group (grp - i) mod 4
                sc[i][g] += __shfl_sync(kFull, tp, ((grp - i) & 3) * 8 + 2 * i);
        }
    }
    if (ntok < BT) {   // slots past the sequence end hold unspecified bits: their scores are replaced
#pragma unroll
        for (int i = 0; i < NQ; ++i)
            if (4 * i + grp >= ntok) {
#pragma unroll
                for (int g = 0; g < GT; ++g) sc[i][g] = kNegBig;
            }
    }
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        float mx = sc[0][g];
#pragma unroll
        for (int i = 1; i < NQ; ++i) mx = fmaxf(mx, sc[i][g]);
        if (mx > m[g]) {
            const float r = fast_exp2(m[g] - mx);
            l[g] *= r;
#pragma unroll
            for (int e = 0; e < NV * 8; ++e) o[g][e] *= r;
            m[g] = mx;
        }
    }
}

// o += softmax weights x V for the GT V tiles (head g's tile is sV + g * TSTRIDE) whose scores are in sc.
template <int D, int GT, int BT, bool BF16, int TSTRIDE>
__device__ __forceinline__ void tile_values(const uint8_t *sV, int ntok, int grp, int sub,
                                            const float (&sc)[BT / 4][GT], float (&o)[GT][(D + 63) / 64 * 8],
                                            const float (&m)[GT], float (&l)[GT]) {
    constexpr int NVF = D / 64, NV = (D + 63) / 64, NQ = BT / 4, ROW = D * 2;
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        const uint8_t *tile = sV + g * TSTRIDE;
        float pwv[NQ];   // the weights of the four passes (used again by the tail step)
#pragma unroll
        for (int i = 0; i < NQ; ++i) {
            const int t = 4 * i + grp;
            pwv[i] = 0.f;
            if (t < ntok) {   // slots past the sequence end hold unspecified bits: never touch them
                pwv[i] = fast_exp2(sc[i][g] - m[g]);
                l[g] += pwv[i];
                const uint4 *vrow = reinterpret_cast<const uint4 *>(tile + t * ROW);
#pragma unroll
                for (int v = 0; v < NVF; ++v) {
                    float vf[8];
                    cvt8<BF16>(vrow[swz(v * 8 + sub, t, D / 8)], vf);
#pragma unroll
                    for (int e = 0; e < 8; e += 2)
                        ffma2(o[g][v * 8 + e], o[g][v * 8 + e + 1], pwv[i], pwv[i], vf[e], vf[e + 1]);
                }
            }
        }
        if (NV > NVF) {
            // The V tails stay with the group that owns the token: their products are added to that group's
            // accumulators, which are scaled by that group's running maximum (no rotation as for the K tails).
            const int pi = sub >> 1, tt = 4 * pi + grp;
            if (tt < ntok) {
                float vf[8];
                cvt8<BF16>(reinterpret_cast<const uint4 *>(tile + tt * ROW)[NVF * 8 + (sub & 1)], vf);
                const float pw = pi == 0 ? pwv[0] : pi == 1 ? pwv[1] : pi == 2 ? pwv[2] : pwv[3];
#pragma unroll
                for (int e = 0; e < 8; e += 2)
                    ffma2(o[g][NVF * 8 + e], o[g][NVF * 8 + e + 1], pw, pw, vf[e], vf[e + 1]);
            }
        }
    }
}

// Stores one row held in group layout (lanes 0..7 cover the row).
template <int D, bool BF16>
__device__ __forceinline__ void store_row_grouped(void *out, float *out_f32, size_t row, int sub,
                                                  const float (&o)[(D + 63) / 64 * 8], float scale) {
#pragma unroll
    for (int v = 0; v < (D + 63) / 64; ++v) {
        if ((v + 1) * 64 > D && v * 64 + sub * 8 >= D) continue;
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = o[v * 8 + e] * scale;
        const size_t idx = row * D + v * 64 + sub * 8;
        if (out_f32) {
            *reinterpret_cast<float4 *>(out_f32 + idx) = make_float4(x[0], x[1], x[2], x[3]);
            *reinterpret_cast<float4 *>(out_f32 + idx + 4) = make_float4(x[4], x[5], x[6], x[7]);
        }
        if (out) {
            uint4 w;
            w.x = pack2<BF16>(x[0], x[1]);
            w.y = pack2<BF16>(x[2], x[3]);
            w.z = pack2<BF16>(x[4], x[5]);
            w.w = pack2<BF16>(x[6], x[7]);
            *reinterpret_cast<uint4 *>(reinterpret_cast<uint16_t *>(out) + idx) = w;
        }
    }
}

// ---------------------------------------------------------------- arithmetic of one warp
//
// The decode kernel is written once; what a warp does with a K tile, a V tile, this step's token and
// its finished (m, l, o) state comes from one of two classes:
//   ScalarMath  CUDA-core arithmetic for multi-head attention: one query head per KV head.  A visit may
//               carry the tiles of HP = 2 adjacent KV heads (they are contiguous in a block), each with its
//               own query head: at head_dim 64 and 80 that halves the per-visit bookkeeping per byte
//   MmaMath     tensor-core arithmetic (mma.sync m16n8k16, fp32 accumulation) for grouped-query
//               attention: the 2..16 query heads that share a KV head are the rows of one 16-row
//               operand, so a KV tile is read once for all of them
// Both keep scores in the log2 domain (the softmax scale is folded in with log2 e) and rescale the
// accumulators lazily, only when a tile raises the running maximum.

template <int D_, int GT_, int BT_, bool BF16_>
struct ScalarMath {
    static constexpr int D = D_, BT = BT_, NVF = D_ / 64, NV = (D_ + 63) / 64, E = NV * 8;   // 8 elements per span and lane
    static constexpr int HP = GT_;            // KV heads (tiles) per visit: query head g of the group reads tile g
    static constexpr int TILE1 = BT_ * D_ * 2;
    static constexpr bool BF16 = BF16_;
    float q[GT_][E], o[GT_][E], m[GT_], l[GT_], sc[BT_ / 4][GT_];
    int grp, sub;

    __device__ __forceinline__ void init(const DecodeParams &, int lane) {
        grp = lane >> 3;
        sub = lane & 7;
    }
    __device__ __forceinline__ int heads() const { return GT_; }

    // New (sequence, head group): load its query rows (pre-scaled) and clear the state.
    __device__ __forceinline__ void begin(const DecodeParams &p, int s, int hg) {
#pragma unroll
        for (int g = 0; g < GT_; ++g) {
            const uint16_t *qrow =
                reinterpret_cast<const uint16_t *>(p.q) + ((size_t)s * p.Hq + (size_t)hg * GT_ + g) * D;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                // complete spans: elements v*64 + sub*8 ..; the tail span: chunk sub & 1 in every lane
                const uint4 r = __ldg(reinterpret_cast<const uint4 *>(qrow + v * 64 + (v < NVF ? sub : (sub & 1)) * 8));
                float qf[8];
                cvt8<BF16>(r, qf);
#pragma unroll
                for (int e = 0; e < 8; ++e) q[g][v * 8 + e] = qf[e] * p.scale_log2;
            }
            m[g] = kNegBig;
            l[g] = 0.f;
#pragma unroll
            for (int e = 0; e < E; ++e) o[g][e] = 0.f;
        }
    }
    __device__ __forceinline__ void k_tile(const uint8_t *tile, int ntok) {
        tile_scores<D, GT_, BT, BF16, TILE1>(tile, ntok, grp, sub, q, sc, o, m, l);
    }
    __device__ __forceinline__ void v_tile(const uint8_t *tile, int ntok) {
        tile_values<D, GT_, BT, BF16, TILE1>(tile, ntok, grp, sub, sc, o, m, l);
    }
    // This step's token, read from the caller's rows (head g's rows are krow + g * D, vrow + g * D): all
    // groups compute its scores (the shuffles need every lane), group 0 keeps it.
    __device__ __forceinline__ void new_token(const uint16_t *krow, const uint16_t *vrow) {
        float a[GT_];
#pragma unroll
        for (int g = 0; g < GT_; ++g) a[g] = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (v * 64 + sub * 8 >= D) continue;   // the tail is counted once: by lanes sub 0 and 1
#pragma unroll
            for (int g = 0; g < GT_; ++g) {
                float kf[8];
                cvt8<BF16>(__ldg(reinterpret_cast<const uint4 *>(krow + g * D + v * 64 + sub * 8)), kf);
#pragma unroll
                for (int e = 0; e < 8; ++e) a[g] = fmaf(q[g][v * 8 + e], kf[e], a[g]);
            }
        }
#pragma unroll
        for (int g = 0; g < GT_; ++g) {
            a[g] += __shfl_xor_sync(kFull, a[g], 4);
            a[g] += __shfl_xor_sync(kFull, a[g], 2);
            a[g] += __shfl_xor_sync(kFull, a[g], 1);
        }
        if (grp == 0) {
            float pw[GT_];
#pragma unroll
            for (int g = 0; g < GT_; ++g) {
                if (a[g] > m[g]) {
                    const float r = exp2f(m[g] - a[g]);
                    l[g] *= r;
#pragma unroll
                    for (int e = 0; e < E; ++e) o[g][e] *= r;
                    m[g] = a[g];
                }
                pw[g] = exp2f(a[g] - m[g]);
                l[g] += pw[g];
            }
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                if (v * 64 + sub * 8 >= D) continue;
#pragma unroll
                for (int g = 0; g < GT_; ++g) {
                    float vf[8];
                    cvt8<BF16>(__ldg(reinterpret_cast<const uint4 *>(vrow + g * D + v * 64 + sub * 8)), vf);
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[g][v * 8 + e] = fmaf(pw[g], vf[e], o[g][v * 8 + e]);
                }
            }
        }
    }
    // End of a unit: merge the four token groups of the warp (every group ends with the merged state).
    __device__ __forceinline__ void finish() {
        if (NV > NVF) {   // tail elements: sum the shares of the lanes with equal sub & 1
#pragma unroll
            for (int g = 0; g < GT_; ++g)
#pragma unroll
                for (int e = NVF * 8; e < E; ++e) {
                    float x = o[g][e];
                    x += __shfl_xor_sync(kFull, x, 2);
                    x += __shfl_xor_sync(kFull, x, 4);
                    o[g][e] = x;
                }
        }
#pragma unroll
        for (int g = 0; g < GT_; ++g) {
            float mm = fmaxf(m[g], __shfl_xor_sync(kFull, m[g], 8));
            mm = fmaxf(mm, __shfl_xor_sync(kFull, mm, 16));
            const float r = exp2f(m[g] - mm);
            float ll = l[g] * r;
            ll += __shfl_xor_sync(kFull, ll, 8);
            ll += __shfl_xor_sync(kFull, ll, 16);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                float x = o[g][e] * r;
                x += __shfl_xor_sync(kFull, x, 8);
                x += __shfl_xor_sync(kFull, x, 16);
                o[g][e] = x;
            }
            m[g] = mm;
            l[g] = ll;
        }
    }
    // Folds the finished state into the running state of rows row0 .. row0 + GT - 1, which this
    // unit alone writes in this launch.
    __device__ __forceinline__ void fold_running(const DecodeParams &p, size_t row0) {
#pragma unroll
        for (int g = 0; g < GT_; ++g) {
            const size_t row = row0 + g;
            const float2 ml = *reinterpret_cast<const float2 *>(&p.acc_ml[row * 2]);
            if (ml.y > 0.f) {
                const float mm = fmaxf(m[g], ml.x);
                const float a1 = exp2f(m[g] - mm), a2 = exp2f(ml.x - mm);
                l[g] = l[g] * a1 + ml.y * a2;
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    if (v * 64 + sub * 8 >= D) continue;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        o[g][v * 8 + e] = o[g][v * 8 + e] * a1 + p.acc_o[row * D + v * 64 + sub * 8 + e] * a2;
                }
                m[g] = mm;
            }
            __syncwarp();   // all lanes have read the old state before group 0 overwrites it
            if (grp == 0) {
                store_row_grouped<D, BF16>(nullptr, p.acc_o, row, sub, o[g], 1.f);
                if (sub == 0) {
                    p.acc_ml[row * 2] = m[g];
                    p.acc_ml[row * 2 + 1] = l[g];
                }
            }
        }
    }
    // Normalised result to out / out_f32, rows row0 .. row0 + GT - 1.
    __device__ __forceinline__ void store_final(const DecodeParams &p, size_t row0) {
        if (grp == 0) {
#pragma unroll
            for (int g = 0; g < GT_; ++g)
                store_row_grouped<D, BF16>(p.out, p.out_f32, row0 + g, sub, o[g], l[g] > 0.f ? 1.f / l[g] : 0.f);
        }
    }
    // Unnormalised (m, l, o) to rows row0 .. of o_dst / ml_dst (a partial slot or the resident result).
    __device__ __forceinline__ void store_state(float *o_dst, float *ml_dst, size_t row0) {
        if (grp == 0) {
#pragma unroll
            for (int g = 0; g < GT_; ++g) {
                store_row_grouped<D, BF16>(nullptr, o_dst, row0 + g, sub, o[g], 1.f);
                if (sub == 0) {
                    ml_dst[(row0 + g) * 2] = m[g];
                    ml_dst[(row0 + g) * 2 + 1] = l[g];
                }
            }
        }
    }
};

// D = A x B + D on one 16 x 8 tile, k = 16, 16-bit operands, fp32 accumulators.
template <bool BF16>
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if (BF16) {
        asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    } else {
        asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
}
// Four 8 x 8 matrices of 16-bit elements from shared memory; lane i gives the address of row i % 8 of
// matrix i / 8 (16 bytes per row).  The transposing form hands out columns instead of rows.
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
template <bool BF16>
__device__ __forceinline__ float2 unpack2(uint32_t w) {
    if (BF16) return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    return __half22float2(*reinterpret_cast<const __half2 *>(&w));
}

// Tensor-core arithmetic for a group of 2..16 query heads that share one KV head (BT = 16).
// Lane = 4 r + c.  Operand layouts of mma.m16n8k16 as used here:
//   scores  S[head][token] = Q[head][dim] . K[token][dim]: A = Q (rows r and r + 8, held in registers
//           for the whole segment), B = K read with ldmatrix (row = token, 8 dims per matrix row);
//   output  O[head][dim] += P[head][token] . V[token][dim]: A = P, taken from the score accumulators
//           (their layout is the A layout), B = V read with the transposing ldmatrix.
// The weights P go to the tensor core as a 16-bit value plus a 16-bit remainder (two products per
// V tile), so that rounding P to 16 bits does not limit the result's accuracy; l sums the fp32 weights.
// Rows at or beyond the group's head count carry zero queries; their results are never stored.
template <int D_, bool BF16_>
struct MmaMath {
    static constexpr int D = D_, BT = 16, ROW = D_ * 2;
    static constexpr int HP = 1;              // one KV head (tile) per visit, shared by the group's query heads
    static constexpr bool BF16 = BF16_;
    uint32_t qa[D_ / 16][4];    // Q as A fragments, one per 16 dims
    float oacc[D_ / 8][4];      // O accumulators: [j][0..1] row r, [j][2..3] row r + 8, dims 8 j + 2 c, + 1
    float m[2], l[2];           // running maximum (same in the 4 lanes of a row) and this lane's share of the sum
    uint32_t ph[4], pl[4];      // weights of the current block as A fragments: 16-bit value and remainder
    float scale;
    int lane, r, c, gt;
    // Byte offsets, inside a tile, of the rows this lane addresses in the matrix loads.  A load of 16-dim step
    // ks wants 16-byte chunk 2 ks + h of token row t (h: the lane's half of the step); with the stored chunk
    // order that is chunk position 8 (ks / 4) + ((2 (ks % 4) + h) ^ (t % 8)): four lane-dependent values per
    // operand, plus 128 bytes per group of eight chunks, which goes into the instruction as an immediate.
    uint32_t koff[4], voff[4];

    __device__ __forceinline__ void init(const DecodeParams &p, int lane_) {
        lane = lane_;
        r = lane_ >> 2;
        c = lane_ & 3;
        gt = p.GT;
        scale = p.scale_log2;
        const int t7 = lane_ & 7;
        const int ktok = ((lane_ >> 4) << 3) + t7, khalf = (lane_ >> 3) & 1;   // K: plain loads
        const int vtok = (((lane_ >> 3) & 1) << 3) + t7, vhi = lane_ >> 4;     // V: transposing loads
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            koff[j] = ktok * ROW + ((((2 * j + khalf) ^ t7) & 7) << 4);
            voff[j] = vtok * ROW + ((((2 * j + vhi) ^ t7) & 7) << 4);
        }
    }
    // Offset of step ks for an operand whose four lane-dependent offsets are off[]: steps inside the complete
    // groups of eight chunks are permuted, a trailing incomplete group (head_dim 80: chunks 8 and 9) is not.
    __device__ __forceinline__ uint32_t step_off(const uint32_t (&off)[4], int ks, int tok_row_bytes, int h) const {
        return (2 * ks < ((D / 8) & ~7)) ? off[ks & 3] + 128 * (ks >> 2) : tok_row_bytes + ((2 * ks + h) << 4);
    }
    __device__ __forceinline__ int heads() const { return gt; }

    __device__ __forceinline__ void begin(const DecodeParams &p, int s, int hg) {
        const uint16_t *qb = reinterpret_cast<const uint16_t *>(p.q) + ((size_t)s * p.Hq + (size_t)hg * gt) * D;
        const uint32_t *q0 = reinterpret_cast<const uint32_t *>(qb + (size_t)r * D + 2 * c);
        const uint32_t *q1 = reinterpret_cast<const uint32_t *>(qb + (size_t)(r + 8) * D + 2 * c);
        const bool v0 = r < gt, v1 = r + 8 < gt;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            qa[ks][0] = v0 ? __ldg(q0 + ks * 8) : 0u;
            qa[ks][1] = v1 ? __ldg(q1 + ks * 8) : 0u;
            qa[ks][2] = v0 ? __ldg(q0 + ks * 8 + 4) : 0u;
            qa[ks][3] = v1 ? __ldg(q1 + ks * 8 + 4) : 0u;
        }
        m[0] = m[1] = kNegBig;
        l[0] = l[1] = 0.f;
#pragma unroll
        for (int j = 0; j < D / 8; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
    }

    // Raises the running maxima to (n0, n1) and rescales l and the accumulators accordingly.
    __device__ __forceinline__ void raise_max(float n0, float n1) {
        const float r0 = fast_exp2(m[0] - n0), r1 = fast_exp2(m[1] - n1);
        l[0] *= r0;
        l[1] *= r1;
#pragma unroll
        for (int j = 0; j < D / 8; ++j) {
            oacc[j][0] *= r0;
            oacc[j][1] *= r0;
            oacc[j][2] *= r1;
            oacc[j][3] *= r1;
        }
        m[0] = n0;
        m[1] = n1;
    }

    __device__ __forceinline__ void k_tile(const uint8_t *tile, int ntok) {
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};   // tokens 0..7 and 8..15
        const uint32_t base = smem_u32(tile);
        const int tok = ((lane >> 4) << 3) + (lane & 7), half = (lane >> 3) & 1;   // (used by the unpermuted tail only)
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4(base + step_off(koff, ks, tok * ROW, half), b0, b1, b2, b3);
            mma16816<BF16>(s0, qa[ks], b0, b1);
            mma16816<BF16>(s1, qa[ks], b2, b3);
        }
        // this lane's scores: rows r (x[0..3]) and r + 8 (y[0..3]) at tokens 2c, 2c+1, 2c+8, 2c+9
        float x[4] = {s0[0] * scale, s0[1] * scale, s1[0] * scale, s1[1] * scale};
        float y[4] = {s0[2] * scale, s0[3] * scale, s1[2] * scale, s1[3] * scale};
        if (ntok < BT) {   // slots past the sequence end hold unspecified bits
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = 2 * c + (i & 1) + 8 * (i >> 1);
                if (t >= ntok) x[i] = y[i] = kNegBig;
            }
        }
        float mx0 = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
        float mx1 = fmaxf(fmaxf(y[0], y[1]), fmaxf(y[2], y[3]));
        mx0 = fmaxf(mx0, __shfl_xor_sync(kFull, mx0, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(kFull, mx1, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(kFull, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(kFull, mx1, 2));
        if (__any_sync(kFull, mx0 > m[0] || mx1 > m[1])) raise_max(fmaxf(m[0], mx0), fmaxf(m[1], mx1));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[i] = fast_exp2(x[i] - m[0]);
            y[i] = fast_exp2(y[i] - m[1]);
        }
        l[0] += (x[0] + x[1]) + (x[2] + x[3]);
        l[1] += (y[0] + y[1]) + (y[2] + y[3]);
        ph[0] = pack2<BF16>(x[0], x[1]);
        ph[1] = pack2<BF16>(y[0], y[1]);
        ph[2] = pack2<BF16>(x[2], x[3]);
        ph[3] = pack2<BF16>(y[2], y[3]);
        const float2 h0 = unpack2<BF16>(ph[0]), h1 = unpack2<BF16>(ph[1]);
        const float2 h2 = unpack2<BF16>(ph[2]), h3 = unpack2<BF16>(ph[3]);
        pl[0] = pack2<BF16>(x[0] - h0.x, x[1] - h0.y);
        pl[1] = pack2<BF16>(y[0] - h1.x, y[1] - h1.y);
        pl[2] = pack2<BF16>(x[2] - h2.x, x[3] - h2.y);
        pl[3] = pack2<BF16>(y[2] - h3.x, y[3] - h3.y);
    }

    __device__ __forceinline__ void v_tile(const uint8_t *tile, int ntok) {
        const uint32_t base = smem_u32(tile);
        const int tok = (((lane >> 3) & 1) << 3) + (lane & 7), hi = lane >> 4;     // (used by the unpermuted tail only)
        uint32_t k0 = 0xffffffffu, k1 = 0xffffffffu;   // keep-masks of the token pairs (2c, 2c+1) and (2c+8, 2c+9)
        if (ntok < BT) {
            k0 = (2 * c < ntok ? 0x0000ffffu : 0u) | (2 * c + 1 < ntok ? 0xffff0000u : 0u);
            k1 = (2 * c + 8 < ntok ? 0x0000ffffu : 0u) | (2 * c + 9 < ntok ? 0xffff0000u : 0u);
        }
#pragma unroll
        for (int jp = 0; jp < D / 16; ++jp) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(base + step_off(voff, jp, tok * ROW, hi), b0, b1, b2, b3);
            if (ntok < BT) {   // never let unspecified bits (possibly NaN patterns) reach a product
                b0 &= k0; b1 &= k1; b2 &= k0; b3 &= k1;
            }
            mma16816<BF16>(oacc[2 * jp], ph, b0, b1);
            mma16816<BF16>(oacc[2 * jp + 1], ph, b2, b3);
            mma16816<BF16>(oacc[2 * jp], pl, b0, b1);
            mma16816<BF16>(oacc[2 * jp + 1], pl, b2, b3);
        }
    }

    // This step's token, read from the caller's rows, in plain fp32 arithmetic.
    __device__ __forceinline__ void new_token(const uint16_t *krow, const uint16_t *vrow) {
        float d0 = 0.f, d1 = 0.f;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const float2 ka = unpack2<BF16>(__ldg(reinterpret_cast<const uint32_t *>(krow + ks * 16 + 2 * c)));
            const float2 kb = unpack2<BF16>(__ldg(reinterpret_cast<const uint32_t *>(krow + ks * 16 + 2 * c + 8)));
            const float2 a0 = unpack2<BF16>(qa[ks][0]), a1 = unpack2<BF16>(qa[ks][1]);
            const float2 a2 = unpack2<BF16>(qa[ks][2]), a3 = unpack2<BF16>(qa[ks][3]);
            d0 = fmaf(a0.x, ka.x, d0); d0 = fmaf(a0.y, ka.y, d0); d0 = fmaf(a2.x, kb.x, d0); d0 = fmaf(a2.y, kb.y, d0);
            d1 = fmaf(a1.x, ka.x, d1); d1 = fmaf(a1.y, ka.y, d1); d1 = fmaf(a3.x, kb.x, d1); d1 = fmaf(a3.y, kb.y, d1);
        }
        d0 += __shfl_xor_sync(kFull, d0, 1);
        d1 += __shfl_xor_sync(kFull, d1, 1);
        d0 += __shfl_xor_sync(kFull, d0, 2);
        d1 += __shfl_xor_sync(kFull, d1, 2);
        d0 *= scale;
        d1 *= scale;
        raise_max(fmaxf(m[0], d0), fmaxf(m[1], d1));
        const float p0 = exp2f(d0 - m[0]), p1 = exp2f(d1 - m[1]);
        if (c == 0) {   // l is summed over the 4 lanes of a row at the end: count the token once
            l[0] += p0;
            l[1] += p1;
        }
#pragma unroll
        for (int j = 0; j < D / 8; ++j) {
            const float2 v = unpack2<BF16>(__ldg(reinterpret_cast<const uint32_t *>(vrow + j * 8 + 2 * c)));
            oacc[j][0] = fmaf(p0, v.x, oacc[j][0]);
            oacc[j][1] = fmaf(p0, v.y, oacc[j][1]);
            oacc[j][2] = fmaf(p1, v.x, oacc[j][2]);
            oacc[j][3] = fmaf(p1, v.y, oacc[j][3]);
        }
    }

    __device__ __forceinline__ void finish() {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            l[i] += __shfl_xor_sync(kFull, l[i], 1);
            l[i] += __shfl_xor_sync(kFull, l[i], 2);
        }
    }

    __device__ __forceinline__ void fold_running(const DecodeParams &p, size_t row0) {
        float2 old[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = r + 8 * i;
            old[i] = make_float2(kNegBig, 0.f);
            if (row < gt) old[i] = *reinterpret_cast<const float2 *>(&p.acc_ml[(row0 + row) * 2]);
        }
        __syncwarp();   // the 4 lanes of a row have read (m, l) before lane c == 0 overwrites it
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = r + 8 * i;
            if (row >= gt) continue;
            float *orow = p.acc_o + (row0 + row) * D + 2 * c;
            float a1 = 1.f, a2 = 0.f;
            if (old[i].y > 0.f) {
                const float mm = fmaxf(m[i], old[i].x);
                a1 = exp2f(m[i] - mm);
                a2 = exp2f(old[i].x - mm);
                l[i] = l[i] * a1 + old[i].y * a2;
                m[i] = mm;
            }
#pragma unroll
            for (int j = 0; j < D / 8; ++j) {
                float2 x = make_float2(oacc[j][2 * i] * a1, oacc[j][2 * i + 1] * a1);
                if (old[i].y > 0.f) {
                    const float2 y = *reinterpret_cast<const float2 *>(orow + j * 8);
                    x.x = fmaf(y.x, a2, x.x);
                    x.y = fmaf(y.y, a2, x.y);
                }
                *reinterpret_cast<float2 *>(orow + j * 8) = x;
            }
            if (c == 0) {
                p.acc_ml[(row0 + row) * 2] = m[i];
                p.acc_ml[(row0 + row) * 2 + 1] = l[i];
            }
        }
    }

    __device__ __forceinline__ void store_final(const DecodeParams &p, size_t row0) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = r + 8 * i;
            if (row >= gt) continue;
            const float inv = l[i] > 0.f ? 1.f / l[i] : 0.f;
            const size_t idx = (row0 + row) * D + 2 * c;
#pragma unroll
            for (int j = 0; j < D / 8; ++j) {
                const float x0 = oacc[j][2 * i] * inv, x1 = oacc[j][2 * i + 1] * inv;
                if (p.out_f32) *reinterpret_cast<float2 *>(p.out_f32 + idx + j * 8) = make_float2(x0, x1);
                if (p.out)
                    *reinterpret_cast<uint32_t *>(reinterpret_cast<uint16_t *>(p.out) + idx + j * 8) =
                        pack2<BF16>(x0, x1);
            }
        }
    }

    __device__ __forceinline__ void store_state(float *o_dst, float *ml_dst, size_t row0) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int row = r + 8 * i;
            if (row >= gt) continue;
            float *orow = o_dst + (row0 + row) * D + 2 * c;
#pragma unroll
            for (int j = 0; j < D / 8; ++j)
                *reinterpret_cast<float2 *>(orow + j * 8) = make_float2(oacc[j][2 * i], oacc[j][2 * i + 1]);
            if (c == 0) {
                ml_dst[(row0 + row) * 2] = m[i];
                ml_dst[(row0 + row) * 2 + 1] = l[i];
            }
        }
    }
};

// Last-arriving contributor of a (sequence, head group): combine the nc partials of
// query head g in fixed order.  Lane owns D/32 consecutive elements.
template <int D, bool BF16>
__device__ __forceinline__ void merge_partials_row(const DecodeParams &p, int wf, int wf_slot, int nc, int g, int GT,
                                                   size_t row, int lane) {
    constexpr int EPL = D > 64 ? 4 : 2;   // lanes 0 .. D / EPL - 1 each own EPL consecutive elements
    const bool own = lane * EPL < D;
    // contributor c is warp wf + c; the first one may have used its second slot, all others used their first
    auto slot_of = [&](int c) { return c == 0 ? 2 * wf + wf_slot : 2 * (wf + c); };
    float mm = kNegBig;
    for (int c = lane; c < nc; c += 32) mm = fmaxf(mm, __ldcg(&p.part_ml[((size_t)slot_of(c) * GT + g) * 2]));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mm = fmaxf(mm, __shfl_xor_sync(kFull, mm, d));
    float ll = 0.f;
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int c = 0; c < nc; ++c) {
        const size_t pr = (size_t)slot_of(c) * GT + g;
        const float2 ml = __ldcg(reinterpret_cast<const float2 *>(&p.part_ml[pr * 2]));
        const float a = exp2f(ml.x - mm);
        ll += ml.y * a;
        const float *po = p.part_o + pr * D + lane * EPL;
        if (!own) continue;
        if (EPL == 4) {
            const float4 x = __ldcg(reinterpret_cast<const float4 *>(po));
            acc[0] = fmaf(a, x.x, acc[0]);
            acc[1] = fmaf(a, x.y, acc[1]);
            acc[2] = fmaf(a, x.z, acc[2]);
            acc[3] = fmaf(a, x.w, acc[3]);
        } else {
            const float2 x = __ldcg(reinterpret_cast<const float2 *>(po));
            acc[0] = fmaf(a, x.x, acc[0]);
            acc[1] = fmaf(a, x.y, acc[1]);
        }
    }
    const size_t idx = row * D + lane * EPL;
    if (!own) return;
    if (p.finalize) {
        const float inv = ll > 0.f ? 1.f / ll : 0.f;
        if (p.out_f32) {
#pragma unroll
            for (int e = 0; e < EPL; ++e) p.out_f32[idx + e] = acc[e] * inv;
        }
        if (p.out) {
            uint16_t *o16 = reinterpret_cast<uint16_t *>(p.out) + idx;
            if (EPL == 4) {
                uint2 w;
                w.x = pack2<BF16>(acc[0] * inv, acc[1] * inv);
                w.y = pack2<BF16>(acc[2] * inv, acc[3] * inv);
                *reinterpret_cast<uint2 *>(o16) = w;
            } else {
                *reinterpret_cast<uint32_t *>(o16) = pack2<BF16>(acc[0] * inv, acc[1] * inv);
            }
        }
    } else {
#pragma unroll
        for (int e = 0; e < EPL; ++e) p.acc_o[idx + e] = acc[e];
        if (lane == 0) {
            p.acc_ml[row * 2] = mm;
            p.acc_ml[row * 2 + 1] = ll;
        }
    }
}

// The same combination for R query heads of the group at once (g0 .. g0 + R - 1, those below GT): the
// loads of all R rows of a contributor are in flight together, so a group of many heads costs a few memory
// round trips instead of a few per head.  Used where the warp's accumulators are no longer live (at the end
// of its range); per head the arithmetic and its order are those of merge_partials_row.
template <int D, bool BF16, int R>
__device__ __forceinline__ void merge_partials_rows(const DecodeParams &p, int wf, int wf_slot, int nc, int g0, int GT,
                                                    size_t row0, int lane) {
    constexpr int EPL = D > 64 ? 4 : 2;
    const bool own = lane * EPL < D;
    auto slot_of = [&](int c) { return c == 0 ? 2 * wf + wf_slot : 2 * (wf + c); };
    float mm[R], ll[R], acc[R][EPL];
#pragma unroll
    for (int j = 0; j < R; ++j) {
        mm[j] = kNegBig;
        ll[j] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[j][e] = 0.f;
    }
    for (int c = 0; c < nc; ++c) {   // every lane reads the same words: broadcast loads
        const float *ml = p.part_ml + ((size_t)slot_of(c) * GT + g0) * 2;
#pragma unroll
        for (int j = 0; j < R; ++j)
            if (g0 + j < GT) mm[j] = fmaxf(mm[j], __ldcg(ml + 2 * j));
    }
    for (int c = 0; c < nc; ++c) {
        const size_t pr = (size_t)slot_of(c) * GT + g0;
        float2 ml[R];
        float x[R][EPL];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            ml[j] = make_float2(kNegBig, 0.f);
#pragma unroll
            for (int e = 0; e < EPL; ++e) x[j][e] = 0.f;
            if (g0 + j < GT) {
                ml[j] = __ldcg(reinterpret_cast<const float2 *>(&p.part_ml[(pr + j) * 2]));
                const float *po = p.part_o + (pr + j) * D + lane * EPL;
                if (!own) continue;
                if (EPL == 4) {
                    const float4 v = __ldcg(reinterpret_cast<const float4 *>(po));
                    x[j][0] = v.x; x[j][1] = v.y; x[j][2] = v.z; x[j][3] = v.w;
                } else {
                    const float2 v = __ldcg(reinterpret_cast<const float2 *>(po));
                    x[j][0] = v.x; x[j][1] = v.y;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const float a = exp2f(ml[j].x - mm[j]);
            ll[j] += ml[j].y * a;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[j][e] = fmaf(a, x[j][e], acc[j][e]);
        }
    }
#pragma unroll
    for (int j = 0; j < R; ++j) {
        if (g0 + j >= GT) continue;
        const size_t row = row0 + g0 + j;
        const size_t idx = row * D + lane * EPL;
        if (!own) continue;
        if (p.finalize) {
            const float inv = ll[j] > 0.f ? 1.f / ll[j] : 0.f;
            if (p.out_f32) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) p.out_f32[idx + e] = acc[j][e] * inv;
            }
            if (p.out) {
                uint16_t *o16 = reinterpret_cast<uint16_t *>(p.out) + idx;
                if (EPL == 4) {
                    uint2 w;
                    w.x = pack2<BF16>(acc[j][0] * inv, acc[j][1] * inv);
                    w.y = pack2<BF16>(acc[j][2] * inv, acc[j][3] * inv);
                    *reinterpret_cast<uint2 *>(o16) = w;
                } else {
                    *reinterpret_cast<uint32_t *>(o16) = pack2<BF16>(acc[j][0] * inv, acc[j][1] * inv);
                }
            }
        } else {
#pragma unroll
            for (int e = 0; e < EPL; ++e) p.acc_o[idx + e] = acc[j][e];
            if (lane == 0) {
                p.acc_ml[row * 2] = mm[j];
                p.acc_ml[row * 2 + 1] = ll[j];
            }
        }
    }
}

// ---------------------------------------------------------------- decode kernel

// A warp's work is a sequence of block visits.  A visit owns two slots of the warp's shared-memory
// ring, one for the block's K tile and one for its V tile (each with its own mbarrier, so the scores
// are computed while the V tile is still arriving), and one metadata record written by the producing
// lane before it arms the K slot.  Visits without tiles (an empty unit, or a unit that consists of this
// step's token only) arm both slots without a copy.
enum { V_INFO = 0, V_SEQ, V_HG, V_NC, V_WF, V_PACK, V_WORDS = 8 };
// V_INFO: bits 0..7 tokens in the block, then the flags
enum { VF_DATA = 0x100,    // the visit has a K and a V tile
       VF_FIRST = 0x200,   // first visit of a segment: load the queries, clear the state
       VF_LAST = 0x400,    // last visit of a segment: store / fold / publish the state
       VF_NEW = 0x800 };   // this step's token follows the block (fused append)

// How the flat list of `total` work items is cut into `n` equal contiguous ranges, one per warp.
// Ranges are numbered in item order, so the ranges that meet any interval are consecutive.
struct Partition {
    long long total;
    int n;
    __device__ int first(int v) const { return (int)(total * v / n); }
    __device__ int end(int v) const { return (int)(total * (v + 1) / n); }
    __device__ int range_of(int x) const { return (int)((((long long)x + 1) * n - 1) / total); }   // holds item x
};

// A split whose partial has been stored but whose arrival has not been
// published yet (publishing needs a fence; it is cheap once the stores have
// landed, so it is done one unit later).
struct PendingArrival {
    int valid, ticket_idx, nc, wf, wf_slot;
    size_t row0;
};

template <class Math, int MODE, int NW>
__global__ void __launch_bounds__(NW * 32, 1) decode_kernel(const DecodeParams p, const int stages) {
    constexpr int D = Math::D, BT = Math::BT;
    constexpr bool BF16 = Math::BF16;
    constexpr int HP = Math::HP;                 // KV heads whose tiles one visit carries (adjacent in a block)
    constexpr uint32_t TILE1 = BT * D * 2;       // one (block, K|V, head) tile
    constexpr uint32_t TILE = TILE1 * HP;        // what a ring slot holds and one bulk copy brings
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    Math mth;
    mth.init(p, lane);
    const int GT = mth.heads();   // query heads of one head group
    const int NVIS = stages >> 1; // visits in flight per warp (stages is even)

    uint8_t *data = smem + (size_t)warp * stages * TILE;
    uint8_t *after_data = smem + (size_t)NW * stages * TILE;
    uint64_t *bars = reinterpret_cast<uint64_t *>(after_data) + warp * stages;
    int32_t *meta = reinterpret_cast<int32_t *>(after_data + (size_t)NW * stages * 8) + warp * stages * V_WORDS;
    // A launch covers NL layers of NSEQ sequences; (layer, sequence) pairs are numbered l * NSEQ + s and are
    // what "sequence" means below wherever q, out, the new rows, tickets or the work list are indexed.
    const int NL = (MODE == MODE_RESIDENT && p.n_layers > 1) ? p.n_layers : 1;
    const int NSEQ = p.n_seqs, NV = NL * NSEQ;
    int32_t *ubase = reinterpret_cast<int32_t *>(after_data + (size_t)NW * stages * (8 + 4 * V_WORDS));   // [NV + 1]
    int32_t *slen = ubase + NV + 1;   // [NV] tokens to attend (resident mode)

    // Programmatic dependent launch.  This kernel may start while its predecessor in the stream is
    // still running; griddepcontrol.wait returns once that predecessor has completed and its writes
    // are visible, and only after its own wait does a CTA let the successor start
    // (griddepcontrol.launch_dependents).  The order matters: a successor begins once every CTA of
    // this grid has released it, so at that moment the predecessor of this grid is complete, and by
    // induction at most two kernels of a chain are ever in flight, whatever the grid sizes.
    // With early_reads the wait is postponed until after the first K/V copies are issued: the host
    // sets the flag only when the immediate predecessor writes neither the lengths, nor the block
    // table, nor this layer's KV slab, and every kernel before that one has completed by the time
    // this one starts; q, the new K/V rows, the scratch and the outputs are touched only after the
    // wait.  The pipeline's ramp-up then overlaps the predecessor's tail.
    if (!p.early_reads) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    const uint32_t spin_limit = p.spin_limit ? p.spin_limit : kSpinLimit;

    const int Hg = p.Hkv * p.P / HP;             // head groups per sequence: what one segment of visits serves
    const uint64_t block_bytes = p.block_bytes;
    const uint64_t v_off = (uint64_t)p.Hkv * TILE1;   // from a block's K tile to its V tile of the same head
    const int fused = (MODE == MODE_RESIDENT && p.k_new != nullptr) ? 1 : 0;

    // ---- this warp's contiguous share of the work.  Resident mode: the flat space of KV blocks
    // ordered by (sequence, head group, block), cut into equal ranges whatever the sequence lengths
    // (an empty sequence counts as one block without tokens so that its zeros get written).
    // Staged mode: whole (chunk unit, head group) items.
    long long NU;
    if (MODE == MODE_RESIDENT) {
        const int len_cap = p.max_blocks * BT;
        for (int s = threadIdx.x; s < NV; s += blockDim.x) {
            // a length the table row does not cover is never followed into the table
            int raw;
            if (NL > 1) {
                const int l = s / NSEQ, la = p.layer0 + l;
                raw = p.lens[(size_t)((p.lens_cur_mask >> la) & 1) * p.lens_copy_stride +
                             (size_t)la * p.lens_layer_stride + (s - l * NSEQ)];
            } else {
                raw = p.lens[s];
            }
            const int len = min(max(raw, 0) + fused, len_cap);
            if (len != raw + fused) atomicOr(p.status, ISV_STATUS_BAD_LENGTH);
            slen[s] = len;
            ubase[s + 1] = max(1, (len + BT - 1) / BT) * Hg;
        }
        if (threadIdx.x == 0) ubase[0] = 0;
        __syncthreads();
        if (warp == 0) {
            int carry = 0;
            for (int base = 0; base < NV; base += 32) {
                const int i = base + lane;
                int v = i < NV ? ubase[i + 1] : 0;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int t = __shfl_up_sync(kFull, v, d);
                    if (lane >= d) v += t;
                }
                if (i < NV) ubase[i + 1] = carry + v;
                carry += __shfl_sync(kFull, v, 31);
            }
        }
        __syncthreads();
        NU = ubase[NV];
    } else {
        NU = (long long)p.cu_count * Hg;
    }
    const int gw = blockIdx.x * NW + warp;
    const int nw_grid = gridDim.x * NW;
    Partition part;
    part.total = NU;
    part.n = (int)min((long long)nw_grid, NU);   // no more ranges than items: every range owns at least one
    const bool idle = gw >= part.n;   // more warps than items: this one only helps with the append
    const int cur_range = gw;
    int u_next = idle ? 0 : part.first(gw);
    const int u_end = idle ? 0 : part.end(gw);
    if (lane == 0) {
        for (int st = 0; st < stages; ++st) mbar_init(smem_u32(&bars[st]), 1);
        fence_barrier_init();
    }
    __syncwarp();

    // ---- producer state (identical in all lanes except the two per-entry values)
    int pu_s = 0, pu_hg = 0, pu_nc = 1, pu_wf = 0, pu_wfslot = 0;
    int pu_row = 0;                                // table row (sequence within the layer) of the open segment
    const uint8_t *pu_pool = p.pool, *pu_tail = p.tail;   // its layer's slabs
    bool pu_first = true, range_first = true;   // the open segment is / the next one will be the first of its range
    bool seg_start = false;                     // the next visit is the first of its segment
    int pu_len = 0, pu_jlast = -1, pu_j0 = 0, pu_n = 0;   // entries of the open unit: [pu_j0, pu_j0 + pu_n)
    int pu_batch = 0, pu_nbatch = 0;
    uint32_t pu_mask = 0;
    const uint8_t *ent_src = nullptr;   // lane i: K tile of entry i of the current batch of 32 entries
    int ent_ntok = BT;                  // lane i: tokens of that block already in the cache, + 256 if it is the
                                        // unit's newest block and this step's token follows it
    bool pu_open = false, pu_done = false;
    const uint8_t *pv_src = nullptr;    // V tile of the visit whose K slot was armed last (NULL: no tiles)
    int prod_vis = 0, inflight = 0;     // ring position of the next visit to emit; visits emitted and not consumed
    bool drop_copy = p.drop_first_copy && blockIdx.x == 0 && warp == 0;   // failure injection, see DecodeParams
    if (MODE == MODE_RESIDENT) {   // sequence of the first unit: largest s with ubase[s] <= u_next
        int lo = 0, hi = NV - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (ubase[mid] <= u_next) lo = mid; else hi = mid - 1;
        }
        pu_s = lo;
    }

    // Decides the next visit, writes its record and arms its K slot; the V slot is armed by produce_v
    // (at once while the ring is being filled, later when the consumer has released that slot).
    // Returns false when this warp's range is exhausted.
    auto produce_k = [&]() -> bool {
        int ntok = 0, flags = 0;
        const uint8_t *ksrc = nullptr;
        while (true) {
            if (pu_mask != 0) {
                const int i = __ffs(pu_mask) - 1;
                pu_mask &= pu_mask - 1;
                const unsigned long long a = __shfl_sync(kFull, (unsigned long long)ent_src, i);
                const int nt = __shfl_sync(kFull, ent_ntok, i);
                const bool last = (pu_mask == 0) && (pu_batch >= pu_nbatch);
                ntok = nt & 255;
                flags = (last ? VF_LAST : 0) | ((nt & 256) ? VF_NEW : 0);
                if (ntok > 0) {
                    flags |= VF_DATA;
                    ksrc = reinterpret_cast<const uint8_t *>(a);
                }
                if (last) pu_open = false;
                break;
            }
            if (pu_open) {
                if (pu_batch < pu_nbatch) {   // next 32 entries of the unit, one per lane
                    const int j = pu_j0 + 32 * pu_batch + lane;
                    ++pu_batch;
                    bool valid = false;
                    const uint8_t *src = nullptr;
                    int nt = BT;
                    if (j < pu_j0 + pu_n) {
                        int32_t e;
                        if (MODE == MODE_RESIDENT) {
                            e = p.table[(size_t)pu_row * p.table_stride + j];
                            if (e != ISV_BLOCK_NONE) {
                                if (e & ISV_BLOCK_HOST_BIT) {   // only the newest block of a sequence is read from its tail slot
                                    valid = (j == pu_jlast) && (pu_tail != nullptr);
                                    src = pu_tail + (uint64_t)pu_row * block_bytes;
                                } else {
                                    valid = e >= 0 && e < p.n_pool_blocks;
                                    if (!valid) atomicOr(p.status, ISV_STATUS_BAD_BLOCK_ID);
                                    src = pu_pool + (uint64_t)e * block_bytes;
                                }
                            }
                            if (j == pu_jlast) nt = (pu_len - j * BT - fused) | (fused ? 256 : 0);
                        } else {
                            e = p.cblk[j];
                            valid = e >= 0 && e < p.n_pool_blocks;
                            if (!valid) atomicOr(p.status, ISV_STATUS_BAD_BLOCK_ID);
                            src = p.pool + (uint64_t)e * block_bytes;
                        }
                    }
                    ent_src = src + (uint64_t)(pu_hg / p.P) * TILE;
                    ent_ntok = nt;
                    pu_mask = __ballot_sync(kFull, valid);
                    continue;
                }
                // no visit carried the end flag (or the unit is empty): explicit end marker
                flags = VF_LAST;
                pu_open = false;
                break;
            }
            if (u_next >= u_end) {
                pu_done = true;
                return false;
            }
            // open the next segment (resident) or unit (staged)
            seg_start = true;
            if (MODE == MODE_RESIDENT) {
                const int x = u_next;
                while (x >= ubase[pu_s + 1]) ++pu_s;
                pu_row = pu_s;
                if (NL > 1) {
                    const int l = pu_s / NSEQ;
                    const int slab = (p.layer0 + l) % p.phys_layers;
                    pu_row = pu_s - l * NSEQ;
                    pu_pool = p.pool + (uint64_t)slab * p.pool_layer_stride;
                    pu_tail = p.tail ? p.tail + (uint64_t)slab * p.tail_layer_stride : nullptr;
                }
                pu_len = slen[pu_s];
                const int nblk = (pu_len + BT - 1) / BT;
                const int nb = max(1, nblk);
                const int r = x - ubase[pu_s];
                pu_hg = r / nb;
                pu_j0 = r - pu_hg * nb;
                const int start = ubase[pu_s] + pu_hg * nb;           // flat range of this (sequence, head group)
                const int seg_end = min(u_end, start + nb);
                const int n = seg_end - x;
                u_next = seg_end;
                pu_n = nblk == 0 ? 0 : n;
                pu_jlast = nblk - 1;
                pu_first = range_first;
                range_first = false;
                if (pu_j0 == 0 && n == nb) {
                    pu_nc = 1;                                        // this range holds all of it
                } else {
                    // the ranges that meet [start, start + nb) each contribute one partial
                    pu_wf = part.range_of(start);
                    pu_nc = part.range_of(start + nb - 1) - pu_wf + 1;
                    pu_wfslot = (part.first(pu_wf) == start) ? 0 : 1;
                }
            } else {
                const int unit = u_next++;
                const int cu = p.cu_first + unit / Hg;
                pu_hg = unit % Hg;
                pu_s = p.cu_seq[cu];
                pu_j0 = p.cu_beg[cu];
                pu_n = p.cu_end[cu] - pu_j0;
                pu_nc = 1;
            }
            pu_nbatch = (pu_n + 31) >> 5;
            pu_batch = 0;
            pu_mask = 0;
            pu_open = true;
        }
        if (seg_start) {
            flags |= VF_FIRST;
            seg_start = false;
        }
        if (lane == 0) {
            int32_t *mt = meta + prod_vis * V_WORDS;
            mt[V_INFO] = ntok | flags;
            if (flags & (VF_FIRST | VF_LAST)) {   // the consumer reads these at segment boundaries only
                mt[V_SEQ] = pu_s;
                mt[V_HG] = pu_hg;
                mt[V_NC] = pu_nc;
                mt[V_WF] = pu_wf;
                mt[V_PACK] = pu_wfslot | (pu_first ? 2 : 0) | (cur_range << 2);   // three fields in one word
            }
            const uint32_t bar = smem_u32(&bars[2 * prod_vis]);
            if (ksrc) {
                mbar_arrive_expect_tx(bar, TILE);
                if (!drop_copy) bulk_g2s(smem_u32(data + (size_t)(2 * prod_vis) * TILE), ksrc, TILE, bar);
                drop_copy = false;
            } else {
                mbar_arrive(bar);
            }
        }
        pv_src = ksrc ? ksrc + v_off : nullptr;
        ++inflight;
        return true;
    };
    auto produce_v = [&]() {   // V slot of the visit produce_k emitted last; advances the ring position
        if (lane == 0) {
            const uint32_t bar = smem_u32(&bars[2 * prod_vis + 1]);
            if (pv_src) {
                mbar_arrive_expect_tx(bar, TILE);
                bulk_g2s(smem_u32(data + (size_t)(2 * prod_vis + 1) * TILE), pv_src, TILE, bar);
            } else {
                mbar_arrive(bar);
            }
        }
        prod_vis = (prod_vis + 1 == NVIS) ? 0 : prod_vis + 1;
    };

    if (!idle)
        for (int i = 0; i < NVIS; ++i) {
            if (!produce_k()) break;
            produce_v();
        }
    if (p.early_reads) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }

    // ---- fused append (placed after the first copies are in flight so that it costs no start-up time):
    // the rows of this step's token go to slot len % BT of block len / BT
    // (pool, or the sequence's tail slot when that block is host-flagged).  Nothing in this launch
    // reads those slots: the new token is attended to from k_new / v_new directly.
    if (fused) {
        const int rows = NV * 2 * p.Hkv;
        const int row_vecs = D * 2 / 16;
        for (int r = blockIdx.x * NW + warp; r < rows; r += gridDim.x * NW) {
            const int s = r / (2 * p.Hkv);
            const int kv = (r / p.Hkv) & 1, h = r % p.Hkv;
            const int len = slen[s] - 1;   // length before this step's token
            const int j = len / BT, slot = len % BT;
            int row = s;                   // table row; the layer's slabs and length copy to write
            uint8_t *pool_w = p.pool_w, *tail_w = p.tail_w;
            int32_t *lens_out = p.lens_out;
            bool store = true;
            if (NL > 1) {
                const int l = s / NSEQ, la = p.layer0 + l;
                const int slab = la % p.phys_layers;
                row = s - l * NSEQ;
                pool_w += (uint64_t)slab * p.pool_layer_stride;
                if (tail_w) tail_w += (uint64_t)slab * p.tail_layer_stride;
                lens_out = p.lens_out + (size_t)(((p.lens_cur_mask >> la) & 1) ^ 1) * p.lens_copy_stride +
                           (size_t)la * p.lens_layer_stride;
                store = l + p.phys_layers >= NL;   // a later layer of this launch writes the same slot
            }
            const int32_t e = p.table[(size_t)row * p.table_stride + j];
            uint8_t *base = nullptr;
            if (e != ISV_BLOCK_NONE) {
                if (e & ISV_BLOCK_HOST_BIT) {
                    if (tail_w) base = tail_w + (uint64_t)row * block_bytes;
                } else if (e >= 0 && e < p.n_pool_blocks) {
                    base = pool_w + (uint64_t)e * block_bytes;
                }
            }
            if (base && !store) {
                // nothing to write
            } else if (base) {
                if (lane < row_vecs) {
                    const uint8_t *src = reinterpret_cast<const uint8_t *>(kv ? p.v_new : p.k_new) +
                                         ((size_t)s * p.Hkv + h) * (D * 2) + lane * 16;
                    uint8_t *dst =
                        base + (size_t)(kv * p.Hkv + h) * TILE1 + (size_t)slot * (D * 2) + swz(lane, slot, row_vecs) * 16;
                    *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
                }
            } else if (lane == 0) {
                atomicOr(p.status, ISV_STATUS_BAD_BLOCK_ID);
            }
            if (kv == 0 && h == 0 && lane == 0) lens_out[row] = len + 1;
        }
        // sequences beyond those of this launch keep their lengths: carry them over to the copy that becomes
        // current, so that a later launch over more sequences finds them
        if (p.lens_count > NSEQ) {
            const int extra = p.lens_count - NSEQ;
            for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < NL * extra; i += gridDim.x * blockDim.x) {
                const int l = i / extra, sx = NSEQ + (i - l * extra);
                if (NL > 1) {
                    const int la = p.layer0 + l;
                    const size_t cur = (size_t)((p.lens_cur_mask >> la) & 1);
                    const size_t at = (size_t)la * p.lens_layer_stride + sx;
                    p.lens_out[(cur ^ 1) * p.lens_copy_stride + at] = p.lens[cur * p.lens_copy_stride + at];
                } else {
                    p.lens_out[sx] = p.lens[sx];
                }
            }
        }
    }

    // Publishes a stored partial: fence, ticket, and the merge if this was the last split to arrive.
    PendingArrival pend{0, 0, 0, 0, 0, 0};
    auto publish = [&](bool at_end) {
        if (!pend.valid) return;
        pend.valid = 0;
        __syncwarp();   // the lanes' partial stores are ordered before lane 0's release below
        int ticket = 0;
        if (lane == 0)
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;"
                         : "=r"(ticket) : "l"(&p.tickets[pend.ticket_idx]) : "memory");
        ticket = __shfl_sync(kFull, ticket, 0);
        __syncwarp();   // orders the other lanes' reads of the partials after lane 0's acquire
        if (ticket == pend.nc - 1) {
            if (lane == 0) p.tickets[pend.ticket_idx] = 0;   // ready for the next launch
            if (at_end && GT > 1) {   // the accumulators are dead: several heads at a time
                for (int g0 = 0; g0 < GT; g0 += 8)
                    merge_partials_rows<D, BF16, 8>(p, pend.wf, pend.wf_slot, pend.nc, g0, GT, pend.row0, lane);
            } else {
                for (int g = 0; g < GT; ++g)
                    merge_partials_row<D, BF16>(p, pend.wf, pend.wf_slot, pend.nc, g, GT, pend.row0 + g, lane);
            }
        }
    };

    // ---- consumer
    int cons_vis = 0;
    uint32_t cons_phase = 0;
    int s = 0, hg = 0;   // sequence and head group of the open segment
    // A bounded wait ran out: report it, give the copies that may still be in flight one more bounded
    // chance to land (slots of visit cons_vis onwards, in ring order), then leave.
    auto give_up = [&]() {
        if (lane == 0) atomicOr(p.status, ISV_STATUS_WAIT_EXPIRED);
        for (int k = 0; k < inflight; ++k) {
            mbar_wait(smem_u32(&bars[2 * cons_vis]), cons_phase, spin_limit);
            mbar_wait(smem_u32(&bars[2 * cons_vis + 1]), cons_phase, spin_limit);
            cons_vis = (cons_vis + 1 == NVIS) ? 0 : cons_vis + 1;
            if (cons_vis == 0) cons_phase ^= 1u;
        }
    };
    while (inflight > 0) {
        bool ok = mbar_wait(smem_u32(&bars[2 * cons_vis]), cons_phase, spin_limit);
        if (!__all_sync(kFull, ok)) {
            give_up();
            return;
        }
        const int32_t *mt = meta + cons_vis * V_WORDS;
        const int info = mt[V_INFO];
        const int ntok = info & 255;
        int nc = 1, mt_wf = 0, mt_pack = 0;
        if (info & VF_FIRST) {
            s = mt[V_SEQ];
            hg = mt[V_HG];
            mth.begin(p, s, hg);
        }
        if (info & VF_LAST) {   // read now: the record is rewritten as soon as the K slot is handed back
            nc = mt[V_NC];
            mt_wf = mt[V_WF];
            mt_pack = mt[V_PACK];
        }
        if (info & VF_DATA) mth.k_tile(data + (size_t)(2 * cons_vis) * TILE, ntok);
        __syncwarp();   // every lane is done with the K slot and the record before they are refilled
        const bool more = !pu_done && produce_k();

        ok = mbar_wait(smem_u32(&bars[2 * cons_vis + 1]), cons_phase, spin_limit);
        if (!__all_sync(kFull, ok)) {
            give_up();
            return;
        }
        if (info & VF_DATA) mth.v_tile(data + (size_t)(2 * cons_vis + 1) * TILE, ntok);
        __syncwarp();   // every lane is done with the V slot before it is refilled
        if (more) produce_v();
        --inflight;
        cons_vis = (cons_vis + 1 == NVIS) ? 0 : cons_vis + 1;
        if (cons_vis == 0) cons_phase ^= 1u;

        if (info & VF_NEW) {   // this step's token, attended to from the caller's rows
            const int kvh = hg / p.P * HP;   // first KV head of the group
            mth.new_token(reinterpret_cast<const uint16_t *>(p.k_new) + ((size_t)s * p.Hkv + kvh) * D,
                          reinterpret_cast<const uint16_t *>(p.v_new) + ((size_t)s * p.Hkv + kvh) * D);
        }
        if (!(info & VF_LAST)) continue;

        // ---- end of unit
        mth.finish();
        const size_t row0 = (size_t)s * p.Hq + (size_t)hg * GT;

        if (MODE == MODE_STAGED) {   // fold into the running state of (s, heads); this unit is its only writer
            mth.fold_running(p, row0);
            continue;
        }

        // ---- resident mode
        if (nc == 1) {   // this warp covered the whole (sequence, head group): no partial needed
            if (p.finalize) mth.store_final(p, row0);
            else mth.store_state(p.acc_o, p.acc_ml, row0);
            continue;
        }
        publish(false);   // the previous partial's arrival; its stores have long landed
        // an incomplete segment is the first or the last of its range: two partial slots per range
        const int slot = 2 * (mt_pack >> 2) + ((mt_pack & 2) ? 0 : 1);
        mth.store_state(p.part_o, p.part_ml, (size_t)slot * GT);
        pend.valid = 1;
        pend.ticket_idx = s * Hg + hg;
        pend.nc = nc;
        pend.wf = mt_wf;
        pend.wf_slot = mt_pack & 1;
        pend.row0 = row0;
    }
    publish(true);
}

// ---------------------------------------------------------------- merge kernel (resident + offloaded)

__global__ void merge_kernel(const MergeParams p) {
    const int warps_per_block = blockDim.x >> 5;
    const int row = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= p.rows) return;
    const float m1 = p.res_ml[row * 2], l1 = p.res_ml[row * 2 + 1];
    float m2 = p.run_ml[row * 2];
    const float l2 = p.run_ml[row * 2 + 1];
    if (!(l2 > 0.f)) m2 = kNegBig;
    const float mm = fmaxf(l1 > 0.f ? m1 : kNegBig, m2);
    const float a1 = l1 > 0.f ? exp2f(m1 - mm) : 0.f;
    const float a2 = l2 > 0.f ? exp2f(m2 - mm) : 0.f;
    const float ll = l1 * a1 + l2 * a2;
    const float inv = ll > 0.f ? 1.f / ll : 0.f;
    for (int e = lane; e < p.D; e += 32) {
        const size_t idx = (size_t)row * p.D + e;
        float x = 0.f;
        if (l1 > 0.f) x += p.res_o[idx] * a1;
        if (l2 > 0.f) x += p.run_o[idx] * a2;
        x *= inv;
        if (p.out_f32) p.out_f32[idx] = x;
        if (p.out) {
            uint16_t *o16 = reinterpret_cast<uint16_t *>(p.out) + idx;
            if (p.bf16) {
                const __nv_bfloat16 h = __float2bfloat16_rn(x);
                *o16 = *reinterpret_cast<const uint16_t *>(&h);
            } else {
                const __half h = __float2half_rn(x);
                *o16 = *reinterpret_cast<const uint16_t *>(&h);
            }
        }
    }
}

// ---------------------------------------------------------------- table update, append, fill, gather

__global__ void table_update_kernel(int32_t *table, const TableUpdateBatch b) {
    for (int i = threadIdx.x; i < b.n; i += blockDim.x) table[b.index[i]] = b.value[i];
}

// One CTA per sequence: K and V rows of the new token go to slot len % BT of
// block len / BT (HBM pool, or the sequence's tail slot when the block is
// host-flagged); then the length is incremented.
__global__ void append_kernel(const AppendParams p) {
    const int s = blockIdx.x;
    const int len = p.lens[s];
    const int j = len / p.BT, slot = len % p.BT;
    const bool in_row = len >= 0 && j < p.max_blocks;   // a length the table row does not cover is not followed
    const int32_t e = in_row ? p.table[(size_t)s * p.table_stride + j] : ISV_BLOCK_NONE;
    uint8_t *base = nullptr;
    if (e != ISV_BLOCK_NONE) {
        if (e & ISV_BLOCK_HOST_BIT) {
            if (p.tail) base = p.tail + (uint64_t)s * p.block_bytes;
        } else if (e >= 0 && e < p.n_pool_blocks) {
            base = p.pool + (uint64_t)e * p.block_bytes;
        }
    }
    const int row_bytes = p.D * 2;
    const int row_vecs = row_bytes / 16;
    const uint32_t tile_bytes = (uint32_t)p.BT * row_bytes;
    const int n = 2 * p.Hkv * row_vecs;
    if (base) {
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int kv = i / (p.Hkv * row_vecs);
            const int r = i - kv * (p.Hkv * row_vecs);
            const int h = r / row_vecs, vec = r - h * row_vecs;
            const uint8_t *src = reinterpret_cast<const uint8_t *>(kv ? p.v : p.k) +
                                 ((size_t)s * p.Hkv + h) * row_bytes + vec * 16;
            uint8_t *dst =
                base + (size_t)(kv * p.Hkv + h) * tile_bytes + (size_t)slot * row_bytes + swz(vec, slot, row_vecs) * 16;
            *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
        }
    } else if (threadIdx.x == 0) {
        atomicOr(p.status, in_row ? ISV_STATUS_BAD_BLOCK_ID : ISV_STATUS_BAD_LENGTH);
    }
    __syncthreads();   // every thread has read the old length
    if (threadIdx.x == 0 && in_row) p.lens[s] = len + 1;
}

// Where block j of sequence s lives for a reader/writer that sees `len`
// tokens: HBM pool, tail slot (host-flagged newest block) or host pool.
__device__ __forceinline__ uint8_t *block_base(int32_t e, int s, int j, int len, int BT, uint8_t *pool, uint8_t *tail,
                                               uint8_t *host, int n_pool, int n_host, uint64_t bb) {
    if (e == ISV_BLOCK_NONE) return nullptr;
    if (e & ISV_BLOCK_HOST_BIT) {
        const int id = e & (ISV_BLOCK_HOST_BIT - 1);
        if (j == (len - 1) / BT) return tail ? tail + (uint64_t)s * bb : nullptr;
        return (host && id < n_host) ? host + (uint64_t)id * bb : nullptr;
    }
    return (e >= 0 && e < n_pool) ? pool + (uint64_t)e * bb : nullptr;
}

__global__ void fill_kernel(const FillParams p) {
    const int j = blockIdx.x, s = blockIdx.y;
    const int len = p.lens[s];
    if (j * p.BT >= len) return;
    const int ntok = min(p.BT, len - j * p.BT);
    const int32_t e = p.table[(size_t)s * p.table_stride + j];
    if (!p.host && e != ISV_BLOCK_NONE && (e & ISV_BLOCK_HOST_BIT) && j != (len - 1) / p.BT) return;   // stored elsewhere
    uint8_t *base = block_base(e, s, j, len, p.BT, p.pool, p.tail, p.host, p.n_pool_blocks, p.n_host_blocks,
                               p.block_bytes);
    if (!base) {
        if (threadIdx.x == 0) atomicOr(p.status, ISV_STATUS_BAD_BLOCK_ID);
        return;
    }
    const int row_bytes = p.D * 2, row_vecs = row_bytes / 16;
    const uint32_t tile_bytes = (uint32_t)p.BT * row_bytes;
    const int per_kv = p.Hkv * ntok * row_vecs;
    for (int i = threadIdx.x; i < 2 * per_kv; i += blockDim.x) {
        const int kv = i / per_kv;
        int r = i - kv * per_kv;
        const int h = r / (ntok * row_vecs);
        r -= h * ntok * row_vecs;
        const int t = r / row_vecs, vec = r - t * row_vecs;
        const uint8_t *src = reinterpret_cast<const uint8_t *>(kv ? p.v : p.k) +
                             (((size_t)s * p.T + (size_t)j * p.BT + t) * p.Hkv + h) * row_bytes + vec * 16;
        uint8_t *dst = base + (size_t)(kv * p.Hkv + h) * tile_bytes + (size_t)t * row_bytes + swz(vec, t, row_vecs) * 16;
        *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
    }
}

__global__ void pack_kernel(const PackParams p) {
    const int b = blockIdx.x;
    const int s = p.owner[2 * (p.first_id + b)], j = p.owner[2 * (p.first_id + b) + 1];
    const int row_bytes = p.D * 2, row_vecs = row_bytes / 16;
    const uint32_t tile_bytes = (uint32_t)p.BT * row_bytes;
    uint8_t *base = p.dst + (uint64_t)b * p.block_bytes;
    const int per_kv = p.Hkv * p.BT * row_vecs;
    for (int i = threadIdx.x; i < 2 * per_kv; i += blockDim.x) {
        const int kv = i / per_kv;
        int r = i - kv * per_kv;
        const int h = r / (p.BT * row_vecs);
        r -= h * p.BT * row_vecs;
        const int t = r / row_vecs, vec = r - t * row_vecs;
        const uint8_t *src = reinterpret_cast<const uint8_t *>(kv ? p.v : p.k) +
                             (((size_t)s * p.T + (size_t)j * p.BT + t) * p.Hkv + h) * row_bytes + vec * 16;
        uint8_t *dst = base + (size_t)(kv * p.Hkv + h) * tile_bytes + (size_t)t * row_bytes + swz(vec, t, row_vecs) * 16;
        *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
    }
}

__global__ void gather_kernel(const GatherParams p) {
    const int j = blockIdx.x;
    if (j * p.BT >= p.len) return;
    const int ntok = min(p.BT, p.len - j * p.BT);
    const int32_t e = p.table[j];
    const uint8_t *base =
        block_base(e, p.seq, j, p.len, p.BT, const_cast<uint8_t *>(p.pool), const_cast<uint8_t *>(p.tail),
                   const_cast<uint8_t *>(p.host), p.n_pool_blocks, p.n_host_blocks, p.block_bytes);
    if (!base) {
        if (threadIdx.x == 0) atomicOr(p.status, ISV_STATUS_BAD_BLOCK_ID);
        return;
    }
    const int row_bytes = p.D * 2, row_vecs = row_bytes / 16;
    const uint32_t tile_bytes = (uint32_t)p.BT * row_bytes;
    const int per_kv = p.Hkv * ntok * row_vecs;
    for (int i = threadIdx.x; i < 2 * per_kv; i += blockDim.x) {
        const int kv = i / per_kv;
        int r = i - kv * per_kv;
        const int h = r / (ntok * row_vecs);
        r -= h * ntok * row_vecs;
        const int t = r / row_vecs, vec = r - t * row_vecs;
        const uint8_t *src =
            base + (size_t)(kv * p.Hkv + h) * tile_bytes + (size_t)t * row_bytes + swz(vec, t, row_vecs) * 16;
        uint8_t *dst = reinterpret_cast<uint8_t *>(kv ? p.v_out : p.k_out) +
                       (((size_t)j * p.BT + t) * p.Hkv + h) * row_bytes + vec * 16;
        *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
    }
}

// ---------------------------------------------------------------- dispatch

#ifndef ISV_WARPS_GT1
#define ISV_WARPS_GT1 16   // warps per CTA when one query head is handled per KV tile
#endif

#ifndef ISV_WARPS_PAIR80
#define ISV_WARPS_PAIR80 12   // warps per CTA when a visit carries two KV heads at head_dim 80 (two heads' queries and
                              // accumulators need more than the 128 registers that 16 warps leave a thread)
#endif

#ifndef ISV_WARPS_MMA
#define ISV_WARPS_MMA 8   // warps per CTA of the tensor-core variant
#endif

typedef void (*DecodeFn)(const DecodeParams, const int);

template <class Math, int NW>
DecodeFn pick_mode(int mode) {
    return mode == MODE_RESIDENT ? decode_kernel<Math, MODE_RESIDENT, NW> : decode_kernel<Math, MODE_STAGED, NW>;
}
template <int D, bool BF16>
DecodeFn pick_gt(int GT, int HP, int mode) {
    if (HP == 2) {   // multi-head attention, two adjacent KV heads per visit (small head dims only)
        if constexpr (D < 128) {
            if (GT == 2) return pick_mode<ScalarMath<D, 2, 16, BF16>, (D == 80 ? ISV_WARPS_PAIR80 : ISV_WARPS_GT1)>(mode);
        }
        return nullptr;
    }
    if (HP != 1) return nullptr;
    if (GT == 1) return pick_mode<ScalarMath<D, 1, 16, BF16>, ISV_WARPS_GT1>(mode);
    if (GT >= 2 && GT <= 16) return pick_mode<MmaMath<D, BF16>, (D == 64 ? 16 : D == 80 ? 12 : ISV_WARPS_MMA)>(mode);
    return nullptr;
}
DecodeFn pick(int D, int GT, int HP, int BT, bool bf16, int mode) {
    if (BT != 16) return nullptr;
    if (D == 64) return bf16 ? pick_gt<64, true>(GT, HP, mode) : pick_gt<64, false>(GT, HP, mode);
    if (D == 80) return bf16 ? pick_gt<80, true>(GT, HP, mode) : pick_gt<80, false>(GT, HP, mode);
    if (D == 128) return bf16 ? pick_gt<128, true>(GT, HP, mode) : pick_gt<128, false>(GT, HP, mode);
    return nullptr;
}

}  // namespace

// The tensor-core variant keeps 96 accumulator and operand registers per thread at head_dim 128 (8 warps),
// 60 at head_dim 80 (12 warps fit without spills); at head_dim 64 it fits 128 registers, and 16 warps hide
// its per-visit latencies (a visit carries only 4 KiB there).
int decode_warps(int GT, int D, int HP) {
    if (HP == 2) return D == 80 ? ISV_WARPS_PAIR80 : ISV_WARPS_GT1;
    return GT == 1 ? ISV_WARPS_GT1 : (D == 64 ? 16 : D == 80 ? 12 : ISV_WARPS_MMA);
}

int decode_default_stages(int D, int BT, int GT, int HP) {
    const int per_stage = decode_warps(GT, D, HP) * BT * D * 2 * HP;
    const int st = ((128 << 10) / per_stage) & ~1;   // slots come in pairs: a K and a V tile per block visit
    return st < 2 ? 2 : (st > 12 ? 12 : st);
}

size_t decode_smem_bytes(int D, int BT, int GT, int HP, int stages, int max_seqs, int mode) {
    const size_t tile = (size_t)BT * D * 2 * HP;
    size_t b = (size_t)decode_warps(GT, D, HP) * stages * (tile + 8 + 4 * V_WORDS);
    if (mode == MODE_RESIDENT) b += (size_t)(2 * max_seqs + 1) * 4;
    return b;
}

cudaError_t decode_configure(int D, int GT, int HP, int BT, bool bf16, int mode, size_t smem) {
    DecodeFn fn = pick(D, GT, HP, BT, bf16, mode);
    if (!fn) return cudaErrorInvalidValue;
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

cudaError_t launch_decode(const DecodeParams &p, int D, int GT, int HP, int BT, bool bf16, int mode, int grid,
                          int stages, size_t smem, cudaStream_t st) {
    DecodeFn fn = pick(D, GT, HP, BT, bf16, mode);
    if (!fn || stages < 2) return cudaErrorInvalidValue;
    stages &= ~1;   // the kernel uses its ring slots in pairs
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(decode_warps(GT, D, HP) * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;   // see the kernel's griddepcontrol pair
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fn, p, stages);
}

cudaError_t launch_table_update(int32_t *table, const TableUpdateBatch &b, cudaStream_t st) {
    table_update_kernel<<<1, 256, 0, st>>>(table, b);
    return cudaGetLastError();
}

cudaError_t launch_append(const AppendParams &p, cudaStream_t st) {
    append_kernel<<<p.n_seqs, 256, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_fill(const FillParams &p, cudaStream_t st) {
    dim3 grid(p.max_blocks, p.n_seqs);
    fill_kernel<<<grid, 256, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_gather(const GatherParams &p, cudaStream_t st) {
    const int nblk = (p.len + p.BT - 1) / p.BT;
    if (nblk == 0) return cudaSuccess;
    gather_kernel<<<nblk, 256, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_pack(const PackParams &p, cudaStream_t st) {
    if (p.n_ids <= 0) return cudaSuccess;
    pack_kernel<<<p.n_ids, 256, 0, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_merge(const MergeParams &p, cudaStream_t st) {
    const int wpb = 8;
    merge_kernel<<<(p.rows + wpb - 1) / wpb, wpb * 32, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace isv
