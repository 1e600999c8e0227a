// Two loophole checks on candidate outputs that need no reference (sm_100a):
//
//   * cross-seed variation: the outputs of K candidates for S input seeds, K * S tensors, in
//     one launch.  For one vector position a thread visits the S outputs of its candidate in
//     turn, so the per-element minimum and maximum across seeds, and seed 0's value, never
//     leave registers; every output byte is read once.  Bound: HBM read bandwidth
//     (K * S * n * element size bytes).  Up to eight seeds take cross_seed_few_kernel (every seed's
//     piece of a position in registers at once, eight 16-byte loads per thread in flight), more
//     take cross_seed_kernel (batches of loads, per-element state carried between batches);
//   * copy of any input: is a candidate's output a bit copy of one of the M operands the
//     kernel received?  16-byte pieces are compared as stored; a block stops comparing
//     against an operand as soon as any block has seen a difference, so only true copies are
//     read to the end.
//
// Reductions are deterministic: integer sums, boolean ands, lexicographic (value descending,
// index ascending) maxima, one partial per block merged in block order.
#include <string.h>

#include <vector>

#include "rkv_internal.h"

namespace rkv {

namespace {

constexpr int kCrossThreads = 256;
constexpr int kCrossBlocksPerSm = 24;      // blocks per SM the grid is sized for (about eight waves: measured best of 3 .. 48)
constexpr int kCrossMaxSeeds = 16;
constexpr int kCopyMaxInputs = 8;
constexpr int kCrossMaxK = 4096;
constexpr uint32_t kFull = 0xFFFFFFFFu;

__device__ __forceinline__ bool finite_bits(uint32_t b) { return (b & 0x7F800000u) != 0x7F800000u; }
__device__ __forceinline__ bool inf_bits(uint32_t b) { return (b & 0x7FFFFFFFu) == 0x7F800000u; }

// 16 storage bits -> the fp32 bit pattern of the same value.
template <int DT>
__device__ __forceinline__ uint32_t widen(uint32_t raw) {
    if (DT == RKV_F32) return raw;
    if (DT == RKV_BF16) return raw << 16;
    float f;
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"((unsigned short)raw));
    return __float_as_uint(f);
}

struct __align__(16) CrossPartial {
    unsigned long long arg;        // first element with the largest spread
    unsigned long long n_nonfin;
    float spread;                  // -1: none
    uint32_t differs;              // bit0: some seed differs from seed 0 in bits; bit1: some seed is not within tolerance
    uint32_t reserved[2];
};
static_assert(sizeof(CrossPartial) == 32, "CrossPartial layout");

struct CrossAcc {
    unsigned long long arg, n_nonfin;
    float spread;
    uint32_t differs;
};

__device__ __forceinline__ void merge(CrossAcc& a, const CrossAcc& b) {
    if (b.spread > a.spread || (b.spread == a.spread && b.arg < a.arg)) { a.spread = b.spread; a.arg = b.arg; }
    a.n_nonfin += b.n_nonfin;
    a.differs |= b.differs;
}

// What one element position contributes, given its value in every seed so far.
struct ElemState {
    uint32_t b0;       // seed 0, widened bits
    float lo, hi;
    bool finite;
};

template <int DT>
__device__ __forceinline__ void visit(ElemState& e, CrossAcc& a, uint32_t raw, uint32_t raw0, bool first,
                                      float atol, float rtol) {
    const uint32_t b = widen<DT>(raw);
    const float x = __uint_as_float(b);
    if (first) {
        e.b0 = b; e.lo = x; e.hi = x; e.finite = finite_bits(b);
        return;
    }
    if (raw != raw0) a.differs |= 1u;
    const float x0 = __uint_as_float(e.b0);
    bool close;
    if (finite_bits(b) && finite_bits(e.b0))
        close = fabsf(__fsub_rn(x, x0)) <= __fadd_rn(atol, __fmul_rn(rtol, fabsf(x0)));
    else
        close = inf_bits(b) && b == e.b0;
    if (!close) a.differs |= 2u;
    e.finite = e.finite && finite_bits(b);
    // (min / max of a NaN leave the other operand: the element is left out anyway)
    e.lo = fminf(e.lo, x);
    e.hi = fmaxf(e.hi, x);
}

__device__ __forceinline__ void finish(const ElemState& e, CrossAcc& a, unsigned long long index) {
    if (!e.finite) { a.n_nonfin++; return; }
    const float d = __fsub_rn(e.hi, e.lo);
    if (d > a.spread) { a.spread = d; a.arg = index; }       // ascending index: the first maximum stays
}

// One vector position by the general rule (values that are not finite included).  Out of line: it
// runs for the rare positions that hold a NaN or an infinity, and its registers stay out of the
// kernel's count.
template <int DT>
__device__ __noinline__ CrossAcc general_position(const void* const* mine, int S, unsigned long long v, float atol,
                                                  float rtol, CrossAcc a) {
    constexpr int VEC = DT == RKV_F32 ? 4 : 8;
    ElemState e[VEC];
    uint32_t raw0[VEC];
    for (int s = 0; s < S; ++s) {
        const uint4 w = __ldcs(reinterpret_cast<const uint4*>(mine[s]) + v);
        const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            const uint32_t raw = DT == RKV_F32 ? words[i] : ((i & 1) ? words[i >> 1] >> 16 : words[i >> 1] & 0xFFFFu);
            if (s == 0) raw0[i] = raw;
            visit<DT>(e[i], a, raw, raw0[i], s == 0, atol, rtol);
        }
    }
#pragma unroll
    for (int i = 0; i < VEC; ++i) finish(e[i], a, v * VEC + i);
    return a;
}

// The end of both kernels: the ragged end of the tensor, then the block's partial.
template <int DT>
__device__ __forceinline__ void cross_block_end(CrossAcc a, const void* const* mine, int k, int S, unsigned long long n,
                                                float atol, float rtol, CrossPartial* __restrict__ partials) {
    constexpr int VEC = DT == RKV_F32 ? 4 : 8;
    const unsigned long long n_vec = n / VEC;
    // the ragged end: fewer elements than a vector, one thread of the first block
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (unsigned long long i = n_vec * VEC; i < n; ++i) {
            ElemState e;
            uint32_t raw0 = 0;
            for (int s = 0; s < S; ++s) {
                const uint32_t raw = DT == RKV_F32 ? reinterpret_cast<const uint32_t*>(mine[s])[i]
                                                   : reinterpret_cast<const unsigned short*>(mine[s])[i];
                if (s == 0) raw0 = raw;
                visit<DT>(e, a, raw, raw0, s == 0, atol, rtol);
            }
            finish(e, a, i);
        }
    }
    // block reduction: shuffle tree, then the warps' results in warp order
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        CrossAcc b;
        b.arg = __shfl_xor_sync(kFull, a.arg, off);
        b.n_nonfin = __shfl_xor_sync(kFull, a.n_nonfin, off);
        b.spread = __shfl_xor_sync(kFull, a.spread, off);
        b.differs = __shfl_xor_sync(kFull, a.differs, off);
        merge(a, b);
    }
    __shared__ CrossAcc warp_acc[kCrossThreads / 32];
    if ((threadIdx.x & 31) == 0) warp_acc[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        CrossAcc t = warp_acc[0];
        for (int w = 1; w < kCrossThreads / 32; ++w) merge(t, warp_acc[w]);
        CrossPartial p;
        p.arg = t.arg; p.n_nonfin = t.n_nonfin; p.spread = t.spread; p.differs = t.differs;
        p.reserved[0] = p.reserved[1] = 0;
        partials[(size_t)k * gridDim.x + blockIdx.x] = p;
    }
}

// One storage word -> element i of it, widened.
template <int DT>
__device__ __forceinline__ float elem_of(const uint4& w, int i) {
    const uint32_t words[4] = {w.x, w.y, w.z, w.w};
    const uint32_t raw = DT == RKV_F32 ? words[i] : ((i & 1) ? words[i >> 1] >> 16 : words[i >> 1] & 0xFFFFu);
    return __uint_as_float(widen<DT>(raw));
}

// Two 16-bit values per 32-bit word at once.  Minimum and maximum select one of their operands, so
// the packed forms give exactly the values the fp32 forms give on the widened operands.
template <int DT>
__device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) {
    uint32_t d;
    if (DT == RKV_BF16) asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    else asm("min.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
template <int DT>
__device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
    uint32_t d;
    if (DT == RKV_BF16) asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    else asm("max.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// chk + x * 0 in both halves: stays a zero while every x is finite, NaN afterwards
template <int DT>
__device__ __forceinline__ uint32_t fma2_zero(uint32_t x, uint32_t chk) {
    uint32_t d;
    const uint32_t zero = 0u;
    if (DT == RKV_BF16) asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(x), "r"(zero), "r"(chk));
    else asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(x), "r"(zero), "r"(chk));
    return d;
}
// x - r in fp32 with one rounding, x the low or high 16-bit value of a word (widening is exact, so
// this is the fp32 subtraction of the widened value)
template <int DT>
__device__ __forceinline__ float sub_half_f32(uint32_t word, int half, float r) {
    float d;
    if (DT == RKV_BF16) {
        if (half) asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, hi, %2;\n\t}" : "=f"(d) : "r"(word), "f"(r));
        else asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, lo, %2;\n\t}" : "=f"(d) : "r"(word), "f"(r));
    } else {
        if (half) asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.f16 %0, hi, %2;\n\t}" : "=f"(d) : "r"(word), "f"(r));
        else asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.f16 %0, lo, %2;\n\t}" : "=f"(d) : "r"(word), "f"(r));
    }
    return d;
}
template <int DT>
__device__ __forceinline__ float half_of(uint32_t word, int half) {
    return __uint_as_float(widen<DT>(half ? word >> 16 : word & 0xFFFFu));
}

// S <= CH: every seed's piece of a position is in registers at once, so nothing is carried from
// seed to seed but the loaded words themselves, and NP positions (one grid stride apart) have their
// loads in flight together: CH * NP 16-byte loads per thread.  A seed slot beyond S repeats seed 0's
// piece, which changes none of the results.  Same rule and same results as cross_seed_kernel.
template <int DT, int CH, int NP, int MINB>
__global__ void __launch_bounds__(kCrossThreads, MINB)
cross_seed_few_kernel(const void* const* __restrict__ outs, int S, unsigned long long n, float atol, float rtol,
                      CrossPartial* __restrict__ partials) {
    constexpr int VEC = DT == RKV_F32 ? 4 : 8;
    const int k = blockIdx.y;
    const void* const* mine = outs + (size_t)k * (size_t)S;
    const unsigned long long n_vec = n / VEC;
    const unsigned long long stride = (unsigned long long)gridDim.x * kCrossThreads;
    CrossAcc a;
    a.arg = RKV_NO_INDEX; a.n_nonfin = 0; a.spread = -1.0f; a.differs = 0;
    const uint4* base[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) base[c] = reinterpret_cast<const uint4*>(mine[c < S ? c : 0]);

    for (unsigned long long v = (unsigned long long)blockIdx.x * kCrossThreads + threadIdx.x; v < n_vec;
         v += NP * stride) {
        uint4 w[NP][CH];
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const unsigned long long vp = v + (unsigned long long)p * stride;
            if (vp < n_vec) {
#pragma unroll
                for (int c = 0; c < CH; ++c) w[p][c] = __ldcs(base[c] + vp);
            }
        }
        // positions in ascending order, so that the first maximum stays
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const unsigned long long vp = v + (unsigned long long)p * stride;
            if (vp >= n_vec) break;
            uint32_t xacc = 0;
#pragma unroll
            for (int c = 1; c < CH; ++c)
                xacc |= (w[p][c].x ^ w[p][0].x) | (w[p][c].y ^ w[p][0].y) | (w[p][c].z ^ w[p][0].z) | (w[p][c].w ^ w[p][0].w);
            // (x * 0 is NaN exactly for NaN and the infinities: chk tells whether every value was finite)
            float chk = 0.0f, best = -1.0f;
            int best_i = 0;
            bool far = false;
            if (DT != RKV_F32) {
                // 16-bit values two at a time: packed minimum, maximum and finiteness check; the
                // tolerance test stays in fp32 (one mixed-precision subtraction per value)
                uint32_t chk2 = 0u;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint32_t w0[4] = {w[p][0].x, w[p][0].y, w[p][0].z, w[p][0].w};
                    const uint32_t first = w0[q];
                    const float x0a = half_of<DT>(first, 0), x0b = half_of<DT>(first, 1);
                    const float thra = __fadd_rn(atol, __fmul_rn(rtol, fabsf(x0a)));
                    const float thrb = __fadd_rn(atol, __fmul_rn(rtol, fabsf(x0b)));
                    uint32_t lo2 = first, hi2 = first;
                    chk2 = fma2_zero<DT>(first, chk2);
#pragma unroll
                    for (int c = 1; c < CH; ++c) {
                        const uint32_t wc[4] = {w[p][c].x, w[p][c].y, w[p][c].z, w[p][c].w};
                        const uint32_t x2 = wc[q];
                        lo2 = min2<DT>(lo2, x2);
                        hi2 = max2<DT>(hi2, x2);
                        chk2 = fma2_zero<DT>(x2, chk2);
                        far |= !(fabsf(sub_half_f32<DT>(x2, 0, x0a)) <= thra);
                        far |= !(fabsf(sub_half_f32<DT>(x2, 1, x0b)) <= thrb);
                    }
                    const float da = __fsub_rn(half_of<DT>(hi2, 0), half_of<DT>(lo2, 0));
                    const float db = __fsub_rn(half_of<DT>(hi2, 1), half_of<DT>(lo2, 1));
                    if (da > best) { best = da; best_i = 2 * q; }
                    if (db > best) { best = db; best_i = 2 * q + 1; }
                }
                chk = (chk2 & 0x7FFF7FFFu) ? 1.0f : 0.0f;
            } else
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                const float x0 = elem_of<DT>(w[p][0], i);
                const float thr = __fadd_rn(atol, __fmul_rn(rtol, fabsf(x0)));
                float lo = x0, hi = x0;
                chk = __fmaf_rn(x0, 0.0f, chk);
#pragma unroll
                for (int c = 1; c < CH; ++c) {
                    const float x = elem_of<DT>(w[p][c], i);
                    far |= !(fabsf(__fsub_rn(x, x0)) <= thr);
                    lo = fminf(lo, x);
                    hi = fmaxf(hi, x);
                    chk = __fmaf_rn(x, 0.0f, chk);
                }
                const float d = __fsub_rn(hi, lo);
                if (d > best) { best = d; best_i = i; }
            }
            if (chk == 0.0f) {
                a.differs |= (xacc ? 1u : 0u) | (far ? 2u : 0u);
                if (best > a.spread) { a.spread = best; a.arg = vp * VEC + best_i; }
            } else {
                // a NaN or an infinity somewhere in the position: the general rule, out of line
                a = general_position<DT>(mine, S, vp, atol, rtol, a);
            }
        }
    }
    cross_block_end<DT>(a, mine, k, S, n, atol, rtol, partials);
}

// grid = (blocks per candidate, K).  outs[k * S + s]: candidate k's output for input seed s.
template <int DT>
__global__ void __launch_bounds__(kCrossThreads, 3)
cross_seed_kernel(const void* const* __restrict__ outs, int S, unsigned long long n, float atol, float rtol,
                  CrossPartial* __restrict__ partials) {
    constexpr int VEC = DT == RKV_F32 ? 4 : 8;
    constexpr int CH = DT == RKV_F32 ? 8 : 4;            // outputs whose loads are issued together
    const int k = blockIdx.y;
    const void* const* mine = outs + (size_t)k * (size_t)S;
    const unsigned long long n_vec = n / VEC;
    CrossAcc a;
    a.arg = RKV_NO_INDEX; a.n_nonfin = 0; a.spread = -1.0f; a.differs = 0;

    for (unsigned long long v = (unsigned long long)blockIdx.x * kCrossThreads + threadIdx.x; v < n_vec;
         v += (unsigned long long)gridDim.x * kCrossThreads) {
        // Common case: every value of the position is finite.  Then "within tolerance of seed 0" is one
        // subtraction and one comparison against a threshold kept from seed 0, "same bits" one
        // exclusive-or per 32-bit word, and one fused multiply-add per value (x * 0 is NaN exactly for
        // NaN and the infinities) tells afterwards whether the assumption held.  If it did not, the
        // position is done again by the general rule.
        float x0[VEC], thr[VEC], lo[VEC], hi[VEC];
        uint32_t w0[4] = {0u, 0u, 0u, 0u};
        uint32_t xacc = 0;
        float chk = 0.0f;
        bool far = false;
        for (int s0 = 0; s0 < S; s0 += CH) {
            uint4 w[CH];
#pragma unroll
            for (int c = 0; c < CH; ++c)
                if (s0 + c < S) w[c] = __ldcs(reinterpret_cast<const uint4*>(mine[s0 + c]) + v);
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                if (s0 + c >= S) break;
                const uint32_t words[4] = {w[c].x, w[c].y, w[c].z, w[c].w};
                if (s0 + c == 0) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) w0[q] = words[q];
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        const uint32_t raw = DT == RKV_F32 ? words[i] : ((i & 1) ? words[i >> 1] >> 16 : words[i >> 1] & 0xFFFFu);
                        const float x = __uint_as_float(widen<DT>(raw));
                        x0[i] = x; lo[i] = x; hi[i] = x;
                        thr[i] = __fadd_rn(atol, __fmul_rn(rtol, fabsf(x)));
                        chk = __fmaf_rn(x, 0.0f, chk);
                    }
                } else {
                    xacc |= (words[0] ^ w0[0]) | (words[1] ^ w0[1]) | (words[2] ^ w0[2]) | (words[3] ^ w0[3]);
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        const uint32_t raw = DT == RKV_F32 ? words[i] : ((i & 1) ? words[i >> 1] >> 16 : words[i >> 1] & 0xFFFFu);
                        const float x = __uint_as_float(widen<DT>(raw));
                        far |= !(fabsf(__fsub_rn(x, x0[i])) <= thr[i]);
                        lo[i] = fminf(lo[i], x);
                        hi[i] = fmaxf(hi[i], x);
                        chk = __fmaf_rn(x, 0.0f, chk);
                    }
                }
            }
        }
        if (chk == 0.0f) {
            a.differs |= (xacc ? 1u : 0u) | (far ? 2u : 0u);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                const float d = __fsub_rn(hi[i], lo[i]);
                if (d > a.spread) { a.spread = d; a.arg = v * VEC + i; }       // ascending index: the first maximum stays
            }
            continue;
        }
        // ---- general rule (a NaN or an infinity somewhere in the position), out of line ----
        a = general_position<DT>(mine, S, v, atol, rtol, a);
    }
    cross_block_end<DT>(a, mine, k, S, n, atol, rtol, partials);
}

// One warp per candidate: the lanes go through the blocks' partials in strides, then a shuffle tree
// (the merge is associative and commutative: integer sums, ors, value-then-first-index maxima).
__global__ void cross_finalize_kernel(const CrossPartial* __restrict__ partials, int K, int S, int blocks,
                                      float spread_lim, rkv_cross_stats* __restrict__ stats_out) {
    const int k = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (k >= K) return;                                  // whole warps leave together
    CrossAcc t;
    t.arg = RKV_NO_INDEX; t.n_nonfin = 0; t.spread = -1.0f; t.differs = 0;
    for (int b = lane; b < blocks; b += 32) {
        const CrossPartial p = partials[(size_t)k * blocks + b];
        CrossAcc q;
        q.arg = p.arg; q.n_nonfin = p.n_nonfin; q.spread = p.spread; q.differs = p.differs;
        merge(t, q);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        CrossAcc q;
        q.arg = __shfl_xor_sync(kFull, t.arg, off);
        q.n_nonfin = __shfl_xor_sync(kFull, t.n_nonfin, off);
        q.spread = __shfl_xor_sync(kFull, t.spread, off);
        q.differs = __shfl_xor_sync(kFull, t.differs, off);
        merge(t, q);
    }
    if (lane != 0) return;
    rkv_cross_stats st;
    memset(&st, 0, sizeof st);
    st.n_nonfinite = t.n_nonfin;
    st.argmax_spread = S >= 2 ? t.arg : RKV_NO_INDEX;
    st.max_spread = S >= 2 ? t.spread : -1.0f;
    uint32_t flags = 0;
    if (S >= 2 && !(t.differs & 1u)) flags |= RKV_CROSS_IDENTICAL;
    if (S >= 2 && !(t.differs & 2u)) flags |= RKV_CROSS_WITHIN_TOL;
    if (S >= 2 && t.spread >= 0.0f && t.spread < spread_lim) flags |= RKV_CROSS_LOW_SPREAD;
    if (t.n_nonfin) flags |= RKV_CROSS_NONFINITE;
    st.flags = flags;
    stats_out[k] = st;
}

// ---- copy of any input ------------------------------------------------------------------
// grid = (blocks per candidate, K).  differs[k]: bit m set once candidate k is known to
// differ from input m.
__global__ void __launch_bounds__(kCrossThreads)
copy_any_kernel(const void* const* __restrict__ inputs, int M, const void* const* __restrict__ cands,
                unsigned long long n_bytes, uint32_t* __restrict__ differs) {
    const int k = blockIdx.y;
    const unsigned char* c = reinterpret_cast<const unsigned char*>(cands[k]);
    const uint32_t all = (1u << M) - 1u;
    const unsigned long long n_vec = n_bytes / 16;
    __shared__ uint32_t s_known;
    uint32_t known = 0;                                  // inputs this block need not look at any more
    uint32_t found = 0;                                  // differences this thread has seen
    unsigned long long v = (unsigned long long)blockIdx.x * kCrossThreads + threadIdx.x;
    const unsigned long long stride = (unsigned long long)gridDim.x * kCrossThreads;
    // the trip count is the same for every thread of the block: barriers inside the loop
    const unsigned long long trips = (n_vec + stride - 1) / stride;
    for (unsigned long long it = 0; it < trips; ++it, v += stride) {
        if ((it & 7u) == 0u) {
            // every eighth round: publish what this block has found, pick up what others have
            const uint32_t warp_found = __reduce_or_sync(kFull, found);
            if ((threadIdx.x & 31) == 0 && warp_found) atomicOr(&differs[k], warp_found);
            found = 0;
            __syncthreads();
            if (threadIdx.x == 0) s_known = atomicOr(&differs[k], 0u);
            __syncthreads();
            known = s_known;
            if (known == all) break;                     // block-uniform
        }
        if (v < n_vec) {
            const uint4 cv = __ldcs(reinterpret_cast<const uint4*>(c) + v);
            for (int m = 0; m < M; ++m) {
                if ((known >> m) & 1u) continue;
                const uint4 iv = __ldg(reinterpret_cast<const uint4*>(inputs[m]) + v);
                if ((cv.x ^ iv.x) | (cv.y ^ iv.y) | (cv.z ^ iv.z) | (cv.w ^ iv.w)) found |= 1u << m;
            }
        }
    }
    // the bytes behind the last whole 16-byte piece
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (unsigned long long b = n_vec * 16; b < n_bytes; ++b)
            for (int m = 0; m < M; ++m)
                if (c[b] != reinterpret_cast<const unsigned char*>(inputs[m])[b]) found |= 1u << m;
    }
    if (found) atomicOr(&differs[k], found);
}

__global__ void copy_finalize_kernel(const uint32_t* __restrict__ differs, int K, int M, uint32_t* __restrict__ mask_out) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < K) mask_out[k] = ~differs[k] & ((1u << M) - 1u);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int blocks_per_candidate(uint64_t units, int K, int sms) {
    uint64_t want = (units + kCrossThreads - 1) / kCrossThreads;
    if (want < 1) want = 1;
    uint64_t cap = ((uint64_t)sms * kCrossBlocksPerSm + (uint64_t)K - 1) / (uint64_t)K;
    if (cap < 1) cap = 1;
    return (int)(want < cap ? want : cap);
}

}  // namespace
}  // namespace rkv

using namespace rkv;

extern "C" {

size_t rkv_cross_workspace_bytes(int K, int S) {
    if (K < 1 || K > kCrossMaxK || S < 1 || S > kCrossMaxSeeds) return 0;
    int sms = 0;
    if (current_num_sms(&sms) != RKV_OK) return 0;
    const size_t ptr_bytes = ((size_t)K * S * sizeof(void*) + 255) / 256 * 256;
    // at most sms * kCrossBlocksPerSm + K blocks in all
    return ptr_bytes + ((size_t)sms * kCrossBlocksPerSm + (size_t)K) * sizeof(CrossPartial);
}

int rkv_cross_seed(const void* const* outs, int K, int S, uint64_t n, int dtype, float atol, float rtol,
                   float spread_lim, rkv_cross_stats* stats_out, void* workspace, size_t workspace_bytes,
                   void* cuda_stream) {
    if (!outs || !stats_out || K < 1 || S < 1 || n < 1) return RKV_ERR_INVALID_ARG;
    if (dtype != RKV_F32 && dtype != RKV_BF16 && dtype != RKV_F16) return RKV_ERR_INVALID_ARG;
    if (!(atol >= 0.0f) || !(rtol >= 0.0f) || !(spread_lim >= 0.0f) || atol > 3.402823466e38f ||
        rtol > 3.402823466e38f)
        return RKV_ERR_INVALID_ARG;
    if (K > kCrossMaxK || S > kCrossMaxSeeds || n >= kMaxN) return RKV_ERR_UNSUPPORTED;
    for (int i = 0; i < K * S; ++i) {
        if (!outs[i]) return RKV_ERR_INVALID_ARG;
        if (!aligned16(outs[i])) return RKV_ERR_ALIGNMENT;
    }
    if (!workspace) return RKV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return RKV_ERR_ALIGNMENT;
    int sms = 0;
    int rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    if (workspace_bytes < rkv_cross_workspace_bytes(K, S)) return RKV_ERR_WORKSPACE;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    rc = refuse_capture(stream);                 // the pointer table travels from host memory of this call
    if (rc != RKV_OK) return rc;
    const size_t ptr_bytes = ((size_t)K * S * sizeof(void*) + 255) / 256 * 256;
    const void** d_ptrs = reinterpret_cast<const void**>(workspace);
    CrossPartial* partials = reinterpret_cast<CrossPartial*>(reinterpret_cast<unsigned char*>(workspace) + ptr_bytes);
    if (cudaMemcpyAsync(d_ptrs, outs, (size_t)K * S * sizeof(void*), cudaMemcpyHostToDevice, stream) != cudaSuccess) {
        cudaGetLastError();
        return RKV_ERR_CUDA;
    }
    const int vec = dtype == RKV_F32 ? 4 : 8;
    const int blocks = blocks_per_candidate(n / vec, K, sms);
    const dim3 grid((unsigned)blocks, (unsigned)K);
    // Up to eight seeds: all of a position's pieces in registers at once, eight 16-byte loads per thread in
    // flight (three blocks per SM for fp32; the 16-bit forms unpack twice the values and get the registers
    // of two blocks per SM, measured faster than three with spills).
#define RKV_CROSS_FEW(DT, CH, NP, MINB) \
    cross_seed_few_kernel<DT, CH, NP, MINB><<<grid, kCrossThreads, 0, stream>>>(d_ptrs, S, n, atol, rtol, partials)
#define RKV_CROSS_BY_S(DT, MINB)                              \
    do {                                                      \
        if (S <= 2) RKV_CROSS_FEW(DT, 2, 4, MINB);            \
        else if (S <= 4) RKV_CROSS_FEW(DT, 4, 2, MINB);       \
        else if (S <= 8) RKV_CROSS_FEW(DT, 8, 1, MINB);       \
        else cross_seed_kernel<DT><<<grid, kCrossThreads, 0, stream>>>(d_ptrs, S, n, atol, rtol, partials); \
    } while (0)
    if (dtype == RKV_F32) RKV_CROSS_BY_S(RKV_F32, 3);
    else if (dtype == RKV_BF16) RKV_CROSS_BY_S(RKV_BF16, 2);
    else RKV_CROSS_BY_S(RKV_F16, 2);
#undef RKV_CROSS_BY_S
#undef RKV_CROSS_FEW
    cross_finalize_kernel<<<(K + 3) / 4, 128, 0, stream>>>(partials, K, S, blocks, spread_lim, stats_out);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

size_t rkv_copy_workspace_bytes(int K, int M) {
    if (K < 1 || K > kCrossMaxK || M < 1 || M > kCopyMaxInputs) return 0;
    return ((size_t)(K + M) * sizeof(void*) + 255) / 256 * 256 + (size_t)K * sizeof(uint32_t);
}

int rkv_copy_of_inputs(const void* const* inputs, int M, const void* const* cands, int K, uint64_t n, int dtype,
                       uint32_t* copy_mask_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!inputs || !cands || !copy_mask_out || K < 1 || M < 1 || n < 1) return RKV_ERR_INVALID_ARG;
    if (dtype != RKV_F32 && dtype != RKV_BF16 && dtype != RKV_F16) return RKV_ERR_INVALID_ARG;
    if (K > kCrossMaxK || M > kCopyMaxInputs || n >= kMaxN) return RKV_ERR_UNSUPPORTED;
    for (int m = 0; m < M; ++m) {
        if (!inputs[m]) return RKV_ERR_INVALID_ARG;
        if (!aligned16(inputs[m])) return RKV_ERR_ALIGNMENT;
    }
    for (int k = 0; k < K; ++k) {
        if (!cands[k]) return RKV_ERR_INVALID_ARG;
        if (!aligned16(cands[k])) return RKV_ERR_ALIGNMENT;
    }
    if (!workspace) return RKV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return RKV_ERR_ALIGNMENT;
    if (workspace_bytes < rkv_copy_workspace_bytes(K, M)) return RKV_ERR_WORKSPACE;
    int sms = 0;
    int rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    rc = refuse_capture(stream);
    if (rc != RKV_OK) return rc;
    const size_t ptr_bytes = ((size_t)(K + M) * sizeof(void*) + 255) / 256 * 256;
    std::vector<const void*> table((size_t)(K + M));
    for (int m = 0; m < M; ++m) table[(size_t)m] = inputs[m];
    for (int k = 0; k < K; ++k) table[(size_t)(M + k)] = cands[k];
    const void** d_ptrs = reinterpret_cast<const void**>(workspace);
    uint32_t* differs = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(workspace) + ptr_bytes);
    if (cudaMemcpyAsync(d_ptrs, table.data(), table.size() * sizeof(void*), cudaMemcpyHostToDevice, stream) !=
            cudaSuccess ||
        cudaMemsetAsync(differs, 0, (size_t)K * sizeof(uint32_t), stream) != cudaSuccess) {
        cudaGetLastError();
        return RKV_ERR_CUDA;
    }
    const uint64_t n_bytes = n * (dtype == RKV_F32 ? 4u : 2u);
    const int blocks = blocks_per_candidate(n_bytes / 16, K, sms);
    copy_any_kernel<<<dim3((unsigned)blocks, (unsigned)K), kCrossThreads, 0, stream>>>(d_ptrs, M, d_ptrs + M, n_bytes,
                                                                                      differs);
    copy_finalize_kernel<<<(K + 127) / 128, 128, 0, stream>>>(differs, K, M, copy_mask_out);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

}  // extern "C"
