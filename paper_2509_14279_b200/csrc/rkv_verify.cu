// Fused single-pass verification kernel and its finalize kernel (sm_100a).
//
// Work decomposition.  Every tensor is cut into slabs (runs of at most ~12-24 K
// elements, a multiple of 128).  A persistent thread block takes slabs round
// robin.  For a slab it stages the reference (and the input tensor, when the
// copy-of-input flag is wanted) in shared memory ONCE -- by a bulk asynchronous
// copy (cp.async.bulk, completion on an mbarrier) or by regenerating it from its
// Philox stream -- and then streams the same slab of all K candidates from HBM
// with 128-bit read-once loads.  Candidate bytes are the only traffic that
// scales with K; the reference costs 1/K of it.
//
// Per element the fast path is: one subtraction, the tolerance product and sum
// (two separately rounded operations), a compare, a running maximum, a filter
// for the relative-error maximum, two xor/or accumulations for the loophole
// flags.  Anything non-finite makes the 4- or 8-element vector sum non-finite,
// which sends that vector down the general path; a slab whose reference holds a
// non-finite value uses the general path throughout.
//
// Reductions are deterministic: integer sums, lexicographic (value descending,
// index ascending) maxima, and a fixed-order fp64 sum.  No float atomics.
#include <type_traits>

#include "rkv_internal.h"
#include "rkv_philox.cuh"

namespace rkv {

namespace {

constexpr int kWarps = kThreads / 32;
constexpr int kGroupK = 2;        // candidates processed per pass over a reference vector
constexpr int kLoadsF32 = 2;      // 16-byte candidate loads per thread, candidate and batch (fp32)
constexpr int kLoadsBf16 = 2;     // same for bf16 candidates
constexpr uint32_t kFullMask = 0xFFFFFFFFu;

// ----------------------------------------------------------------------------
// shared-memory layout
// ----------------------------------------------------------------------------
constexpr int kOffMbar = 0;                               // 8 bytes
constexpr int kOffHintE = 64;
constexpr int kOffHintQ = kOffHintE + kHintK * 4;
constexpr int kOffHintF = kOffHintQ + kHintK * 4;
constexpr int kOffWarpPart = kOffHintF + kHintK * 4;      // 16-aligned
constexpr int kOffCandPtr = kOffWarpPart + kChunkK * kWarps * (int)sizeof(Partial);
constexpr int kOffCandFirst = kOffCandPtr + kPreK * 8;
constexpr int kOffDataRaw = kOffCandFirst + kPreK * 4;
constexpr int kOffData = (kOffDataRaw + 127) / 128 * 128;
static_assert(kOffWarpPart % 16 == 0, "warp partials must be 16-byte aligned");

// ----------------------------------------------------------------------------
// small PTX helpers
// ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count));
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t mbar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(mbar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bulk asynchronous copy global -> this block's shared memory; bytes is a
// multiple of 16, both addresses 16-byte aligned.  No multicast.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(mbar)
        : "memory");
}

// 128-bit read-once load of candidate data: no L1 allocation.
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ bool bits_finite(uint32_t b) { return (b & 0x7F800000u) != 0x7F800000u; }
__device__ __forceinline__ bool bits_inf(uint32_t b) { return (b & 0x7FFFFFFFu) == 0x7F800000u; }
__device__ __forceinline__ bool bits_nan(uint32_t b) { return (b & 0x7FFFFFFFu) > 0x7F800000u; }

// ----------------------------------------------------------------------------
// per-thread accumulators for one (slab, candidate)
// ----------------------------------------------------------------------------
struct Acc {
    uint32_t n_over;
    float emax; uint32_t eidx; float ethr;
    float qmax; uint32_t qidx; float qthr;
    double sum;
    uint32_t cacc, pacc;
    // four 8-bit counters (a thread sees < 256 elements of one slab):
    // byte 0 non-comparable, 1 NaN, 2 Inf, 3 infinity mismatch
    uint32_t rare;
};

__device__ __forceinline__ void acc_reset(Acc& a, float hint_e, float hint_q) {
    a.n_over = 0;
    a.emax = -1.0f; a.eidx = 0xFFFFFFFFu; a.ethr = hint_e;
    a.qmax = -1.0f; a.qidx = 0xFFFFFFFFu; a.qthr = hint_q;
    a.sum = 0.0;
    a.cacc = 0; a.pacc = 0;
    a.rare = 0;
}

// The comparison rule for one element, every case included.
__device__ __forceinline__ void elem_general(Acc& a, uint32_t cb, uint32_t rb, uint32_t idx, float atol,
                                             float rtol) {
    if (bits_nan(cb)) a.rare += 1u << 8;
    if (bits_inf(cb)) a.rare += 1u << 16;
    if (bits_finite(cb) && bits_finite(rb)) {
        const float c = __uint_as_float(cb), r = __uint_as_float(rb);
        const float e = fabsf(__fsub_rn(c, r));
        const float thr = __fadd_rn(atol, __fmul_rn(rtol, fabsf(r)));
        if (!(e <= thr)) a.n_over++;
        if (e > a.emax) { a.emax = e; a.eidx = idx; }
        if (r != 0.0f) {
            const float q = __fdiv_rn(e, fabsf(r));
            if (q > a.qmax) { a.qmax = q; a.qidx = idx; }
        }
        a.sum += (double)e;
    } else if (bits_inf(cb) && cb == rb) {
        a.rare += 1u;
    } else {
        a.rare += 1u;
        a.n_over++;
        if (bits_inf(cb) || bits_inf(rb)) a.rare += 1u << 24;
    }
}

// Per-vector values that depend on the reference only; computed once and used
// for every candidate of a group.
template <int VEC>
struct RefVec {
    uint32_t r[VEC];      // reference bits (fp32 patterns)
    float thr[VEC];       // atol + rtol*|r|, product and sum each rounded
    float minarp;         // smallest non-zero |r| of the vector, +inf if all are zero
};

template <int VEC>
__device__ __forceinline__ void refvec_prepare(RefVec<VEC>& rv, float atol, float rtol) {
    // |r| as an integer orders like the float; subtracting one wraps zero to the top
    uint32_t mn = 0xFFFFFFFFu;
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        const uint32_t ab = rv.r[j] & 0x7FFFFFFFu;
        rv.thr[j] = __fadd_rn(atol, __fmul_rn(rtol, __uint_as_float(ab)));
        mn = min(mn, ab - 1u);
    }
    rv.minarp = mn == 0xFFFFFFFFu ? __int_as_float(0x7F800000) : __uint_as_float(mn + 1u);
}

// The rarely taken parts of a vector step live out of line, so that the hot loop
// stays small enough for the instruction cache.  Arguments travel by value.
struct Best {
    float emax; uint32_t eidx;
    float qmax; uint32_t qidx;
};

template <int VEC>
struct VecErr {
    float e[VEC];
    uint32_t r[VEC];
};

// All values finite: new running maxima of |c - r| and of |c - r| / |r|.
template <int VEC>
__device__ __noinline__ Best rare_finite(Best b, float qthr, VecErr<VEC> x, uint32_t idx0) {
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        if (x.e[j] > b.emax) { b.emax = x.e[j]; b.eidx = idx0 + j; }
        const float ar = fabsf(__uint_as_float(x.r[j]));
        if (ar != 0.0f && x.e[j] > __fmul_rd(qthr, ar)) {
            const float q = __fdiv_rn(x.e[j], ar);
            if (q > b.qmax) { b.qmax = q; b.qidx = idx0 + j; }
        }
    }
    return b;
}

template <int VEC>
struct VecBits {
    uint32_t c[VEC];
    uint32_t r[VEC];
};

struct GenState {
    Best b;
    uint32_t n_over;
    uint32_t rare;
    double sum;
};

// A vector with a non-finite value somewhere: the general rule, element by element.
template <int VEC>
__device__ __noinline__ GenState rare_general(GenState g, VecBits<VEC> x, uint32_t idx0, float atol,
                                              float rtol) {
    Acc a;
    a.n_over = g.n_over; a.rare = g.rare; a.sum = g.sum;
    a.emax = g.b.emax; a.eidx = g.b.eidx; a.qmax = g.b.qmax; a.qidx = g.b.qidx;
    a.ethr = 0.0f; a.qthr = 0.0f; a.cacc = 0; a.pacc = 0;
#pragma unroll
    for (int j = 0; j < VEC; ++j) elem_general(a, x.c[j], x.r[j], idx0 + j, atol, rtol);
    g.n_over = a.n_over; g.rare = a.rare; g.sum = a.sum;
    g.b.emax = a.emax; g.b.eidx = a.eidx; g.b.qmax = a.qmax; g.b.qidx = a.qidx;
    return g;
}

// VEC consecutive elements of one candidate: bits c[] against the prepared
// reference vector; idx0 is the slab-local index of the first element.
//
// The common path only evaluates predicates; everything behind them sits in one
// rarely taken region:
//   !(s < s_limit)                          a non-finite value somewhere in the
//                                           vector (or a slab whose reference
//                                           has one: s_limit = -1) -> general rule
//   over : !(e <= thr)                      -> recount the vector
//   abs  : e > ethr, ethr >= running max    -> update (max, first index)
//   rel  : max e > RD(qthr * min|r|)        -> per element e > RD(qthr*|r|): divide, update
// RD is the product rounded toward -inf.  If fl(e/|r|) > qthr then, rounding
// being monotone, e/|r| > qthr exactly, so e > qthr*|r| >= RD(qthr*|r|): the
// test never skips an element that beats qthr.  Thresholds always come from
// elements with SMALLER indices (the thread's own earlier elements, earlier
// rounds of the warp, earlier slabs of the block), so a tie may be skipped: the
// first index keeps the maximum.
template <int VEC>
__device__ __forceinline__ void step_vec(Acc& a, const uint32_t (&c)[VEC], const RefVec<VEC>& rv,
                                         uint32_t idx0, float atol, float rtol, float s_limit) {
    float e[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j)
        e[j] = fabsf(__fsub_rn(__uint_as_float(c[j]), __uint_as_float(rv.r[j])));
    float s;
    if (VEC == 4) {
        s = __fadd_rn(__fadd_rn(e[0], e[1]), __fadd_rn(e[2], e[3]));
    } else {
        s = __fadd_rn(__fadd_rn(__fadd_rn(e[0], e[1]), __fadd_rn(e[2], e[3])),
                      __fadd_rn(__fadd_rn(e[4 % VEC], e[5 % VEC]), __fadd_rn(e[6 % VEC], e[7 % VEC])));
    }
    const bool finite = s < s_limit;
    bool rare = !finite;
    float m = e[0];
#pragma unroll
    for (int j = 1; j < VEC; ++j) m = fmaxf(m, e[j]);
    rare |= m > a.ethr;
    // vector-level relative-error filter: e_j > qthr*|r_j| for some j implies m > qthr*min|r|
    rare |= m > __fmul_rd(a.qthr, rv.minarp);
    // over-tolerance elements are common in failing candidates: counted unconditionally
#pragma unroll
    for (int j = 0; j < VEC; ++j)
        if (!(e[j] <= rv.thr[j]) && finite) a.n_over++;
    a.sum += (double)(finite ? s : 0.0f);
    if (rare) {
        if (!finite) {
            GenState g;
            g.b.emax = a.emax; g.b.eidx = a.eidx; g.b.qmax = a.qmax; g.b.qidx = a.qidx;
            g.n_over = a.n_over; g.rare = a.rare; g.sum = a.sum;
            VecBits<VEC> x;
#pragma unroll
            for (int j = 0; j < VEC; ++j) { x.c[j] = c[j]; x.r[j] = rv.r[j]; }
            g = rare_general<VEC>(g, x, idx0, atol, rtol);
            a.emax = g.b.emax; a.eidx = g.b.eidx; a.qmax = g.b.qmax; a.qidx = g.b.qidx;
            a.n_over = g.n_over; a.rare = g.rare; a.sum = g.sum;
        } else {
            Best b;
            b.emax = a.emax; b.eidx = a.eidx; b.qmax = a.qmax; b.qidx = a.qidx;
            VecErr<VEC> x;
#pragma unroll
            for (int j = 0; j < VEC; ++j) { x.e[j] = e[j]; x.r[j] = rv.r[j]; }
            b = rare_finite<VEC>(b, a.qthr, x, idx0);
            a.emax = b.emax; a.eidx = b.eidx; a.qmax = b.qmax; a.qidx = b.qidx;
        }
        a.ethr = fmaxf(a.ethr, a.emax);
        a.qthr = fmaxf(a.qthr, a.qmax);
    }
}

// ----------------------------------------------------------------------------
// warp reduction of the accumulators -> one Partial in shared memory
// ----------------------------------------------------------------------------
__device__ __forceinline__ void warp_reduce_store(const Acc& a, Partial* dst, int lane) {
    const uint32_t n_over = __reduce_add_sync(kFullMask, a.n_over);
    uint32_t n_noncomp = 0, n_nan = 0, n_inf = 0, n_infmis = 0;
    if (__any_sync(kFullMask, a.rare != 0)) {
        n_noncomp = __reduce_add_sync(kFullMask, a.rare & 0xFFu);
        n_nan = __reduce_add_sync(kFullMask, (a.rare >> 8) & 0xFFu);
        n_inf = __reduce_add_sync(kFullMask, (a.rare >> 16) & 0xFFu);
        n_infmis = __reduce_add_sync(kFullMask, a.rare >> 24);
    }
    // non-negative floats (and the -1 sentinel) order like their bit patterns as signed ints
    const int eb = __float_as_int(a.emax);
    const int ebm = __reduce_max_sync(kFullMask, eb);
    const uint32_t eidx = __reduce_min_sync(kFullMask, eb == ebm ? a.eidx : 0xFFFFFFFFu);
    const int qb = __float_as_int(a.qmax);
    const int qbm = __reduce_max_sync(kFullMask, qb);
    const uint32_t qidx = __reduce_min_sync(kFullMask, qb == qbm ? a.qidx : 0xFFFFFFFFu);
    const uint32_t cacc = __reduce_or_sync(kFullMask, a.cacc);
    const uint32_t pacc = __reduce_or_sync(kFullMask, a.pacc);
    double sum = a.sum;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(kFullMask, sum, off);
    if (lane == 0) {
        Partial p;
        p.n_over = n_over; p.n_noncomp = n_noncomp; p.n_nan = n_nan; p.n_inf = n_inf;
        p.n_infmis = n_infmis;
        p.mismatch = (cacc ? 1u : 0u) | (pacc ? 2u : 0u);
        p.emax = __int_as_float(ebm); p.eidx = eidx;
        p.qmax = __int_as_float(qbm); p.qidx = qidx;
        p.sum = sum;
        *dst = p;
    }
}

__device__ __forceinline__ void partial_merge(Partial& a, const Partial& b) {
    a.n_over += b.n_over; a.n_noncomp += b.n_noncomp; a.n_nan += b.n_nan; a.n_inf += b.n_inf;
    a.n_infmis += b.n_infmis; a.mismatch |= b.mismatch;
    if (b.emax > a.emax || (b.emax == a.emax && b.eidx < a.eidx)) { a.emax = b.emax; a.eidx = b.eidx; }
    if (b.qmax > a.qmax || (b.qmax == a.qmax && b.qidx < a.qidx)) { a.qmax = b.qmax; a.qidx = b.qidx; }
    a.sum += b.sum;
}

// ----------------------------------------------------------------------------
// staging of the reference / input slab
// ----------------------------------------------------------------------------

// Generate `len` elements starting at tensor element `start` (a multiple of 4)
// into shared memory, as fp32 bit patterns or as bf16 bit patterns.
template <bool OUT_BF16, bool ROUND_BF16>
__device__ __forceinline__ void stage_generated(unsigned char* dst, uint64_t seed, uint64_t stream_id,
                                                int dist, uint64_t start, uint32_t len, int tid) {
    const PhiloxKey key = philox_key(seed);
    const uint32_t n_blocks = (len + 3u) >> 2;
    for (uint32_t b = tid; b < n_blocks; b += kThreads) {
        float v[4];
        gen_block_dyn(dist, (start >> 2) + b, stream_id, key, v);
        if (OUT_BF16) {
            uint2 w;
            w.x = bf16_rne_bits(v[0]) | (bf16_rne_bits(v[1]) << 16);
            w.y = bf16_rne_bits(v[2]) | (bf16_rne_bits(v[3]) << 16);
            *reinterpret_cast<uint2*>(dst + (size_t)b * 8) = w;
        } else {
            uint4 w;
            w.x = __float_as_uint(v[0]); w.y = __float_as_uint(v[1]);
            w.z = __float_as_uint(v[2]); w.w = __float_as_uint(v[3]);
            if (ROUND_BF16) {
                w.x = bf16_rne_bits(v[0]) << 16; w.y = bf16_rne_bits(v[1]) << 16;
                w.z = bf16_rne_bits(v[2]) << 16; w.w = bf16_rne_bits(v[3]) << 16;
            }
            *reinterpret_cast<uint4*>(dst + (size_t)b * 16) = w;
        }
    }
}

// Element 0 of a tensor as an fp32 bit pattern (upcast), from memory or generated.
__device__ __forceinline__ uint32_t first_elem_bits(const void* ptr, int src, int dtype, uint64_t seed,
                                                    uint64_t stream_id, int dist) {
    if (src == RKV_SRC_POINTER) {
        if (dtype == RKV_BF16) return (uint32_t)(*reinterpret_cast<const uint16_t*>(ptr)) << 16;
        return *reinterpret_cast<const uint32_t*>(ptr);
    }
    const PhiloxKey key = philox_key(seed);
    float v[4];
    gen_block_dyn(dist, 0, stream_id, key, v);
    if (dtype == RKV_BF16) return bf16_rne_bits(v[0]) << 16;
    return __float_as_uint(v[0]);
}

template <bool B16>
__device__ __forceinline__ uint32_t smem_elem_bits(const unsigned char* base, uint32_t i) {
    if (B16) return (uint32_t)reinterpret_cast<const uint16_t*>(base)[i] << 16;
    return reinterpret_cast<const uint32_t*>(base)[i];
}

// ----------------------------------------------------------------------------
// one slab, all candidates
//   CB16   candidates (and the staged input) are bf16
//   RB16   the staged reference is bf16 (only a bf16 reference read from memory)
//   HAS_IN an input tensor is staged and the copy flag computed
// ----------------------------------------------------------------------------
template <bool CB16, bool RB16, bool HAS_IN, int KB, int U>
__device__ __forceinline__ bool process_item(const DevTensor& D, uint32_t item, int K, int k_begin, int k_end,
                                             Partial* __restrict__ partials, unsigned char* smem,
                                             uint32_t& phase, int32_t* status) {
    constexpr int VEC = CB16 ? 8 : 4;
    constexpr int CSZ = CB16 ? 2 : 4;
    constexpr int RSZ = RB16 ? 2 : 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t S = D.slab_elems;
    const uint32_t slab = item - D.first_item;
    const uint64_t start = (uint64_t)slab * S;
    const uint32_t len = (uint32_t)((D.n - start) < (uint64_t)S ? (D.n - start) : (uint64_t)S);
    const float atol = D.atol, rtol = D.rtol;

    unsigned char* ref_s = smem + kOffData;
    unsigned char* in_s = ref_s + (((size_t)S * RSZ + 127) & ~(size_t)127);
    const uint32_t mbar = smem_u32(smem + kOffMbar);
    float* hint_e = reinterpret_cast<float*>(smem + kOffHintE);
    float* hint_q = reinterpret_cast<float*>(smem + kOffHintQ);
    uint32_t* hint_f = reinterpret_cast<uint32_t*>(smem + kOffHintF);
    Partial* warp_part = reinterpret_cast<Partial*>(smem + kOffWarpPart);

    // ---- stage reference and input -------------------------------------------------
    uint32_t bulk_total = 0;
    const uint32_t ref_bulk = (D.ref_src == RKV_SRC_POINTER) ? (len * RSZ) & ~15u : 0u;
    const uint32_t in_bulk = (HAS_IN && D.input_src == RKV_SRC_POINTER) ? (len * CSZ) & ~15u : 0u;
    bulk_total = ref_bulk + in_bulk;
    if (tid == 0 && bulk_total) {
        mbar_expect_tx(mbar, bulk_total);
        const unsigned char* g = reinterpret_cast<const unsigned char*>(D.ref) + start * RSZ;
        for (uint32_t off = 0; off < ref_bulk; off += 32768u) {
            const uint32_t bytes = (ref_bulk - off) < 32768u ? (ref_bulk - off) : 32768u;
            bulk_g2s(smem_u32(ref_s + off), g + off, bytes, mbar);
        }
        if (in_bulk) {
            const unsigned char* gi = reinterpret_cast<const unsigned char*>(D.input) + start * CSZ;
            for (uint32_t off = 0; off < in_bulk; off += 32768u) {
                const uint32_t bytes = (in_bulk - off) < 32768u ? (in_bulk - off) : 32768u;
                bulk_g2s(smem_u32(in_s + off), gi + off, bytes, mbar);
            }
        }
    }
    if (D.ref_src == RKV_SRC_POINTER) {
        // the last (< 16) bytes of a ragged slab come by plain loads
        for (uint32_t i = ref_bulk / RSZ + tid; i < len; i += kThreads) {
            if (RB16)
                reinterpret_cast<uint16_t*>(ref_s)[i] =
                    reinterpret_cast<const uint16_t*>(D.ref)[start + i];
            else
                reinterpret_cast<uint32_t*>(ref_s)[i] =
                    reinterpret_cast<const uint32_t*>(D.ref)[start + i];
        }
    } else {
        if (D.ref_dtype == RKV_BF16)
            stage_generated<false, true>(ref_s, D.ref_seed, D.ref_stream, D.ref_dist, start, len, tid);
        else
            stage_generated<false, false>(ref_s, D.ref_seed, D.ref_stream, D.ref_dist, start, len, tid);
    }
    if (HAS_IN) {
        if (D.input_src == RKV_SRC_POINTER) {
            for (uint32_t i = in_bulk / CSZ + tid; i < len; i += kThreads) {
                if (CB16)
                    reinterpret_cast<uint16_t*>(in_s)[i] =
                        reinterpret_cast<const uint16_t*>(D.input)[start + i];
                else
                    reinterpret_cast<uint32_t*>(in_s)[i] =
                        reinterpret_cast<const uint32_t*>(D.input)[start + i];
            }
        } else {
            stage_generated<CB16, false>(in_s, D.in_seed, D.in_stream, D.in_dist, start, len, tid);
        }
    }
    bool waited_ok = true;
    if (bulk_total) {
        waited_ok = false;
        const long long t0 = clock64();
        for (uint32_t spin = 0; spin < (1u << 24); ++spin) {
            if (mbar_try_wait(mbar, phase)) { waited_ok = true; break; }
            if (clock64() - t0 > 2000000000LL) break;      // about a second
        }
        phase ^= 1u;
    }
    if (__syncthreads_or(!waited_ok)) {
        if (tid == 0) atomicExch(status, (int32_t)RKV_ERR_TIMEOUT);
        return false;
    }

    // ---- scan the staged slab: non-finite reference values, reference flags ---------
    const uint32_t r_first = first_elem_bits(D.ref, D.ref_src, D.ref_dtype, D.ref_seed, D.ref_stream,
                                             D.ref_dist);
    uint32_t r_nonfinite = 0, r_cacc = 0, r_pacc = 0;
    for (uint32_t i = tid; i < len; i += kThreads) {
        const uint32_t rb = smem_elem_bits<RB16>(ref_s, i);
        r_nonfinite |= bits_finite(rb) ? 0u : 1u;
        r_cacc |= rb ^ r_first;
        if (HAS_IN) r_pacc |= rb ^ smem_elem_bits<CB16>(in_s, i);
    }
    // __syncthreads_or is a boolean any(), one call per flag
    const bool general = __syncthreads_or((int)r_nonfinite) != 0;
    const bool ref_differs_first = __syncthreads_or(r_cacc != 0u) != 0;
    const bool ref_differs_input = HAS_IN ? (__syncthreads_or(r_pacc != 0u) != 0) : false;
    if (tid == 0 && k_begin == 0) {
        Partial p = {};
        p.mismatch = (ref_differs_first ? 1u : 0u) | (ref_differs_input ? 2u : 0u);
        p.emax = -1.0f; p.qmax = -1.0f; p.eidx = 0xFFFFFFFFu; p.qidx = 0xFFFFFFFFu;
        partials[(size_t)item * (K + 1) + K] = p;
    }

    // ---- stream the candidates -------------------------------------------------------
    // Candidates are taken KB at a time: the reference vector is read from shared
    // memory and prepared once per KB candidate vectors.  Each thread keeps U
    // 16-byte loads per candidate in flight: a register slot is reloaded with the
    // vector U rounds ahead right after it has been consumed.
    const uint32_t nvec = len / VEC;
    const uint32_t tail0 = nvec * VEC;
    // this thread's vectors are v = tid + i*kThreads, i < n_mine; the first lane of a
    // warp has the most (n_first), which gives the warp-uniform trip count
    const uint32_t n_mine = nvec > (uint32_t)tid ? (nvec - tid + kThreads - 1) / kThreads : 0u;
    const uint32_t tid_first = (uint32_t)tid & ~31u;
    const uint32_t n_first = nvec > tid_first ? (nvec - tid_first + kThreads - 1) / kThreads : 0u;
    const float s_limit = general ? -1.0f : __int_as_float(0x7F800000);
    const unsigned char* const* cptr_s = reinterpret_cast<const unsigned char* const*>(smem + kOffCandPtr);
    const uint32_t* cfirst_s = reinterpret_cast<const uint32_t*>(smem + kOffCandFirst);
    for (int kc0 = k_begin; kc0 < k_end; kc0 += kChunkK) {
        const int kc1 = (kc0 + kChunkK) < k_end ? (kc0 + kChunkK) : k_end;
        for (int kg = kc0; kg < kc1; kg += KB) {
            const unsigned char* cp[KB];
            uint32_t c_first[KB];
            Acc a[KB];
#pragma unroll
            for (int i = 0; i < KB; ++i) {
                // a group that runs past the chunk repeats its last candidate (result dropped)
                const int k = (kg + i) < kc1 ? (kg + i) : (kc1 - 1);
                if (k < kPreK) {
                    cp[i] = cptr_s[k];
                    c_first[i] = cfirst_s[k];
                } else {
                    cp[i] = reinterpret_cast<const unsigned char*>(D.cands[k]);
                    c_first[i] = CB16 ? (uint32_t)(*reinterpret_cast<const uint16_t*>(cp[i]))
                                      : *reinterpret_cast<const uint32_t*>(cp[i]);
                }
                if (CB16) c_first[i] = (c_first[i] & 0xFFFFu) * 0x10001u;
                cp[i] += start * CSZ + (size_t)tid * 16;
                acc_reset(a[i], k < kHintK ? hint_e[k] : -1.0f, k < kHintK ? hint_q[k] : -1.0f);
            }

            // The loophole flags are OR-reductions over the whole tensor: once an earlier
            // slab of this block has reported "differs" for every candidate of the group,
            // the xor/or work is skipped and the settled value reported again.
            uint32_t settled = 3u;
#pragma unroll
            for (int i = 0; i < KB; ++i) {
                const int k = (kg + i) < kc1 ? (kg + i) : (kc1 - 1);
                settled &= k < kHintK ? hint_f[k] : 0u;
            }
            constexpr uint32_t kWanted = HAS_IN ? 3u : 1u;
            const bool need_flags = (settled & kWanted) != kWanted;
            if (!need_flags) {
#pragma unroll
                for (int i = 0; i < KB; ++i) { a[i].cacc = 1u; a[i].pacc = 1u; }
            }

            // Two register buffers of U vectors per candidate.  All loads of a batch are
            // issued together, one batch ahead of their use, and consumed together.
            uint4 bufA[KB][U], bufB[KB][U];
            auto load_batch = [&](uint4 (&buf)[KB][U], const uint32_t r0) {
#pragma unroll
                for (int i = 0; i < KB; ++i)
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (r0 + u < n_mine)
                            buf[i][u] = ldg_stream(cp[i] + (size_t)(r0 + u) * (kThreads * 16));
            };

            // one vector position of this thread: round r (v = tid + r*kThreads)
            auto do_vector = [&](const uint4 (&buf)[KB][U], const int u, const uint32_t r) {
                const uint32_t v = (uint32_t)tid + r * kThreads;
                RefVec<VEC> rv;
                if (!CB16) {
                    if (RB16) {
                        const uint2 t = *reinterpret_cast<const uint2*>(ref_s + (size_t)v * 8);
                        rv.r[0] = t.x << 16; rv.r[1] = t.x & 0xFFFF0000u;
                        rv.r[2] = t.y << 16; rv.r[3] = t.y & 0xFFFF0000u;
                    } else {
                        const uint4 t = *reinterpret_cast<const uint4*>(ref_s + (size_t)v * 16);
                        rv.r[0] = t.x; rv.r[1] = t.y; rv.r[2] = t.z; rv.r[3] = t.w;
                    }
                } else {
                    if (RB16) {
                        const uint4 t = *reinterpret_cast<const uint4*>(ref_s + (size_t)v * 16);
                        const uint32_t rw[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            rv.r[(2 * q) % VEC] = rw[q] << 16;
                            rv.r[(2 * q + 1) % VEC] = rw[q] & 0xFFFF0000u;
                        }
                    } else {
                        const uint4 t0 = *reinterpret_cast<const uint4*>(ref_s + (size_t)v * 32);
                        const uint4 t1 = *reinterpret_cast<const uint4*>(ref_s + (size_t)v * 32 + 16);
                        rv.r[0] = t0.x; rv.r[1] = t0.y; rv.r[2] = t0.z; rv.r[3] = t0.w;
                        rv.r[4 % VEC] = t1.x; rv.r[5 % VEC] = t1.y;
                        rv.r[6 % VEC] = t1.z; rv.r[7 % VEC] = t1.w;
                    }
                }
                refvec_prepare<VEC>(rv, atol, rtol);
                if (need_flags) {
                    uint4 iv = make_uint4(0, 0, 0, 0);
                    if (HAS_IN) iv = *reinterpret_cast<const uint4*>(in_s + (size_t)v * 16);
#pragma unroll
                    for (int i = 0; i < KB; ++i) {
                        const uint4 w = buf[i][u];
                        a[i].cacc |= (w.x ^ c_first[i]) | (w.y ^ c_first[i]) | (w.z ^ c_first[i]) |
                                     (w.w ^ c_first[i]);
                        if (HAS_IN) a[i].pacc |= (w.x ^ iv.x) | (w.y ^ iv.y) | (w.z ^ iv.z) | (w.w ^ iv.w);
                    }
                }
#pragma unroll
                for (int i = 0; i < KB; ++i) {
                    const uint32_t w[4] = {buf[i][u].x, buf[i][u].y, buf[i][u].z, buf[i][u].w};
                    uint32_t c[VEC];
                    if (!CB16) {
                        c[0] = w[0]; c[1] = w[1]; c[2] = w[2]; c[3] = w[3];
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            c[(2 * q) % VEC] = w[q] << 16;
                            c[(2 * q + 1) % VEC] = w[q] & 0xFFFF0000u;
                        }
                    }
                    step_vec<VEC>(a[i], c, rv, v * VEC, atol, rtol, s_limit);
                }
            };

            auto compute_batch = [&](const uint4 (&buf)[KB][U], const uint32_t r0) {
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (r0 + u < n_mine) do_vector(buf, u, r0 + u);
                if (r0 < 2 * U) {
                    // share the running maxima across the warp: every element seen so far has
                    // a smaller index than every element of the batches to come
#pragma unroll
                    for (int i = 0; i < KB; ++i) {
                        a[i].ethr = fmaxf(a[i].ethr, __int_as_float(__reduce_max_sync(
                                                         kFullMask, __float_as_int(a[i].emax))));
                        a[i].qthr = fmaxf(a[i].qthr, __int_as_float(__reduce_max_sync(
                                                         kFullMask, __float_as_int(a[i].qmax))));
                    }
                }
            };

            // n_first rounds: what the first lane of the warp needs (the most), so that the
            // trip count is uniform across the warp
            load_batch(bufA, 0);
            for (uint32_t r0 = 0; r0 < n_first; r0 += 2 * U) {
                load_batch(bufB, r0 + U);
                compute_batch(bufA, r0);
                load_batch(bufA, r0 + 2 * U);
                if (r0 + U < n_first) compute_batch(bufB, r0 + U);
            }
            // ragged end of the tensor: fewer than VEC elements, one thread, element by element
            if (tid == 0) {
#pragma unroll
                for (int i = 0; i < KB; ++i) {
                    for (uint32_t e = tail0; e < len; ++e) {
                        uint32_t cb;
                        if (CB16) cb = (uint32_t)reinterpret_cast<const uint16_t*>(cp[i])[e] << 16;
                        else cb = reinterpret_cast<const uint32_t*>(cp[i])[e];
                        const uint32_t cf = CB16 ? (c_first[i] << 16) : c_first[i];
                        a[i].cacc |= cb ^ cf;
                        if (HAS_IN) a[i].pacc |= cb ^ smem_elem_bits<CB16>(in_s, e);
                        elem_general(a[i], cb, smem_elem_bits<RB16>(ref_s, e), e, atol, rtol);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < KB; ++i)
                if (kg + i < kc1) warp_reduce_store(a[i], &warp_part[(kg + i - kc0) * kWarps + warp], lane);
        }
        __syncthreads();
        if (tid < kc1 - kc0) {
            const int k = kc0 + tid;
            Partial p = warp_part[tid * kWarps];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) partial_merge(p, warp_part[tid * kWarps + w]);
            partials[(size_t)item * (K + 1) + k] = p;
            if (k < kHintK) {
                hint_e[k] = fmaxf(hint_e[k], p.emax);
                hint_q[k] = fmaxf(hint_q[k], p.qmax);
                hint_f[k] |= p.mismatch;
            }
        }
        __syncthreads();
    }
    return true;
}

__device__ __forceinline__ int variant_of(const DevTensor& D) {
    const int cb16 = D.cand_dtype == RKV_BF16;
    const int rb16 = D.ref_dtype == RKV_BF16 && D.ref_src == RKV_SRC_POINTER;
    const int has_in = D.input_src != RKV_SRC_NONE;
    return cb16 * 4 + rb16 * 2 + has_in;
}

// One kernel per storage variant (candidate dtype, staged reference dtype,
// input present), so that each gets its own register allocation.  A launch
// handles the slabs of every tensor of its variant; `n_items` counts them.
template <bool CB16, bool RB16, bool HAS_IN>
__global__ void __launch_bounds__(kThreads, kBlocksPerSm)
verify_kernel(const DevTensor* __restrict__ tensors, int T, int K, int k_begin, int k_end,
              uint32_t n_items, Partial* __restrict__ partials, int32_t* status) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kVariant = (CB16 ? 4 : 0) + (RB16 ? 2 : 0) + (HAS_IN ? 1 : 0);
    const int tid = threadIdx.x;
    if (tid == 0) {
        mbar_init(smem_u32(smem + kOffMbar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t phase = 0;
    int cur_t = -1;
    for (uint32_t it = blockIdx.x; it < n_items; it += gridDim.x) {
        // it-th slab among the tensors of this variant
        int t = 0;
        uint32_t slab = it;
        for (; t < T; ++t) {
            if (variant_of(tensors[t]) != kVariant) continue;
            const uint32_t ns = tensors[t].n_slabs;
            if (slab < ns) break;
            slab -= ns;
        }
        if (t >= T) return;
        const DevTensor D = tensors[t];
        const uint32_t item = D.first_item + slab;
        if (t != cur_t) {
            // per-tensor block state: thresholds carried from earlier slabs, and the
            // candidates' base pointers and first elements (the constant-output test)
            float* hint_e = reinterpret_cast<float*>(smem + kOffHintE);
            float* hint_q = reinterpret_cast<float*>(smem + kOffHintQ);
            const unsigned char** cptr_s = reinterpret_cast<const unsigned char**>(smem + kOffCandPtr);
            uint32_t* cfirst_s = reinterpret_cast<uint32_t*>(smem + kOffCandFirst);
            __syncthreads();
            uint32_t* hint_f = reinterpret_cast<uint32_t*>(smem + kOffHintF);
            for (int i = tid; i < kHintK; i += kThreads) { hint_e[i] = -1.0f; hint_q[i] = -1.0f; hint_f[i] = 0u; }
            for (int k = tid; k < K && k < kPreK; k += kThreads) {
                const unsigned char* p = reinterpret_cast<const unsigned char*>(D.cands[k]);
                cptr_s[k] = p;
                cfirst_s[k] = CB16 ? (uint32_t)(*reinterpret_cast<const uint16_t*>(p))
                                   : *reinterpret_cast<const uint32_t*>(p);
            }
            cur_t = t;
        }
        if (!process_item<CB16, RB16, HAS_IN, kGroupK, CB16 ? kLoadsBf16 : kLoadsF32>(
                D, item, K, k_begin, k_end, partials, smem, phase, status))
            return;
    }
}

// ----------------------------------------------------------------------------
// finalize: merge the per-slab partials of each (candidate, tensor) in a fixed
// order, derive flags and verdict, and the joint verdict over tensors
// ----------------------------------------------------------------------------
constexpr int kFinThreads = 128;

struct Wide {
    uint64_t n_over, n_noncomp, n_nan, n_inf, n_infmis;
    uint64_t eidx, qidx;
    double sum;
    float emax, qmax;
    uint32_t mismatch;
};

__device__ __forceinline__ void wide_merge(Wide& a, const Wide& b) {
    a.n_over += b.n_over; a.n_noncomp += b.n_noncomp; a.n_nan += b.n_nan; a.n_inf += b.n_inf;
    a.n_infmis += b.n_infmis; a.mismatch |= b.mismatch;
    if (b.emax > a.emax || (b.emax == a.emax && b.eidx < a.eidx)) { a.emax = b.emax; a.eidx = b.eidx; }
    if (b.qmax > a.qmax || (b.qmax == a.qmax && b.qidx < a.qidx)) { a.qmax = b.qmax; a.qidx = b.qidx; }
    a.sum += b.sum;
}

__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(const DevTensor* __restrict__ tensors, int T, int K, const Partial* __restrict__ partials,
                rkv_stats* __restrict__ stats_out, uint32_t* __restrict__ joint_pass) {
    __shared__ Wide red[kFinThreads];
    __shared__ uint32_t ref_mismatch_s;
    const int k = blockIdx.x, tid = threadIdx.x;
    uint32_t all_pass = 1;
    for (int t = 0; t < T; ++t) {
        const DevTensor D = tensors[t];
        Wide w = {};
        w.emax = -1.0f; w.qmax = -1.0f; w.eidx = RKV_NO_INDEX; w.qidx = RKV_NO_INDEX;
        uint32_t ref_mm = 0;
        for (uint32_t s = tid; s < D.n_slabs; s += kFinThreads) {
            const size_t row = (size_t)(D.first_item + s) * (K + 1);
            const Partial p = partials[row + k];
            Wide b;
            b.n_over = p.n_over; b.n_noncomp = p.n_noncomp; b.n_nan = p.n_nan; b.n_inf = p.n_inf;
            b.n_infmis = p.n_infmis; b.mismatch = p.mismatch;
            const uint64_t base = (uint64_t)s * D.slab_elems;
            b.emax = p.emax; b.eidx = p.emax < 0.0f ? RKV_NO_INDEX : base + p.eidx;
            b.qmax = p.qmax; b.qidx = p.qmax < 0.0f ? RKV_NO_INDEX : base + p.qidx;
            b.sum = p.sum;
            wide_merge(w, b);
            ref_mm |= partials[row + K].mismatch;
        }
        red[tid] = w;
        if (tid == 0) ref_mismatch_s = 0;
        __syncthreads();
        if (ref_mm) atomicOr(&ref_mismatch_s, ref_mm);
        for (int off = kFinThreads / 2; off > 0; off >>= 1) {
            if (tid < off) {
                Wide a = red[tid];
                wide_merge(a, red[tid + off]);
                red[tid] = a;
            }
            __syncthreads();
        }
        if (tid == 0) {
            const Wide r = red[0];
            const uint32_t ref_mismatch = ref_mismatch_s;
            rkv_stats st;
            st.n_over_tol = r.n_over;
            st.n_nan = r.n_nan;
            st.n_inf = r.n_inf;
            st.n_inf_mismatch = r.n_infmis;
            st.n_comparable = D.n - r.n_noncomp;
            st.argmax_abs_err = r.emax < 0.0f ? RKV_NO_INDEX : r.eidx;
            st.argmax_rel_err = r.qmax < 0.0f ? RKV_NO_INDEX : r.qidx;
            st.sum_abs_err = r.sum;
            st.max_abs_err = r.emax < 0.0f ? 0.0f : r.emax;
            st.max_rel_err = r.qmax < 0.0f ? 0.0f : r.qmax;
            st.mean_abs_err = st.n_comparable ? (float)(r.sum / (double)st.n_comparable) : 0.0f;
            st.reserved = 0;
            const bool has_in = D.input_src != RKV_SRC_NONE;
            uint32_t flags = 0;
            if (!(r.mismatch & 1u)) flags |= RKV_FLAG_CAND_CONST;
            if (has_in && !(r.mismatch & 2u)) flags |= RKV_FLAG_CAND_COPY_OF_INPUT;
            if (!(ref_mismatch & 1u)) flags |= RKV_FLAG_REF_CONST;
            if (has_in && !(ref_mismatch & 2u)) flags |= RKV_FLAG_REF_COPY_OF_INPUT;
            if (r.n_nan) flags |= RKV_FLAG_HAS_NAN;
            if (r.n_inf) flags |= RKV_FLAG_HAS_INF;
            uint32_t verdict = 0;
            if (r.n_over) verdict |= RKV_FAIL_TOL;
            if (r.n_nan) verdict |= RKV_FAIL_NAN;
            if (r.n_infmis) verdict |= RKV_FAIL_INF_MISMATCH;
            if ((flags & RKV_FLAG_CAND_CONST) && !(flags & RKV_FLAG_REF_CONST) && D.n > 1)
                verdict |= RKV_FAIL_LOOPHOLE_CONST;
            if ((flags & RKV_FLAG_CAND_COPY_OF_INPUT) && !(flags & RKV_FLAG_REF_COPY_OF_INPUT))
                verdict |= RKV_FAIL_LOOPHOLE_COPY;
            st.flags = flags;
            st.verdict = verdict;
            stats_out[(size_t)k * T + t] = st;
            if (verdict) all_pass = 0;
        }
        __syncthreads();
    }
    if (tid == 0 && joint_pass) joint_pass[k] = all_pass;
}

}  // namespace

template <bool CB16, bool RB16, bool HAS_IN>
static int launch_variant(const DevTensor* d_tensors, int T, int K, int k_begin, int k_end, uint32_t n_items,
                          int num_sms, Partial* partials, int32_t* status, cudaStream_t stream) {
    const int smem = kOffData + kSmemDataBudget + 256;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RKV_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(verify_kernel<CB16, RB16, HAS_IN>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return RKV_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    uint32_t grid = (uint32_t)num_sms * kBlocksPerSm;
    if (grid > n_items) grid = n_items;
    verify_kernel<CB16, RB16, HAS_IN><<<grid, kThreads, smem, stream>>>(d_tensors, T, K, k_begin, k_end,
                                                                      n_items, partials, status);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

int launch_verify(const DevTensor* d_tensors, int T, int K, int k_begin, int k_end,
                  const uint32_t variant_items[8], int num_sms, Partial* partials, int32_t* status,
                  cudaStream_t stream) {
    int rc = RKV_OK;
    for (int v = 0; v < 8 && rc == RKV_OK; ++v) {
        const uint32_t n = variant_items[v];
        if (!n) continue;
#define RKV_LAUNCH(CB, RB, IN) \
    launch_variant<CB, RB, IN>(d_tensors, T, K, k_begin, k_end, n, num_sms, partials, status, stream)
        switch (v) {
            case 0: rc = RKV_LAUNCH(false, false, false); break;
            case 1: rc = RKV_LAUNCH(false, false, true); break;
            case 2: rc = RKV_LAUNCH(false, true, false); break;
            case 3: rc = RKV_LAUNCH(false, true, true); break;
            case 4: rc = RKV_LAUNCH(true, false, false); break;
            case 5: rc = RKV_LAUNCH(true, false, true); break;
            case 6: rc = RKV_LAUNCH(true, true, false); break;
            default: rc = RKV_LAUNCH(true, true, true); break;
        }
#undef RKV_LAUNCH
    }
    return rc;
}

int launch_finalize(const DevTensor* d_tensors, int T, int K, const Partial* partials,
                    rkv_stats* stats_out, uint32_t* joint_pass, cudaStream_t stream) {
    finalize_kernel<<<K, kFinThreads, 0, stream>>>(d_tensors, T, K, partials, stats_out, joint_pass);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

}  // namespace rkv
