// Fused single-pass verification kernel and its finalize kernel (sm_100a).
//
// Work decomposition.  A tensor is cut into tiles of 14336 candidate bytes (3584 fp32 or
// 7168 bf16 elements); the K candidates into parts of at most 64.  A work item is
// (tensor, group, part, tile).  A persistent thread block starts with the item of its own
// number and then draws further items from a ticket counter.  It has two roles:
//
//   * one producer warp: a single thread issues bulk asynchronous copies
//     (cp.async.bulk, completion counted on an mbarrier) that bring, for the
//     item, the reference tile and then the same tile of every candidate of the
//     part into a ring of shared-memory stages.  Several stages are in flight,
//     so the copies of later candidates overlap the comparison of earlier ones;
//   * seven consumer warps: each thread owns 64 bytes of every candidate tile (16 fp32
//     or 32 bf16 elements).  It keeps their reference values (and, for fp32 candidates,
//     the tolerance thresholds) IN REGISTERS for the whole item and meets every
//     candidate tile as it lands in the ring.
//
// Candidate bytes are read from HBM exactly once; the reference once per part.
// When the reference is "generated" the threads regenerate their values from
// the Philox stream instead of reading them (fused generate + verify).
//
// Per element the common path is one subtraction, one running maximum and one
// addition (bf16 candidates: one fused multiply-add and one more maximum, see
// process_candidate_b16).  Counting the elements over tolerance, locating maxima,
// dividing for the relative error and everything about non-finite values sit behind
// tests evaluated once per thread, candidate and tile and one warp vote:
//   m > min thr              some element may be over tolerance  -> count them
//   !(sum < inf)             a non-finite value                  -> general rule
//   m beats/ties the hint    a new maximum is possible           -> locate it
// The hints are running maxima that all blocks publish in global memory with
// their tile number.  A hint only ever lets a thread skip elements that cannot
// be the first maximum (see Hint), so results do not depend on when a hint
// becomes visible.
//
// Reductions are deterministic: integer sums, lexicographic (value descending,
// index ascending) maxima, fixed-order floating-point sums.  No float atomics.
#include "rkv_internal.h"
#include "rkv_philox.cuh"

namespace rkv {

namespace {

constexpr uint32_t kFullMask = 0xFFFFFFFFu;
constexpr float kInf = __builtin_huge_valf();
enum : uint32_t { kNoItem = 0xFFFFFFFFu };     // the producer's "no more items" mark

// ----------------------------------------------------------------------------
// shared-memory layout (dynamic)
// ----------------------------------------------------------------------------
// Per (warp, candidate of the part) running result.
struct __align__(16) WarpRec {
    float emax; uint32_t etile;
    float qmax; uint32_t qtile;
    uint32_t offs;           // eoff | qoff << 16 : element offsets inside their tiles
    uint32_t n_over;
    double sum;
};
static_assert(sizeof(WarpRec) == 32, "WarpRec layout");

// Per candidate of the part, rebuilt from the published state at the start of an item.
// With (te, te_tile) the published maximum of |c - r| and the tile it was found in, an
// element can still be the FIRST maximum only if it is larger, or equal and in a tile at or
// before te_tile.  For the item's tile that is one comparison against te_x:
//     te_x = tile <= te_tile ? (largest float below te) : te          (-1 if nothing published)
// tq_x is the same for the relative error.
struct __align__(16) Hint {
    float te_x;
    float tq_x;
    uint32_t settled;                // bit0: known to differ from element 0; bit1: from the input
    uint32_t first;                  // element 0 of the candidate as an fp32 bit pattern
};
static_assert(sizeof(Hint) == 16, "Hint layout");

constexpr int kOffFull = 0;                                   // kStages mbarriers
constexpr int kOffEmpty = kOffFull + 8 * kStages;
constexpr int kOffAbort = kOffEmpty + 8 * kStages;         // uint32
constexpr int kOffRefState = kOffAbort + 16;                  // 2 x uint32 settled bits of the reference (item parity)
constexpr int kOffIds = kOffRefState + 8;                     // kStages x uint32: item id that starts in a stage
constexpr int kOffPtrC = 256;                                 // consumer copy of the pointers
constexpr int kOffPtrP = kOffPtrC + kPartK * 8;               // producer copy
constexpr int kOffHint = kOffPtrP + kPartK * 8;               // two tables (item parity)
constexpr int kOffRec = kOffHint + 2 * kPartK * (int)sizeof(Hint);
constexpr int kOffStage = (kOffRec + kConsumerWarps * kPartK * (int)sizeof(WarpRec) + 1023) / 1024 * 1024;
constexpr int kSmemBytes = kOffStage + kStages * kStageBytes;
static_assert(kOffPtrC >= kOffIds + 4 * kStages, "layout");
static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two blocks per SM must fit");

// Geometry of a tile.  A thread owns 64 bytes of each candidate tile, so a candidate tile
// always fills exactly one ring stage: 16 fp32 elements or 32 bf16 elements.  Their
// reference values stay in registers for the whole item.  With fp32 candidates the
// tolerance thresholds do too; with bf16 candidates they are recomputed in the rare case
// that needs them (see process_candidate_b16).
template <bool CB16>
struct Geo {
    static constexpr int E = CB16 ? 32 : 16;            // elements per thread
    static constexpr int VEC = CB16 ? 8 : 4;            // elements per 16-byte piece
    static constexpr int NW = 16;                       // 32-bit words per thread and candidate tile
    static constexpr int kTile = kConsumers * E;        // elements per tile
};

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

__device__ __forceinline__ void mbar_arrive(uint32_t mbar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
}

// Arrive from the threads for which `on` holds, as one predicated instruction (no branch).
__device__ __forceinline__ void mbar_arrive_if(uint32_t mbar, bool on) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(mbar), "r"((uint32_t)on)
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

// Bounded wait.  Returns false when the wait ran out (about a second) or when
// another thread of the block has already given up; the block then drains: every
// later wait returns at once, all barriers are still reached, and the status
// word tells the host that the results are void.
__device__ __noinline__ bool mbar_wait_slow(uint32_t mbar, uint32_t parity, volatile uint32_t* abort_flag) {
    const long long t0 = clock64();
    for (uint32_t spin = 0; spin < (1u << 26); ++spin) {
        if (mbar_try_wait(mbar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > 2000000000LL) break;
    }
    *abort_flag = 1u;
    return false;
}

__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity, volatile uint32_t* abort_flag) {
    if (mbar_try_wait(mbar, parity)) return true;
    return mbar_wait_slow(mbar, parity, abort_flag);
}

// Bulk asynchronous copy global -> this block's shared memory; bytes is a
// multiple of 16, both addresses 16-byte aligned.  No multicast.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(mbar)
        : "memory");
}

// Barrier among the consumer threads only (the producer warp never joins).
__device__ __forceinline__ void consumer_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
}

// The same barrier, returning whether any consumer thread passed a non-zero value.
__device__ __forceinline__ bool consumer_sync_or(uint32_t v) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "barrier.red.or.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"(v), "n"(kConsumers)
        : "memory");
    return out != 0;
}

__device__ __forceinline__ bool bits_finite(uint32_t b) { return (b & 0x7F800000u) != 0x7F800000u; }
__device__ __forceinline__ bool bits_inf(uint32_t b) { return (b & 0x7FFFFFFFu) == 0x7F800000u; }
__device__ __forceinline__ bool bits_nan(uint32_t b) { return (b & 0x7FFFFFFFu) > 0x7F800000u; }

__device__ __forceinline__ uint32_t ld_elem_bits(const void* base, int dtype, uint64_t i) {
    if (dtype == RKV_BF16) return (uint32_t)reinterpret_cast<const uint16_t*>(base)[i] << 16;
    return reinterpret_cast<const uint32_t*>(base)[i];
}

// ----------------------------------------------------------------------------
// work items
// ----------------------------------------------------------------------------
struct Item {
    int t;
    uint32_t group;          // 0 = A (leading tiles, small parts), 1 = B, 2 = C (last tiles, small parts)
    uint32_t part, tile;     // tile is the tensor-wide tile index
    uint32_t n_parts;        // candidate parts of this group
    uint32_t first_item;     // first item of this (tensor, group) in this launch
    uint32_t n_items;        // items of this (tensor, group)
};

// Item `id` of this launch among the tensors of `variant`; false past the end.
__device__ __forceinline__ bool decode_item(const DevTensor* __restrict__ tensors, int T, uint32_t variant,
                                            uint32_t k_count, uint32_t id, Item& it) {
    uint32_t base = 0;
    for (uint32_t g = 0; g < 3; ++g) {
        for (int t = 0; t < T; ++t) {
            if (tensors[t].variant != variant) continue;
            const uint32_t warm = tensors[t].warm_tiles, tail = tensors[t].tail_tiles;
            const uint32_t nt = group_tiles(g, tensors[t].n_tiles, warm, tail);
            if (nt == 0) continue;
            const uint32_t parts = group_parts(g, nt, k_count, gridDim.x, tensors[t].tail_div);
            const uint32_t cnt = nt * parts;
            if (id - base < cnt) {
                it.t = t;
                it.group = g;
                it.part = (id - base) / nt;
                it.tile = (id - base) % nt + group_first_tile(g, tensors[t].n_tiles, warm, tail);
                it.n_parts = parts;
                it.first_item = base;
                it.n_items = cnt;
                return true;
            }
            base += cnt;
        }
    }
    return false;
}

// ----------------------------------------------------------------------------
// producer warp: feeds the ring
// ----------------------------------------------------------------------------
struct Ring {
    uint32_t full0, empty0;      // shared-memory addresses of the first full / empty mbarrier
    uint32_t stage0;             // shared-memory address of stage 0
    volatile uint32_t* abort_flag;
};

template <bool CB16, bool RB16>
__device__ __forceinline__ void producer_loop(const DevTensor* __restrict__ tensors, int T, int k_begin,
                                              int k_end, uint32_t n_items, unsigned char* smem,
                                              const Ring& ring, WorkspaceHeader* header) {
    constexpr uint32_t CSZ = CB16 ? 2 : 4, RSZ = RB16 ? 2 : 4;
    constexpr uint32_t kVariant = (CB16 ? 2u : 0u) + (RB16 ? 1u : 0u);
    constexpr uint32_t kTile = Geo<CB16>::kTile;
    constexpr uint32_t kRefStages = (CB16 && !RB16) ? 2 : 1;      // an fp32 tile under bf16 candidates
    const int lane = threadIdx.x & 31;
    const unsigned char** ptrs = reinterpret_cast<const unsigned char**>(smem + kOffPtrP);
    volatile uint32_t* ids = reinterpret_cast<volatile uint32_t*>(smem + kOffIds);
    uint32_t n_issued = 0;
    int cur_t = -1;
    uint32_t cur_part = 0xFFFFFFFFu;

    // mark: the id of the item that starts in this stage (kNoItem at the very end), else none
    auto issue = [&](const unsigned char* src, uint32_t bytes, bool starts_item, uint32_t id) {
        const uint32_t s = n_issued % kStages;
        const uint32_t ph = (n_issued / kStages) & 1u;
        // the stage is free once every consumer warp has released its previous use
        mbar_wait(ring.empty0 + 8 * s, ph ^ 1u, ring.abort_flag);
        if (starts_item) ids[s] = id;          // ordered before the arrive below
        if (bytes) {
            mbar_expect_tx(ring.full0 + 8 * s, bytes);
            bulk_g2s(ring.stage0 + s * kStageBytes, src, bytes, ring.full0 + 8 * s);
        } else {
            mbar_arrive(ring.full0 + 8 * s);
        }
        ++n_issued;
    };

    // Every block starts with item blockIdx.x; after that lane 0 draws tickets, one ahead of
    // the item it is issuing, so that the atomic's latency is never waited for.
    uint32_t id = blockIdx.x;
    for (;;) {
        id = __shfl_sync(kFullMask, id, 0);
        if (id >= n_items) break;
        uint32_t next_id = 0;
        if (lane == 0) next_id = gridDim.x + atomicAdd(&header->next_ticket, 1u);
        Item it;
        if (!decode_item(tensors, T, kVariant, (uint32_t)(k_end - k_begin), id, it)) break;
        const DevTensor& D = tensors[it.t];
        const uint32_t k_count = (uint32_t)(k_end - k_begin);
        const int k0 = k_begin + (int)part_begin(it.part, it.n_parts, k_count);
        const int k1 = k_begin + (int)part_begin(it.part + 1, it.n_parts, k_count);
        const uint32_t part_key = (it.group << 30) | it.part;
        if (it.t != cur_t || part_key != cur_part) {
            __syncwarp();
            for (int k = k0 + lane; k < k1; k += 32)
                ptrs[k - k0] = reinterpret_cast<const unsigned char*>(D.cands[k]);
            __syncwarp();
            cur_t = it.t;
            cur_part = part_key;
        }
        if (lane == 0) {
            const uint64_t start = (uint64_t)it.tile * kTile;
            const uint32_t len = (uint32_t)min((uint64_t)kTile, D.n - start);
            bool first = true;
            if (D.ref_src == RKV_SRC_POINTER) {
                const unsigned char* src = reinterpret_cast<const unsigned char*>(D.ref) + start * RSZ;
                const uint32_t rbytes = (len * RSZ) & ~15u;
                for (uint32_t rs = 0; rs < kRefStages; ++rs) {
                    const uint32_t lo = rs * kStageBytes;
                    const uint32_t b = rbytes > lo ? min(rbytes - lo, (uint32_t)kStageBytes) : 0u;
                    issue(src + lo, b, first, id);
                    first = false;
                }
            }
            const uint32_t cbytes = (len * CSZ) & ~15u;
            for (int k = k0; k < k1; ++k) {
                issue(ptrs[k - k0] + start * CSZ, cbytes, first, id);
                first = false;
            }
        }
        id = next_id;
    }
    if (lane == 0) {
        issue(nullptr, 0u, true, kNoItem);                     // tell the consumers to stop
        // the last block to get here clears the ticket counter for the next launch
        __threadfence();
        if (atomicAdd(&header->blocks_done, 1u) == gridDim.x - 1u) {
            header->next_ticket = 0u;
            header->blocks_done = 0u;
        }
    }
    // A block that gave up must not retire with copies still landing in its shared
    // memory: wait (bounded) for the copies issued last.
    if (lane == 0 && *ring.abort_flag) {
        const uint32_t pending = n_issued < kStages ? n_issued : kStages;
        for (uint32_t i = 0; i < pending; ++i) {
            const uint32_t q = n_issued - 1 - i;
            const uint32_t s = q % kStages, ph = (q / kStages) & 1u;
            const long long t0 = clock64();
            for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
                if (mbar_try_wait(ring.full0 + 8 * s, ph)) break;
                if (clock64() - t0 > 200000000LL) break;
            }
        }
    }
}

// ----------------------------------------------------------------------------
// consumer side: per-thread view of a tile
// ----------------------------------------------------------------------------
// A thread owns E elements of the tile (see Geo) as vectors of VEC elements
// (one 16-byte piece of a candidate each): vector jv of thread tid is vector
// jv * 224 + tid of the tile.  Element j = jv * VEC + i of the thread has the
// tile offset below; offsets grow with j.
template <int VEC>
__device__ __forceinline__ uint32_t elem_off(int j, int tid) {
    return (uint32_t)(((j / VEC) * kConsumers + tid) * VEC + (j % VEC));
}

// What a thread keeps for the whole item.
template <bool CB16>
struct RefRegs;

template <>
struct RefRegs<false> {
    float r[16];       // reference values
    float thr[16];     // atol + rtol*|r|, product and sum each rounded
    float thr_min;     // smallest threshold of the thread's elements
    float minarp;      // smallest non-zero |r|, +inf if all are zero
    bool general;      // a non-finite reference value: element-by-element rule
};

template <>
struct RefRegs<true> {
    float r[32];          // reference values
    float atol, rtol;     // (thresholds are recomputed where they are needed)
    float thr_min;        // smallest threshold of the thread's elements
    bool general;         // a non-finite reference value: element-by-element rule
    bool warp_has_zero;   // some thread of the warp holds a reference value of exactly 0
};

// The comparison rule for one element, every case included.
struct LaneGen {
    uint32_t n_over, n_noncomp, n_nan, n_inf, n_infmis;
    float emax; uint32_t eoff;
    float qmax; uint32_t qoff;
    double sum;
};

__device__ __forceinline__ void elem_general(LaneGen& a, uint32_t cb, uint32_t rb, uint32_t off, float atol,
                                             float rtol) {
    if (bits_nan(cb)) a.n_nan++;
    if (bits_inf(cb)) a.n_inf++;
    if (bits_finite(cb) && bits_finite(rb)) {
        const float c = __uint_as_float(cb), r = __uint_as_float(rb);
        const float e = fabsf(__fsub_rn(c, r));
        const float thr = __fadd_rn(atol, __fmul_rn(rtol, fabsf(r)));
        if (!(e <= thr)) a.n_over++;
        if (e > a.emax) { a.emax = e; a.eoff = off; }
        if (r != 0.0f) {
            const float q = __fdiv_rn(e, fabsf(r));
            if (q > a.qmax) { a.qmax = q; a.qoff = off; }
        }
        a.sum += (double)e;
    } else if (bits_inf(cb) && cb == rb) {
        a.n_noncomp++;
    } else {
        a.n_noncomp++;
        a.n_over++;
        if (bits_inf(cb) || bits_inf(rb)) a.n_infmis++;
    }
}

// Four consecutive elements (tile offset off0, a multiple of 4) of a generated
// tensor, as fp32 bit patterns; bf16 == true rounds them to bf16 first.
__device__ __forceinline__ void gen_group(uint64_t seed, uint64_t stream_id, int dist, uint64_t start,
                                          uint32_t off0, bool bf16, uint32_t out[4]) {
    const PhiloxKey key = philox_key(seed);
    float v[4];
    gen_block_dyn(dist, (start + off0) >> 2, stream_id, key, v);
#pragma unroll
    for (int i = 0; i < 4; ++i)
        out[i] = bf16 ? (bf16_rne_bits(v[i]) << 16) : __float_as_uint(v[i]);
}

// Four consecutive elements of the input tensor as fp32 bit patterns (the input
// has the candidates' dtype); elements at or beyond `len` come back as 0.
template <bool CB16>
__device__ __forceinline__ void input_group(const DevTensor& D, uint64_t start, uint32_t off0, uint32_t len,
                                            uint32_t out[4]) {
    if (D.input_src == RKV_SRC_GENERATED) {
        gen_group(D.in_seed, D.in_stream, D.in_dist, start, off0, CB16, out);
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            out[i] = (off0 + i < len) ? ld_elem_bits(D.input, CB16 ? RKV_BF16 : RKV_F32, start + off0 + i) : 0u;
    }
}

// Element 0 of a tensor as an fp32 bit pattern (upcast), from memory or generated.
__device__ __forceinline__ uint32_t first_elem_bits(const void* ptr, int src, int dtype, uint64_t seed,
                                                    uint64_t stream_id, int dist) {
    if (src == RKV_SRC_POINTER) return ld_elem_bits(ptr, dtype, 0);
    uint32_t g[4];
    gen_group(seed, stream_id, dist, 0, 0, dtype == RKV_BF16, g);
    return g[0];
}

// Load (or regenerate) the thread's reference values for a tile and derive what
// depends on them alone.  The bulk-copied part of the tile sits in ring stage
// `stage_a` (and, for an fp32 reference under bf16 candidates, continues in
// `stage_b`); anything beyond comes from global memory.  `rb` returns all E values as
// fp32 bit patterns (for the reference's own loophole flags); `ref_s` is the thread's
// shared-memory home for them with bf16 candidates.
template <bool CB16, bool RB16>
__device__ __forceinline__ void load_ref(RefRegs<CB16>& R, uint32_t (&rb)[Geo<CB16>::E], const DevTensor& D,
                                         uint64_t start, uint32_t len, const unsigned char* stage_a,
                                         const unsigned char* stage_b, int tid) {
    constexpr int E = Geo<CB16>::E, VEC = Geo<CB16>::VEC;
    constexpr uint32_t RSZ = RB16 ? 2 : 4;
    const bool full = len == (uint32_t)Geo<CB16>::kTile;
    // byte `b` of the reference tile in the ring
    auto at = [&](uint32_t b) -> const unsigned char* {
        return b < (uint32_t)kStageBytes ? stage_a + b : stage_b + (b - kStageBytes);
    };
    if (D.ref_src == RKV_SRC_GENERATED) {
#pragma unroll
        for (int g = 0; g < E / 4; ++g) {
            uint32_t v[4];
            gen_group(D.ref_seed, D.ref_stream, D.ref_dist, start, elem_off<VEC>(4 * g, tid),
                      D.ref_dtype == RKV_BF16, v);
#pragma unroll
            for (int i = 0; i < 4; ++i) rb[4 * g + i] = v[i];
        }
    } else if (full) {
#pragma unroll
        for (int g = 0; g < E / 4; ++g) {
            const uint32_t off0 = elem_off<VEC>(4 * g, tid);
            if (RB16) {
                const uint2 t = *reinterpret_cast<const uint2*>(at(off0 * 2));
                rb[4 * g + 0] = t.x << 16; rb[4 * g + 1] = t.x & 0xFFFF0000u;
                rb[4 * g + 2] = t.y << 16; rb[4 * g + 3] = t.y & 0xFFFF0000u;
            } else {
                const uint4 t = *reinterpret_cast<const uint4*>(at(off0 * 4));
                rb[4 * g + 0] = t.x; rb[4 * g + 1] = t.y; rb[4 * g + 2] = t.z; rb[4 * g + 3] = t.w;
            }
        }
    } else {
        const uint32_t copied = ((len * RSZ) & ~15u) / RSZ;
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const uint32_t off = elem_off<VEC>(j, tid);
            uint32_t b = 0;
            if (off < copied) b = ld_elem_bits(at(off * RSZ), RB16 ? RKV_BF16 : RKV_F32, 0);
            else if (off < len) b = ld_elem_bits(D.ref, RB16 ? RKV_BF16 : RKV_F32, start + off);
            rb[j] = b;
        }
    }
    if (!full) {
        // positions past the end of the tensor hold 0 (the candidates get 0 there as well)
#pragma unroll
        for (int j = 0; j < E; ++j)
            if (elem_off<VEC>(j, tid) >= len) rb[j] = 0u;
    }
    const float atol = D.atol, rtol = D.rtol;
    bool nonfinite = false, has_zero = false;
    uint32_t mn = 0xFFFFFFFFu;
    float tmin = kInf;
#pragma unroll
    for (int j = 0; j < E; ++j) {
        const uint32_t ab = rb[j] & 0x7FFFFFFFu;
        nonfinite |= !bits_finite(rb[j]);
        const float thr = __fadd_rn(atol, __fmul_rn(rtol, __uint_as_float(ab)));
        R.r[j] = __uint_as_float(rb[j]);
        tmin = fminf(tmin, thr);
        if constexpr (CB16) {
            has_zero |= ab == 0u;
        } else {
            R.thr[j] = thr;
            mn = min(mn, ab - 1u);   // |r| orders like its bits; zero wraps to the top
        }
    }
    R.thr_min = tmin;
    R.general = nonfinite;
    if constexpr (CB16) {
        R.atol = atol;
        R.rtol = rtol;
        R.warp_has_zero = __any_sync(kFullMask, has_zero);
    } else {
        R.minarp = mn == 0xFFFFFFFFu ? kInf : __uint_as_float(mn + 1u);
    }
}

__device__ __forceinline__ unsigned long long hint_key(float v, uint32_t tile) {
    return ((unsigned long long)(__float_as_uint(v) + 1u) << 32) | (unsigned long long)(~tile);
}

// Candidate bits of element j of the thread, as an fp32 pattern.
template <bool CB16, int NW>
__device__ __forceinline__ uint32_t cand_bits(const uint32_t (&w)[NW], int j) {
    if (!CB16) return w[j];
    return (j & 1) ? (w[j >> 1] & 0xFFFF0000u) : (w[j >> 1] << 16);
}

// Loophole flags of one candidate tile, until a difference has been seen.
template <bool CB16>
__device__ __forceinline__ void candidate_flags(const uint32_t (&w)[16], const Hint& h, Hint* h_smem,
                                                CandState* st, const DevTensor& D, const void* cand_g,
                                                uint64_t start, uint32_t len, uint32_t wanted_flags, int tid,
                                                int lane) {
    constexpr int E = Geo<CB16>::E, VEC = Geo<CB16>::VEC, NW = Geo<CB16>::NW;
    constexpr uint32_t CSZ = CB16 ? 2 : 4;
    // `settled` is the one hint field other warps update while this warp reads it: take
    // lane 0's copy so that the branch below is uniform across the warp.
    const uint32_t need = wanted_flags & ~__shfl_sync(kFullMask, h.settled, 0);
    if (need) {
        uint32_t acc1 = 0, acc2 = 0;
        const bool full = len == (uint32_t)Geo<CB16>::kTile;
        if (full && (need & 1u)) {
            const uint32_t f = CB16 ? (h.first >> 16) * 0x10001u : h.first;
#pragma unroll
            for (int i = 0; i < NW; ++i) acc1 |= w[i] ^ f;
        }
        if (full && (need & 2u) && D.input_src == RKV_SRC_POINTER) {
            // the input has the candidates' dtype: compare the 16-byte pieces as stored
            const uint4* in = reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(D.input) +
                                                             start * CSZ) + tid;
#pragma unroll
            for (int jv = 0; jv < E / VEC; ++jv) {
                const uint4 t = __ldg(in + jv * kConsumers);
                acc2 |= (w[4 * jv] ^ t.x) | (w[4 * jv + 1] ^ t.y) | (w[4 * jv + 2] ^ t.z) | (w[4 * jv + 3] ^ t.w);
            }
        } else if (!full || (need & 2u)) {
            const uint32_t copied = ((len * CSZ) & ~15u) / CSZ;
            // Regenerating the input is the expensive part.  A candidate that is no copy
            // of it almost surely shows that in the first four elements of every thread,
            // so the warp stops generating once a difference has been seen.
            bool with_input = (need & 2u) != 0u;
#pragma unroll
            for (int g = 0; g < E / 4; ++g) {
                if (g == 1 && with_input) with_input = !__any_sync(kFullMask, acc2 != 0u);
                if (full && !with_input) break;
                const uint32_t off0 = elem_off<VEC>(4 * g, tid);
                uint32_t in[4] = {0, 0, 0, 0};
                if (with_input && off0 < len) input_group<CB16>(D, start, off0, len, in);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t off = off0 + i;
                    if (off < len) {
                        uint32_t cb = cand_bits<CB16, NW>(w, 4 * g + i);
                        if (off >= copied) cb = ld_elem_bits(cand_g, CB16 ? RKV_BF16 : RKV_F32, start + off);
                        if (!full) acc1 |= cb ^ h.first;
                        if (with_input) acc2 |= cb ^ in[i];
                    }
                }
            }
        }
        uint32_t seen = (__any_sync(kFullMask, acc1 != 0u) ? 1u : 0u) |
                        (__any_sync(kFullMask, acc2 != 0u) ? 2u : 0u);
        seen &= need;
        if (lane == 0 && seen) {
            atomicOr(&st->mismatch, seen);
            atomicOr(&h_smem->settled, seen);
        }
    }
}

// One candidate tile against the thread's reference registers.
//   w        the thread's 16-byte pieces of the candidate tile (from the ring)
//   h        the candidate's hint entry (a snapshot; see the file header)
//   rec      the warp's running result for this candidate (shared memory; lane 0 writes)
//   st       the candidate's global state
//   cand_g   the candidate tensor in global memory (only the last < 16 bytes of a
//            ragged tensor are read from there)
template <bool CB16>
__device__ __forceinline__ void process_candidate(const RefRegs<CB16>& R, const uint32_t (&w)[16],
                                                  const Hint& h, Hint* h_smem, WarpRec* rec, CandState* st,
                                                  const DevTensor& D, const void* cand_g, uint32_t tile,
                                                  uint64_t start, uint32_t len, uint32_t wanted_flags,
                                                  int tid, int lane) {
    static_assert(!CB16, "bf16 candidates take process_candidate_b16");
    constexpr int E = Geo<CB16>::E, VEC = Geo<CB16>::VEC, NW = Geo<CB16>::NW;
    constexpr uint32_t CSZ = CB16 ? 2 : 4;

    // ---- common path ---------------------------------------------------------------
    float e[E];
#pragma unroll
    for (int j = 0; j < E; ++j)
        e[j] = fabsf(__fsub_rn(__uint_as_float(cand_bits<CB16, NW>(w, j)), R.r[j]));
    float m = fmaxf(fmaxf(fmaxf(e[0], e[1]), fmaxf(e[2], e[3])), fmaxf(fmaxf(e[4], e[5]), fmaxf(e[6], e[7])));
    m = fmaxf(m, fmaxf(fmaxf(fmaxf(e[8], e[9]), fmaxf(e[10], e[11])),
                       fmaxf(fmaxf(e[12], e[13]), fmaxf(e[14], e[15]))));
    float s4[4];
#pragma unroll
    for (int g = 0; g < 4; ++g)
        s4[g] = __fadd_rn(__fadd_rn(e[4 * g], e[4 * g + 1]), __fadd_rn(e[4 * g + 2], e[4 * g + 3]));
    const float s = __fadd_rn(__fadd_rn(s4[0], s4[1]), __fadd_rn(s4[2], s4[3]));

    // a NaN or an infinity anywhere makes the sum non-finite
    const bool lane_gen = R.general || !(s < kInf);
    // One vote settles the common case: nothing over tolerance, no possible first maximum,
    // nothing non-finite (the tests are explained below).
    if (!__any_sync(kFullMask, lane_gen || m > R.thr_min || m > h.te_x || m > __fmul_rd(h.tq_x, R.minarp))) {
        float sf = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sf = __fadd_rn(sf, __shfl_xor_sync(kFullMask, sf, off));
        const double total = rec->sum + (double)sf;       // every lane computes it, one stores
        if (lane == 0) rec->sum = total;
        candidate_flags<CB16>(w, h, h_smem, st, D, cand_g, start, len, wanted_flags, tid, lane);
        return;
    }
    // m <= thr_min means e_j <= m <= thr_min <= thr_j for every element: none over
    uint32_t cnt = 0;
    const bool any_over = __any_sync(kFullMask, m > R.thr_min);
    if (any_over) {
#pragma unroll
        for (int j = 0; j < E; ++j) cnt += (e[j] > R.thr[j]) ? 1u : 0u;
    }
    // Can one of these elements be the first maximum?  See Hint.
    bool rare = (m > h.te_x) || lane_gen;
    // Relative error.  fl(e/|r|) > t implies e > t*|r| >= RD(t*|r|) for a representable
    // t >= 0.  First a test on the thread's largest e and smallest non-zero |r|; only if
    // that passes somewhere in the warp, the same test element by element (errors
    // proportional to |r|, as in an all-zero output, pass the first test everywhere).
    if (__any_sync(kFullMask, m > __fmul_rd(h.tq_x, R.minarp))) {
        bool hit = false;
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const float ar = fabsf(R.r[j]);
            hit |= (ar != 0.0f) && (e[j] > __fmul_rd(h.tq_x, ar));
        }
        rare |= hit;
    }

    const bool any_gen = __any_sync(kFullMask, lane_gen);
    if (__any_sync(kFullMask, rare)) {
        // ---- locate maxima; general rule where needed ------------------------------
        const float rec_q = rec->qmax;
        LaneGen a;
        a.n_over = cnt; a.n_noncomp = 0; a.n_nan = 0; a.n_inf = 0; a.n_infmis = 0;
        a.emax = -1.0f; a.eoff = 0xFFFFu; a.qmax = -1.0f; a.qoff = 0xFFFFu; a.sum = (double)s;
        if (lane_gen) {
            a.n_over = 0; a.sum = 0.0;
            const uint32_t copied = ((len * CSZ) & ~15u) / CSZ;
#pragma unroll
            for (int j = 0; j < E; ++j) {
                const uint32_t off = elem_off<VEC>(j, tid);
                if (off < len) {
                    uint32_t cb = cand_bits<CB16, NW>(w, j);
                    if (off >= copied) cb = ld_elem_bits(cand_g, CB16 ? RKV_BF16 : RKV_F32, start + off);
                    elem_general(a, cb, __float_as_uint(R.r[j]), off, D.atol, D.rtol);
                }
            }
            if (a.n_noncomp) atomicAdd(&st->n_noncomp, (unsigned long long)a.n_noncomp);
            if (a.n_nan) atomicAdd(&st->n_nan, (unsigned long long)a.n_nan);
            if (a.n_inf) atomicAdd(&st->n_inf, (unsigned long long)a.n_inf);
            if (a.n_infmis) atomicAdd(&st->n_infmis, (unsigned long long)a.n_infmis);
        } else {
#pragma unroll
            for (int j = 0; j < E; ++j) {
                // (positions past the end of a ragged tile hold zeros and never count)
                if (e[j] > a.emax && elem_off<VEC>(j, tid) < len) { a.emax = e[j]; a.eoff = elem_off<VEC>(j, tid); }
                const float ar = fabsf(R.r[j]);
                // the warp's own record comes from earlier tiles: only a strictly larger
                // quotient can replace it
                if (ar != 0.0f && e[j] > __fmul_rd(fmaxf(rec_q, a.qmax), ar)) {
                    const float q = __fdiv_rn(e[j], ar);
                    if (q > a.qmax) { a.qmax = q; a.qoff = elem_off<VEC>(j, tid); }
                }
            }
        }
        cnt = a.n_over;
        // warp-wide first maximum: largest value, then smallest offset.  Non-negative
        // floats (and the -1 sentinel) order like their bit patterns as signed ints.
        const int eb = __float_as_int(a.emax);
        const int ebm = __reduce_max_sync(kFullMask, eb);
        const uint32_t eoff = __reduce_min_sync(kFullMask, eb == ebm ? a.eoff : 0xFFFFu);
        const int qb = __float_as_int(a.qmax);
        const int qbm = __reduce_max_sync(kFullMask, qb);
        const uint32_t qoff = __reduce_min_sync(kFullMask, qb == qbm ? a.qoff : 0xFFFFu);
        double sd = a.sum;
        if (any_gen) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sd += __shfl_xor_sync(kFullMask, sd, off);
        } else {
            float sf = s;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sf = __fadd_rn(sf, __shfl_xor_sync(kFullMask, sf, off));
            sd = (double)sf;
        }
        if (lane == 0) {
            WarpRec r = *rec;
            const float em = __int_as_float(ebm), qm = __int_as_float(qbm);
            if (em > r.emax) {
                r.emax = em; r.etile = tile; r.offs = (r.offs & 0xFFFF0000u) | eoff;
                atomicMax(&st->hint_e, hint_key(em, tile));
            }
            if (qm > r.qmax) {
                r.qmax = qm; r.qtile = tile; r.offs = (r.offs & 0x0000FFFFu) | (qoff << 16);
                atomicMax(&st->hint_q, hint_key(qm, tile));
            }
            r.sum += sd;
            *rec = r;
        }
    } else {
        float sf = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sf = __fadd_rn(sf, __shfl_xor_sync(kFullMask, sf, off));
        if (lane == 0) rec->sum += (double)sf;
    }
    if (any_over || any_gen) {
        const uint32_t tot = __reduce_add_sync(kFullMask, cnt);
        if (lane == 0 && tot) rec->n_over += tot;
    }

    candidate_flags<CB16>(w, h, h_smem, st, D, cand_g, start, len, wanted_flags, tid, lane);
}

// c - r for the bf16 value c in the low (half = 0) or high 16 bits of x: the bf16 value
// widened exactly, one fp32 subtraction rounded to nearest (a mixed-precision instruction
// of sm_100).
__device__ __forceinline__ float sub_bf16_f32(uint32_t x, int half, float r) {
    float d;
    if (half)
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, hi, %2;\n\t}" : "=f"(d) : "r"(x), "f"(r));
    else
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, lo, %2;\n\t}" : "=f"(d) : "r"(x), "f"(r));
    return d;
}

// One pass over a thread's 32 elements of a bf16 candidate tile: largest and summed
// e_j = |c_j - r_j|, and the largest d_j, where d_j = fma(-t, |r_j|, e_j) for the
// relative-error threshold t (see process_candidate_b16).  HAS_ZERO: reference values of
// exactly 0 may occur; they take no part in the relative error, and d_j = e_j - atol there,
// positive exactly when the element is over tolerance.
template <bool HAS_ZERO>
__device__ __forceinline__ void pass_b16(const RefRegs<true>& R, const uint32_t (&w)[16], float t, float& m_out,
                                         float& s_out, float& dm_out) {
    float m = 0.0f, dm = -kInf;
    float sg[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        float e[4], d[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = 4 * g + i;
            e[i] = fabsf(sub_bf16_f32(w[j >> 1], j & 1, R.r[j]));
            const float ar = fabsf(R.r[j]);
            if (HAS_ZERO && ar == 0.0f) d[i] = __fsub_rn(e[i], R.atol);
            else d[i] = __fmaf_rn(-t, ar, e[i]);
        }
        m = fmaxf(fmaxf(m, fmaxf(e[0], e[1])), fmaxf(e[2], e[3]));
        dm = fmaxf(fmaxf(dm, fmaxf(d[0], d[1])), fmaxf(d[2], d[3]));
        sg[g] = __fadd_rn(__fadd_rn(e[0], e[1]), __fadd_rn(e[2], e[3]));
    }
    m_out = m;
    dm_out = dm;
    s_out = __fadd_rn(__fadd_rn(__fadd_rn(sg[0], sg[1]), __fadd_rn(sg[2], sg[3])),
                      __fadd_rn(__fadd_rn(sg[4], sg[5]), __fadd_rn(sg[6], sg[7])));
}

// One tile of a bf16 candidate (32 elements per thread) against the thread's reference
// registers.  Same results as process_candidate; the tests that keep the rare work rare
// are arranged for errors proportional to |r|, the normal case of a rounded bf16 output,
// against which a test on the thread's largest error is powerless.
//
// Relative error.  With t = h.tq_x, element j can be a first maximum only if
// fl(e_j / |r_j|) > t, which implies e_j > t * |r_j| exactly (t is representable, rounding
// is monotone).  d_j = fma(-t, |r_j|, e_j) has the sign of that exact difference, except
// that a positive difference below the subnormal range rounds to zero; such a difference
// needs e_j < 2^-100 (the product has 48 significant bits).  So the elements pass as a
// whole when max_j d_j < 0, or = 0 with the thread's largest error 0 or at least 2^-100.
// A negative t says that nothing is published yet, or that a tie at 0 could still win;
// the hint table holds -inf then, which makes every d_j with r_j != 0 equal +inf.
//
// Over tolerance.  thr_j = fl(atol + fl(rtol * |r_j|)) >= fl(rtol * |r_j|), and a float
// e_j above fl(P) is above P itself, so e_j > thr_j implies e_j > rtol * |r_j| >= t * |r_j|
// whenever 0 <= t <= rtol: while the published relative maximum is at most rtol, an element
// over tolerance also fails the test above.  Where r_j = 0 the pass takes d_j = e_j - atol,
// the over-tolerance test itself; that such an element also counts as a possible maximum
// costs a look, not a result.
// Otherwise: m <= thr_min means e_j <= m <= thr_min <= thr_j for every element.
__device__ __forceinline__ void process_candidate_b16(const RefRegs<true>& R, const uint32_t (&w)[16],
                                                      const Hint& h, Hint* h_smem, WarpRec* rec,
                                                      CandState* st, const DevTensor& D, const void* cand_g,
                                                      uint32_t tile, uint64_t start, uint32_t len,
                                                      uint32_t wanted_flags, int tid, int lane) {
    constexpr int VEC = 8;
    constexpr float kTiny = 7.8886090522101181e-31f;      // 2^-100
    // candidate element j as an fp32 bit pattern
    auto cbits = [&](int j) -> uint32_t {
        const uint32_t x = w[j >> 1];
        return (j & 1) ? (x & 0xFFFF0000u) : (x << 16);
    };

    // ---- common path ---------------------------------------------------------------
    float m, s, dm;
    if (R.warp_has_zero) pass_b16<true>(R, w, h.tq_x, m, s, dm);
    else pass_b16<false>(R, w, h.tq_x, m, s, dm);

    const bool lane_gen = R.general || !(s < kInf);
    const bool hit = dm > 0.0f || (dm == 0.0f && m != 0.0f && m < kTiny);
    const bool rare = (m > h.te_x) || lane_gen || hit;
    const bool rel_covers = h.tq_x >= 0.0f && h.tq_x <= R.rtol;
    const bool maybe_over = rel_covers ? hit : (m > R.thr_min);

    if (!__any_sync(kFullMask, rare || maybe_over)) {
        // nothing but the sum to record (every lane computes it, one stores)
        float sf = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sf = __fadd_rn(sf, __shfl_xor_sync(kFullMask, sf, off));
        const double total = rec->sum + (double)sf;
        if (lane == 0) rec->sum = total;
    } else {
        uint32_t cnt = 0;
        const bool any_over = __any_sync(kFullMask, maybe_over);
        if (any_over) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float e = fabsf(__fsub_rn(__uint_as_float(cbits(j)), R.r[j]));
                cnt += (e > __fadd_rn(R.atol, __fmul_rn(R.rtol, fabsf(R.r[j])))) ? 1u : 0u;
            }
        }
        const bool any_gen = __any_sync(kFullMask, lane_gen);
        // ---- locate maxima; general rule where needed ----------------------------------
        const float rec_q = rec->qmax;
        LaneGen a;
        a.n_over = cnt; a.n_noncomp = 0; a.n_nan = 0; a.n_inf = 0; a.n_infmis = 0;
        a.emax = -1.0f; a.eoff = 0xFFFFu; a.qmax = -1.0f; a.qoff = 0xFFFFu; a.sum = (double)s;
        if (lane_gen) {
            a.n_over = 0; a.sum = 0.0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const uint32_t off = elem_off<VEC>(j, tid);
                // (a ragged tile's tail was patched into w by the caller)
                if (off < len) elem_general(a, cbits(j), __float_as_uint(R.r[j]), off, R.atol, R.rtol);
            }
            if (a.n_noncomp) atomicAdd(&st->n_noncomp, (unsigned long long)a.n_noncomp);
            if (a.n_nan) atomicAdd(&st->n_nan, (unsigned long long)a.n_nan);
            if (a.n_inf) atomicAdd(&st->n_inf, (unsigned long long)a.n_inf);
            if (a.n_infmis) atomicAdd(&st->n_infmis, (unsigned long long)a.n_infmis);
        } else if (rare) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float e = fabsf(__fsub_rn(__uint_as_float(cbits(j)), R.r[j]));
                const uint32_t off = elem_off<VEC>(j, tid);
                // (positions past the end of a ragged tile hold zeros and never count)
                if (e > a.emax && off < len) { a.emax = e; a.eoff = off; }
                const float ar = fabsf(R.r[j]);
                // the warp's own record comes from earlier tiles: only a strictly larger
                // quotient can replace it
                if (ar != 0.0f && e > __fmul_rd(fmaxf(rec_q, a.qmax), ar)) {
                    const float q = __fdiv_rn(e, ar);
                    if (q > a.qmax) { a.qmax = q; a.qoff = off; }
                }
            }
        }
        cnt = a.n_over;
        // warp-wide first maximum: largest value, then smallest offset.  Non-negative
        // floats (and the -1 sentinel) order like their bit patterns as signed ints.
        const int eb = __float_as_int(a.emax);
        const int ebm = __reduce_max_sync(kFullMask, eb);
        const uint32_t eoff = __reduce_min_sync(kFullMask, eb == ebm ? a.eoff : 0xFFFFu);
        const int qb = __float_as_int(a.qmax);
        const int qbm = __reduce_max_sync(kFullMask, qb);
        const uint32_t qoff = __reduce_min_sync(kFullMask, qb == qbm ? a.qoff : 0xFFFFu);
        double sd = a.sum;
        if (any_gen) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sd += __shfl_xor_sync(kFullMask, sd, off);
        } else {
            float sf = s;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sf = __fadd_rn(sf, __shfl_xor_sync(kFullMask, sf, off));
            sd = (double)sf;
        }
        const uint32_t tot = (any_over || any_gen) ? __reduce_add_sync(kFullMask, cnt) : 0u;
        if (lane == 0) {
            WarpRec r = *rec;
            const float em = __int_as_float(ebm), qm = __int_as_float(qbm);
            if (em > r.emax) {
                r.emax = em; r.etile = tile; r.offs = (r.offs & 0xFFFF0000u) | eoff;
                atomicMax(&st->hint_e, hint_key(em, tile));
            }
            if (qm > r.qmax) {
                r.qmax = qm; r.qtile = tile; r.offs = (r.offs & 0x0000FFFFu) | (qoff << 16);
                atomicMax(&st->hint_q, hint_key(qm, tile));
            }
            r.sum += sd;
            r.n_over += tot;
            *rec = r;
        }
    }
    candidate_flags<true>(w, h, h_smem, st, D, cand_g, start, len, wanted_flags, tid, lane);
}

// Merge the warp records of every candidate of a part into the block's
// Partial row and clear them.  Called by all consumer threads between two
// consumer barriers.
__device__ __forceinline__ void flush_records(WarpRec* recs, const DevTensor& D, int K, int k0, int kc,
                                              uint32_t slot, Partial* __restrict__ partials, int tid,
                                              uint32_t tile_elems) {
    if (tid < kc) {
        Partial p;
        p.n_over = 0; p.eidx = RKV_NO_INDEX; p.qidx = RKV_NO_INDEX; p.sum = 0.0;
        p.emax = -1.0f; p.qmax = -1.0f; p.valid = 1u; p.reserved = 0u;
#pragma unroll
        for (int wp = 0; wp < kConsumerWarps; ++wp) {
            WarpRec& r = recs[wp * kPartK + tid];
            p.n_over += r.n_over;
            p.sum += r.sum;
            if (r.emax >= 0.0f) {
                const uint64_t idx = (uint64_t)r.etile * tile_elems + (r.offs & 0xFFFFu);
                if (r.emax > p.emax || (r.emax == p.emax && idx < p.eidx)) { p.emax = r.emax; p.eidx = idx; }
            }
            if (r.qmax >= 0.0f) {
                const uint64_t idx = (uint64_t)r.qtile * tile_elems + (r.offs >> 16);
                if (r.qmax > p.qmax || (r.qmax == p.qmax && idx < p.qidx)) { p.qmax = r.qmax; p.qidx = idx; }
            }
            r.emax = -1.0f; r.etile = 0; r.qmax = -1.0f; r.qtile = 0; r.offs = 0; r.n_over = 0; r.sum = 0.0;
        }
        // the block may have written this slot before (group A, then group B): merge
        Partial* dst = &partials[((size_t)D.slot_base + slot) * (size_t)K + (size_t)(k0 + tid)];
        const Partial old = *dst;
        if (old.valid) {
            p.n_over += old.n_over;
            p.sum = old.sum + p.sum;
            if (old.emax > p.emax || (old.emax == p.emax && old.eidx < p.eidx)) { p.emax = old.emax; p.eidx = old.eidx; }
            if (old.qmax > p.qmax || (old.qmax == p.qmax && old.qidx < p.qidx)) { p.qmax = old.qmax; p.qidx = old.qidx; }
        }
        *dst = p;
    }
}

// Published (maximum, tile) -> the threshold an element of `tile` has to exceed to
// be able to become the first maximum (see Hint).
__device__ __forceinline__ float hint_threshold(unsigned long long key, uint32_t tile) {
    if (!(key >> 32)) return -1.0f;
    const uint32_t bits = (uint32_t)(key >> 32) - 1u;
    const uint32_t at_tile = ~(uint32_t)key;
    if (tile > at_tile) return __uint_as_float(bits);
    return bits ? __uint_as_float(bits - 1u) : -1.0f;       // the float below; below +0 anything goes
}

template <bool CB16, bool RB16>
__device__ __forceinline__ void consumer_loop(const DevTensor* __restrict__ tensors, int T, int K, int k_begin,
                                              int k_end, uint32_t n_items, CandState* __restrict__ state,
                                              Partial* __restrict__ partials, unsigned char* smem,
                                              const Ring& ring) {
    constexpr int E = Geo<CB16>::E, VEC = Geo<CB16>::VEC, NW = Geo<CB16>::NW;
    constexpr int NV = E / VEC;
    constexpr uint32_t kTile = Geo<CB16>::kTile;
    constexpr int kRefStages = (CB16 && !RB16) ? 2 : 1;
    constexpr uint32_t kVariant = (CB16 ? 2u : 0u) + (RB16 ? 1u : 0u);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned char** ptrs = reinterpret_cast<const unsigned char**>(smem + kOffPtrC);
    Hint* hints = reinterpret_cast<Hint*>(smem + kOffHint);
    WarpRec* recs = reinterpret_cast<WarpRec*>(smem + kOffRec);
    volatile uint32_t* ref_state = reinterpret_cast<volatile uint32_t*>(smem + kOffRefState);
    const unsigned char* stages = smem + kOffStage;

    // clear the records once; flush_records leaves them cleared
    for (int i = tid; i < kConsumerWarps * kPartK; i += kConsumers) {
        WarpRec& r = recs[i];
        r.emax = -1.0f; r.etile = 0; r.qmax = -1.0f; r.qtile = 0; r.offs = 0; r.n_over = 0; r.sum = 0.0;
    }

    // next ring stage to consume and the parity of its current use (same order as the producer issues)
    uint32_t cstage = 0, cphase = 0;
    uint32_t ord = 0;               // items this block has started
    int cur_t = -1, cur_k0 = 0, cur_kc = 0;
    uint32_t cur_part = 0xFFFFFFFFu, cur_slot = 0;

    volatile uint32_t* ids = reinterpret_cast<volatile uint32_t*>(smem + kOffIds);
    for (;; ++ord) {
        // The next item announces itself in the first ring stage it uses (which stays full
        // until it is consumed below).  All consumers agree on stopping: at the producer's
        // end mark, or when any thread of the block has given up on a wait.
        const uint32_t s0 = cstage;
        const bool got = mbar_wait(ring.full0 + 8 * s0, cphase, ring.abort_flag);
        const uint32_t id = got ? ids[s0] : kNoItem;
        if (consumer_sync_or((id == kNoItem || id >= n_items || *ring.abort_flag) ? 1u : 0u)) break;
        Item it;
        if (!decode_item(tensors, T, kVariant, (uint32_t)(k_end - k_begin), id, it)) break;
        const DevTensor& D = tensors[it.t];
        const uint32_t k_count = (uint32_t)(k_end - k_begin);
        const int k0 = k_begin + (int)part_begin(it.part, it.n_parts, k_count);
        const int kc = k_begin + (int)part_begin(it.part + 1, it.n_parts, k_count) - k0;
        const uint32_t part_key = (it.group << 30) | it.part;
        const uint64_t start = (uint64_t)it.tile * kTile;
        const uint32_t len = (uint32_t)min((uint64_t)kTile, D.n - start);
        const uint32_t wanted = D.input_src != RKV_SRC_NONE ? 3u : 1u;
        CandState* st_t = state + (size_t)it.t * (size_t)(K + 1);
        Hint* H = hints + (ord & 1u) * kPartK;

        if (it.t != cur_t || part_key != cur_part) {
            consumer_sync();                      // every warp is done with the previous part
            if (cur_t >= 0) flush_records(recs, tensors[cur_t], K, cur_k0, cur_kc, cur_slot, partials, tid, kTile);
            if (tid < kc) ptrs[tid] = reinterpret_cast<const unsigned char*>(D.cands[k0 + tid]);
            cur_t = it.t; cur_part = part_key; cur_k0 = k0; cur_kc = kc;
            cur_slot = blockIdx.x;                // one Partial row per block and tensor
        }
        // refresh the hints of this part from the published state
        if (tid < kc) {
            const CandState* sc = st_t + k0 + tid;
            Hint h;
            h.te_x = hint_threshold(__ldcg(&sc->hint_e), it.tile);
            h.tq_x = hint_threshold(__ldcg(&sc->hint_q), it.tile);
            if (CB16 && h.tq_x < 0.0f) h.tq_x = -kInf;     // see process_candidate_b16
            h.settled = __ldcg(&sc->mismatch);
            h.first = ld_elem_bits(ptrs[tid], CB16 ? RKV_BF16 : RKV_F32, 0);
            H[tid] = h;
        }
        if (tid == kPartK) ref_state[ord & 1u] = __ldcg(&st_t[K].mismatch);

        // ---- the thread's reference values --------------------------------------------
        RefRegs<CB16> R;
        uint32_t rb[E];
        if (D.ref_src == RKV_SRC_POINTER) {
            // the reference tile fills one ring stage, or two (fp32 under bf16 candidates)
            const uint32_t sa = cstage, pha = cphase;
            mbar_wait(ring.full0 + 8 * sa, pha, ring.abort_flag);
            if (++cstage == kStages) { cstage = 0; cphase ^= 1u; }
            uint32_t sb = sa;
            if (kRefStages == 2) {
                sb = cstage;
                mbar_wait(ring.full0 + 8 * sb, cphase, ring.abort_flag);
                if (++cstage == kStages) { cstage = 0; cphase ^= 1u; }
            }
            load_ref<CB16, RB16>(R, rb, D, start, len, stages + (size_t)sa * kStageBytes,
                                 stages + (size_t)sb * kStageBytes, tid);
            __syncwarp();
            mbar_arrive_if(ring.empty0 + 8 * sa, lane == 0);
            if (kRefStages == 2) mbar_arrive_if(ring.empty0 + 8 * sb, lane == 0);
        } else {
            load_ref<CB16, RB16>(R, rb, D, start, len, nullptr, nullptr, tid);
        }
        consumer_sync();                          // hints, pointers and cleared records are visible

        // reference flags (constant / copy of the input), until a difference has been seen
        {
            const uint32_t need = wanted & ~ref_state[ord & 1u];
            if (need) {
                const uint32_t r_first = first_elem_bits(D.ref, D.ref_src, D.ref_dtype, D.ref_seed,
                                                         D.ref_stream, D.ref_dist);
                uint32_t acc1 = 0, acc2 = 0;
#pragma unroll
                for (int g = 0; g < E / 4; ++g) {
                    const uint32_t off0 = elem_off<VEC>(4 * g, tid);
                    uint32_t in[4] = {0, 0, 0, 0};
                    if ((need & 2u) && off0 < len) input_group<CB16>(D, start, off0, len, in);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (off0 + i < len) {
                            acc1 |= rb[4 * g + i] ^ r_first;
                            acc2 |= rb[4 * g + i] ^ in[i];
                        }
                    }
                }
                uint32_t seen = (__any_sync(kFullMask, acc1 != 0u) ? 1u : 0u) |
                                (__any_sync(kFullMask, acc2 != 0u) ? 2u : 0u);
                seen &= need;
                if (lane == 0 && seen) atomicOr(&st_t[K].mismatch, seen);
            }
        }

        // ---- every candidate of the part ----------------------------------------------
        for (int kk = 0; kk < kc; ++kk) {
            const uint32_t s = cstage;
            const Hint h = H[kk];
            mbar_wait(ring.full0 + 8 * s, cphase, ring.abort_flag);
            const unsigned char* stage = stages + (size_t)s * kStageBytes;
            uint32_t w[NW];
#pragma unroll
            for (int jv = 0; jv < NV; ++jv) {
                const uint4 t = *reinterpret_cast<const uint4*>(stage + (size_t)(jv * kConsumers + tid) * 16);
                w[4 * jv + 0] = t.x; w[4 * jv + 1] = t.y; w[4 * jv + 2] = t.z; w[4 * jv + 3] = t.w;
            }
            __syncwarp();
            mbar_arrive_if(ring.empty0 + 8 * s, lane == 0);
            if (++cstage == kStages) { cstage = 0; cphase ^= 1u; }
            if (len != kTile) {
                // Ragged last tile: the copy brought whole 16-byte pieces only.  The few
                // elements behind them come from global memory; positions past the end of the
                // tensor get 0 against a reference of 0 (see load_ref): no error, never over
                // tolerance, excluded from the relative error, and never the first maximum,
                // because their offsets are larger than every real element's.
                constexpr uint32_t CSZ = CB16 ? 2 : 4;
                const uint32_t copied = ((len * CSZ) & ~15u) / CSZ;
#pragma unroll
                for (int j = 0; j < E; ++j) {
                    const uint32_t off = elem_off<VEC>(j, tid);
                    if (off >= copied) {
                        const uint32_t cb = off < len ? ld_elem_bits(ptrs[kk], CB16 ? RKV_BF16 : RKV_F32, start + off) : 0u;
                        if (!CB16) w[j] = cb;
                        else w[j >> 1] = (j & 1) ? ((w[j >> 1] & 0x0000FFFFu) | cb) : ((w[j >> 1] & 0xFFFF0000u) | (cb >> 16));
                    }
                }
            }
            if constexpr (CB16)
                process_candidate_b16(R, w, h, &H[kk], &recs[warp * kPartK + kk], st_t + k0 + kk, D, ptrs[kk],
                                      it.tile, start, len, wanted, tid, lane);
            else
                process_candidate<false>(R, w, h, &H[kk], &recs[warp * kPartK + kk], st_t + k0 + kk, D, ptrs[kk],
                                         it.tile, start, len, wanted, tid, lane);
        }
    }
    consumer_sync();
    if (cur_t >= 0) flush_records(recs, tensors[cur_t], K, cur_k0, cur_kc, cur_slot, partials, tid, kTile);
}

// One kernel per storage variant (candidate dtype, stored reference dtype), so
// that each gets its own register allocation.  A launch handles the items of
// every tensor of its variant; `n_items` counts them.
template <bool CB16, bool RB16>
__global__ void __launch_bounds__(kThreads, kBlocksPerSm)
verify_kernel(const DevTensor* __restrict__ tensors, int T, int K, int k_begin, int k_end, uint32_t n_items,
              CandState* __restrict__ state, Partial* __restrict__ partials, WorkspaceHeader* header) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x;
    Ring ring;
    ring.full0 = smem_u32(smem + kOffFull);
    ring.empty0 = smem_u32(smem + kOffEmpty);
    ring.stage0 = smem_u32(smem + kOffStage);
    ring.abort_flag = reinterpret_cast<volatile uint32_t*>(smem + kOffAbort);
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(ring.full0 + 8 * s, 1);                    // the producer's arrive + its bytes
            mbar_init(ring.empty0 + 8 * s, kConsumerWarps);      // one release per consumer warp
        }
        *ring.abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid >= kConsumers) {
        producer_loop<CB16, RB16>(tensors, T, k_begin, k_end, n_items, smem, ring, header);
    } else {
        consumer_loop<CB16, RB16>(tensors, T, K, k_begin, k_end, n_items, state, partials, smem, ring);
        if (tid == 0 && *ring.abort_flag) atomicExch(&header->status, (int32_t)RKV_ERR_TIMEOUT);
    }
}

// ----------------------------------------------------------------------------
// finalize: merge the per-block partials of each (candidate, tensor) in a fixed
// order, derive flags and verdict, and the joint verdict over tensors
// ----------------------------------------------------------------------------
constexpr int kFinThreads = 128;

struct Wide {
    uint64_t n_over;
    uint64_t eidx, qidx;
    double sum;
    float emax, qmax;
};

__device__ __forceinline__ void wide_merge(Wide& a, const Wide& b) {
    a.n_over += b.n_over;
    if (b.emax > a.emax || (b.emax == a.emax && b.eidx < a.eidx)) { a.emax = b.emax; a.eidx = b.eidx; }
    if (b.qmax > a.qmax || (b.qmax == a.qmax && b.qidx < a.qidx)) { a.qmax = b.qmax; a.qidx = b.qidx; }
    a.sum += b.sum;
}

__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(const DevTensor* __restrict__ tensors, int T, int K, const CandState* __restrict__ state,
                const Partial* __restrict__ partials, rkv_stats* __restrict__ stats_out,
                uint32_t* __restrict__ joint_pass) {
    __shared__ Wide red[kFinThreads];
    const int k = blockIdx.x, tid = threadIdx.x;
    uint32_t all_pass = 1;
    for (int t = 0; t < T; ++t) {
        const DevTensor D = tensors[t];
        Wide w;
        w.n_over = 0; w.sum = 0.0;
        w.emax = -1.0f; w.qmax = -1.0f; w.eidx = RKV_NO_INDEX; w.qidx = RKV_NO_INDEX;
        for (uint32_t s = tid; s < D.n_slots; s += kFinThreads) {
            const Partial p = partials[((size_t)D.slot_base + s) * (size_t)K + (size_t)k];
            if (!p.valid) continue;
            Wide b;
            b.n_over = p.n_over; b.sum = p.sum;
            b.emax = p.emax; b.eidx = p.eidx; b.qmax = p.qmax; b.qidx = p.qidx;
            wide_merge(w, b);
        }
        red[tid] = w;
        __syncthreads();
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
            const CandState cs = state[(size_t)t * (size_t)(K + 1) + (size_t)k];
            const uint32_t ref_mismatch = state[(size_t)t * (size_t)(K + 1) + (size_t)K].mismatch;
            rkv_stats st;
            st.n_over_tol = r.n_over;
            st.n_nan = cs.n_nan;
            st.n_inf = cs.n_inf;
            st.n_inf_mismatch = cs.n_infmis;
            st.n_comparable = D.n - cs.n_noncomp;
            st.argmax_abs_err = r.emax < 0.0f ? RKV_NO_INDEX : r.eidx;
            st.argmax_rel_err = r.qmax < 0.0f ? RKV_NO_INDEX : r.qidx;
            st.sum_abs_err = r.sum;
            st.max_abs_err = r.emax < 0.0f ? 0.0f : r.emax;
            st.max_rel_err = r.qmax < 0.0f ? 0.0f : r.qmax;
            st.mean_abs_err = st.n_comparable ? (float)(r.sum / (double)st.n_comparable) : 0.0f;
            st.reserved = 0;
            const bool has_in = D.input_src != RKV_SRC_NONE;
            uint32_t flags = 0;
            if (!(cs.mismatch & 1u)) flags |= RKV_FLAG_CAND_CONST;
            if (has_in && !(cs.mismatch & 2u)) flags |= RKV_FLAG_CAND_COPY_OF_INPUT;
            if (!(ref_mismatch & 1u)) flags |= RKV_FLAG_REF_CONST;
            if (has_in && !(ref_mismatch & 2u)) flags |= RKV_FLAG_REF_COPY_OF_INPUT;
            if (cs.n_nan) flags |= RKV_FLAG_HAS_NAN;
            if (cs.n_inf) flags |= RKV_FLAG_HAS_INF;
            uint32_t verdict = 0;
            if (r.n_over) verdict |= RKV_FAIL_TOL;
            if (cs.n_nan) verdict |= RKV_FAIL_NAN;
            if (cs.n_infmis) verdict |= RKV_FAIL_INF_MISMATCH;
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

template <bool CB16, bool RB16>
static int launch_variant(const DevTensor* d_tensors, int T, int K, int k_begin, int k_end, uint32_t n_items,
                          int grid_max, CandState* state, Partial* partials, WorkspaceHeader* header,
                          cudaStream_t stream) {
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RKV_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(verify_kernel<CB16, RB16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemBytes) != cudaSuccess)
            return RKV_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    // the grid is always the full resident grid: Partial rows are numbered by block
    verify_kernel<CB16, RB16><<<grid_max, kThreads, kSmemBytes, stream>>>(d_tensors, T, K, k_begin, k_end,
                                                                         n_items, state, partials, header);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

int launch_verify(const DevTensor* d_tensors, int T, int K, int k_begin, int k_end,
                  const uint32_t variant_items[4], int grid, CandState* state, Partial* partials,
                  WorkspaceHeader* header, cudaStream_t stream) {
    int rc = RKV_OK;
    for (int v = 0; v < 4 && rc == RKV_OK; ++v) {
        const uint32_t n = variant_items[v];
        if (!n) continue;
#define RKV_LAUNCH(CB, RB) \
    launch_variant<CB, RB>(d_tensors, T, K, k_begin, k_end, n, grid, state, partials, header, stream)
        switch (v) {
            case 0: rc = RKV_LAUNCH(false, false); break;
            case 1: rc = RKV_LAUNCH(false, true); break;
            case 2: rc = RKV_LAUNCH(true, false); break;
            default: rc = RKV_LAUNCH(true, true); break;
        }
#undef RKV_LAUNCH
    }
    return rc;
}

int launch_finalize(const DevTensor* d_tensors, int T, int K, const CandState* state,
                    const Partial* partials, rkv_stats* stats_out, uint32_t* joint_pass,
                    cudaStream_t stream) {
    finalize_kernel<<<K, kFinThreads, 0, stream>>>(d_tensors, T, K, state, partials, stats_out, joint_pass);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

}  // namespace rkv
