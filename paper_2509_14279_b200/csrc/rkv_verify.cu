// Fused single-pass verification kernel and its finalize kernels (sm_100a).
//
// Work decomposition.  A tensor is cut into tiles of 14336 candidate bytes (3584 fp32 or
// 7168 bf16 / fp16 elements); the K candidates into parts of at most 64.  A work item is
// (tensor, group, part, tile); the items of every tensor of a call -- whatever its storage
// types -- form one list (see Segment), and one launch of persistent thread blocks works
// through it: a block starts with the item of its own number and then draws further items
// from a ticket counter.
//
// A block has two roles:
//
//   * one producer warp: it takes the block's items one after the other -- the ticket for the
//     next one is drawn while the current one is being issued -- decodes them, publishes their
//     description, fetches the part's candidate pointers (all 32 lanes, one round trip) and
//     then one lane issues the bulk asynchronous copies (cp.async.bulk, completion counted on
//     an mbarrier) that bring, for the item, the reference tile and then the same tile of
//     every candidate of the part into a ring of shared-memory stages.  Several stages are in
//     flight, across item boundaries, so the copies of later candidates overlap the
//     comparison of earlier ones;
//   * seven consumer warps: each thread owns 64 bytes of every candidate tile (16 fp32 or 32
//     16-bit elements).  It keeps their reference values (and, for fp32 candidates, the
//     tolerance thresholds) IN REGISTERS for the whole item and meets every candidate tile as
//     it lands in the ring.
//
// Candidate bytes are read from HBM exactly once; the reference once per part.
// When the reference is "generated" the threads regenerate their values from
// the Philox stream instead of reading them (fused generate + verify).
//
// Per element the common path is one subtraction, one running maximum and one
// addition (16-bit candidates: one fused multiply-add and one more maximum, see
// process_candidate_16; whole tiles of 16-bit candidates are taken two candidates at a
// time, straight from their ring stages, see pair_common_16: the waits, votes, warp
// reductions and loop overhead of a step are then paid once per two candidates).
// Counting the elements over tolerance, locating maxima,
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
// Reductions are deterministic: integer sums; lexicographic (value descending, index
// ascending) maxima; the error sum of a (tile, candidate) is a fixed tree over the tile's
// elements and is stored per tile, and the finalize kernel adds the tile sums in tile
// order -- whichever block verified whichever tile, the bits of the sum are the same.
// No float atomics.
#include "rkv_internal.h"
#include "rkv_philox.cuh"

namespace rkv {

namespace {

constexpr uint32_t kFullMask = 0xFFFFFFFFu;
constexpr float kInf = __builtin_huge_valf();
enum : uint32_t { kNoItem = 0xFFFFFFFFu };     // the producer's "no more items" mark
constexpr int kInfoRing = 16;                  // item descriptions kept per block (> kStages + 1: an item uses >= 1 stage)
constexpr long long kWaitCycles = 2000000000LL;

// ----------------------------------------------------------------------------
// range checks of a debug build
// ----------------------------------------------------------------------------
// With RKV_DEBUG_BOUNDS every index into global memory and into the shared-memory tables
// is checked before it is used; a violation records its site and value in the workspace
// header, sets the status word and skips the access.  Nothing traps or asserts.
#ifdef RKV_DEBUG_BOUNDS
__device__ __noinline__ void bounds_fail(WorkspaceHeader* header, uint32_t site, unsigned long long value) {
    if (atomicCAS(&header->bounds_site, 0u, site) == 0u) header->bounds_value = value;
    atomicExch(&header->status, (int32_t)RKV_ERR_BOUNDS);
}
#define RKV_IN_BOUNDS(header, site, cond, value) \
    ((cond) ? true : (bounds_fail((header), (site), (unsigned long long)(value)), false))
#else
#define RKV_IN_BOUNDS(header, site, cond, value) (true)
#endif

// ----------------------------------------------------------------------------
// shared-memory layout (dynamic)
// ----------------------------------------------------------------------------
// Per (warp, candidate of the part) running result.
struct __align__(16) WarpRec {
    float emax; uint32_t etile;
    float qmax; uint32_t qtile;
    uint32_t offs;           // eoff | qoff << 16 : element offsets inside their tiles
    uint32_t n_over;
    double sum;              // of the current item's tile only
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
    uint32_t first;                  // element 0 of the candidate, storage bits
};
static_assert(sizeof(Hint) == 16, "Hint layout");

// What the producer tells the consumers about an item, before it arms the item's first stage.
struct __align__(16) ItemInfo {
    uint32_t id;             // kNoItem: no more items
    uint32_t t;
    uint32_t tile;           // tensor-wide tile index
    uint32_t k0, kc;         // candidates [k0, k0 + kc) of the call
    uint32_t reserved[3];
};
static_assert(sizeof(ItemInfo) == 32, "ItemInfo layout");

constexpr int kOffFull = 0;                                   // kStages mbarriers: the stage's copy has landed
constexpr int kOffEmpty = kOffFull + 8 * kStages;             // kStages mbarriers: every consumer warp has read the stage
constexpr int kOffAbort = kOffEmpty + 8 * kStages;            // uint32
constexpr int kOffRefState = kOffAbort + 8;                   // 2 x uint32 settled bits of the reference (item parity)
constexpr int kOffWaitLimit = kOffRefState + 8;               // long long: cycles a wait may take
constexpr int kOffInfo = 128;
constexpr int kOffPtrC = kOffInfo + kInfoRing * (int)sizeof(ItemInfo);   // consumer copy of the part's candidate pointers
constexpr int kOffPtrP = kOffPtrC + kPartK * 8;                          // producer copy (it runs an item ahead)
constexpr int kOffFirst = kOffPtrP + kPartK * 8;                         // element 0 of the part's candidates, storage bits
constexpr int kOffHint = kOffFirst + kPartK * 4;                         // two tables (item parity)
constexpr int kOffRec = kOffHint + 2 * kPartK * (int)sizeof(Hint);
constexpr int kOffStage = (kOffRec + kConsumerWarps * kPartK * (int)sizeof(WarpRec) + 1023) / 1024 * 1024;
constexpr int kSmemBytes = kOffStage + kStages * kStageBytes;
static_assert(kOffWaitLimit + 8 <= kOffInfo && kOffWaitLimit % 8 == 0 && kOffEmpty % 8 == 0 && kOffInfo % 16 == 0 &&
              kOffPtrC % 8 == 0 && kOffPtrP % 8 == 0 && kOffHint % 16 == 0 && kOffRec % 16 == 0, "layout");
static_assert(kInfoRing > kStages + 1 && (kInfoRing & (kInfoRing - 1)) == 0, "item ring");
static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two blocks per SM must fit");

// Candidate storage kinds the comparison is compiled for.
enum : int { CK_F32 = 0, CK_BF16 = 1, CK_F16 = 2 };

// Geometry of a tile.  A thread owns 64 bytes of each candidate tile, so a candidate tile
// always fills exactly one ring stage: 16 fp32 elements or 32 16-bit elements.  Their
// reference values stay in registers for the whole item.  With fp32 candidates the
// tolerance thresholds do too; with 16-bit candidates they are recomputed in the rare case
// that needs them (see process_candidate_16).
template <int CK>
struct Geo {
    static constexpr bool C16 = CK != CK_F32;
    static constexpr int E = C16 ? 32 : 16;             // elements per thread
    static constexpr int VEC = C16 ? 8 : 4;             // elements per 16-byte piece
    static constexpr int NW = 16;                       // 32-bit words per thread and candidate tile
    static constexpr int kTile = kConsumers * E;        // elements per tile
    static constexpr int DTYPE = CK == CK_F32 ? RKV_F32 : CK == CK_BF16 ? RKV_BF16 : RKV_F16;
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

// What every wait of a block shares: the flag that says "a wait ran out, drain" and the
// number of clock cycles a wait may take.
struct WaitCtl {
    volatile uint32_t* abort_flag;
    const volatile long long* limit;
};

// Bounded wait.  Returns false when the wait ran out (about a second) or when
// another thread of the block has already given up; the block then drains: every
// later wait returns at once, all barriers are still reached, and the status
// word tells the host that the results are void.
__device__ __noinline__ bool mbar_wait_slow(uint32_t mbar, uint32_t parity, WaitCtl ctl) {
    const long long t0 = clock64();
    const long long limit = *ctl.limit;
    for (uint32_t spin = 0; spin < (1u << 26); ++spin) {
        if (mbar_try_wait(mbar, parity)) return true;
        if (*ctl.abort_flag) return false;
        if (clock64() - t0 > limit) break;
    }
    *ctl.abort_flag = 1u;
    return false;
}

__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity, WaitCtl ctl) {
    if (mbar_try_wait(mbar, parity)) return true;
    return mbar_wait_slow(mbar, parity, ctl);
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

// 16 storage bits -> the fp32 bit pattern of the same value (exact for both kinds).
__device__ __forceinline__ uint32_t upcast16(uint32_t raw, int dtype) {
    if (dtype == RKV_BF16) return raw << 16;
    float f;
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"((unsigned short)raw));
    return __float_as_uint(f);
}

// Element i of a stored tensor as an fp32 bit pattern.
__device__ __forceinline__ uint32_t ld_elem_bits(const void* base, int dtype, uint64_t i) {
    if (dtype == RKV_F32) return reinterpret_cast<const uint32_t*>(base)[i];
    return upcast16(reinterpret_cast<const uint16_t*>(base)[i], dtype);
}

// Element i of a stored tensor, storage bits.
__device__ __forceinline__ uint32_t ld_elem_raw(const void* base, int dtype, uint64_t i) {
    if (dtype == RKV_F32) return reinterpret_cast<const uint32_t*>(base)[i];
    return reinterpret_cast<const uint16_t*>(base)[i];
}

// ----------------------------------------------------------------------------
// what the kernel gets
// ----------------------------------------------------------------------------
struct Args {
    const DevTensor* tensors;
    const Segment* segments;
    CandState* state;
    Partial* partials;
    double* sums;
    WorkspaceHeader* header;
    int T, K, k_begin, k_end;
    uint32_t n_items, n_segments;
};

// ----------------------------------------------------------------------------
// the producer warp: feeds the ring
// ----------------------------------------------------------------------------
struct Ring {
    uint32_t full0, empty0;      // shared-memory addresses of the first full / empty mbarrier
    uint32_t stage0;             // ... of stage 0
    WaitCtl ctl;
};

// Item `id` of the launch: which tensor, tile and candidates.  One lane runs this.
__device__ __forceinline__ bool decode_item(const Args& A, uint32_t id, uint32_t& seg_cache, ItemInfo& info) {
    if (id >= A.n_items) return false;
    const uint32_t n_seg = A.n_segments;
    uint32_t s = seg_cache;
    if (!(s < n_seg && A.segments[s].first_id <= id && id < A.segments[s + 1].first_id)) {
        uint32_t lo = 0, hi = n_seg;          // the segment with first_id <= id < next first_id
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (A.segments[mid].first_id <= id) lo = mid; else hi = mid;
        }
        s = lo;
        seg_cache = s;
    }
    const Segment sg = A.segments[s];
    if (!RKV_IN_BOUNDS(A.header, 1, sg.tensor < (uint32_t)A.T && sg.group < 3u, sg.tensor)) return false;
    const DevTensor& D = A.tensors[sg.tensor];
    const uint32_t local = sg.first_local + (id - sg.first_id);
    const uint32_t nt = group_tiles(sg.group, D.n_tiles, D.warm_tiles, D.tail_tiles);
    const uint32_t parts = D.parts[sg.group];
    const uint32_t part = local / nt;
    if (!RKV_IN_BOUNDS(A.header, 2, nt > 0 && part < parts, local)) return false;
    const uint32_t k_count = (uint32_t)(A.k_end - A.k_begin);
    const uint32_t k0 = part_begin(part, parts, k_count);
    info.id = id;
    info.t = sg.tensor;
    info.tile = local % nt + group_first_tile(sg.group, D.n_tiles, D.warm_tiles, D.tail_tiles);
    info.k0 = (uint32_t)A.k_begin + k0;
    info.kc = part_begin(part + 1, parts, k_count) - k0;
    return true;
}

// The producer warp.  Per item: draw the ticket for the one after it (its latency hides
// behind the rest), decode, fetch the part's candidate pointers with all lanes, publish the
// item's description, then lane 0 issues the item's copies in ring order, each as soon as
// every consumer warp has released the stage's previous use.
__device__ __forceinline__ void producer_loop(const Args& A, unsigned char* smem, const Ring& ring) {
    const int lane = threadIdx.x & 31;
    const void** table = reinterpret_cast<const void**>(smem + kOffPtrP);
    ItemInfo* infos = reinterpret_cast<ItemInfo*>(smem + kOffInfo);
    const uint32_t drill = blockIdx.x == 0u ? A.header->drill_issue : 0u;
    uint32_t n_issued = 0, stage = 0, phase = 0, seg = 0, ord = 0;
    uint32_t withheld = 0xFFFFFFFFu;          // ring stage a fault drill left unarmed

    auto issue = [&](const unsigned char* src, uint32_t bytes) {
        // the stage is free once every consumer warp has released its previous use; once a
        // wait of the block has run out nothing more is issued
        if (!mbar_wait(ring.empty0 + 8 * stage, phase ^ 1u, ring.ctl)) return;
        const uint32_t full = ring.full0 + 8 * stage;
        if (n_issued + 1u == drill) {
            // the fault drill of a test: this stage is neither armed nor filled, so whoever waits
            // for it runs into the wait limit; nothing is in flight because of it
            withheld = stage;
        } else if (bytes) {
            mbar_expect_tx(full, bytes);
            bulk_g2s(ring.stage0 + stage * kStageBytes, src, bytes, full);
        } else {
            mbar_arrive(full);
        }
        ++n_issued;
        if (++stage == (uint32_t)kStages) { stage = 0; phase ^= 1u; }
    };

    uint32_t id = blockIdx.x;                 // every block starts with the item of its own number
    for (;;) {
        id = __shfl_sync(kFullMask, id, 0);
        if (id >= A.n_items || *ring.ctl.abort_flag) break;
        uint32_t next_id = 0, ok = 0;
        ItemInfo info;
        info.id = kNoItem; info.t = 0; info.tile = 0; info.k0 = 0; info.kc = 0;
        info.reserved[0] = info.reserved[1] = info.reserved[2] = 0;
        if (lane == 0) {
            next_id = gridDim.x + atomicAdd(&A.header->next_ticket, 1u);
            ok = decode_item(A, id, seg, info) ? 1u : 0u;
        }
        if (!__shfl_sync(kFullMask, ok, 0)) break;
        const uint32_t t = __shfl_sync(kFullMask, info.t, 0);
        const uint32_t k0 = __shfl_sync(kFullMask, info.k0, 0);
        const uint32_t kc = __shfl_sync(kFullMask, info.kc, 0);
        const DevTensor& D = A.tensors[t];
        {
            const void* const* src = D.cands + k0;
            for (uint32_t i = (uint32_t)lane; i < kc; i += 32u)
                if (RKV_IN_BOUNDS(A.header, 6, i < (uint32_t)kPartK && k0 + i < (uint32_t)A.K, k0 + i)) table[i] = src[i];
        }
        __syncwarp();
        if (lane == 0) {
            infos[ord & (kInfoRing - 1)] = info;      // ordered before the arrive of the item's first stage
            const uint32_t csz = elem_bytes(D.cand_dtype), rsz = elem_bytes(D.ref_dtype);
            const uint32_t te = tile_elems(D.cand_dtype);
            const uint64_t start = (uint64_t)info.tile * te;
            const uint32_t len = (uint32_t)min((uint64_t)te, D.n - start);
            if (D.ref_src == RKV_SRC_POINTER) {
                const uint32_t nref = (te * rsz + kStageBytes - 1) / kStageBytes;
                const uint32_t rbytes = (len * rsz) & ~15u;
                const unsigned char* src = reinterpret_cast<const unsigned char*>(D.ref) + start * rsz;
                for (uint32_t r = 0; r < nref; ++r) {
                    const uint32_t lo = r * kStageBytes;
                    uint32_t b = rbytes > lo ? min(rbytes - lo, (uint32_t)kStageBytes) : 0u;
                    if (b && !RKV_IN_BOUNDS(A.header, 7, start * rsz + lo + b <= D.n * rsz, start)) b = 0u;
                    issue(src + lo, b);
                }
            }
            uint32_t cbytes = (len * csz) & ~15u;
            const uint64_t c_off = start * csz;
            if (cbytes && !RKV_IN_BOUNDS(A.header, 8, c_off + cbytes <= D.n * csz && cbytes <= (uint32_t)kStageBytes, c_off)) cbytes = 0u;
            for (uint32_t i = 0; i < kc; ++i)
                issue(reinterpret_cast<const unsigned char*>(table[i]) + c_off, cbytes);
        }
        __syncwarp();
        ++ord;
        id = next_id;
    }
    if (lane == 0) {
        ItemInfo end;
        end.id = kNoItem; end.t = 0; end.tile = 0; end.k0 = 0; end.kc = 0;
        end.reserved[0] = end.reserved[1] = end.reserved[2] = 0;
        infos[ord & (kInfoRing - 1)] = end;
        issue(nullptr, 0u);                              // tell the consumers to stop
        // the last block to get here clears the ticket counter for the next launch
        __threadfence();
        if (atomicAdd(&A.header->blocks_done, 1u) == gridDim.x - 1u) {
            A.header->next_ticket = 0u;
            A.header->blocks_done = 0u;
        }
        // A block that gave up must not retire with copies still landing in its shared
        // memory: wait (bounded) for the copies issued last.
        if (*ring.ctl.abort_flag) {
            const uint32_t pending = n_issued < (uint32_t)kStages ? n_issued : (uint32_t)kStages;
            for (uint32_t i = 0; i < pending; ++i) {
                const uint32_t q = n_issued - 1 - i;
                const uint32_t s = q % kStages, ph = (q / kStages) & 1u;
                if (s == withheld) continue;
                const long long t0 = clock64();
                for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
                    if (mbar_try_wait(ring.full0 + 8 * s, ph)) break;
                    if (clock64() - t0 > 200000000LL) break;
                }
            }
        }
    }
}

// A consumer warp has read ring stage `s`: release it.
__device__ __forceinline__ void release_stage(const Ring& ring, uint32_t s, int lane) {
    __syncwarp();
    mbar_arrive_if(ring.empty0 + 8 * s, lane == 0);
}

// ----------------------------------------------------------------------------
// per-thread view of a tile
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
template <bool C16>
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
__device__ __forceinline__ void input_group(const DevTensor& D, uint64_t start, uint32_t off0, uint32_t len,
                                            uint32_t out[4]) {
    if (D.input_src == RKV_SRC_GENERATED) {
        gen_group(D.in_seed, D.in_stream, D.in_dist, start, off0, D.cand_dtype == RKV_BF16, out);
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            out[i] = (off0 + i < len) ? ld_elem_bits(D.input, D.cand_dtype, start + off0 + i) : 0u;
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

// The thread's E elements of a tile of a generated tensor (distribution DIST), as fp32 bit
// patterns; bf16 == true rounds them to bf16 first.
template <int CK, int DIST>
__device__ __forceinline__ void gen_thread_tile(uint64_t seed, uint64_t stream_id, uint64_t start, int tid, bool bf16,
                                                uint32_t (&rb)[Geo<CK>::E]) {
    constexpr int E = Geo<CK>::E, VEC = Geo<CK>::VEC;
    const PhiloxKey key = philox_key(seed);
#pragma unroll
    for (int g = 0; g < E / 4; ++g) {
        float v[4];
        gen_block<DIST>((start + elem_off<VEC>(4 * g, tid)) >> 2, stream_id, key, v);
#pragma unroll
        for (int i = 0; i < 4; ++i) rb[4 * g + i] = bf16 ? (bf16_rne_bits(v[i]) << 16) : __float_as_uint(v[i]);
    }
}

// Load (or regenerate) the thread's reference values for a tile and derive what
// depends on them alone.  The bulk-copied part of the tile sits in ring stage
// `stage_a` (and, for an fp32 reference under 16-bit candidates, continues in
// `stage_b`); anything beyond comes from global memory.  `rb` returns all E values as
// fp32 bit patterns (for the reference's own loophole flags).
template <int CK>
__device__ __forceinline__ void load_ref(RefRegs<Geo<CK>::C16>& R, uint32_t (&rb)[Geo<CK>::E], const DevTensor& D,
                                         uint64_t start, uint32_t len, const unsigned char* stage_a,
                                         const unsigned char* stage_b, int tid) {
    constexpr int E = Geo<CK>::E, VEC = Geo<CK>::VEC;
    constexpr bool C16 = Geo<CK>::C16;
    const int rdt = D.ref_dtype;
    const uint32_t rsz = elem_bytes(rdt);
    const bool full = len == (uint32_t)Geo<CK>::kTile;
    // byte `b` of the reference tile in the ring
    auto at = [&](uint32_t b) -> const unsigned char* {
        return b < (uint32_t)kStageBytes ? stage_a + b : stage_b + (b - kStageBytes);
    };
    if (D.ref_src == RKV_SRC_GENERATED) {
        // the distribution is chosen once, outside the loop over the thread's Philox blocks: the
        // blocks are independent, and as straight-line code their long dependent chains overlap
        switch (D.ref_dist) {
            case 0: gen_thread_tile<CK, 0>(D.ref_seed, D.ref_stream, start, tid, rdt == RKV_BF16, rb); break;
            case 1: gen_thread_tile<CK, 1>(D.ref_seed, D.ref_stream, start, tid, rdt == RKV_BF16, rb); break;
            case 2: gen_thread_tile<CK, 2>(D.ref_seed, D.ref_stream, start, tid, rdt == RKV_BF16, rb); break;
            case 3: gen_thread_tile<CK, 3>(D.ref_seed, D.ref_stream, start, tid, rdt == RKV_BF16, rb); break;
            default: gen_thread_tile<CK, 4>(D.ref_seed, D.ref_stream, start, tid, rdt == RKV_BF16, rb); break;
        }
    } else if (full) {
#pragma unroll
        for (int g = 0; g < E / 4; ++g) {
            const uint32_t off0 = elem_off<VEC>(4 * g, tid);
            if (rdt != RKV_F32) {
                const uint2 t = *reinterpret_cast<const uint2*>(at(off0 * 2));
                rb[4 * g + 0] = upcast16(t.x & 0xFFFFu, rdt); rb[4 * g + 1] = upcast16(t.x >> 16, rdt);
                rb[4 * g + 2] = upcast16(t.y & 0xFFFFu, rdt); rb[4 * g + 3] = upcast16(t.y >> 16, rdt);
            } else {
                const uint4 t = *reinterpret_cast<const uint4*>(at(off0 * 4));
                rb[4 * g + 0] = t.x; rb[4 * g + 1] = t.y; rb[4 * g + 2] = t.z; rb[4 * g + 3] = t.w;
            }
        }
    } else {
        const uint32_t copied = ((len * rsz) & ~15u) / rsz;
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const uint32_t off = elem_off<VEC>(j, tid);
            uint32_t b = 0;
            if (off < copied) b = ld_elem_bits(at(off * rsz), rdt, 0);
            else if (off < len) b = ld_elem_bits(D.ref, rdt, start + off);
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
        if constexpr (C16) {
            has_zero |= ab == 0u;
        } else {
            R.thr[j] = thr;
            mn = min(mn, ab - 1u);   // |r| orders like its bits; zero wraps to the top
        }
    }
    R.thr_min = tmin;
    R.general = nonfinite;
    if constexpr (C16) {
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

// Candidate element j of the thread as an fp32 bit pattern.
template <int CK>
__device__ __forceinline__ uint32_t cand_bits(const uint32_t (&w)[16], int j) {
    if constexpr (CK == CK_F32) return w[j];
    else if constexpr (CK == CK_BF16) return (j & 1) ? (w[j >> 1] & 0xFFFF0000u) : (w[j >> 1] << 16);
    else return upcast16((j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xFFFFu), RKV_F16);
}

// Loophole flags of one candidate tile, until a difference has been seen.
template <int CK>
__device__ __forceinline__ void candidate_flags(const uint32_t (&w)[16], const Hint& h, Hint* h_smem,
                                                CandState* st, const DevTensor& D, const unsigned char* const* cand_p,
                                                uint64_t start, uint32_t len, uint32_t wanted_flags, int tid,
                                                int lane) {
    constexpr int E = Geo<CK>::E, VEC = Geo<CK>::VEC, NW = Geo<CK>::NW, DT = Geo<CK>::DTYPE;
    constexpr bool C16 = Geo<CK>::C16;
    constexpr uint32_t CSZ = C16 ? 2 : 4;
    // `settled` is the one hint field other warps update while this warp reads it: take
    // lane 0's copy so that the branch below is uniform across the warp.
    const uint32_t need = wanted_flags & ~__shfl_sync(kFullMask, h.settled, 0);
    if (need) {
        uint32_t acc1 = 0, acc2 = 0;
        const bool full = len == (uint32_t)Geo<CK>::kTile;
        if (full && (need & 1u)) {
            const uint32_t f = C16 ? h.first * 0x10001u : h.first;
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
            const uint32_t first_up = C16 ? upcast16(h.first, DT) : h.first;
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
                if (with_input && off0 < len) input_group(D, start, off0, len, in);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t off = off0 + i;
                    if (off < len) {
                        uint32_t cb = cand_bits<CK>(w, 4 * g + i);
                        if (off >= copied) cb = ld_elem_bits(*cand_p, DT, start + off);
                        if (!full) acc1 |= cb ^ first_up;
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

// One tile of an fp32 candidate against the thread's reference registers.
//   w        the thread's 16-byte pieces of the candidate tile (from the ring)
//   h        the candidate's hint entry (a snapshot; see the file header)
//   rec      the warp's running result for this candidate (shared memory; lane 0 writes)
//   st       the candidate's global state
//   cand_p   where the pointer to the candidate tensor in global memory is kept (only the last < 16 bytes of a
//            ragged tensor are read from there)
__device__ __forceinline__ void process_candidate_32(const RefRegs<false>& R, const uint32_t (&w)[16],
                                                     const Hint& h, Hint* h_smem, WarpRec* rec, CandState* st,
                                                     const DevTensor& D, const unsigned char* const* cand_p, uint32_t tile,
                                                     uint64_t start, uint32_t len, uint32_t wanted_flags,
                                                     int tid, int lane) {
    constexpr int CK = CK_F32;
    constexpr int E = Geo<CK>::E, VEC = Geo<CK>::VEC;
    constexpr uint32_t CSZ = 4;

    // ---- common path ---------------------------------------------------------------
    float e[E];
#pragma unroll
    for (int j = 0; j < E; ++j)
        e[j] = fabsf(__fsub_rn(__uint_as_float(w[j]), R.r[j]));
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
        if (lane == 0) rec->sum = (double)sf;
        candidate_flags<CK>(w, h, h_smem, st, D, cand_p, start, len, wanted_flags, tid, lane);
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
                    uint32_t cb = w[j];
                    if (off >= copied) cb = ld_elem_bits(*cand_p, RKV_F32, start + off);
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
            r.sum = sd;
            *rec = r;
        }
    } else {
        float sf = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sf = __fadd_rn(sf, __shfl_xor_sync(kFullMask, sf, off));
        if (lane == 0) rec->sum = (double)sf;
    }
    if (any_over || any_gen) {
        const uint32_t tot = __reduce_add_sync(kFullMask, cnt);
        if (lane == 0 && tot) rec->n_over += tot;
    }

    candidate_flags<CK>(w, h, h_smem, st, D, cand_p, start, len, wanted_flags, tid, lane);
}

// c - r for the 16-bit value c in the low (half = 0) or high 16 bits of x: the value
// widened exactly, one fp32 subtraction rounded to nearest (a mixed-precision instruction
// of sm_100).
template <int CK>
__device__ __forceinline__ float sub16_f32(uint32_t x, int half, float r) {
    float d;
    if constexpr (CK == CK_BF16) {
        if (half)
            asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, hi, %2;\n\t}" : "=f"(d) : "r"(x), "f"(r));
        else
            asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.bf16 %0, lo, %2;\n\t}" : "=f"(d) : "r"(x), "f"(r));
    } else {
        if (half)
            asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.f16 %0, hi, %2;\n\t}" : "=f"(d) : "r"(x), "f"(r));
        else
            asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tsub.rn.f32.f16 %0, lo, %2;\n\t}" : "=f"(d) : "r"(x), "f"(r));
    }
    return d;
}

// One pass over a thread's 32 elements of a 16-bit candidate tile: largest and summed
// e_j = |c_j - r_j|, and the largest d_j, where d_j = fma(-t, |r_j|, e_j) for the
// relative-error threshold t (see process_candidate_16).  HAS_ZERO: reference values of
// exactly 0 may occur; they take no part in the relative error, and d_j = e_j - atol there,
// positive exactly when the element is over tolerance.
template <int CK, bool HAS_ZERO>
__device__ __forceinline__ void pass_16(const RefRegs<true>& R, const uint32_t (&w)[16], float t, float& m_out,
                                        float& s_out, float& dm_out) {
    float m = 0.0f, dm = -kInf;
    float sg[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        float e[4], d[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = 4 * g + i;
            e[i] = fabsf(sub16_f32<CK>(w[j >> 1], j & 1, R.r[j]));
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

// Eight elements (one 16-byte piece) of each of two 16-bit candidates against reference
// values r[0..8): the work of pass_16 for both, sharing |r_j| and the test for a reference
// of zero.  acc = {m_a, dm_a, m_b, dm_b}; returns the two partial sums of the piece.
template <int CK, bool HAS_ZERO>
__device__ __forceinline__ void piece_16x2(const float* r, float atol, const uint4& a, const uint4& b, float ta,
                                           float tb, float (&acc)[4], float& sum_a, float& sum_b) {
    const uint32_t wa[4] = {a.x, a.y, a.z, a.w}, wb[4] = {b.x, b.y, b.z, b.w};
    float sa[2], sb[2];
#pragma unroll
    for (int g = 0; g < 2; ++g) {
        float ea[4], da[4], eb[4], db[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = 4 * g + i;
            ea[i] = fabsf(sub16_f32<CK>(wa[j >> 1], j & 1, r[j]));
            eb[i] = fabsf(sub16_f32<CK>(wb[j >> 1], j & 1, r[j]));
            const float ar = fabsf(r[j]);
            if (HAS_ZERO && ar == 0.0f) {
                da[i] = __fsub_rn(ea[i], atol);
                db[i] = __fsub_rn(eb[i], atol);
            } else {
                da[i] = __fmaf_rn(-ta, ar, ea[i]);
                db[i] = __fmaf_rn(-tb, ar, eb[i]);
            }
        }
        acc[0] = fmaxf(fmaxf(acc[0], fmaxf(ea[0], ea[1])), fmaxf(ea[2], ea[3]));
        acc[1] = fmaxf(fmaxf(acc[1], fmaxf(da[0], da[1])), fmaxf(da[2], da[3]));
        acc[2] = fmaxf(fmaxf(acc[2], fmaxf(eb[0], eb[1])), fmaxf(eb[2], eb[3]));
        acc[3] = fmaxf(fmaxf(acc[3], fmaxf(db[0], db[1])), fmaxf(db[2], db[3]));
        sa[g] = __fadd_rn(__fadd_rn(ea[0], ea[1]), __fadd_rn(ea[2], ea[3]));
        sb[g] = __fadd_rn(__fadd_rn(eb[0], eb[1]), __fadd_rn(eb[2], eb[3]));
    }
    sum_a = __fadd_rn(sa[0], sa[1]);
    sum_b = __fadd_rn(sb[0], sb[1]);
}

// Two whole tiles of 16-bit candidates straight from their ring stages (pa, pb: the thread's
// first 16-byte piece of each), common case only.  The pieces are read one ahead of the
// arithmetic; both stages are released once the last piece has been read.  Returns true when
// neither candidate needs anything but its error sum recorded (then rec[0].sum and rec[1].sum
// are written); false leaves both candidates to process_candidate_16.
template <int CK, bool HAS_ZERO>
__device__ __forceinline__ bool pair_common_16(const RefRegs<true>& R, const unsigned char* pa,
                                               const unsigned char* pb, uint32_t empty_a, uint32_t empty_b,
                                               const Hint& ha, const Hint& hb, WarpRec* rec, int lane) {
    constexpr float kTiny = 7.8886090522101181e-31f;      // 2^-100
    constexpr int kStep = kConsumers * 16;                // bytes from a thread's piece to its next one
    float acc[4] = {0.0f, -kInf, 0.0f, -kInf};
    float ca[4], cb[4];
    uint4 a = *reinterpret_cast<const uint4*>(pa), b = *reinterpret_cast<const uint4*>(pb);
#pragma unroll
    for (int jv = 0; jv < 4; ++jv) {
        uint4 an = a, bn = b;
        if (jv < 3) {
            an = *reinterpret_cast<const uint4*>(pa + (jv + 1) * kStep);
            bn = *reinterpret_cast<const uint4*>(pb + (jv + 1) * kStep);
        }
        if (jv == 2) {
            // every piece of both tiles has been read
            __syncwarp();
            mbar_arrive_if(empty_a, lane == 0);
            mbar_arrive_if(empty_b, lane == 0);
        }
        piece_16x2<CK, HAS_ZERO>(&R.r[8 * jv], R.atol, a, b, ha.tq_x, hb.tq_x, acc, ca[jv], cb[jv]);
        a = an; b = bn;
    }
    const float s_a = __fadd_rn(__fadd_rn(ca[0], ca[1]), __fadd_rn(ca[2], ca[3]));
    const float s_b = __fadd_rn(__fadd_rn(cb[0], cb[1]), __fadd_rn(cb[2], cb[3]));
    bool slow = R.general;
    {
        const float m = acc[0], dm = acc[1];
        const bool hit = dm > 0.0f || (dm == 0.0f && m != 0.0f && m < kTiny);
        const bool rel_covers = ha.tq_x >= 0.0f && ha.tq_x <= R.rtol;
        slow |= !(s_a < kInf) || (m > ha.te_x) || hit || (!rel_covers && m > R.thr_min);
    }
    {
        const float m = acc[2], dm = acc[3];
        const bool hit = dm > 0.0f || (dm == 0.0f && m != 0.0f && m < kTiny);
        const bool rel_covers = hb.tq_x >= 0.0f && hb.tq_x <= R.rtol;
        slow |= !(s_b < kInf) || (m > hb.te_x) || hit || (!rel_covers && m > R.thr_min);
    }
    if (__any_sync(kFullMask, slow)) return false;
    // both warp sums with one butterfly: lanes 0..15 end up with candidate a's, lanes 16..31 with
    // candidate b's; every level adds the same two values as the butterfly of one candidate
    const bool up = (lane & 16) != 0;
    const float keep = up ? s_b : s_a, give = up ? s_a : s_b;
    float v = __fadd_rn(keep, __shfl_xor_sync(kFullMask, give, 16));
#pragma unroll
    for (int off = 8; off > 0; off >>= 1) v = __fadd_rn(v, __shfl_xor_sync(kFullMask, v, off));
    if ((lane & 15) == 0) rec[lane >> 4].sum = (double)v;
    return true;
}

// One tile of a bf16 or fp16 candidate (32 elements per thread) against the thread's
// reference registers.  Same results as process_candidate_32; the tests that keep the rare
// work rare are arranged for errors proportional to |r|, the normal case of a rounded
// 16-bit output, against which a test on the thread's largest error is powerless.
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
template <int CK>
__device__ __forceinline__ void process_candidate_16(const RefRegs<true>& R, const uint32_t (&w)[16],
                                                     const Hint& h, Hint* h_smem, WarpRec* rec,
                                                     CandState* st, const DevTensor& D, const unsigned char* const* cand_p,
                                                     uint32_t tile, uint64_t start, uint32_t len,
                                                     uint32_t wanted_flags, int tid, int lane) {
    constexpr int VEC = 8;
    constexpr float kTiny = 7.8886090522101181e-31f;      // 2^-100

    // ---- common path ---------------------------------------------------------------
    float m, s, dm;
    if (R.warp_has_zero) pass_16<CK, true>(R, w, h.tq_x, m, s, dm);
    else pass_16<CK, false>(R, w, h.tq_x, m, s, dm);

    const bool lane_gen = R.general || !(s < kInf);
    const bool hit = dm > 0.0f || (dm == 0.0f && m != 0.0f && m < kTiny);
    const bool rare = (m > h.te_x) || lane_gen || hit;
    const bool rel_covers = h.tq_x >= 0.0f && h.tq_x <= R.rtol;
    const bool maybe_over = rel_covers ? hit : (m > R.thr_min);

    if (!__any_sync(kFullMask, rare || maybe_over)) {
        // nothing but the sum to record
        float sf = s;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sf = __fadd_rn(sf, __shfl_xor_sync(kFullMask, sf, off));
        if (lane == 0) rec->sum = (double)sf;
    } else {
        uint32_t cnt = 0;
        const bool any_over = __any_sync(kFullMask, maybe_over);
        if (any_over) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float e = fabsf(__fsub_rn(__uint_as_float(cand_bits<CK>(w, j)), R.r[j]));
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
                if (off < len) elem_general(a, cand_bits<CK>(w, j), __float_as_uint(R.r[j]), off, R.atol, R.rtol);
            }
            if (a.n_noncomp) atomicAdd(&st->n_noncomp, (unsigned long long)a.n_noncomp);
            if (a.n_nan) atomicAdd(&st->n_nan, (unsigned long long)a.n_nan);
            if (a.n_inf) atomicAdd(&st->n_inf, (unsigned long long)a.n_inf);
            if (a.n_infmis) atomicAdd(&st->n_infmis, (unsigned long long)a.n_infmis);
        } else if (rare) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float e = fabsf(__fsub_rn(__uint_as_float(cand_bits<CK>(w, j)), R.r[j]));
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
            r.sum = sd;
            r.n_over += tot;
            *rec = r;
        }
    }
    candidate_flags<CK>(w, h, h_smem, st, D, cand_p, start, len, wanted_flags, tid, lane);
}

// The error sums of the item just finished: for every candidate of its part, the warps'
// tile sums added in warp order, stored in the (tile, candidate) slot, and cleared.
// Called by all consumer threads between two consumer barriers.
__device__ __forceinline__ void flush_sums(WarpRec* recs, const Args& A, const DevTensor& D, uint32_t tile, int k0,
                                           int kc, int tid) {
    if (tid < kc) {
        double s = 0.0;
#pragma unroll
        for (int wp = 0; wp < kConsumerWarps; ++wp) {
            WarpRec& r = recs[wp * kPartK + tid];
            s += r.sum;
            r.sum = 0.0;
        }
        const unsigned long long at = D.sum_base + (unsigned long long)tile * (unsigned long long)A.K +
                                      (unsigned long long)(k0 + tid);
        if (RKV_IN_BOUNDS(A.header, 3, tile < D.n_tiles && k0 + tid < A.K, at)) A.sums[at] = s;
    }
}

// Merge the warp records of every candidate of a part into the Partial row and clear
// them.  Called by all consumer threads between two consumer barriers.
__device__ __forceinline__ void flush_records(WarpRec* recs, const Args& A, const DevTensor& D, int k0, int kc,
                                              uint32_t slot, int tid, uint32_t tile_elems_) {
    if (tid < kc) {
        Partial p;
        p.n_over = 0; p.eidx = RKV_NO_INDEX; p.qidx = RKV_NO_INDEX;
        p.emax = -1.0f; p.qmax = -1.0f; p.valid = 1u; p.reserved[0] = p.reserved[1] = p.reserved[2] = 0u;
#pragma unroll
        for (int wp = 0; wp < kConsumerWarps; ++wp) {
            WarpRec& r = recs[wp * kPartK + tid];
            p.n_over += r.n_over;
            if (r.emax >= 0.0f) {
                const uint64_t idx = (uint64_t)r.etile * tile_elems_ + (r.offs & 0xFFFFu);
                if (r.emax > p.emax || (r.emax == p.emax && idx < p.eidx)) { p.emax = r.emax; p.eidx = idx; }
            }
            if (r.qmax >= 0.0f) {
                const uint64_t idx = (uint64_t)r.qtile * tile_elems_ + (r.offs >> 16);
                if (r.qmax > p.qmax || (r.qmax == p.qmax && idx < p.qidx)) { p.qmax = r.qmax; p.qidx = idx; }
            }
            r.emax = -1.0f; r.etile = 0; r.qmax = -1.0f; r.qtile = 0; r.offs = 0; r.n_over = 0;
        }
        if (RKV_IN_BOUNDS(A.header, 4, slot < D.n_slots && k0 + tid < A.K, slot)) {
            // the slot may have been written before (another group, or an earlier launch of a
            // chunked call): merge
            Partial* dst = &A.partials[((size_t)D.slot_base + slot) * (size_t)A.K + (size_t)(k0 + tid)];
            const Partial old = *dst;
            if (old.valid) {
                p.n_over += old.n_over;
                if (old.emax > p.emax || (old.emax == p.emax && old.eidx < p.eidx)) { p.emax = old.emax; p.eidx = old.eidx; }
                if (old.qmax > p.qmax || (old.qmax == p.qmax && old.qidx < p.qidx)) { p.qmax = old.qmax; p.qidx = old.qidx; }
            }
            *dst = p;
        }
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

// What a block carries from item to item.
struct BlockState {
    uint32_t cstage, cphase;     // next ring stage to consume and the parity of its current use
    uint32_t ord;                // items this block has started
};

// Wait for the next ring stage.
__device__ __forceinline__ bool wait_stage(const Ring& ring, const BlockState& B, uint32_t& stage_out) {
    stage_out = B.cstage;
    return mbar_wait(ring.full0 + 8 * B.cstage, B.cphase, ring.ctl);
}

__device__ __forceinline__ void advance_stage(BlockState& B) {
    if (++B.cstage == (uint32_t)kStages) { B.cstage = 0; B.cphase ^= 1u; }
}

// One item: every candidate of the part against the tile's reference values.
template <int CK>
__device__ __forceinline__ void run_item(const Args& A, unsigned char* smem, const Ring& ring, BlockState& B,
                                         const ItemInfo& it, const DevTensor& D, bool same_part) {
    constexpr int E = Geo<CK>::E, VEC = Geo<CK>::VEC, NW = Geo<CK>::NW;
    constexpr int NV = E / VEC;
    constexpr bool C16 = Geo<CK>::C16;
    constexpr uint32_t kTile = Geo<CK>::kTile;
    constexpr uint32_t CSZ = C16 ? 2 : 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned char** ptrs = reinterpret_cast<const unsigned char**>(smem + kOffPtrC);
    uint32_t* firsts = reinterpret_cast<uint32_t*>(smem + kOffFirst);
    Hint* H = reinterpret_cast<Hint*>(smem + kOffHint) + (B.ord & 1u) * kPartK;
    WarpRec* recs = reinterpret_cast<WarpRec*>(smem + kOffRec);
    volatile uint32_t* ref_state = reinterpret_cast<volatile uint32_t*>(smem + kOffRefState);
    const unsigned char* stages = smem + kOffStage;

    const int k0 = (int)it.k0, kc = (int)it.kc;
    const uint64_t start = (uint64_t)it.tile * kTile;
    const uint32_t len = (uint32_t)min((uint64_t)kTile, D.n - start);
    // flags looked for: bit0 constant, bit1 copy of the input.  The reference is always checked for
    // both; with defer_copy the candidates are compared with the (regenerated) input on the warm-up
    // tiles only, and copy_check_kernel settles whoever is still bit-equal to it after them.
    const uint32_t wanted_ref = D.input_src != RKV_SRC_NONE ? 3u : 1u;
    const uint32_t wanted = (D.defer_copy && it.tile >= D.warm_tiles) ? 1u : wanted_ref;
    CandState* st_t = A.state + D.state_base;

    // (range checks of a debug build: the tile lies inside the tensor; the state, hint and
    // record tables are indexed by k0 + kk < K and kk < kPartK, checked with the item)
    if (!RKV_IN_BOUNDS(A.header, 9, start < D.n && it.tile < D.n_tiles, it.tile)) return;
    // the part's pointers (kept while the block stays with the part) and hints, from the
    // published state
    if (tid < kc) {
        const unsigned char* p;
        if (same_part) {
            p = ptrs[tid];
        } else {
            p = reinterpret_cast<const unsigned char*>(D.cands[k0 + tid]);
            ptrs[tid] = p;
            firsts[tid] = ld_elem_raw(p, Geo<CK>::DTYPE, 0);
        }
        const CandState* sc = st_t + k0 + tid;
        Hint h;
        h.te_x = hint_threshold(__ldcg(&sc->hint_e), it.tile);
        h.tq_x = hint_threshold(__ldcg(&sc->hint_q), it.tile);
        if (C16 && h.tq_x < 0.0f) h.tq_x = -kInf;     // see process_candidate_16
        h.settled = __ldcg(&sc->mismatch);
        h.first = firsts[tid];
        H[tid] = h;
    }
    if (tid == kPartK) ref_state[B.ord & 1u] = __ldcg(&st_t[A.K].mismatch);

    // ---- the thread's reference values --------------------------------------------
    RefRegs<C16> R;
    uint32_t rb[E];
    if (D.ref_src == RKV_SRC_POINTER) {
        // the reference tile fills one ring stage, or two (fp32 under 16-bit candidates)
        const bool two = (kTile * elem_bytes(D.ref_dtype)) > (uint32_t)kStageBytes;
        uint32_t sa, sb;
        wait_stage(ring, B, sa);
        advance_stage(B);
        sb = sa;
        if (two) {
            wait_stage(ring, B, sb);
            advance_stage(B);
        }
        load_ref<CK>(R, rb, D, start, len, stages + (size_t)sa * kStageBytes, stages + (size_t)sb * kStageBytes, tid);
        release_stage(ring, sa, lane);
        if (two) release_stage(ring, sb, lane);
    } else {
        load_ref<CK>(R, rb, D, start, len, nullptr, nullptr, tid);
    }
    consumer_sync();                          // hints, pointers and cleared records are visible

    // reference flags (constant / copy of the input), until a difference has been seen
    {
        const uint32_t need = wanted_ref & ~ref_state[B.ord & 1u];
        if (need) {
            const uint32_t r_first = first_elem_bits(D.ref, D.ref_src, D.ref_dtype, D.ref_seed,
                                                     D.ref_stream, D.ref_dist);
            uint32_t acc1 = 0, acc2 = 0;
#pragma unroll
            for (int g = 0; g < E / 4; ++g) {
                const uint32_t off0 = elem_off<VEC>(4 * g, tid);
                uint32_t in[4] = {0, 0, 0, 0};
                if ((need & 2u) && off0 < len) input_group(D, start, off0, len, in);
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
            if (lane == 0 && seen) atomicOr(&st_t[A.K].mismatch, seen);
        }
    }

    // ---- every candidate of the part ----------------------------------------------
    int kk = 0;
    if constexpr (C16) {
        // Whole tiles: two candidates per step while the common case holds.  The rare work
        // reads the candidate's pieces again, from global memory (the stages are released).
        if (len == kTile) {
            for (; kk + 1 < kc; kk += 2) {
                const Hint ha = H[kk], hb = H[kk + 1];
                uint32_t sa, sb;
                wait_stage(ring, B, sa);
                advance_stage(B);
                wait_stage(ring, B, sb);
                advance_stage(B);
                if (!RKV_IN_BOUNDS(A.header, 11, sa < (uint32_t)kStages && sb < (uint32_t)kStages, sa)) sa = sb = 0;
                WarpRec* rec = &recs[warp * kPartK + kk];
                const unsigned char* pa = stages + (size_t)sa * kStageBytes + (size_t)tid * 16;
                const unsigned char* pb = stages + (size_t)sb * kStageBytes + (size_t)tid * 16;
                const bool common =
                    R.warp_has_zero
                        ? pair_common_16<CK, true>(R, pa, pb, ring.empty0 + 8 * sa, ring.empty0 + 8 * sb, ha, hb, rec, lane)
                        : pair_common_16<CK, false>(R, pa, pb, ring.empty0 + 8 * sa, ring.empty0 + 8 * sb, ha, hb, rec, lane);
                const uint32_t settled = __shfl_sync(kFullMask, ha.settled & hb.settled, 0);
                if (!common || (wanted & ~settled)) {
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
                        uint32_t w[NW];
                        // (a whole tile: its kStageBytes lie inside the tensor)
                        const uint4* gp = reinterpret_cast<const uint4*>(ptrs[kk + c] + start * CSZ) + tid;
#pragma unroll
                        for (int jv = 0; jv < NV; ++jv) {
                            uint4 t = make_uint4(0u, 0u, 0u, 0u);
                            if (RKV_IN_BOUNDS(A.header, 12, (start + kTile) * CSZ <= D.n * CSZ, start)) t = __ldcg(gp + jv * kConsumers);
                            w[4 * jv + 0] = t.x; w[4 * jv + 1] = t.y; w[4 * jv + 2] = t.z; w[4 * jv + 3] = t.w;
                        }
                        const Hint h = c ? hb : ha;
                        if (!common)
                            process_candidate_16<CK>(R, w, h, &H[kk + c], rec + c, st_t + k0 + kk + c, D, &ptrs[kk + c],
                                                     it.tile, start, len, wanted, tid, lane);
                        else
                            candidate_flags<CK>(w, h, &H[kk + c], st_t + k0 + kk + c, D, &ptrs[kk + c], start, len, wanted,
                                                tid, lane);
                    }
                }
            }
        }
    }
    for (; kk < kc; ++kk) {
        const Hint h = H[kk];
        uint32_t s;
        wait_stage(ring, B, s);
        if (!RKV_IN_BOUNDS(A.header, 10, s < (uint32_t)kStages, s)) s = 0;
        const unsigned char* stage = stages + (size_t)s * kStageBytes;
        uint32_t w[NW];
#pragma unroll
        for (int jv = 0; jv < NV; ++jv) {
            const uint4 t = *reinterpret_cast<const uint4*>(stage + (size_t)(jv * kConsumers + tid) * 16);
            w[4 * jv + 0] = t.x; w[4 * jv + 1] = t.y; w[4 * jv + 2] = t.z; w[4 * jv + 3] = t.w;
        }
        release_stage(ring, s, lane);
        advance_stage(B);
        if (len != kTile) {
            // Ragged last tile: the copy brought whole 16-byte pieces only.  The few
            // elements behind them come from global memory; positions past the end of the
            // tensor get 0 against a reference of 0 (see load_ref): no error, never over
            // tolerance, excluded from the relative error, and never the first maximum,
            // because their offsets are larger than every real element's.
            const uint32_t copied = ((len * CSZ) & ~15u) / CSZ;
#pragma unroll
            for (int j = 0; j < E; ++j) {
                const uint32_t off = elem_off<VEC>(j, tid);
                if (off >= copied) {
                    const uint32_t cb = off < len ? ld_elem_raw(ptrs[kk], Geo<CK>::DTYPE, start + off) : 0u;
                    if (!C16) w[j] = cb;
                    else w[j >> 1] = (j & 1) ? ((w[j >> 1] & 0x0000FFFFu) | (cb << 16)) : ((w[j >> 1] & 0xFFFF0000u) | cb);
                }
            }
        }
        if constexpr (C16)
            process_candidate_16<CK>(R, w, h, &H[kk], &recs[warp * kPartK + kk], st_t + k0 + kk, D, &ptrs[kk],
                                     it.tile, start, len, wanted, tid, lane);
        else
            process_candidate_32(R, w, h, &H[kk], &recs[warp * kPartK + kk], st_t + k0 + kk, D, &ptrs[kk],
                                 it.tile, start, len, wanted, tid, lane);
    }
}

// The consumer warps: item after item, as the producer announces them.
__device__ __forceinline__ void consumer_loop(const Args& A, unsigned char* smem, const Ring& ring) {
    const int tid = threadIdx.x;
    WarpRec* recs = reinterpret_cast<WarpRec*>(smem + kOffRec);
    const ItemInfo* infos = reinterpret_cast<const ItemInfo*>(smem + kOffInfo);
    // clear the records once; the flushes leave them cleared
    for (int i = tid; i < kConsumerWarps * kPartK; i += kConsumers) {
        WarpRec& r = recs[i];
        r.emax = -1.0f; r.etile = 0; r.qmax = -1.0f; r.qtile = 0; r.offs = 0; r.n_over = 0; r.sum = 0.0;
    }
    BlockState B;
    B.cstage = 0; B.cphase = 0; B.ord = 0;

    int cur_t = -1, cur_k0 = 0, cur_kc = 0;
    uint32_t cur_slot = 0, cur_tile = 0, cur_te = 0;
    for (;; ++B.ord) {
        // The next item announces itself before its first ring stage is armed (that stage stays
        // full until it is consumed in run_item).  All consumers agree on stopping: at the
        // producer's end mark, or when any thread of the block has given up on a wait.
        uint32_t s0;
        const bool got = wait_stage(ring, B, s0);
        ItemInfo it = infos[B.ord & (kInfoRing - 1)];
        if (!got) it.id = kNoItem;
        if (consumer_sync_or((it.id == kNoItem || *ring.ctl.abort_flag) ? 1u : 0u)) break;
        if (!RKV_IN_BOUNDS(A.header, 5, it.t < (uint32_t)A.T && it.kc >= 1u && it.kc <= (uint32_t)kPartK &&
                                            it.k0 + it.kc <= (uint32_t)A.K, it.t))
            break;
        const DevTensor& D = A.tensors[it.t];
        // every warp is done with the previous item: its sums, and, when the tensor or the
        // candidates change, its records
        if (cur_t >= 0) {
            flush_sums(recs, A, A.tensors[cur_t], cur_tile, cur_k0, cur_kc, tid);
            if ((int)it.t != cur_t || (int)it.k0 != cur_k0 || (int)it.kc != cur_kc ||
                (A.tensors[cur_t].slot_by_tile && it.tile != cur_tile))
                flush_records(recs, A, A.tensors[cur_t], cur_k0, cur_kc, cur_slot, tid, cur_te);
        }
        const bool same_part = (int)it.t == cur_t && (int)it.k0 == cur_k0 && (int)it.kc == cur_kc;
        cur_t = (int)it.t; cur_k0 = (int)it.k0; cur_kc = (int)it.kc; cur_tile = it.tile;
        cur_slot = D.slot_by_tile ? it.tile : blockIdx.x;
        cur_te = tile_elems(D.cand_dtype);
        // (the stage waited for above is consumed inside run_item: it holds the item's reference
        // tile or its first candidate)
        switch (D.cand_dtype) {
            case RKV_F32: run_item<CK_F32>(A, smem, ring, B, it, D, same_part); break;
            case RKV_BF16: run_item<CK_BF16>(A, smem, ring, B, it, D, same_part); break;
            default: run_item<CK_F16>(A, smem, ring, B, it, D, same_part); break;
        }
    }
    consumer_sync();
    if (cur_t >= 0) {
        flush_sums(recs, A, A.tensors[cur_t], cur_tile, cur_k0, cur_kc, tid);
        flush_records(recs, A, A.tensors[cur_t], cur_k0, cur_kc, cur_slot, tid, cur_te);
    }
    if (tid == 0 && *ring.ctl.abort_flag) atomicCAS(&A.header->status, (int32_t)RKV_OK, (int32_t)RKV_ERR_TIMEOUT);
}

// Persistent blocks, kBlocksPerSm per SM.
__global__ void __launch_bounds__(kThreads, kBlocksPerSm) verify_kernel(const __grid_constant__ Args A) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x;
    Ring ring;
    ring.full0 = smem_u32(smem + kOffFull);
    ring.empty0 = smem_u32(smem + kOffEmpty);
    ring.stage0 = smem_u32(smem + kOffStage);
    ring.ctl.abort_flag = reinterpret_cast<volatile uint32_t*>(smem + kOffAbort);
    ring.ctl.limit = reinterpret_cast<const volatile long long*>(smem + kOffWaitLimit);
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(ring.full0 + 8 * s, 1);                    // the producer's arrive + the copy's bytes
            mbar_init(ring.empty0 + 8 * s, kConsumerWarps);      // one release per consumer warp
        }
        *ring.ctl.abort_flag = 0u;
        const unsigned long long lim = A.header->drill_issue ? A.header->drill_wait_cycles : 0ull;
        *reinterpret_cast<volatile long long*>(smem + kOffWaitLimit) = lim ? (long long)lim : kWaitCycles;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid >= kConsumers) producer_loop(A, smem, ring);
    else consumer_loop(A, smem, ring);
}

// ----------------------------------------------------------------------------
// copy check: candidates still bit-equal to a regenerated input after the warm-up tiles
// ----------------------------------------------------------------------------
// The whole grid compares one such candidate with the input, regenerated Philox block by
// Philox block (four elements of the candidate per thread and step), and stops at the
// first difference any thread finds.  Only true copies are read to the end.
constexpr int kCopyThreads = 256;

template <int DIST, bool BF16>
__device__ __noinline__ void copy_check_scan(const DevTensor& D, const unsigned char* cand, CandState* st) {
    const PhiloxKey key = philox_key(D.in_seed);
    // one Philox block = four elements per thread and step: 16 bytes of an fp32 candidate, 8 of a bf16 one
    const uint64_t n = D.n, stream_id = D.in_stream;
    const uint64_t n_whole = n >> 2;
    const uint64_t stride = (uint64_t)gridDim.x * kCopyThreads;
    uint64_t u = (uint64_t)blockIdx.x * kCopyThreads + threadIdx.x;
    while (u < n_whole) {
        // somebody has found a difference: done (looked at every 8th step)
        if (__ldcg(&st->mismatch) & 2u) return;
#pragma unroll 1
        for (int j = 0; j < 8 && u < n_whole; ++j, u += stride) {
            // the candidate's piece is asked for first: its latency hides behind the generation
            uint4 c = make_uint4(0u, 0u, 0u, 0u);
            if (BF16) {
                const uint2 h = __ldcs(reinterpret_cast<const uint2*>(cand) + u);
                c.x = h.x; c.y = h.y;
            } else {
                c = __ldcs(reinterpret_cast<const uint4*>(cand) + u);
            }
            float v[4];
            gen_block<DIST>(u, stream_id, key, v);
            uint32_t diff;
            if (BF16) diff = (c.x ^ (bf16_rne_bits(v[0]) | (bf16_rne_bits(v[1]) << 16))) |
                             (c.y ^ (bf16_rne_bits(v[2]) | (bf16_rne_bits(v[3]) << 16)));
            else diff = (c.x ^ __float_as_uint(v[0])) | (c.y ^ __float_as_uint(v[1])) |
                        (c.z ^ __float_as_uint(v[2])) | (c.w ^ __float_as_uint(v[3]));
            if (diff) {
                atomicOr(&st->mismatch, 2u);
                return;
            }
        }
    }
    // the last one to three elements of a tensor whose length is no multiple of four
    if ((n & 3u) && blockIdx.x == 0 && threadIdx.x == 0) {
        float v[4];
        gen_block<DIST>(n_whole, stream_id, key, v);
        uint32_t diff = 0;
        for (uint32_t q = 0; q < (uint32_t)(n & 3u); ++q)
            diff |= ld_elem_raw(cand, BF16 ? RKV_BF16 : RKV_F32, (n_whole << 2) + q) ^
                    (BF16 ? bf16_rne_bits(v[q]) : __float_as_uint(v[q]));
        if (diff) atomicOr(&st->mismatch, 2u);
    }
}

// Every block goes through the same (tensor, candidate) pairs, found 256 at a time by all its
// threads at once (one global read per thread instead of one after the other), and takes its
// share of each pair's pieces.
__global__ void __launch_bounds__(kCopyThreads)
copy_check_kernel(const DevTensor* __restrict__ tensors, int T, int k_begin, int k_end, CandState* state) {
    __shared__ unsigned char t_flag[kCopyThreads], k_flag[kCopyThreads];
    const int tid = threadIdx.x;
    for (int t0 = 0; t0 < T; t0 += kCopyThreads) {
        const int mine_t = (t0 + tid < T && tensors[t0 + tid].defer_copy) ? 1 : 0;
        t_flag[tid] = (unsigned char)mine_t;
        if (!__syncthreads_or(mine_t)) continue;
        const int t_end = min(T - t0, kCopyThreads);
        for (int ti = 0; ti < t_end; ++ti) {
            if (!t_flag[ti]) continue;
            const DevTensor& D = tensors[t0 + ti];
            const bool b16 = D.cand_dtype == RKV_BF16;
            for (int kb = k_begin; kb < k_end; kb += kCopyThreads) {
                const int k = kb + tid;
                const int mine_k = (k < k_end && !(__ldcg(&state[D.state_base + k].mismatch) & 2u)) ? 1 : 0;
                __syncthreads();                       // the previous round's flags have been read
                k_flag[tid] = (unsigned char)mine_k;
                if (!__syncthreads_or(mine_k)) continue;
                const int k_cnt = min(k_end - kb, kCopyThreads);
                for (int ki = 0; ki < k_cnt; ++ki) {
                    if (!k_flag[ki]) continue;
                    CandState* st = state + D.state_base + kb + ki;
                    const unsigned char* cand = reinterpret_cast<const unsigned char*>(D.cands[kb + ki]);
                    switch (D.in_dist) {
                        case 0: b16 ? copy_check_scan<0, true>(D, cand, st) : copy_check_scan<0, false>(D, cand, st); break;
                        case 1: b16 ? copy_check_scan<1, true>(D, cand, st) : copy_check_scan<1, false>(D, cand, st); break;
                        case 2: b16 ? copy_check_scan<2, true>(D, cand, st) : copy_check_scan<2, false>(D, cand, st); break;
                        case 3: b16 ? copy_check_scan<3, true>(D, cand, st) : copy_check_scan<3, false>(D, cand, st); break;
                        default: b16 ? copy_check_scan<4, true>(D, cand, st) : copy_check_scan<4, false>(D, cand, st); break;
                    }
                }
            }
        }
        __syncthreads();                               // t_flag is rewritten by the next round
    }
}

// ----------------------------------------------------------------------------
// finalize: merge the per-block partials of each (candidate, tensor) in a fixed
// order, add the tile sums in tile order, derive flags and verdict; then the joint
// verdicts over the tensors of a case and over the cases
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

// The result of candidate k on tensor t, by one block; returns the verdict (in thread 0).
__device__ __forceinline__ uint32_t finalize_one(Wide* red, const DevTensor* __restrict__ tensors, int t, int k, int K,
                                                 const CandState* __restrict__ state,
                                                 const Partial* __restrict__ partials,
                                                 const double* __restrict__ sums,
                                                 rkv_stats* __restrict__ stats_out) {
    const int tid = threadIdx.x;
    uint32_t verdict_out = 0;
    const DevTensor D = tensors[t];
    Wide w;
    w.n_over = 0; w.sum = 0.0;
    w.emax = -1.0f; w.qmax = -1.0f; w.eidx = RKV_NO_INDEX; w.qidx = RKV_NO_INDEX;
    for (uint32_t s = tid; s < D.n_slots; s += kFinThreads) {
        const Partial p = partials[((size_t)D.slot_base + s) * (size_t)K + (size_t)k];
        if (!p.valid) continue;
        Wide b;
        b.n_over = p.n_over; b.sum = 0.0;
        b.emax = p.emax; b.eidx = p.eidx; b.qmax = p.qmax; b.qidx = p.qidx;
        wide_merge(w, b);
    }
    // tile sums: thread i adds tiles i, i + 128, ... in that order; the tree below is fixed
    for (uint32_t tile = tid; tile < D.n_tiles; tile += kFinThreads)
        w.sum += sums[D.sum_base + (unsigned long long)tile * (unsigned long long)K + (unsigned long long)k];
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
        const CandState cs = state[(size_t)D.state_base + (size_t)k];
        const uint32_t ref_mismatch = state[(size_t)D.state_base + (size_t)K].mismatch;
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
        stats_out[D.out_base + (unsigned long long)k * D.out_stride] = st;
        verdict_out = verdict;
    }
    __syncthreads();                  // `red` is free for the next tensor
    return verdict_out;
}

// One block per (tensor, candidate); the verdicts of a case meet in its fail words (a sweep).
__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(const DevTensor* __restrict__ tensors, int T, int K, const CandState* __restrict__ state,
                const Partial* __restrict__ partials, const double* __restrict__ sums,
                rkv_stats* __restrict__ stats_out, uint32_t* __restrict__ fail) {
    __shared__ Wide red[kFinThreads];
    const int t = blockIdx.x / K, k = blockIdx.x % K;
    if (t >= T) return;
    const uint32_t verdict = finalize_one(red, tensors, t, k, K, state, partials, sums, stats_out);
    if (threadIdx.x == 0 && verdict)
        atomicOr(&fail[(size_t)tensors[t].case_index * (size_t)K + (size_t)k], 1u);
}

// One case: one block per candidate goes through the case's tensors and writes the joint verdict.
__global__ void __launch_bounds__(kFinThreads)
finalize_case_kernel(const DevTensor* __restrict__ tensors, int T, int K, const CandState* __restrict__ state,
                     const Partial* __restrict__ partials, const double* __restrict__ sums,
                     rkv_stats* __restrict__ stats_out, uint32_t* __restrict__ joint_pass) {
    __shared__ Wide red[kFinThreads];
    const int k = blockIdx.x;
    uint32_t failed = 0;
    for (int t = 0; t < T; ++t) failed |= finalize_one(red, tensors, t, k, K, state, partials, sums, stats_out);
    if (threadIdx.x == 0 && joint_pass) joint_pass[k] = failed ? 0u : 1u;
}

// case_pass[c][k] = candidate k passed on every tensor of case c; all_pass[k] = on every case.
__global__ void joint_kernel(const uint32_t* __restrict__ fail, int K, uint32_t n_cases,
                             uint32_t* __restrict__ case_pass, uint32_t* __restrict__ all_pass) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    uint32_t all = 1u;
    for (uint32_t c = 0; c < n_cases; ++c) {
        const uint32_t ok = fail[(size_t)c * (size_t)K + (size_t)k] ? 0u : 1u;
        if (case_pass) case_pass[(size_t)c * (size_t)K + (size_t)k] = ok;
        all &= ok;
    }
    if (all_pass) all_pass[k] = all;
}

}  // namespace

int launch_verify(const Layout& L, int T, int K, int k_begin, int k_end, uint32_t n_items, uint32_t n_segments,
                  int grid, cudaStream_t stream) {
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RKV_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) !=
            cudaSuccess)
            return RKV_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    Args A;
    A.tensors = L.d_tensors; A.segments = L.d_segments; A.state = L.state; A.partials = L.partials;
    A.sums = L.sums; A.header = L.header;
    A.T = T; A.K = K; A.k_begin = k_begin; A.k_end = k_end; A.n_items = n_items; A.n_segments = n_segments;
    // the grid is always the full resident grid: Partial rows of large tensors are numbered by block
    verify_kernel<<<grid, kThreads, kSmemBytes, stream>>>(A);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

// Resident blocks per SM the device grants the verification kernel (0 on error).
int verify_occupancy() {
    int n = 0;
    if (cudaFuncSetAttribute(verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, verify_kernel, kThreads, kSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

int launch_copy_check(const Layout& L, int T, int K, int k_begin, int k_end, int num_sms, cudaStream_t stream) {
    (void)K;
    copy_check_kernel<<<(unsigned)num_sms * 3u, kCopyThreads, 0, stream>>>(L.d_tensors, T, k_begin, k_end, L.state);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

int launch_finalize(const Layout& L, int T, int K, uint32_t n_cases, rkv_stats* stats_out, uint32_t* case_pass,
                    uint32_t* all_pass, cudaStream_t stream) {
    if (n_cases == 1 && !case_pass && T <= kMaxTensors) {
        // one case: no second kernel for the joint verdict
        finalize_case_kernel<<<(unsigned)K, kFinThreads, 0, stream>>>(L.d_tensors, T, K, L.state, L.partials, L.sums,
                                                                     stats_out, all_pass);
        return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
    }
    finalize_kernel<<<(unsigned)T * (unsigned)K, kFinThreads, 0, stream>>>(L.d_tensors, T, K, L.state, L.partials,
                                                                          L.sums, stats_out, L.fail);
    if (cudaGetLastError() != cudaSuccess) return RKV_ERR_CUDA;
    if (case_pass || all_pass) {
        joint_kernel<<<(K + 127) / 128, 128, 0, stream>>>(L.fail, K, n_cases, case_pass, all_pass);
        if (cudaGetLastError() != cudaSuccess) return RKV_ERR_CUDA;
    }
    return RKV_OK;
}

}  // namespace rkv
