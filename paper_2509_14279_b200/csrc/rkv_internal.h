// Internal declarations shared by the translation units of librkv (host side).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "rkv.h"

namespace rkv {

// ---- verification kernel geometry ------------------------------------------------
constexpr int kConsumerWarps = 7;                    // warps that compare
constexpr int kConsumers = kConsumerWarps * 32;      // 224 threads
constexpr int kThreads = kConsumers + 32;            // + one warp that issues the bulk copies = 256
constexpr int kBlocksPerSm = 2;                      // resident verification blocks per SM
constexpr int kStageBytes = kConsumers * 64;         // a ring stage: 64 bytes of a candidate per thread
// A thread owns 64 bytes of each candidate tile: 16 fp32 or 32 16-bit elements.
constexpr int kTileElems32 = kStageBytes / 4;        // 3584 elements per tile of fp32 candidates
constexpr int kTileElems16 = kStageBytes / 2;        // 7168 elements per tile of bf16 / fp16 candidates
__host__ __device__ constexpr bool is16(int dtype) { return dtype != RKV_F32; }
__host__ __device__ constexpr uint32_t elem_bytes(int dtype) { return dtype == RKV_F32 ? 4u : 2u; }
__host__ __device__ constexpr uint32_t tile_elems(int cand_dtype) {
    return is16(cand_dtype) ? kTileElems16 : kTileElems32;
}
constexpr int kStages = 5;                           // ring depth (bulk copies in flight)
constexpr int kPartK = 64;                           // candidates a block tracks at a time
constexpr int kWarmTiles = 18;                       // leading tiles of a tensor that are verified first: the square root of its tiles, at most this
constexpr int kTailDiv = 4;                          // a tail item covers a quarter of a part's candidates ...
constexpr int kTailDivGenerated = 2;                 // ... half, when every item regenerates its reference tile
constexpr int kMaxTensors = 64;                      // rkv_verify_multi
constexpr int kMaxSweepTensors = 4096;               // rkv_verify_sweep, over all its cases
constexpr uint64_t kMaxN = 1ull << 40;

// Result of one thread block (or, for a small tensor, of one tile) for one (tensor,
// candidate); merged by the finalize kernel.  The error sum is not here: it goes to the
// tile sums, one per (tile, candidate), so that its value does not depend on which block
// verified which tile.
struct __align__(16) Partial {
    uint64_t n_over;
    uint64_t eidx;       // tensor-wide element index of the first maximum of |c - r|
    uint64_t qidx;       // same for |c - r| / |r|
    float emax;          // -1 when the block saw no comparable element
    float qmax;
    uint32_t valid;      // 0 in the zero-filled workspace, 1 once a block has written the slot
    uint32_t reserved[3];
};
static_assert(sizeof(Partial) == 48, "Partial layout");

// Global per-(tensor, candidate) state, zero-filled before the launch.  Slot K of
// a tensor belongs to the reference (only `mismatch` is used there).
struct __align__(16) CandState {
    // Running maxima published by all blocks, only ever used to skip work:
    // ((bits(max) + 1) << 32) | ~tile, 0 = nothing published yet.
    unsigned long long hint_e;
    unsigned long long hint_q;
    unsigned long long n_noncomp;   // elements that are not comparable
    unsigned long long n_nan;
    unsigned long long n_inf;
    unsigned long long n_infmis;
    uint32_t mismatch;              // bit0: some element differs from element 0; bit1: from the input
    uint32_t reserved[3];
};
static_assert(sizeof(CandState) == 64, "CandState layout");

// Device-side description of one tensor of a launch.
//
// Work items.  A large tensor has three groups of items: group 0 covers its first
// warm_tiles tiles with small candidate parts (so that all blocks take part), group 1
// the tiles after them with parts of up to kPartK candidates, group 2 its last
// tail_tiles tiles with smaller parts.  Group 0 runs first: the maxima and loophole flags
// it publishes let the rest skip almost all rare-path work.  Group 2 runs last: its
// short items even out the finishing times of the blocks.  A short tensor warms up on
// the square root of its tiles; in a launch whose tiles all fit the first wave of
// blocks every tile is in group 0.  Within a group, local item = part * tiles + tile.  The launch-wide item
// numbering is given by the segment table (see Segment).
struct DevTensor {
    uint64_t n;
    const void* ref;
    const void* input;
    const void* const* cands;   // device array of K device pointers
    uint64_t ref_seed, ref_stream;
    uint64_t in_seed, in_stream;
    int32_t ref_dist, in_dist;
    int32_t cand_dtype, ref_dtype;
    int32_t ref_src, input_src;
    float atol, rtol;
    uint32_t n_tiles;       // ceil(n / tile_elems(cand_dtype))
    uint32_t warm_tiles;    // tiles in group 0 (== n_tiles when there are no other groups)
    uint32_t tail_tiles;    // tiles in group 2
    uint32_t parts[3];      // candidate parts of each group in this launch
    uint32_t n_slots;       // Partial rows of this tensor: one per block, or one per tile (small tensors)
    uint32_t slot_base;     // first Partial row (K entries per row) of this tensor
    uint32_t slot_by_tile;  // 1: Partial row = tile index; 0: Partial row = block index
    uint32_t state_base;    // first CandState of this tensor (K + 1 entries)
    uint32_t out_stride;    // rkv_stats index step from candidate k to k + 1 (tensors of the tensor's case)
    uint32_t case_index;    // the case this tensor belongs to (0 unless a sweep)
    // 1: the input is regenerated and the tensor has tiles beyond its warm-up group.  The
    // verification kernel then compares candidates with the input on the warm-up tiles only
    // (which settles every candidate that is no copy); the few candidates still bit-equal to
    // the input after them are compared over the whole tensor by copy_check_kernel.
    uint32_t defer_copy;
    uint32_t reserved0;
    uint64_t sum_base;      // first tile sum (n_tiles x K doubles, [tile][k]) of this tensor
    uint64_t out_base;      // rkv_stats index of candidate 0 of this tensor
};

// A run of consecutive launch-wide item ids that map to consecutive local items of one
// (tensor, group).  Sorted by first_id; the last entry is a sentinel with first_id = total.
struct Segment {
    uint32_t first_id;
    uint32_t first_local;
    uint32_t tensor;
    uint32_t group;
};

struct WorkspaceHeader {
    int32_t status;        // rkv_status written by the device
    // Work distribution of the verification kernel: every block starts with item blockIdx.x
    // and then draws tickets; item = grid + ticket.  The last block to finish clears both
    // words again, so that the next launch on the workspace starts from zero.
    uint32_t next_ticket;
    uint32_t blocks_done;
    uint32_t reserved2;
    // Fault drill (a test makes a bounded wait run out without any memory fault):
    // when drill_issue != 0, block 0 skips its drill_issue-th copy (the ring stage is neither
    // armed nor filled), and every wait gives up after drill_wait_cycles clock cycles.
    uint32_t drill_issue;
    uint32_t reserved0;
    unsigned long long drill_wait_cycles;
    // First failed range check of a build with RKV_DEBUG_BOUNDS (site number, offending value).
    uint32_t bounds_site;
    uint32_t reserved1;
    unsigned long long bounds_value;
    uint32_t reserved[52];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header size");

// How a launch is cut into work items, and where everything lives in the workspace:
//   header | tensor descriptors | segment table | pointer tables | per-case fail words |
//   CandState[T][K+1] | Partial[rows][K] | tile sums
// The two tables live in storage the caller provides (vectors, or arrays on the stack of
// the entry point that must not allocate).
struct Plan {
    DevTensor* tensors = nullptr;        // T entries; planning fields filled in, pointers set by the caller
    Segment* segments = nullptr;         // n_segments + 1 entries (the last one is the sentinel)
    size_t segment_capacity = 0;         // entries `segments` has room for
    int T = 0;
    uint32_t n_segments = 0;
    uint32_t grid = 0;                   // blocks per launch (num_sms * kBlocksPerSm)
    uint32_t n_items = 0;
    uint32_t n_cases = 1;
    bool any_deferred = false;           // some tensor has defer_copy set: copy_check_kernel runs after verify_kernel
    size_t off_tensors = 0, off_segments = 0, off_ptrs = 0, off_fail = 0, off_state = 0, off_partials = 0,
           off_sums = 0;
    size_t upload_bytes = 0;             // header + descriptors + segments + pointer tables
    size_t clear_bytes = 0;              // fail words + CandState + Partials (from off_fail)
    size_t total_bytes = 0;
};

// Entries a segment table needs at most for T tensors (sentinel included).
size_t segment_bound(int T);

int validate_tensors(const rkv_tensor_desc* tensors, int T, int K, int max_tensors);
// Fills plan->tensors[0..T) (every field except the pointer `cands`, which the caller sets
// once the workspace address is known), the segment table for a launch over k_count
// candidates, and the workspace layout.
//   case_of[t], out_base[t], out_stride[t]   where a sweep puts tensor t (null: one case,
//                                            results at [k * T + t])
int make_plan(const rkv_tensor_desc* tensors, int T, int K, int k_count, int num_sms, const uint32_t* case_of,
              const uint64_t* out_base, const uint32_t* out_stride, uint32_t n_cases, Plan* plan);
// Candidate parts and item numbering for a launch over k_count candidates (the chunked
// host form calls this again for a shorter last chunk).
void plan_items(Plan* plan, int k_count);
int current_num_sms(int* num_sms);   // RKV_ERR_CUDA without a device
int refuse_capture(cudaStream_t stream);   // RKV_ERR_UNSUPPORTED while `stream` is being captured

// Number of candidate parts for a group in a launch over k_count candidates: enough parts
// that none holds more than kPartK candidates, and, when the launch's group has fewer tiles
// (`launch_tiles`, over all its tensors) than there are blocks, enough that every block gets
// an item where k_count allows.  Part p of `parts` covers the candidates
// [p * k_count / parts, (p + 1) * k_count / parts): sizes differ by at most one.
__host__ __device__ inline uint32_t part_count(uint32_t launch_tiles, uint32_t k_count, uint32_t grid) {
    uint32_t parts = (k_count + kPartK - 1) / kPartK;
    if (launch_tiles < grid) {
        const uint32_t want = (grid + launch_tiles - 1) / launch_tiles;
        if (want > parts) parts = want;
    }
    return parts > k_count ? k_count : parts;
}

// Tiles and first tile of group g (0, 1, 2) of a tensor.
__host__ __device__ inline uint32_t group_tiles(uint32_t g, uint32_t n_tiles, uint32_t warm, uint32_t tail) {
    return g == 0 ? warm : g == 1 ? n_tiles - warm - tail : tail;
}
__host__ __device__ inline uint32_t group_first_tile(uint32_t g, uint32_t n_tiles, uint32_t warm, uint32_t tail) {
    return g == 0 ? 0u : g == 1 ? warm : n_tiles - tail;
}
// Tiles in group 2: half a tile per block, for tensors long enough that the blocks'
// finishing times would otherwise differ by up to a whole item.
__host__ __device__ inline uint32_t tail_tiles_of(uint32_t n_tiles, uint32_t warm, uint32_t grid) {
    return (n_tiles - warm >= 4u * grid && grid >= 2u) ? grid / 2u : 0u;
}

__host__ __device__ inline uint32_t part_begin(uint32_t part, uint32_t parts, uint32_t k_count) {
    return (uint32_t)(((uint64_t)part * k_count) / parts);
}

// Pieces of a workspace.
struct Layout {
    WorkspaceHeader* header;
    DevTensor* d_tensors;
    Segment* d_segments;
    const void** d_ptrs;
    uint32_t* fail;          // [n_cases][K] words: non-zero once candidate k failed on a tensor of the case
    CandState* state;
    Partial* partials;
    double* sums;
};

// kernels (rkv_verify.cu / rkv_gen.cu)
int launch_verify(const Layout& L, int T, int K, int k_begin, int k_end, uint32_t n_items, uint32_t n_segments,
                  int grid, cudaStream_t stream);
int verify_occupancy();   // resident verification blocks per SM on the current device
// Candidates [k_begin, k_end) of every tensor with defer_copy set that are still bit-equal to the
// regenerated input after the warm-up tiles: compared with it over the whole tensor.
int launch_copy_check(const Layout& L, int T, int K, int k_begin, int k_end, int num_sms, cudaStream_t stream);
int launch_finalize(const Layout& L, int T, int K, uint32_t n_cases, rkv_stats* stats_out, uint32_t* case_pass,
                    uint32_t* all_pass, cudaStream_t stream);
int launch_gen(uint64_t seed, uint64_t stream_id, int dist, uint64_t n, uint64_t first_elem,
               int dtype, void* out, int num_sms, cudaStream_t stream);

}  // namespace rkv
