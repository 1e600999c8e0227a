// Internal declarations shared by the translation units of librkv (host side).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "rkv.h"

namespace rkv {

// ---- verification kernel geometry ------------------------------------------------
constexpr int kConsumerWarps = 7;                    // warps that compare
constexpr int kConsumers = kConsumerWarps * 32;      // 224 threads
constexpr int kThreads = kConsumers + 32;            // + one warp that issues the bulk copies = 256
constexpr int kBlocksPerSm = 2;                      // resident verification blocks per SM
constexpr int kStageBytes = kConsumers * 64;         // a ring stage: 64 bytes of a candidate per thread
// A thread owns 64 bytes of each candidate tile: 16 fp32 or 32 bf16 elements.
constexpr int kTileElemsF32 = kStageBytes / 4;       // 3584 elements per tile of fp32 candidates
constexpr int kTileElemsBF16 = kStageBytes / 2;      // 7168 elements per tile of bf16 candidates
__host__ __device__ constexpr uint32_t tile_elems(int cand_dtype) {
    return cand_dtype == RKV_BF16 ? kTileElemsBF16 : kTileElemsF32;
}
constexpr int kStages = 5;                           // ring depth (bulk copies in flight)
constexpr int kPartK = 64;                           // candidates a block tracks at a time
constexpr int kWarmTiles = 18;                       // leading tiles of a large tensor that are verified first
constexpr int kWarmMinTiles = 2048;                  // tensors with fewer tiles have no warm-up group
constexpr int kTailDiv = 4;                          // a tail item covers a quarter of a part's candidates ...
constexpr int kTailDivGenerated = 2;                 // ... half, when every item regenerates its reference tile
constexpr int kMaxTensors = 64;
constexpr uint64_t kMaxN = 1ull << 40;

// Result of one thread block for one (tensor, candidate); merged by the finalize kernel.
struct __align__(16) Partial {
    uint64_t n_over;
    uint64_t eidx;       // tensor-wide element index of the first maximum of |c - r|
    uint64_t qidx;       // same for |c - r| / |r|
    double sum;
    float emax;          // -1 when the block saw no comparable element
    float qmax;
    uint32_t valid;      // 0 in the zero-filled workspace, 1 once a block has written the slot
    uint32_t reserved;
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

// Device-side description of one tensor of a case.
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
    // Work items.  A large tensor has three groups of items: group A covers its first
    // warm_tiles tiles with small candidate parts (so that all blocks take part), group B
    // the tiles after them with parts of up to kPartK candidates, group C its last
    // tail_tiles tiles with parts a quarter that size.  Group A runs first: the maxima and
    // loophole flags it publishes let the rest skip almost all rare-path work.  Group C runs
    // last: its short items even out the finishing times of the blocks.  Smaller tensors
    // only have group A.  Within a group item = part * tiles + tile, with group_parts()
    // parts per group.
    // Items of the tensors of one storage variant are numbered consecutively, all A
    // groups, then all B groups, then all C groups; blocks take them in this order (see
    // WorkspaceHeader).
    uint32_t n_tiles;       // ceil(n / tile_elems(cand_dtype))
    uint32_t warm_tiles;    // tiles in group A (== n_tiles when there is no group B)
    uint32_t n_slots;       // Partial rows of this tensor: one per block of the grid
    uint32_t slot_base;     // first Partial row (K entries per row) of this tensor
    uint32_t variant;       // 2 * (candidates bf16) + (reference stored as bf16)
    uint32_t tail_tiles;    // tiles in group C
    uint32_t tail_div;      // group C cuts the candidates into this many times the parts of group B
    uint32_t reserved;
};

struct WorkspaceHeader {
    int32_t status;        // rkv_status written by the device
    // Work distribution of the verification kernel: every block starts with item blockIdx.x
    // and then draws tickets; item = grid + ticket.  The last block to finish clears both
    // words again, so that the next launch on the workspace starts from zero.
    uint32_t next_ticket;
    uint32_t blocks_done;
    uint32_t reserved[61];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header size");

// How a case is cut into work items, and where everything lives in the workspace:
//   header | tensor descriptors + pointer tables | CandState[T][K+1] | Partial[rows][K]
struct Plan {
    uint32_t n_tiles[kMaxTensors];
    uint32_t warm_tiles[kMaxTensors];
    uint32_t tail_tiles[kMaxTensors];
    uint32_t tail_div[kMaxTensors];
    uint32_t n_slots[kMaxTensors];
    uint32_t slot_base[kMaxTensors];
    uint32_t variant[kMaxTensors];
    uint32_t grid;          // blocks per launch (num_sms * kBlocksPerSm)
    size_t table_bytes;     // descriptors + pointer tables, rounded to 256
    size_t state_bytes;     // CandState region, rounded to 256
    size_t partial_bytes;
    size_t total_bytes;
};

int validate_tensors(const rkv_tensor_desc* tensors, int T, int K);
// k_count: candidates one launch covers (K, or the chunk length of the host-buffer form)
int make_plan(const rkv_tensor_desc* tensors, int T, int K, int k_count, int num_sms, Plan* plan);
int current_num_sms(int* num_sms);   // RKV_ERR_CUDA without a device
int refuse_capture(cudaStream_t stream);   // RKV_ERR_UNSUPPORTED while `stream` is being captured

// Number of candidate parts for a group of `tiles` tiles in a launch over k_count
// candidates: enough parts that none holds more than kPartK candidates, and, when the
// group has fewer tiles than there are blocks, enough that every block gets an item
// (tiles * parts >= grid where k_count allows).  Part p of `parts` covers the candidates
// [p * k_count / parts, (p + 1) * k_count / parts): sizes differ by at most one.
// The kernels and the host use this one rule.
__host__ __device__ inline uint32_t part_count(uint32_t tiles, uint32_t k_count, uint32_t grid) {
    uint32_t parts = (k_count + kPartK - 1) / kPartK;
    if (tiles < grid) {
        const uint32_t want = (grid + tiles - 1) / tiles;
        if (want > parts) parts = want;
    }
    return parts > k_count ? k_count : parts;
}

// Tiles, first tile and candidate parts of group g (0: A, 1: B, 2: C) of a tensor.
__host__ __device__ inline uint32_t group_tiles(uint32_t g, uint32_t n_tiles, uint32_t warm, uint32_t tail) {
    return g == 0 ? warm : g == 1 ? n_tiles - warm - tail : tail;
}
__host__ __device__ inline uint32_t group_first_tile(uint32_t g, uint32_t n_tiles, uint32_t warm, uint32_t tail) {
    return g == 0 ? 0u : g == 1 ? warm : n_tiles - tail;
}
__host__ __device__ inline uint32_t group_parts(uint32_t g, uint32_t tiles, uint32_t k_count, uint32_t grid,
                                                uint32_t tail_div) {
    if (g != 2) return part_count(tiles, k_count, grid);
    const uint32_t parts = (k_count + kPartK - 1) / kPartK * tail_div;
    return parts > k_count ? k_count : parts;
}
// Tiles in group C: half a tile per block, for tensors long enough that the blocks'
// finishing times would otherwise differ by up to a whole item.
__host__ __device__ inline uint32_t tail_tiles_of(uint32_t n_tiles, uint32_t warm, uint32_t grid) {
    return (n_tiles - warm >= 4u * grid && grid >= 2u) ? grid / 2u : 0u;
}

__host__ __device__ inline uint32_t part_begin(uint32_t part, uint32_t parts, uint32_t k_count) {
    return (uint32_t)(((uint64_t)part * k_count) / parts);
}

// kernels (rkv_verify.cu / rkv_gen.cu)
int launch_verify(const DevTensor* d_tensors, int T, int K, int k_begin, int k_end,
                  const uint32_t variant_items[4], int grid, CandState* state, Partial* partials,
                  WorkspaceHeader* header, cudaStream_t stream);
int launch_finalize(const DevTensor* d_tensors, int T, int K, const CandState* state,
                    const Partial* partials, rkv_stats* stats_out, uint32_t* joint_pass,
                    cudaStream_t stream);
int launch_gen(uint64_t seed, uint64_t stream_id, int dist, uint64_t n, uint64_t first_elem,
               int dtype, void* out, int num_sms, cudaStream_t stream);

}  // namespace rkv
