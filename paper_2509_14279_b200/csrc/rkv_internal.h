// Internal declarations shared by the translation units of librkv (host side).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "rkv.h"

namespace rkv {

constexpr int kThreads = 256;          // threads per verification block
constexpr int kBlocksPerSm = 2;        // resident verification blocks per SM
constexpr int kSlabGranule = 128;      // slab lengths are multiples of this many elements
constexpr int kSmemDataBudget = 96 * 1024;  // bytes of reference + input one block stages
constexpr int kChunkK = 16;            // candidates between two block-level merges
constexpr int kPreK = 512;             // candidates whose pointer and first element are preloaded
constexpr int kHintK = 256;            // candidates with a cross-slab threshold hint
constexpr int kMaxTensors = 64;
constexpr uint64_t kMaxN = 1ull << 40;

// Per (slab, candidate) partial result; also the per-warp record in shared memory.
struct __align__(16) Partial {
    uint32_t n_over;
    uint32_t n_noncomp;
    uint32_t n_nan;
    uint32_t n_inf;
    uint32_t n_infmis;
    uint32_t mismatch;   // bit0: some element differs from element 0; bit1: differs from input
    float emax;          // -1 when no comparable element beat the hint
    uint32_t eidx;       // slab-local index
    float qmax;
    uint32_t qidx;
    double sum;
};
static_assert(sizeof(Partial) == 48, "Partial layout");

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
    uint32_t slab_elems;
    uint32_t n_slabs;
    uint32_t first_item;
    uint32_t reserved;
};

struct WorkspaceHeader {
    int32_t status;        // rkv_status written by the device
    uint32_t reserved[63];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header size");

struct Plan {
    uint32_t slab_elems[kMaxTensors];
    uint32_t n_slabs[kMaxTensors];
    uint32_t first_item[kMaxTensors];
    uint32_t total_items;
    uint32_t variant_items[8];
    size_t table_bytes;     // descriptors + pointer tables, rounded to 256
    size_t partial_bytes;
    size_t total_bytes;
};

int smem_bytes_per_elem(const rkv_tensor_desc& t);
int validate_tensors(const rkv_tensor_desc* tensors, int T, int K);
int make_plan(const rkv_tensor_desc* tensors, int T, int K, int num_sms, Plan* plan);
int current_num_sms(int* num_sms);   // RKV_ERR_CUDA without a device

// kernels (rkv_verify.cu / rkv_gen.cu)
// variant_items[v]: slabs of the tensors whose storage variant is v =
// 4*(candidates bf16) + 2*(reference staged as bf16) + (input present)
int launch_verify(const DevTensor* d_tensors, int T, int K, int k_begin, int k_end,
                  const uint32_t variant_items[8], int num_sms, Partial* partials, int32_t* status,
                  cudaStream_t stream);
int launch_finalize(const DevTensor* d_tensors, int T, int K, const Partial* partials,
                    rkv_stats* stats_out, uint32_t* joint_pass, cudaStream_t stream);
int launch_gen(uint64_t seed, uint64_t stream_id, int dist, uint64_t n, uint64_t first_elem,
               int dtype, void* out, int num_sms, cudaStream_t stream);

}  // namespace rkv
