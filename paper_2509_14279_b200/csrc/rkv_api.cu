// Host side of librkv: argument validation, work-item planning, workspace layout,
// launches, and the host-buffer end-to-end form.  No torch types anywhere.
#include <math.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "rkv_internal.h"

namespace rkv {

// ----------------------------------------------------------------------------
// planning
// ----------------------------------------------------------------------------

// How one tensor is cut: tiles of tile_elems(cand_dtype) elements; its first tiles, up to
// kWarmTiles of them, form the warm-up group (see DevTensor).
static int plan_one(uint64_t n, int cand_dtype, uint32_t* n_tiles, uint32_t* warm_tiles) {
    if (n == 0 || n >= kMaxN) return RKV_ERR_INVALID_ARG;
    const uint64_t te = tile_elems(cand_dtype);
    const uint64_t tiles = (n + te - 1) / te;
    if (tiles > 0x3FFFFFFFull) return RKV_ERR_UNSUPPORTED;
    *n_tiles = (uint32_t)tiles;
    // The tiles that run at the same time as the first ones of the main group see what the
    // warm-up tiles published and nothing else: with w warm-up tiles about 1 in w + 1 of them
    // still has to locate a maximum, so w + c / (w + 1) tiles take the slow path, c the tiles
    // running at once (the blocks of the grid, or all the tiles of a short tensor): least near
    // w = sqrt(c).  kWarmTiles is that for two blocks on each of 148 SMs.
    uint32_t w = 1;
    while (w < (uint32_t)kWarmTiles && (uint64_t)(w + 1) * (w + 1) <= tiles) ++w;
    *warm_tiles = w;
    return RKV_OK;
}

// The descriptor tables of a call travel to the device from host memory that dies with the
// call.  A stream capture would record that copy with its host address and every replay of
// the graph would read freed memory, so the verification entry points refuse a capturing
// stream instead of enqueueing anything.
int refuse_capture(cudaStream_t stream) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &st) != cudaSuccess) { cudaGetLastError(); return RKV_ERR_CUDA; }
    return st == cudaStreamCaptureStatusNone ? RKV_OK : RKV_ERR_UNSUPPORTED;
}

static bool finite_nonneg(float x) { return x >= 0.0f && x <= 3.402823466e38f; }
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool dtype_ok(int d) { return d == RKV_F32 || d == RKV_BF16 || d == RKV_F16; }
static bool dist_ok(int d) { return d >= RKV_DIST_NORMAL && d <= RKV_DIST_NORMAL_1E4; }
static size_t round_up(size_t b, size_t a) { return (b + a - 1) / a * a; }

// Checks of one tensor descriptor that do not depend on where its buffers live.
static int validate_desc(const rkv_tensor_desc& d, int K) {
    if (d.n < 1) return RKV_ERR_INVALID_ARG;
    if (d.n >= kMaxN) return RKV_ERR_UNSUPPORTED;
    if (!dtype_ok(d.cand_dtype) || !dtype_ok(d.ref_dtype)) return RKV_ERR_INVALID_ARG;
    if (!finite_nonneg(d.atol) || !finite_nonneg(d.rtol)) return RKV_ERR_INVALID_ARG;
    if (d.ref_src == RKV_SRC_POINTER) {
        if (!d.ref) return RKV_ERR_INVALID_ARG;
    } else if (d.ref_src == RKV_SRC_GENERATED) {
        if (!dist_ok(d.ref_gen.dist)) return RKV_ERR_INVALID_ARG;
        if (d.ref_dtype == RKV_F16) return RKV_ERR_UNSUPPORTED;       // the generator has no fp16 rounding
    } else {
        return RKV_ERR_INVALID_ARG;
    }
    if (d.input_src == RKV_SRC_POINTER) {
        if (!d.input) return RKV_ERR_INVALID_ARG;
    } else if (d.input_src == RKV_SRC_GENERATED) {
        if (!dist_ok(d.input_gen.dist)) return RKV_ERR_INVALID_ARG;
        if (d.cand_dtype == RKV_F16) return RKV_ERR_UNSUPPORTED;
    } else if (d.input_src != RKV_SRC_NONE) {
        return RKV_ERR_INVALID_ARG;
    }
    if (!d.cands) return RKV_ERR_INVALID_ARG;
    for (int k = 0; k < K; ++k)
        if (!d.cands[k]) return RKV_ERR_INVALID_ARG;
    return RKV_OK;
}

int validate_tensors(const rkv_tensor_desc* tensors, int T, int K, int max_tensors) {
    if (!tensors || T < 1 || K < 1) return RKV_ERR_INVALID_ARG;
    if (T > max_tensors) return RKV_ERR_UNSUPPORTED;
    for (int t = 0; t < T; ++t) {
        const rkv_tensor_desc& d = tensors[t];
        const int rc = validate_desc(d, K);
        if (rc != RKV_OK) return rc;
        if (d.ref_src == RKV_SRC_POINTER && !aligned16(d.ref)) return RKV_ERR_ALIGNMENT;
        if (d.input_src == RKV_SRC_POINTER && !aligned16(d.input)) return RKV_ERR_ALIGNMENT;
        for (int k = 0; k < K; ++k)
            if (!aligned16(d.cands[k])) return RKV_ERR_ALIGNMENT;
    }
    return RKV_OK;
}

size_t segment_bound(int T) { return 3 * (size_t)T + 1; }

void plan_items(Plan* plan, int k_count) {
    const uint32_t grid = plan->grid, kc = (uint32_t)k_count;
    // candidate parts of every group: by the tiles the whole launch has in that group
    uint32_t launch_tiles[3] = {0, 0, 0};
    for (int t = 0; t < plan->T; ++t)
        for (uint32_t g = 0; g < 3; ++g) {
            const DevTensor& d = plan->tensors[t];
            const uint64_t sum = (uint64_t)launch_tiles[g] + group_tiles(g, d.n_tiles, d.warm_tiles, d.tail_tiles);
            launch_tiles[g] = sum > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)sum;
        }
    for (int t = 0; t < plan->T; ++t) {
        DevTensor& d = plan->tensors[t];
        d.parts[0] = part_count(launch_tiles[0] ? launch_tiles[0] : 1u, kc, grid);
        d.parts[1] = part_count(launch_tiles[1] ? launch_tiles[1] : 1u, kc, grid);
        const uint32_t tail_div = d.ref_src == RKV_SRC_GENERATED ? kTailDivGenerated : kTailDiv;
        const uint32_t p2 = (kc + kPartK - 1) / kPartK * tail_div;
        d.parts[2] = p2 > kc ? kc : p2;
    }
    // Item numbering: group 0 of every tensor, then group 1 of every tensor, then group 2;
    // inside a group the tensors of one storage type one after the other, then those of the
    // next type.  The kernel has one instantiation of its item code per candidate storage type,
    // and a block that changes type with every item runs out of its instruction cache: a sweep
    // of alternating fp32 / bf16 / fp16 cases took twice the time of the same sweep in one
    // type.  (Dealing the items of an fp32 and of a 16-bit tensor out in turn, so that
    // HBM-bound and issue-bound items share every SM, was measured 11 % slower than one tensor
    // after the other.)
    uint32_t n_seg = 0;
    uint64_t id = 0;
    static const int32_t kTypeOrder[3] = {RKV_F32, RKV_BF16, RKV_F16};
    for (uint32_t g = 0; g < 3; ++g) {
        for (int ty = 0; ty < 3; ++ty) {
            for (int t = 0; t < plan->T; ++t) {
                const DevTensor& d = plan->tensors[t];
                if (d.cand_dtype != kTypeOrder[ty]) continue;
                const uint64_t cnt = (uint64_t)group_tiles(g, d.n_tiles, d.warm_tiles, d.tail_tiles) * d.parts[g];
                if (!cnt) continue;
                if ((size_t)n_seg + 1 >= plan->segment_capacity || id + cnt > 0x7FFFFFFFull) {
                    id = 0x100000000ull;          // cannot be numbered: the caller refuses the case
                    continue;
                }
                Segment& s = plan->segments[n_seg++];
                s.first_id = (uint32_t)id;
                s.first_local = 0;
                s.tensor = (uint32_t)t;
                s.group = g;
                id += cnt;
            }
        }
    }
    const bool too_many = id > 0x7FFFFFFFull;
    Segment& end = plan->segments[n_seg];
    end.first_id = too_many ? 0u : (uint32_t)id; end.first_local = 0; end.tensor = 0; end.group = 0;
    plan->n_segments = n_seg;
    plan->n_items = too_many ? 0xFFFFFFFFu : (uint32_t)id;
}

int make_plan(const rkv_tensor_desc* tensors, int T, int K, int k_count, int num_sms, const uint32_t* case_of,
              const uint64_t* out_base, const uint32_t* out_stride, uint32_t n_cases, Plan* plan) {
    if (k_count < 1 || k_count > K) return RKV_ERR_INVALID_ARG;
    const uint32_t grid = (uint32_t)(num_sms * kBlocksPerSm);
    plan->grid = grid;
    plan->T = T;
    plan->n_cases = n_cases;
    plan->any_deferred = false;
    uint64_t rows = 0, sums = 0;
    // A launch whose tiles all fit the first wave of blocks has nobody to warm up for: what a
    // block publishes comes too late for the others, so every tile is a warm-up tile.
    uint64_t launch_tiles = 0;
    for (int t = 0; t < T; ++t) {
        uint32_t nt = 0, wt = 0;
        const int rc = plan_one(tensors[t].n, tensors[t].cand_dtype, &nt, &wt);
        if (rc != RKV_OK) return rc;
        launch_tiles += nt;
    }
    const bool one_wave = launch_tiles <= (uint64_t)grid;
    for (int t = 0; t < T; ++t) {
        const rkv_tensor_desc& s = tensors[t];
        DevTensor& d = plan->tensors[t];
        memset(&d, 0, sizeof d);
        const int rc = plan_one(s.n, s.cand_dtype, &d.n_tiles, &d.warm_tiles);
        if (rc != RKV_OK) return rc;
        if (one_wave) d.warm_tiles = d.n_tiles;
        d.tail_tiles = tail_tiles_of(d.n_tiles, d.warm_tiles, grid);
        d.n = s.n;
        d.ref = s.ref_src == RKV_SRC_POINTER ? s.ref : nullptr;
        d.input = s.input_src == RKV_SRC_POINTER ? s.input : nullptr;
        d.ref_seed = s.ref_gen.seed; d.ref_stream = s.ref_gen.stream_id; d.ref_dist = s.ref_gen.dist;
        d.in_seed = s.input_gen.seed; d.in_stream = s.input_gen.stream_id; d.in_dist = s.input_gen.dist;
        d.cand_dtype = s.cand_dtype; d.ref_dtype = s.ref_dtype;
        d.ref_src = s.ref_src; d.input_src = s.input_src;
        d.atol = s.atol; d.rtol = s.rtol;
        // a tensor of no more tiles than there are blocks keeps one Partial row per tile
        d.slot_by_tile = d.n_tiles <= grid ? 1u : 0u;
        d.n_slots = d.slot_by_tile ? d.n_tiles : grid;
        d.slot_base = (uint32_t)rows;
        rows += d.n_slots;
        if (rows > 0x7FFFFFFFull) return RKV_ERR_UNSUPPORTED;
        d.state_base = (uint32_t)((uint64_t)t * (uint64_t)(K + 1));
        d.sum_base = sums;
        sums += (uint64_t)d.n_tiles * (uint64_t)K;
        d.case_index = case_of ? case_of[t] : 0u;
        d.defer_copy = (s.input_src == RKV_SRC_GENERATED && d.warm_tiles < d.n_tiles) ? 1u : 0u;
        if (d.defer_copy) plan->any_deferred = true;
        d.out_base = out_base ? out_base[t] : (uint64_t)t;
        d.out_stride = out_stride ? out_stride[t] : (uint32_t)T;
    }
    plan_items(plan, k_count);
    if (plan->n_items == 0xFFFFFFFFu) return RKV_ERR_UNSUPPORTED;     // more items than a 32-bit id numbers
    plan->off_tensors = sizeof(WorkspaceHeader);
    plan->off_segments = round_up(plan->off_tensors + (size_t)T * sizeof(DevTensor), 16);
    plan->off_ptrs = round_up(plan->off_segments + ((size_t)plan->n_segments + 1) * sizeof(Segment), 16);
    plan->upload_bytes = round_up(plan->off_ptrs + (size_t)T * (size_t)K * sizeof(void*), 256);
    plan->off_fail = plan->upload_bytes;
    plan->off_state = round_up(plan->off_fail + (size_t)n_cases * (size_t)K * sizeof(uint32_t), 256);
    plan->off_partials = round_up(plan->off_state + (size_t)T * (size_t)(K + 1) * sizeof(CandState), 256);
    plan->off_sums = round_up(plan->off_partials + (size_t)rows * (size_t)K * sizeof(Partial), 256);
    plan->clear_bytes = plan->off_sums - plan->off_fail;
    plan->total_bytes = plan->off_sums + (size_t)sums * sizeof(double);
    return RKV_OK;
}

int current_num_sms(int* num_sms) {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return RKV_ERR_CUDA; }
    if (dev >= 0 && dev < 64 && cached[dev]) { *num_sms = cached[dev]; return RKV_OK; }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
        cudaGetLastError();
        return RKV_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) cached[dev] = n;
    *num_sms = n;
    return RKV_OK;
}

// ----------------------------------------------------------------------------
// library-owned buffers for the forms that take no workspace
// ----------------------------------------------------------------------------
namespace {

struct DeviceCache {
    void* workspace = nullptr;
    size_t workspace_bytes = 0;
    void* staging = nullptr;      // host-buffer form: reference + candidate chunks + stats
    size_t staging_bytes = 0;
    cudaStream_t copy_stream[2] = {nullptr, nullptr};
    cudaEvent_t copied[2] = {nullptr, nullptr};
    cudaEvent_t consumed[2] = {nullptr, nullptr};
};

std::mutex g_mutex;
DeviceCache g_cache[64];
cudaStream_t g_stream = nullptr;

// Fault drill armed by rkv_debug_fault_drill: applies to the next verification call only.
uint32_t g_drill_issue = 0;
unsigned long long g_drill_wait_cycles = 0;

int ensure(void** buf, size_t* have, size_t want) {
    if (*have >= want) return RKV_OK;
    if (*buf) { cudaFree(*buf); *buf = nullptr; *have = 0; }
    size_t bytes = (want + (size_t(1) << 20) - 1) >> 20 << 20;
    if (cudaMalloc(buf, bytes) != cudaSuccess) { cudaGetLastError(); return RKV_ERR_CUDA; }
    *have = bytes;
    return RKV_OK;
}

Layout layout_of(void* workspace, const Plan& plan) {
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    Layout L;
    L.header = reinterpret_cast<WorkspaceHeader*>(ws);
    L.d_tensors = reinterpret_cast<DevTensor*>(ws + plan.off_tensors);
    L.d_segments = reinterpret_cast<Segment*>(ws + plan.off_segments);
    L.d_ptrs = reinterpret_cast<const void**>(ws + plan.off_ptrs);
    L.fail = reinterpret_cast<uint32_t*>(ws + plan.off_fail);
    L.state = reinterpret_cast<CandState*>(ws + plan.off_state);
    L.partials = reinterpret_cast<Partial*>(ws + plan.off_partials);
    L.sums = reinterpret_cast<double*>(ws + plan.off_sums);
    return L;
}

// The image of the first plan.upload_bytes of the workspace: header, descriptors (with
// their device pointer tables), segment table, pointer tables.  `blob` has upload_bytes.
void build_blob(unsigned char* blob, const rkv_tensor_desc* tensors, int K, const Plan& plan, const Layout& L) {
    memset(blob, 0, plan.upload_bytes);
    WorkspaceHeader* h = reinterpret_cast<WorkspaceHeader*>(blob);
    h->drill_issue = g_drill_issue;
    h->drill_wait_cycles = g_drill_wait_cycles;
    g_drill_issue = 0;
    g_drill_wait_cycles = 0;
    DevTensor* h_t = reinterpret_cast<DevTensor*>(blob + plan.off_tensors);
    const void** h_p = reinterpret_cast<const void**>(blob + plan.off_ptrs);
    for (int t = 0; t < plan.T; ++t) {
        h_t[t] = plan.tensors[t];
        h_t[t].cands = L.d_ptrs + (size_t)t * K;
        for (int k = 0; k < K; ++k) h_p[(size_t)t * K + k] = tensors[t].cands[k];
    }
    memcpy(blob + plan.off_segments, plan.segments, ((size_t)plan.n_segments + 1) * sizeof(Segment));
}

// Send the tables (and clear what must start at zero), launch verify over candidates
// [k_begin, k_end) and, when asked, finalize.
//   upload  0: the tables are in place; 1: send them again (a chunk cut differently);
//           2: send them, with the header, and clear the results
int run_case(const rkv_tensor_desc* tensors, int K, int k_begin, int k_end, bool finalize, int upload,
             const Plan& plan, rkv_stats* stats_out, uint32_t* case_pass, uint32_t* all_pass, void* workspace,
             cudaStream_t stream) {
    const Layout L = layout_of(workspace, plan);
    if (upload) {
        std::vector<unsigned char> blob(plan.upload_bytes);
        build_blob(blob.data(), tensors, K, plan, L);
        // (in a chunked call the status word and the ticket counter of the first upload stay)
        const size_t skip = upload == 2 ? 0 : sizeof(WorkspaceHeader);
        if (cudaMemcpyAsync(reinterpret_cast<unsigned char*>(workspace) + skip, blob.data() + skip,
                            blob.size() - skip, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
            (upload == 2 && cudaMemsetAsync(L.fail, 0, plan.clear_bytes, stream) != cudaSuccess)) {
            cudaGetLastError();
            return RKV_ERR_CUDA;
        }
    }
    int rc = launch_verify(L, plan.T, K, k_begin, k_end, plan.n_items, plan.n_segments, (int)plan.grid, stream);
    if (rc != RKV_OK) return rc;
    if (plan.any_deferred) {
        rc = launch_copy_check(L, plan.T, K, k_begin, k_end, (int)plan.grid / kBlocksPerSm, stream);
        if (rc != RKV_OK) return rc;
    }
    if (finalize) rc = launch_finalize(L, plan.T, K, plan.n_cases, stats_out, case_pass, all_pass, stream);
    return rc;
}

// Plan storage for the entry points that may allocate on the host.
struct PlanStore {
    std::vector<DevTensor> tensors;
    std::vector<Segment> segments;
    Plan plan;
    explicit PlanStore(int T) : tensors((size_t)T), segments(segment_bound(T)) {
        plan.tensors = tensors.data();
        plan.segments = segments.data();
        plan.segment_capacity = segments.size();
    }
};

}  // namespace
}  // namespace rkv

using namespace rkv;

// ----------------------------------------------------------------------------
// C ABI
// ----------------------------------------------------------------------------
extern "C" {

int rkv_version(void) { return 200; }

const char* rkv_status_string(int status) {
    switch (status) {
        case RKV_OK: return "ok";
        case RKV_ERR_INVALID_ARG: return "invalid argument";
        case RKV_ERR_UNSUPPORTED: return "unsupported size or combination";
        case RKV_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case RKV_ERR_WORKSPACE: return "workspace missing or too small";
        case RKV_ERR_CUDA: return "CUDA runtime error";
        case RKV_ERR_TIMEOUT: return "device-side bounded wait ran out";
        case RKV_ERR_BOUNDS: return "device-side range check failed (debug build)";
        default: return "unknown status";
    }
}

int rkv_set_stream(void* cuda_stream) {
    g_stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    return RKV_OK;
}

// Not part of the public interface (rkv.h does not declare it): arms a fault drill for the
// next verification call of this process.  Block 0 of that call's kernel skips its issue-th
// copy (1-based; the ring stage is neither armed nor filled), and every bounded wait of
// the launch gives up after wait_cycles clock cycles instead of about a second.  Nothing
// is in flight because of it and nothing faults: the block times out, drains and reports
// RKV_ERR_TIMEOUT through the status word.  issue == 0 disarms.
int rkv_debug_fault_drill(unsigned int issue, unsigned long long wait_cycles) {
    std::lock_guard<std::mutex> lock(g_mutex);
    g_drill_issue = issue;
    g_drill_wait_cycles = issue ? wait_cycles : 0ull;
    return RKV_OK;
}

// Not part of the public interface either: 1 when the library was built with
// RKV_DEBUG_BOUNDS (every device-side index range-checked), else 0.
int rkv_debug_bounds_build(void) {
#ifdef RKV_DEBUG_BOUNDS
    return 1;
#else
    return 0;
#endif
}

// Not part of the public interface: resident verification blocks per SM on the current
// device (the kernel is written for kBlocksPerSm = 2).
int rkv_debug_occupancy(void) { return verify_occupancy(); }

int rkv_plan_items(uint64_t n, int cand_dtype, int K, int num_sms, uint32_t* tile_elems_out, uint32_t* n_tiles,
                   uint32_t* warm_tiles, uint32_t* parts_warm, uint32_t* parts_main, uint32_t* tail_tiles,
                   uint32_t* parts_tail) {
    if (!tile_elems_out || !n_tiles || !warm_tiles || !parts_warm || !parts_main || !tail_tiles || !parts_tail)
        return RKV_ERR_INVALID_ARG;
    if (!dtype_ok(cand_dtype)) return RKV_ERR_INVALID_ARG;
    if (n >= kMaxN) return RKV_ERR_UNSUPPORTED;
    if (n < 1 || K < 1 || num_sms < 1 || num_sms > (1 << 20)) return RKV_ERR_INVALID_ARG;
    rkv_tensor_desc d;
    memset(&d, 0, sizeof d);
    d.n = n; d.cand_dtype = cand_dtype; d.ref_dtype = RKV_F32; d.ref_src = RKV_SRC_POINTER;
    DevTensor dt;
    Segment seg[8];
    Plan plan;
    plan.tensors = &dt; plan.segments = seg; plan.segment_capacity = 8;
    const int rc = make_plan(&d, 1, K, K, num_sms, nullptr, nullptr, nullptr, 1, &plan);
    if (rc != RKV_OK) return rc;
    *tile_elems_out = tile_elems(cand_dtype);
    *n_tiles = dt.n_tiles;
    *warm_tiles = dt.warm_tiles;
    *tail_tiles = dt.tail_tiles;
    *parts_warm = dt.parts[0];
    *parts_main = (dt.n_tiles - dt.warm_tiles - dt.tail_tiles) ? dt.parts[1] : 0u;
    *parts_tail = dt.tail_tiles ? dt.parts[2] : 0u;
    return RKV_OK;
}

int rkv_gen_inputs_ex(uint64_t seed, uint64_t stream_id, int dist, uint64_t n, uint64_t first_elem,
                      int dtype, void* out, void* cuda_stream) {
    if (!out || n < 1 || !dist_ok(dist) || (dtype != RKV_F32 && dtype != RKV_BF16) || (first_elem & 3u))
        return RKV_ERR_INVALID_ARG;
    if (n >= kMaxN) return RKV_ERR_UNSUPPORTED;
    if (!aligned16(out)) return RKV_ERR_ALIGNMENT;
    int sms = 0;
    const int rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    return launch_gen(seed, stream_id, dist, n, first_elem, dtype, out, sms,
                      reinterpret_cast<cudaStream_t>(cuda_stream));
}

int rkv_gen_inputs(uint64_t seed, int dist, const int64_t* shape, int ndim, int dtype, void* out) {
    if (!shape || ndim < 1) return RKV_ERR_INVALID_ARG;
    uint64_t n = 1;
    for (int i = 0; i < ndim; ++i) {
        if (shape[i] < 1) return RKV_ERR_INVALID_ARG;
        if ((uint64_t)shape[i] >= kMaxN || n * (uint64_t)shape[i] >= kMaxN) return RKV_ERR_UNSUPPORTED;
        n *= (uint64_t)shape[i];
    }
    return rkv_gen_inputs_ex(seed, 0, dist, n, 0, dtype, out, g_stream);
}

size_t rkv_workspace_bytes(const rkv_tensor_desc* tensors, int T, int K) {
    if (!tensors || T < 1 || T > kMaxTensors || K < 1) return 0;
    for (int t = 0; t < T; ++t)
        if (tensors[t].n < 1 || tensors[t].n >= kMaxN || !dtype_ok(tensors[t].cand_dtype)) return 0;
    int sms = 0;
    if (current_num_sms(&sms) != RKV_OK) return 0;
    PlanStore ps(T);
    if (make_plan(tensors, T, K, K, sms, nullptr, nullptr, nullptr, 1, &ps.plan) != RKV_OK) return 0;
    return ps.plan.total_bytes;
}

int rkv_verify_multi(const rkv_tensor_desc* tensors, int T, int K, rkv_stats* stats_out,
                     uint32_t* joint_pass, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = validate_tensors(tensors, T, K, kMaxTensors);
    if (rc != RKV_OK) return rc;
    if (!stats_out) return RKV_ERR_INVALID_ARG;
    if (!workspace) return RKV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return RKV_ERR_ALIGNMENT;
    int sms = 0;
    rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    PlanStore ps(T);
    rc = make_plan(tensors, T, K, K, sms, nullptr, nullptr, nullptr, 1, &ps.plan);
    if (rc != RKV_OK) return rc;
    if (workspace_bytes < ps.plan.total_bytes) return RKV_ERR_WORKSPACE;
    rc = refuse_capture(reinterpret_cast<cudaStream_t>(cuda_stream));
    if (rc != RKV_OK) return rc;
    return run_case(tensors, K, 0, K, true, 2, ps.plan, stats_out, nullptr, joint_pass, workspace,
                    reinterpret_cast<cudaStream_t>(cuda_stream));
}

// Flatten the cases of a sweep into one tensor list.
static int flatten_sweep(const rkv_case_desc* cases, int C, int K, std::vector<rkv_tensor_desc>* flat,
                         std::vector<uint32_t>* case_of, std::vector<uint64_t>* out_base,
                         std::vector<uint32_t>* out_stride) {
    if (!cases || C < 1 || K < 1) return RKV_ERR_INVALID_ARG;
    uint64_t total = 0;
    for (int c = 0; c < C; ++c) {
        if (!cases[c].tensors || cases[c].T < 1) return RKV_ERR_INVALID_ARG;
        if (cases[c].T > kMaxTensors) return RKV_ERR_UNSUPPORTED;
        total += (uint64_t)cases[c].T;
        if (total > (uint64_t)kMaxSweepTensors) return RKV_ERR_UNSUPPORTED;
    }
    uint64_t at = 0;
    for (int c = 0; c < C; ++c) {
        for (int t = 0; t < cases[c].T; ++t) {
            flat->push_back(cases[c].tensors[t]);
            case_of->push_back((uint32_t)c);
            out_base->push_back(at + (uint64_t)t);
            out_stride->push_back((uint32_t)cases[c].T);
        }
        at += (uint64_t)K * (uint64_t)cases[c].T;
    }
    return RKV_OK;
}

size_t rkv_sweep_workspace_bytes(const rkv_case_desc* cases, int C, int K) {
    std::vector<rkv_tensor_desc> flat;
    std::vector<uint32_t> case_of, out_stride;
    std::vector<uint64_t> out_base;
    if (flatten_sweep(cases, C, K, &flat, &case_of, &out_base, &out_stride) != RKV_OK) return 0;
    for (const rkv_tensor_desc& d : flat)
        if (d.n < 1 || d.n >= kMaxN || !dtype_ok(d.cand_dtype)) return 0;
    int sms = 0;
    if (current_num_sms(&sms) != RKV_OK) return 0;
    PlanStore ps((int)flat.size());
    if (make_plan(flat.data(), (int)flat.size(), K, K, sms, case_of.data(), out_base.data(), out_stride.data(),
                  (uint32_t)C, &ps.plan) != RKV_OK)
        return 0;
    return ps.plan.total_bytes;
}

int rkv_verify_sweep(const rkv_case_desc* cases, int C, int K, rkv_stats* stats_out, uint32_t* case_pass,
                     uint32_t* all_pass, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    std::vector<rkv_tensor_desc> flat;
    std::vector<uint32_t> case_of, out_stride;
    std::vector<uint64_t> out_base;
    int rc = flatten_sweep(cases, C, K, &flat, &case_of, &out_base, &out_stride);
    if (rc != RKV_OK) return rc;
    const int T = (int)flat.size();
    rc = validate_tensors(flat.data(), T, K, kMaxSweepTensors);
    if (rc != RKV_OK) return rc;
    if (!stats_out) return RKV_ERR_INVALID_ARG;
    if (!workspace) return RKV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return RKV_ERR_ALIGNMENT;
    int sms = 0;
    rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    PlanStore ps(T);
    rc = make_plan(flat.data(), T, K, K, sms, case_of.data(), out_base.data(), out_stride.data(), (uint32_t)C,
                   &ps.plan);
    if (rc != RKV_OK) return rc;
    if (workspace_bytes < ps.plan.total_bytes) return RKV_ERR_WORKSPACE;
    rc = refuse_capture(reinterpret_cast<cudaStream_t>(cuda_stream));
    if (rc != RKV_OK) return rc;
    return run_case(flat.data(), K, 0, K, true, 2, ps.plan, stats_out, case_pass, all_pass, workspace,
                    reinterpret_cast<cudaStream_t>(cuda_stream));
}

int rkv_verify_batch(const void* ref, const void* const* cands, int K, uint64_t n, int dtype, float atol,
                     float rtol, rkv_stats* stats_out) {
    rkv_tensor_desc d;
    memset(&d, 0, sizeof d);
    d.n = n; d.ref = ref; d.cands = cands;
    d.cand_dtype = dtype; d.ref_dtype = dtype;
    d.ref_src = RKV_SRC_POINTER; d.input_src = RKV_SRC_NONE;
    d.atol = atol; d.rtol = rtol;
    int rc = validate_tensors(&d, 1, K, kMaxTensors);
    if (rc != RKV_OK) return rc;
    if (!stats_out) return RKV_ERR_INVALID_ARG;
    int sms = 0;
    rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    PlanStore ps(1);
    rc = make_plan(&d, 1, K, K, sms, nullptr, nullptr, nullptr, 1, &ps.plan);
    if (rc != RKV_OK) return rc;
    rc = refuse_capture(g_stream);
    if (rc != RKV_OK) return rc;
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCache& c = g_cache[dev & 63];
    rc = ensure(&c.workspace, &c.workspace_bytes, ps.plan.total_bytes);
    if (rc != RKV_OK) return rc;
    return run_case(&d, K, 0, K, true, 2, ps.plan, stats_out, nullptr, nullptr, c.workspace, g_stream);
}

int rkv_device_status(const void* workspace, void* cuda_stream) {
    if (!workspace) return RKV_ERR_INVALID_ARG;
    int32_t st = 0;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(&st, workspace, sizeof st, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return RKV_ERR_CUDA;
    }
    return st;
}

int rkv_verify_multi_host(const rkv_tensor_desc* tensors, int T, int K, rkv_stats* stats_host,
                          uint32_t* joint_host) {
    if (!tensors || !stats_host || T < 1 || K < 1) return RKV_ERR_INVALID_ARG;
    if (T > kMaxTensors) return RKV_ERR_UNSUPPORTED;
    for (int t = 0; t < T; ++t) {
        const int rc = validate_desc(tensors[t], K);
        if (rc != RKV_OK) return rc;
    }
    int sms = 0;
    int rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    rc = refuse_capture(g_stream);
    if (rc != RKV_OK) return rc;
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCache& c = g_cache[dev & 63];

    // staging layout: references and inputs | two buffers of kc candidates of every tensor | results
    size_t fixed_bytes = 0, per_cand = 0;
    for (int t = 0; t < T; ++t) {
        const rkv_tensor_desc& d = tensors[t];
        if (d.ref_src == RKV_SRC_POINTER) fixed_bytes += round_up((size_t)d.n * elem_bytes(d.ref_dtype), 256);
        if (d.input_src == RKV_SRC_POINTER) fixed_bytes += round_up((size_t)d.n * elem_bytes(d.cand_dtype), 256);
        per_cand += round_up((size_t)d.n * elem_bytes(d.cand_dtype), 256);
    }
    // candidates travel in chunks of kc, two chunks in flight
    size_t kc = (size_t(512) << 20) / per_cand;
    if (kc < 1) kc = 1;
    if (kc > (size_t)K) kc = (size_t)K;
    if (kc > 16) kc = 16;
    const size_t stats_bytes = round_up((size_t)K * (size_t)T * sizeof(rkv_stats), 256);
    const size_t joint_bytes = round_up((size_t)K * sizeof(uint32_t), 256);
    rc = ensure(&c.staging, &c.staging_bytes, fixed_bytes + 2 * kc * per_cand + stats_bytes + joint_bytes);
    if (rc != RKV_OK) return rc;
    for (int i = 0; i < 2; ++i) {
        if (!c.copy_stream[i] &&
            (cudaStreamCreateWithFlags(&c.copy_stream[i], cudaStreamNonBlocking) != cudaSuccess ||
             cudaEventCreateWithFlags(&c.copied[i], cudaEventDisableTiming) != cudaSuccess ||
             cudaEventCreateWithFlags(&c.consumed[i], cudaEventDisableTiming) != cudaSuccess)) {
            cudaGetLastError();
            return RKV_ERR_CUDA;
        }
    }
    unsigned char* base = reinterpret_cast<unsigned char*>(c.staging);
    unsigned char* d_chunk[2] = {base + fixed_bytes, base + fixed_bytes + kc * per_cand};
    rkv_stats* d_stats = reinterpret_cast<rkv_stats*>(base + fixed_bytes + 2 * kc * per_cand);
    uint32_t* d_joint = reinterpret_cast<uint32_t*>(base + fixed_bytes + 2 * kc * per_cand + stats_bytes);

    // device-side descriptors: candidate k of tensor t lives in slot k % kc of buffer (k / kc) % 2
    std::vector<rkv_tensor_desc> dd(tensors, tensors + T);
    std::vector<const void*> ptrs((size_t)T * (size_t)K);
    cudaStream_t main = g_stream;
    bool fail = false;
    size_t fixed_at = 0, tensor_at = 0;
    for (int t = 0; t < T; ++t) {
        rkv_tensor_desc& d = dd[(size_t)t];
        if (d.ref_src == RKV_SRC_POINTER) {
            const size_t b = (size_t)d.n * elem_bytes(d.ref_dtype);
            fail |= cudaMemcpyAsync(base + fixed_at, tensors[t].ref, b, cudaMemcpyHostToDevice, main) != cudaSuccess;
            d.ref = base + fixed_at;
            fixed_at += round_up(b, 256);
        }
        if (d.input_src == RKV_SRC_POINTER) {
            const size_t b = (size_t)d.n * elem_bytes(d.cand_dtype);
            fail |= cudaMemcpyAsync(base + fixed_at, tensors[t].input, b, cudaMemcpyHostToDevice, main) != cudaSuccess;
            d.input = base + fixed_at;
            fixed_at += round_up(b, 256);
        }
        for (int k = 0; k < K; ++k)
            ptrs[(size_t)t * K + k] = d_chunk[((size_t)k / kc) & 1] + ((size_t)k % kc) * per_cand + tensor_at;
        d.cands = ptrs.data() + (size_t)t * K;
        tensor_at += round_up((size_t)d.n * elem_bytes(d.cand_dtype), 256);
    }
    PlanStore ps(T);
    rc = make_plan(dd.data(), T, K, (int)kc, sms, nullptr, nullptr, nullptr, 1, &ps.plan);
    if (rc != RKV_OK) return rc;
    rc = ensure(&c.workspace, &c.workspace_bytes, ps.plan.total_bytes);
    if (rc != RKV_OK) return rc;

    const int n_chunks = (int)(((size_t)K + kc - 1) / kc);
    for (int ch = 0; ch < n_chunks && !fail; ++ch) {
        const int b = ch & 1;
        const int k0 = ch * (int)kc;
        const int k1 = (k0 + (int)kc) < K ? (k0 + (int)kc) : K;
        // the buffer may be overwritten once the verification of chunk ch-2 is done
        if (ch >= 2) fail |= cudaStreamWaitEvent(c.copy_stream[b], c.consumed[b], 0) != cudaSuccess;
        for (int k = k0; k < k1; ++k)
            for (int t = 0; t < T; ++t)
                fail |= cudaMemcpyAsync(const_cast<void*>(ptrs[(size_t)t * K + k]), tensors[t].cands[k],
                                        (size_t)tensors[t].n * elem_bytes(tensors[t].cand_dtype),
                                        cudaMemcpyHostToDevice, c.copy_stream[b]) != cudaSuccess;
        fail |= cudaEventRecord(c.copied[b], c.copy_stream[b]) != cudaSuccess;
        fail |= cudaStreamWaitEvent(main, c.copied[b], 0) != cudaSuccess;
        if (fail) break;
        // a shorter last chunk is cut into parts of its own: send the tables again
        int upload = ch == 0 ? 2 : 0;
        if (ch > 0 && k1 - k0 != (int)kc) {
            plan_items(&ps.plan, k1 - k0);
            upload = 1;
        }
        rc = run_case(dd.data(), K, k0, k1, k1 == K, upload, ps.plan, d_stats, nullptr, d_joint, c.workspace, main);
        if (rc != RKV_OK) { fail = true; break; }
        fail |= cudaEventRecord(c.consumed[b], main) != cudaSuccess;
    }
    if (!fail) {
        fail |= cudaMemcpyAsync(stats_host, d_stats, (size_t)K * (size_t)T * sizeof(rkv_stats),
                                cudaMemcpyDeviceToHost, main) != cudaSuccess;
        if (joint_host)
            fail |= cudaMemcpyAsync(joint_host, d_joint, (size_t)K * sizeof(uint32_t), cudaMemcpyDeviceToHost,
                                    main) != cudaSuccess;
    }
    const bool sync_fail = cudaStreamSynchronize(main) != cudaSuccess;
    cudaStreamSynchronize(c.copy_stream[0]);
    cudaStreamSynchronize(c.copy_stream[1]);
    if (fail || sync_fail) { cudaGetLastError(); return rc != RKV_OK ? rc : RKV_ERR_CUDA; }
    return RKV_OK;
}

int rkv_verify_batch_host(const void* ref_host, const void* const* cands_host, int K, uint64_t n,
                          int dtype, float atol, float rtol, rkv_stats* stats_host) {
    if (!cands_host) return RKV_ERR_INVALID_ARG;
    rkv_tensor_desc d;
    memset(&d, 0, sizeof d);
    d.n = n; d.ref = ref_host; d.cands = cands_host;
    d.cand_dtype = dtype; d.ref_dtype = dtype;
    d.ref_src = RKV_SRC_POINTER; d.input_src = RKV_SRC_NONE;
    d.atol = atol; d.rtol = rtol;
    return rkv_verify_multi_host(&d, 1, K, stats_host, nullptr);
}

// ----------------------------------------------------------------------------
// rkv_verify_batch_static: the same verification with its scratch in a fixed
// device array that is part of the library image -- nothing is allocated.
// ----------------------------------------------------------------------------
}  // extern "C"

namespace rkv {
namespace {

constexpr size_t kStaticScratchBytes = size_t(8) << 20;
constexpr int kStaticMaxK = 256;

// Lives in the global memory of every device that loads the library, until the
// process exits.  On the host this name is only a handle for
// cudaGetSymbolAddress: it is not a device address and is never passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch on each device, looked up once per device
// with that device current.
void* g_static_scratch_addr[64] = {};

int static_scratch_address(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return RKV_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return RKV_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return RKV_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return RKV_OK;
}

}  // namespace
}  // namespace rkv

extern "C" {

int rkv_verify_batch_static(const void* ref, const void* const* cands, int K, uint64_t n, int dtype,
                            float atol, float rtol, rkv_stats* stats_out, void* cuda_stream) {
    rkv_tensor_desc d;
    memset(&d, 0, sizeof d);
    d.n = n; d.ref = ref; d.cands = cands;
    d.cand_dtype = dtype; d.ref_dtype = dtype;
    d.ref_src = RKV_SRC_POINTER; d.input_src = RKV_SRC_NONE;
    d.atol = atol; d.rtol = rtol;
    int rc = validate_tensors(&d, 1, K, kMaxTensors);
    if (rc != RKV_OK) return rc;
    if (!stats_out) return RKV_ERR_INVALID_ARG;
    if (K > kStaticMaxK) return RKV_ERR_UNSUPPORTED;
    int sms = 0;
    rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    // the plan's two tables on the stack: one tensor, at most three segments and the sentinel
    DevTensor dt;
    Segment seg[8];
    Plan plan;
    plan.tensors = &dt; plan.segments = seg; plan.segment_capacity = 8;
    rc = make_plan(&d, 1, K, K, sms, nullptr, nullptr, nullptr, 1, &plan);
    if (rc != RKV_OK) return rc;
    if (plan.total_bytes > kStaticScratchBytes) return RKV_ERR_UNSUPPORTED;
    rc = refuse_capture(reinterpret_cast<cudaStream_t>(cuda_stream));
    if (rc != RKV_OK) return rc;
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != RKV_OK) return rc;

    // header (status word = 0) + descriptor + segments + pointer table, built on the stack
    constexpr size_t kBlobMax = 4096;
    static_assert(sizeof(WorkspaceHeader) + sizeof(DevTensor) + 8 * sizeof(Segment) + kStaticMaxK * sizeof(void*) +
                          3 * 256 <= kBlobMax, "the static form's tables fit its stack buffer");
    alignas(16) unsigned char blob[kBlobMax];
    if (plan.upload_bytes > kBlobMax) return RKV_ERR_UNSUPPORTED;
    const Layout L = layout_of(scratch, plan);
    {
        std::lock_guard<std::mutex> lock(g_mutex);     // (the fault-drill words are shared state)
        build_blob(blob, &d, K, plan, L);
    }

    // what must start at zero in the shared array: the status word (in the blob), the fail
    // words, the per-candidate state and the partial results; the tile sums are all rewritten
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(scratch, blob, plan.upload_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemsetAsync(L.fail, 0, plan.clear_bytes, stream) != cudaSuccess) {
        cudaGetLastError();
        return RKV_ERR_CUDA;
    }
    rc = launch_verify(L, 1, K, 0, K, plan.n_items, plan.n_segments, (int)plan.grid, stream);
    if (rc != RKV_OK) return rc;
    return launch_finalize(L, 1, K, 1, stats_out, nullptr, nullptr, stream);
}

int rkv_release_cached(void) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int cur = 0;
    const bool have_dev = cudaGetDevice(&cur) == cudaSuccess;
    for (int dev = 0; dev < 64; ++dev) {
        DeviceCache& c = g_cache[dev];
        if (!c.workspace && !c.staging && !c.copy_stream[0]) continue;
        cudaSetDevice(dev);
        if (c.workspace) cudaFree(c.workspace);
        if (c.staging) cudaFree(c.staging);
        for (int i = 0; i < 2; ++i) {
            if (c.copy_stream[i]) cudaStreamDestroy(c.copy_stream[i]);
            if (c.copied[i]) cudaEventDestroy(c.copied[i]);
            if (c.consumed[i]) cudaEventDestroy(c.consumed[i]);
        }
        c = DeviceCache();
    }
    if (have_dev) cudaSetDevice(cur);
    cudaGetLastError();
    return RKV_OK;
}

}  // extern "C"
