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

// How one tensor is cut: tiles of tile_elems(cand_dtype) elements; a large tensor's first
// kWarmTiles tiles form the warm-up group (see DevTensor).
static int plan_one(uint64_t n, int cand_dtype, uint32_t* n_tiles, uint32_t* warm_tiles) {
    if (n == 0 || n >= kMaxN) return RKV_ERR_INVALID_ARG;
    const uint64_t te = tile_elems(cand_dtype);
    const uint64_t tiles = (n + te - 1) / te;
    if (tiles > 0x3FFFFFFFull) return RKV_ERR_UNSUPPORTED;
    *n_tiles = (uint32_t)tiles;
    *warm_tiles = tiles >= (uint64_t)kWarmMinTiles ? (uint32_t)kWarmTiles : (uint32_t)tiles;
    return RKV_OK;
}

// Work items of one tensor for a launch over k_count candidates.
static uint64_t items_of(uint32_t n_tiles, uint32_t warm_tiles, uint32_t tail_tiles, uint32_t tail_div,
                         uint32_t k_count, uint32_t grid) {
    uint64_t items = 0;
    for (uint32_t g = 0; g < 3; ++g) {
        const uint32_t nt = group_tiles(g, n_tiles, warm_tiles, tail_tiles);
        if (!nt) continue;
        items += (uint64_t)nt * group_parts(g, nt, k_count, grid, tail_div);
    }
    return items;
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
static bool dtype_ok(int d) { return d == RKV_F32 || d == RKV_BF16; }
static bool dist_ok(int d) { return d >= RKV_DIST_NORMAL && d <= RKV_DIST_NORMAL_1E4; }

int validate_tensors(const rkv_tensor_desc* tensors, int T, int K) {
    if (!tensors || T < 1 || K < 1) return RKV_ERR_INVALID_ARG;
    if (T > kMaxTensors) return RKV_ERR_UNSUPPORTED;
    for (int t = 0; t < T; ++t) {
        const rkv_tensor_desc& d = tensors[t];
        if (d.n < 1) return RKV_ERR_INVALID_ARG;
        if (d.n >= kMaxN) return RKV_ERR_UNSUPPORTED;
        if (!dtype_ok(d.cand_dtype) || !dtype_ok(d.ref_dtype)) return RKV_ERR_INVALID_ARG;
        if (!finite_nonneg(d.atol) || !finite_nonneg(d.rtol)) return RKV_ERR_INVALID_ARG;
        if (d.ref_src == RKV_SRC_POINTER) {
            if (!d.ref) return RKV_ERR_INVALID_ARG;
            if (!aligned16(d.ref)) return RKV_ERR_ALIGNMENT;
        } else if (d.ref_src == RKV_SRC_GENERATED) {
            if (!dist_ok(d.ref_gen.dist)) return RKV_ERR_INVALID_ARG;
        } else {
            return RKV_ERR_INVALID_ARG;
        }
        if (d.input_src == RKV_SRC_POINTER) {
            if (!d.input) return RKV_ERR_INVALID_ARG;
            if (!aligned16(d.input)) return RKV_ERR_ALIGNMENT;
        } else if (d.input_src == RKV_SRC_GENERATED) {
            if (!dist_ok(d.input_gen.dist)) return RKV_ERR_INVALID_ARG;
        } else if (d.input_src != RKV_SRC_NONE) {
            return RKV_ERR_INVALID_ARG;
        }
        if (!d.cands) return RKV_ERR_INVALID_ARG;
        for (int k = 0; k < K; ++k) {
            if (!d.cands[k]) return RKV_ERR_INVALID_ARG;
            if (!aligned16(d.cands[k])) return RKV_ERR_ALIGNMENT;
        }
    }
    return RKV_OK;
}

static uint32_t variant_of(const rkv_tensor_desc& d) {
    return (d.cand_dtype == RKV_BF16 ? 2u : 0u) +
           ((d.ref_dtype == RKV_BF16 && d.ref_src == RKV_SRC_POINTER) ? 1u : 0u);
}

int make_plan(const rkv_tensor_desc* tensors, int T, int K, int k_count, int num_sms, Plan* plan) {
    if (k_count < 1 || k_count > K) return RKV_ERR_INVALID_ARG;
    const uint32_t grid = (uint32_t)(num_sms * kBlocksPerSm);
    plan->grid = grid;
    uint64_t rows = 0, total_items[4] = {0, 0, 0, 0};
    for (int t = 0; t < T; ++t) {
        uint32_t tiles, warm;
        const int rc = plan_one(tensors[t].n, tensors[t].cand_dtype, &tiles, &warm);
        if (rc != RKV_OK) return rc;
        plan->n_tiles[t] = tiles;
        plan->warm_tiles[t] = warm;
        const uint32_t tail = tail_tiles_of(tiles, warm, grid);
        plan->tail_tiles[t] = tail;
        const uint32_t tail_div = tensors[t].ref_src == RKV_SRC_GENERATED ? kTailDivGenerated : kTailDiv;
        plan->tail_div[t] = tail_div;
        plan->variant[t] = variant_of(tensors[t]);
        const uint64_t items = items_of(tiles, warm, tail, tail_div, (uint32_t)k_count, grid);
        total_items[plan->variant[t]] += items;
        if (total_items[plan->variant[t]] > 0x7FFFFFFFull) return RKV_ERR_UNSUPPORTED;
        plan->n_slots[t] = grid;                 // one Partial row per block
        plan->slot_base[t] = (uint32_t)rows;
        rows += plan->n_slots[t];
    }
    size_t table = (size_t)T * sizeof(DevTensor) + (size_t)T * (size_t)K * sizeof(void*);
    plan->table_bytes = (table + 255) / 256 * 256;
    plan->state_bytes = ((size_t)T * (size_t)(K + 1) * sizeof(CandState) + 255) / 256 * 256;
    plan->partial_bytes = (size_t)rows * (size_t)K * sizeof(Partial);
    plan->total_bytes = sizeof(WorkspaceHeader) + plan->table_bytes + plan->state_bytes + plan->partial_bytes;
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

int ensure(void** buf, size_t* have, size_t want) {
    if (*have >= want) return RKV_OK;
    if (*buf) { cudaFree(*buf); *buf = nullptr; *have = 0; }
    size_t bytes = (want + (size_t(1) << 20) - 1) >> 20 << 20;
    if (cudaMalloc(buf, bytes) != cudaSuccess) { cudaGetLastError(); return RKV_ERR_CUDA; }
    *have = bytes;
    return RKV_OK;
}

// Fill the device-side descriptor of tensor t.
void fill_dev_tensor(DevTensor& d, const rkv_tensor_desc& s, const Plan& plan, int t, const void** d_ptrs, int K) {
    memset(&d, 0, sizeof d);
    d.n = s.n;
    d.ref = s.ref_src == RKV_SRC_POINTER ? s.ref : nullptr;
    d.input = s.input_src == RKV_SRC_POINTER ? s.input : nullptr;
    d.cands = d_ptrs + (size_t)t * K;
    d.ref_seed = s.ref_gen.seed; d.ref_stream = s.ref_gen.stream_id; d.ref_dist = s.ref_gen.dist;
    d.in_seed = s.input_gen.seed; d.in_stream = s.input_gen.stream_id; d.in_dist = s.input_gen.dist;
    d.cand_dtype = s.cand_dtype; d.ref_dtype = s.ref_dtype;
    d.ref_src = s.ref_src; d.input_src = s.input_src;
    d.atol = s.atol; d.rtol = s.rtol;
    d.n_tiles = plan.n_tiles[t]; d.warm_tiles = plan.warm_tiles[t]; d.tail_tiles = plan.tail_tiles[t]; d.tail_div = plan.tail_div[t];
    d.n_slots = plan.n_slots[t]; d.slot_base = plan.slot_base[t];
    d.variant = plan.variant[t];
}

// Workspace pieces.
struct Layout {
    WorkspaceHeader* header;
    DevTensor* d_tensors;
    const void** d_ptrs;
    CandState* state;
    Partial* partials;
};

Layout layout_of(void* workspace, const Plan& plan, int T) {
    unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
    Layout L;
    L.header = reinterpret_cast<WorkspaceHeader*>(ws);
    L.d_tensors = reinterpret_cast<DevTensor*>(ws + sizeof(WorkspaceHeader));
    L.d_ptrs = reinterpret_cast<const void**>(ws + sizeof(WorkspaceHeader) + (size_t)T * sizeof(DevTensor));
    L.state = reinterpret_cast<CandState*>(ws + sizeof(WorkspaceHeader) + plan.table_bytes);
    L.partials = reinterpret_cast<Partial*>(ws + sizeof(WorkspaceHeader) + plan.table_bytes + plan.state_bytes);
    return L;
}

// Launch verify over candidates [k_begin, k_end) (+ finalize); the tables must be in place.
int launch_case(const rkv_tensor_desc* tensors, int T, int K, int k_begin, int k_end, bool finalize,
                const Plan& plan, const Layout& L, rkv_stats* stats_out, uint32_t* joint_pass,
                cudaStream_t stream) {
    uint32_t items[4] = {0, 0, 0, 0};
    const uint32_t kcount = (uint32_t)(k_end - k_begin);
    for (int t = 0; t < T; ++t)
        items[plan.variant[t]] += (uint32_t)items_of(plan.n_tiles[t], plan.warm_tiles[t], plan.tail_tiles[t], plan.tail_div[t], kcount, plan.grid);
    (void)tensors;
    int rc = launch_verify(L.d_tensors, T, K, k_begin, k_end, items, (int)plan.grid, L.state, L.partials,
                           L.header, stream);
    if (rc != RKV_OK) return rc;
    if (finalize) rc = launch_finalize(L.d_tensors, T, K, L.state, L.partials, stats_out, joint_pass, stream);
    return rc;
}

// Build the device tables in the workspace, clear the per-candidate state and the
// partials, and launch verify (+ finalize).
int run_case(const rkv_tensor_desc* tensors, int T, int K, int k_begin, int k_end, bool finalize,
             bool upload, const Plan& plan, rkv_stats* stats_out, uint32_t* joint_pass, void* workspace,
             cudaStream_t stream) {
    const Layout L = layout_of(workspace, plan, T);
    if (upload) {
        std::vector<unsigned char> blob(sizeof(WorkspaceHeader) + plan.table_bytes, 0);
        DevTensor* h_t = reinterpret_cast<DevTensor*>(blob.data() + sizeof(WorkspaceHeader));
        const void** h_p = reinterpret_cast<const void**>(blob.data() + sizeof(WorkspaceHeader) +
                                                          (size_t)T * sizeof(DevTensor));
        for (int t = 0; t < T; ++t) {
            fill_dev_tensor(h_t[t], tensors[t], plan, t, L.d_ptrs, K);
            for (int k = 0; k < K; ++k) h_p[(size_t)t * K + k] = tensors[t].cands[k];
        }
        if (cudaMemcpyAsync(workspace, blob.data(), blob.size(), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
            cudaMemsetAsync(L.state, 0, plan.state_bytes + plan.partial_bytes, stream) != cudaSuccess) {
            cudaGetLastError();
            return RKV_ERR_CUDA;
        }
    }
    return launch_case(tensors, T, K, k_begin, k_end, finalize, plan, L, stats_out, joint_pass, stream);
}

}  // namespace
}  // namespace rkv

using namespace rkv;

// ----------------------------------------------------------------------------
// C ABI
// ----------------------------------------------------------------------------
extern "C" {

int rkv_version(void) { return 100; }

const char* rkv_status_string(int status) {
    switch (status) {
        case RKV_OK: return "ok";
        case RKV_ERR_INVALID_ARG: return "invalid argument";
        case RKV_ERR_UNSUPPORTED: return "unsupported size or combination";
        case RKV_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case RKV_ERR_WORKSPACE: return "workspace missing or too small";
        case RKV_ERR_CUDA: return "CUDA runtime error";
        case RKV_ERR_TIMEOUT: return "device-side bounded wait ran out";
        default: return "unknown status";
    }
}

int rkv_set_stream(void* cuda_stream) {
    g_stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    return RKV_OK;
}

int rkv_plan_items(uint64_t n, int cand_dtype, int K, int num_sms, uint32_t* tile_elems_out, uint32_t* n_tiles,
                   uint32_t* warm_tiles, uint32_t* parts_warm, uint32_t* parts_main, uint32_t* tail_tiles,
                   uint32_t* parts_tail) {
    if (!tile_elems_out || !n_tiles || !warm_tiles || !parts_warm || !parts_main || !tail_tiles || !parts_tail)
        return RKV_ERR_INVALID_ARG;
    if (!dtype_ok(cand_dtype)) return RKV_ERR_INVALID_ARG;
    if (n >= kMaxN) return RKV_ERR_UNSUPPORTED;
    if (K < 1 || num_sms < 1 || num_sms > (1 << 20)) return RKV_ERR_INVALID_ARG;
    const int rc = plan_one(n, cand_dtype, n_tiles, warm_tiles);
    if (rc != RKV_OK) return rc;
    const uint32_t grid = (uint32_t)(num_sms * kBlocksPerSm);
    *tile_elems_out = tile_elems(cand_dtype);
    *tail_tiles = tail_tiles_of(*n_tiles, *warm_tiles, grid);
    const uint32_t main_tiles = group_tiles(1, *n_tiles, *warm_tiles, *tail_tiles);
    *parts_warm = group_parts(0, *warm_tiles, (uint32_t)K, grid, kTailDiv);
    *parts_main = main_tiles ? group_parts(1, main_tiles, (uint32_t)K, grid, kTailDiv) : 0u;
    *parts_tail = *tail_tiles ? group_parts(2, *tail_tiles, (uint32_t)K, grid, kTailDiv) : 0u;
    return RKV_OK;
}

int rkv_gen_inputs_ex(uint64_t seed, uint64_t stream_id, int dist, uint64_t n, uint64_t first_elem,
                      int dtype, void* out, void* cuda_stream) {
    if (!out || n < 1 || !dist_ok(dist) || !dtype_ok(dtype) || (first_elem & 3u))
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
        if (tensors[t].n < 1 || tensors[t].n >= kMaxN) return 0;
    int sms = 0;
    if (current_num_sms(&sms) != RKV_OK) return 0;
    Plan plan;
    if (make_plan(tensors, T, K, K, sms, &plan) != RKV_OK) return 0;
    return plan.total_bytes;
}

int rkv_verify_multi(const rkv_tensor_desc* tensors, int T, int K, rkv_stats* stats_out,
                     uint32_t* joint_pass, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = validate_tensors(tensors, T, K);
    if (rc != RKV_OK) return rc;
    if (!stats_out) return RKV_ERR_INVALID_ARG;
    if (!workspace) return RKV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return RKV_ERR_ALIGNMENT;
    int sms = 0;
    rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    Plan plan;
    rc = make_plan(tensors, T, K, K, sms, &plan);
    if (rc != RKV_OK) return rc;
    if (workspace_bytes < plan.total_bytes) return RKV_ERR_WORKSPACE;
    rc = refuse_capture(reinterpret_cast<cudaStream_t>(cuda_stream));
    if (rc != RKV_OK) return rc;
    return run_case(tensors, T, K, 0, K, true, true, plan, stats_out, joint_pass, workspace,
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
    int rc = validate_tensors(&d, 1, K);
    if (rc != RKV_OK) return rc;
    if (!stats_out) return RKV_ERR_INVALID_ARG;
    int sms = 0;
    rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    Plan plan;
    rc = make_plan(&d, 1, K, K, sms, &plan);
    if (rc != RKV_OK) return rc;
    rc = refuse_capture(g_stream);
    if (rc != RKV_OK) return rc;
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceCache& c = g_cache[dev & 63];
    rc = ensure(&c.workspace, &c.workspace_bytes, plan.total_bytes);
    if (rc != RKV_OK) return rc;
    return run_case(&d, 1, K, 0, K, true, true, plan, stats_out, nullptr, c.workspace, g_stream);
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
        const rkv_tensor_desc& d = tensors[t];
        if (d.n < 1 || !dtype_ok(d.cand_dtype) || !dtype_ok(d.ref_dtype) || !finite_nonneg(d.atol) ||
            !finite_nonneg(d.rtol) || !d.cands)
            return RKV_ERR_INVALID_ARG;
        if (d.n >= kMaxN) return RKV_ERR_UNSUPPORTED;
        if (d.ref_src == RKV_SRC_POINTER ? !d.ref : (d.ref_src != RKV_SRC_GENERATED || !dist_ok(d.ref_gen.dist)))
            return RKV_ERR_INVALID_ARG;
        if (d.input_src == RKV_SRC_POINTER ? !d.input
                                           : (d.input_src == RKV_SRC_GENERATED ? !dist_ok(d.input_gen.dist)
                                                                               : d.input_src != RKV_SRC_NONE))
            return RKV_ERR_INVALID_ARG;
        for (int k = 0; k < K; ++k)
            if (!d.cands[k]) return RKV_ERR_INVALID_ARG;
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
    auto round256 = [](size_t b) { return (b + 255) / 256 * 256; };
    auto esz = [](int dtype) { return (size_t)(dtype == RKV_BF16 ? 2 : 4); };
    size_t fixed_bytes = 0, per_cand = 0;
    for (int t = 0; t < T; ++t) {
        const rkv_tensor_desc& d = tensors[t];
        if (d.ref_src == RKV_SRC_POINTER) fixed_bytes += round256((size_t)d.n * esz(d.ref_dtype));
        if (d.input_src == RKV_SRC_POINTER) fixed_bytes += round256((size_t)d.n * esz(d.cand_dtype));
        per_cand += round256((size_t)d.n * esz(d.cand_dtype));
    }
    // candidates travel in chunks of kc, two chunks in flight
    size_t kc = (size_t(512) << 20) / per_cand;
    if (kc < 1) kc = 1;
    if (kc > (size_t)K) kc = (size_t)K;
    if (kc > 16) kc = 16;
    const size_t stats_bytes = round256((size_t)K * (size_t)T * sizeof(rkv_stats));
    const size_t joint_bytes = round256((size_t)K * sizeof(uint32_t));
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
            const size_t b = (size_t)d.n * esz(d.ref_dtype);
            fail |= cudaMemcpyAsync(base + fixed_at, tensors[t].ref, b, cudaMemcpyHostToDevice, main) != cudaSuccess;
            d.ref = base + fixed_at;
            fixed_at += round256(b);
        }
        if (d.input_src == RKV_SRC_POINTER) {
            const size_t b = (size_t)d.n * esz(d.cand_dtype);
            fail |= cudaMemcpyAsync(base + fixed_at, tensors[t].input, b, cudaMemcpyHostToDevice, main) != cudaSuccess;
            d.input = base + fixed_at;
            fixed_at += round256(b);
        }
        const size_t cb = round256((size_t)d.n * esz(d.cand_dtype));
        for (int k = 0; k < K; ++k)
            ptrs[(size_t)t * K + k] = d_chunk[((size_t)k / kc) & 1] + ((size_t)k % kc) * per_cand + tensor_at;
        d.cands = ptrs.data() + (size_t)t * K;
        tensor_at += cb;
    }
    Plan plan;
    rc = make_plan(dd.data(), T, K, (int)kc, sms, &plan);
    if (rc != RKV_OK) return rc;
    rc = ensure(&c.workspace, &c.workspace_bytes, plan.total_bytes);
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
                                        (size_t)tensors[t].n * esz(tensors[t].cand_dtype), cudaMemcpyHostToDevice,
                                        c.copy_stream[b]) != cudaSuccess;
        fail |= cudaEventRecord(c.copied[b], c.copy_stream[b]) != cudaSuccess;
        fail |= cudaStreamWaitEvent(main, c.copied[b], 0) != cudaSuccess;
        if (fail) break;
        rc = run_case(dd.data(), T, K, k0, k1, k1 == K, ch == 0, plan, d_stats, d_joint, c.workspace, main);
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
    int rc = validate_tensors(&d, 1, K);
    if (rc != RKV_OK) return rc;
    if (!stats_out) return RKV_ERR_INVALID_ARG;
    if (K > kStaticMaxK) return RKV_ERR_UNSUPPORTED;
    int sms = 0;
    rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    Plan plan;
    rc = make_plan(&d, 1, K, K, sms, &plan);
    if (rc != RKV_OK) return rc;
    if (plan.total_bytes > kStaticScratchBytes) return RKV_ERR_UNSUPPORTED;
    rc = refuse_capture(reinterpret_cast<cudaStream_t>(cuda_stream));
    if (rc != RKV_OK) return rc;
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != RKV_OK) return rc;

    // header (status word = 0) + descriptor + pointer table, built on the stack
    constexpr size_t kBlobMax = sizeof(WorkspaceHeader) +
                                (sizeof(DevTensor) + kStaticMaxK * sizeof(void*) + 255) / 256 * 256;
    alignas(16) unsigned char blob[kBlobMax];
    const size_t blob_bytes = sizeof(WorkspaceHeader) + plan.table_bytes;
    if (blob_bytes > kBlobMax) return RKV_ERR_UNSUPPORTED;
    memset(blob, 0, blob_bytes);
    const Layout L = layout_of(scratch, plan, 1);
    fill_dev_tensor(*reinterpret_cast<DevTensor*>(blob + sizeof(WorkspaceHeader)), d, plan, 0, L.d_ptrs, K);
    const void** h_p = reinterpret_cast<const void**>(blob + sizeof(WorkspaceHeader) + sizeof(DevTensor));
    for (int k = 0; k < K; ++k) h_p[k] = cands[k];

    // what must start at zero in the shared array: the status word (in the blob), the
    // per-candidate state and the partial results
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(scratch, blob, blob_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemsetAsync(L.state, 0, plan.state_bytes + plan.partial_bytes, stream) != cudaSuccess) {
        cudaGetLastError();
        return RKV_ERR_CUDA;
    }
    return launch_case(&d, 1, K, 0, K, true, plan, L, stats_out, nullptr, stream);
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
