// Task-soundness screens over the reference outputs of one task for S seeds (sm_100a):
// one streaming pass that reads every output byte once and yields the range, mean and
// standard deviation of all values, the largest per-element spread across the seeds and
// whether the outputs are uniform along an axis; then a small merge kernel.
//
// Bound: HBM read bandwidth (S * n * element size bytes, each read once).  No tensor
// cores: about ten operations per element.
//
// Layout of the work: a thread takes 16-byte vectors (4 fp32 or 8 bf16 elements) at a
// grid stride; for one vector position it visits the S outputs in turn, so the per-element
// minimum and maximum across seeds never leave registers (up to three fp32 outputs:
// screen_few_kernel, which has the pieces of two positions in flight).  Sums are fp64, taken about a
// pivot (the mean of the first finite values of the first output, computed identically by
// every block) so that a large common offset costs the variance no digits.  Reductions are
// deterministic: fixed shuffle trees, one partial per block, merged in block order;
// maxima are lexicographic (value descending, index ascending).
#include <string.h>

#include "rkv_internal.h"

namespace rkv {

namespace {

constexpr int kScreenThreads = 256;
constexpr int kScreenBlocksPerSm = 3;         // resident blocks per SM, fp32 outputs
constexpr int kScreenBlocksPerSmB16 = 3;
constexpr int kScreenMaxSeeds = 16;
constexpr int kPivotSample = 256;
constexpr uint32_t kFull = 0xFFFFFFFFu;
constexpr float kInfF = __builtin_huge_valf();

struct ScreenArgs {
    const void* outs[kScreenMaxSeeds];
    uint64_t rows, cols, n;
    int32_t S;
};

struct __align__(16) ScreenPartial {
    double sum;            // of (x - pivot) over the finite values
    double sumsq;          // of (x - pivot)^2
    unsigned long long n_fin;
    unsigned long long n_nonfin;
    unsigned long long arg;          // first element with the largest spread
    float vmin, vmax;
    float spread;          // -1: none
    uint32_t nonuniform;   // bit0: some column is not constant; bit1: some row is not constant
};
static_assert(sizeof(ScreenPartial) == 64, "ScreenPartial layout");

struct ScreenHeader {
    double pivot;
    uint32_t grid;
    uint32_t reserved[13];
};
static_assert(sizeof(ScreenHeader) == 64, "ScreenHeader layout");

__device__ __forceinline__ bool finite_bits(uint32_t b) { return (b & 0x7F800000u) != 0x7F800000u; }

template <bool B16>
__device__ __forceinline__ uint32_t load_elem_bits(const void* p, uint64_t i) {
    if (B16) return (uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p) + i) << 16;
    return __ldg(reinterpret_cast<const uint32_t*>(p) + i);
}

struct Acc {
    double sum, sumsq;
    unsigned long long n_fin, n_nonfin, arg;     // n_fin: values visited until the thread is done, then the finite ones
    float vmin, vmax, spread;
    uint32_t nonuniform;
};

__device__ __forceinline__ void acc_value(Acc& a, uint32_t b, double pivot, float& lo, float& hi, bool& ok) {
    if (finite_bits(b)) {
        const float x = __uint_as_float(b);
        const double d = (double)x - pivot;
        a.sum += d;
        a.sumsq = fma(d, d, a.sumsq);
        lo = fminf(lo, x);
        hi = fmaxf(hi, x);
    } else {
        a.n_nonfin++;
        ok = false;
    }
}

// lexicographic merge of (spread, arg): larger spread, then smaller index
__device__ __forceinline__ void merge_spread(float& s, unsigned long long& arg, float s2, unsigned long long arg2) {
    if (s2 > s || (s2 == s && arg2 < arg)) { s = s2; arg = arg2; }
}

__device__ __forceinline__ void merge_acc(Acc& a, const Acc& b) {
    a.sum += b.sum;
    a.sumsq += b.sumsq;
    a.n_fin += b.n_fin;
    a.n_nonfin += b.n_nonfin;
    a.vmin = fminf(a.vmin, b.vmin);
    a.vmax = fmaxf(a.vmax, b.vmax);
    merge_spread(a.spread, a.arg, b.spread, b.arg);
    a.nonuniform |= b.nonuniform;
}

__device__ __forceinline__ Acc shfl_acc(const Acc& a, int off) {
    Acc b;
    b.sum = __shfl_xor_sync(kFull, a.sum, off);
    b.sumsq = __shfl_xor_sync(kFull, a.sumsq, off);
    b.n_fin = __shfl_xor_sync(kFull, a.n_fin, off);
    b.n_nonfin = __shfl_xor_sync(kFull, a.n_nonfin, off);
    b.arg = __shfl_xor_sync(kFull, a.arg, off);
    b.vmin = __shfl_xor_sync(kFull, a.vmin, off);
    b.vmax = __shfl_xor_sync(kFull, a.vmax, off);
    b.spread = __shfl_xor_sync(kFull, a.spread, off);
    b.nonuniform = __shfl_xor_sync(kFull, a.nonuniform, off);
    return b;
}

// One element position across all seeds, scalar loads, any shape (the ragged end of a
// tensor, and shapes whose rows do not hold whole 16-byte vectors).
template <bool B16>
__device__ __forceinline__ void screen_element(const ScreenArgs& A, Acc& a, double pivot, uint64_t i,
                                               bool check_axes) {
    float lo = kInfF, hi = -kInfF;
    bool ok = true;
    const uint64_t r = i / A.cols, c = i - r * A.cols;
    a.n_fin += (unsigned long long)A.S;
    for (int s = 0; s < A.S; ++s) {
        const uint32_t b = load_elem_bits<B16>(A.outs[s], i);
        acc_value(a, b, pivot, lo, hi, ok);
        if (check_axes) {
            if (b != load_elem_bits<B16>(A.outs[s], c)) a.nonuniform |= 1u;
            if (b != load_elem_bits<B16>(A.outs[s], r * A.cols)) a.nonuniform |= 2u;
        }
    }
    a.vmin = fminf(a.vmin, lo);
    a.vmax = fmaxf(a.vmax, hi);
    if (A.S >= 2 && ok) {
        const float d = fabsf(__fsub_rn(hi, lo));
        if (d > a.spread) { a.spread = d; a.arg = i; }
    }
}

// The work of screen_chunk on N outputs whose pieces q[0 .. N-1] are already in registers.
template <bool B16, int N>
__device__ __forceinline__ void screen_chunk_loaded(const ScreenArgs& A, Acc& a, double pivot, int s0,
                                                    const uint4 (&q)[N], uint32_t need, uint64_t r, uint64_t c0,
                                                    float (&lo)[B16 ? 8 : 4], float (&hi)[B16 ? 8 : 4],
                                                    bool (&ok)[B16 ? 8 : 4]) {
    constexpr int VEC = B16 ? 8 : 4;
    uint32_t b[N][VEC];
#pragma unroll
    for (int u = 0; u < N; ++u) {
        const uint32_t wv[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
        for (int j = 0; j < VEC; ++j)
            b[u][j] = B16 ? ((j & 1) ? (wv[j >> 1] & 0xFFFF0000u) : (wv[j >> 1] << 16)) : wv[j];
    }
    float chk = 0.0f;
#pragma unroll
    for (int u = 0; u < N; ++u)
#pragma unroll
        for (int j = 0; j < VEC; ++j) chk = __fmaf_rn(__uint_as_float(b[u][j]), 0.0f, chk);
    if (chk == 0.0f) {
#pragma unroll
        for (int u = 0; u < N; ++u)
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
                const float x = __uint_as_float(b[u][j]);
                lo[j] = fminf(lo[j], x);
                hi[j] = fmaxf(hi[j], x);
                const double d = (double)x - pivot;
                a.sum += d;
                a.sumsq = fma(d, d, a.sumsq);
            }
    } else {
#pragma unroll
        for (int u = 0; u < N; ++u)
#pragma unroll
            for (int j = 0; j < VEC; ++j) acc_value(a, b[u][j], pivot, lo[j], hi[j], ok[j]);
    }
    if (need) {
#pragma unroll
        for (int u = 0; u < N; ++u) {
            if (need & 1u) {
                // the same columns of row 0, as stored
                const uint4 f = __ldg(reinterpret_cast<const uint4*>(A.outs[s0 + u]) + c0 / VEC);
                if ((q[u].x ^ f.x) | (q[u].y ^ f.y) | (q[u].z ^ f.z) | (q[u].w ^ f.w)) a.nonuniform |= 1u;
            }
            if (need & 2u) {
                const uint32_t first = load_elem_bits<B16>(A.outs[s0 + u], r * A.cols);
                uint32_t diff = 0;
#pragma unroll
                for (int j = 0; j < VEC; ++j) diff |= b[u][j] ^ first;
                if (diff) a.nonuniform |= 2u;
            }
        }
    }
}


// N outputs (s0 .. s0+N-1) at one vector position: their loads are issued together, then one
// test tells whether all N * VEC values are finite (x * 0 is a zero for a finite x and NaN
// otherwise) and the branch-free path can run.
template <bool B16, int N>
__device__ __forceinline__ void screen_chunk(const ScreenArgs& A, Acc& a, double pivot, int s0, uint64_t v,
                                             uint32_t need, uint64_t r, uint64_t c0,
                                             float (&lo)[B16 ? 8 : 4], float (&hi)[B16 ? 8 : 4],
                                             bool (&ok)[B16 ? 8 : 4]) {
    uint4 q[N];
#pragma unroll
    for (int u = 0; u < N; ++u) q[u] = __ldg(reinterpret_cast<const uint4*>(A.outs[s0 + u]) + v);
    screen_chunk_loaded<B16, N>(A, a, pivot, s0, q, need, r, c0, lo, hi, ok);
}

// The pivot: mean of the finite values among the first elements of the first output, computed
// identically by every block (warp 0), handed to all threads through shared memory.
template <bool B16>
__device__ __forceinline__ double block_pivot(const ScreenArgs& A, double* s_pivot) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (warp == 0) {
        double ps = 0.0;
        uint32_t pc = 0;
        uint32_t pb[kPivotSample / 32];
#pragma unroll
        for (int t = 0; t < kPivotSample / 32; ++t) {       // independent loads, issued together
            const uint64_t i = (uint64_t)(lane + 32 * t);
            pb[t] = i < A.n ? load_elem_bits<B16>(A.outs[0], i) : 0x7FC00000u;
        }
#pragma unroll
        for (int t = 0; t < kPivotSample / 32; ++t)
            if (finite_bits(pb[t])) { ps += (double)__uint_as_float(pb[t]); pc++; }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            ps += __shfl_xor_sync(kFull, ps, off);
            pc += __shfl_xor_sync(kFull, pc, off);
        }
        if (lane == 0) *s_pivot = pc ? ps / (double)pc : 0.0;
    }
    __syncthreads();
    return *s_pivot;
}

__device__ __forceinline__ void acc_clear(Acc& a) {
    a.sum = 0.0; a.sumsq = 0.0; a.n_fin = 0; a.n_nonfin = 0; a.arg = RKV_NO_INDEX;
    a.vmin = kInfF; a.vmax = -kInfF; a.spread = -1.0f; a.nonuniform = 0u;
}

// Block reduction (fixed shuffle tree, then the warps in order) and the block's partial.
__device__ __forceinline__ void block_end(Acc a, uint32_t axes_wanted, double pivot, Acc* s_acc,
                                          ScreenHeader* __restrict__ header, ScreenPartial* __restrict__ partials) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    a.nonuniform &= axes_wanted;
    a.n_fin -= a.n_nonfin;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const Acc b = shfl_acc(a, off);
        merge_acc(a, b);
    }
    if (lane == 0) s_acc[warp] = a;
    __syncthreads();
    if (tid == 0) {
        Acc t = s_acc[0];
        for (int w = 1; w < kScreenThreads / 32; ++w) merge_acc(t, s_acc[w]);
        ScreenPartial p;
        p.sum = t.sum; p.sumsq = t.sumsq; p.n_fin = t.n_fin; p.n_nonfin = t.n_nonfin; p.arg = t.arg;
        p.vmin = t.vmin; p.vmax = t.vmax; p.spread = t.spread; p.nonuniform = t.nonuniform;
        partials[blockIdx.x] = p;
        if (blockIdx.x == 0) { header->pivot = pivot; header->grid = gridDim.x; }
    }
}

template <bool B16>
__global__ void __launch_bounds__(kScreenThreads, B16 ? kScreenBlocksPerSmB16 : kScreenBlocksPerSm)
screen_kernel(const ScreenArgs A, ScreenHeader* __restrict__ header, ScreenPartial* __restrict__ partials) {
    constexpr int VEC = B16 ? 8 : 4;
    __shared__ double s_pivot;
    __shared__ Acc s_acc[kScreenThreads / 32];
    const int tid = threadIdx.x;

    const double pivot = block_pivot<B16>(A, &s_pivot);

    Acc a;
    acc_clear(a);

    const bool vec_rows = (A.cols % VEC) == 0;       // every 16-byte vector lies inside one row
    const uint64_t nvec = A.n / VEC;
    const uint64_t stride = (uint64_t)gridDim.x * kScreenThreads;
    const uint32_t axes_wanted = (A.rows >= 2 ? 1u : 0u) | (A.cols >= 2 ? 2u : 0u);

    if (vec_rows) {
        for (uint64_t v = (uint64_t)blockIdx.x * kScreenThreads + tid; v < nvec; v += stride) {
            const uint64_t i0 = v * VEC;
            a.n_fin += (unsigned long long)(VEC * A.S);
            float lo[VEC], hi[VEC];
            bool ok[VEC];
#pragma unroll
            for (int j = 0; j < VEC; ++j) { lo[j] = kInfF; hi[j] = -kInfF; ok[j] = true; }
            // a mismatch, once seen, settles an axis for good: stop looking
            const uint32_t need = axes_wanted & ~a.nonuniform;
            uint64_t r = 0, c0 = 0;
            if (need) { r = i0 / A.cols; c0 = i0 - r * A.cols; }
            // the outputs in chunks of 8, 4, 3 (fp32 only), 2 and 1
            int s0 = 0;
            if (!B16) {
                for (; A.S - s0 >= 8; s0 += 8) screen_chunk<B16, B16 ? 1 : 8>(A, a, pivot, s0, v, need, r, c0, lo, hi, ok);
                if (A.S - s0 >= 4) { screen_chunk<B16, B16 ? 1 : 4>(A, a, pivot, s0, v, need, r, c0, lo, hi, ok); s0 += 4; }
            }
            if (!B16 && A.S - s0 == 3) { screen_chunk<B16, B16 ? 1 : 3>(A, a, pivot, s0, v, need, r, c0, lo, hi, ok); s0 += 3; }
            for (; A.S - s0 >= 2; s0 += 2) screen_chunk<B16, 2>(A, a, pivot, s0, v, need, r, c0, lo, hi, ok);
            if (A.S - s0 >= 1) screen_chunk<B16, 1>(A, a, pivot, s0, v, need, r, c0, lo, hi, ok);
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
                a.vmin = fminf(a.vmin, lo[j]);
                a.vmax = fmaxf(a.vmax, hi[j]);
            }
            if (A.S >= 2) {
#pragma unroll
                for (int j = 0; j < VEC; ++j) {
                    if (ok[j]) {
                        const float d = fabsf(__fsub_rn(hi[j], lo[j]));
                        if (d > a.spread) { a.spread = d; a.arg = i0 + j; }
                    }
                }
            }
        }
        // the last n % VEC elements
        if (blockIdx.x == 0 && tid == 0)
            for (uint64_t i = nvec * VEC; i < A.n; ++i) screen_element<B16>(A, a, pivot, i, true);
    } else {
        for (uint64_t i = (uint64_t)blockIdx.x * kScreenThreads + tid; i < A.n; i += stride)
            screen_element<B16>(A, a, pivot, i, (axes_wanted & ~a.nonuniform) != 0u);
    }
    block_end(a, axes_wanted, pivot, s_acc, header, partials);
}

// One vector position of fp32 outputs whose N = S pieces are already in registers: everything the
// general kernel does for a position.
template <int N>
__device__ __forceinline__ void screen_position_loaded(const ScreenArgs& A, Acc& a, double pivot, uint64_t v,
                                                       uint32_t axes_wanted, const uint4 (&q)[N]) {
    constexpr int VEC = 4;
    const uint64_t i0 = v * VEC;
    a.n_fin += (unsigned long long)(VEC * N);
    float lo[VEC], hi[VEC];
    bool ok[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) { lo[j] = kInfF; hi[j] = -kInfF; ok[j] = true; }
    const uint32_t need = axes_wanted & ~a.nonuniform;
    uint64_t r = 0, c0 = 0;
    if (need) { r = i0 / A.cols; c0 = i0 - r * A.cols; }
    screen_chunk_loaded<false, N>(A, a, pivot, 0, q, need, r, c0, lo, hi, ok);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        a.vmin = fminf(a.vmin, lo[j]);
        a.vmax = fmaxf(a.vmax, hi[j]);
    }
    if (N >= 2) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            if (ok[j]) {
                const float d = fabsf(__fsub_rn(hi[j], lo[j]));
                if (d > a.spread) { a.spread = d; a.arg = i0 + j; }
            }
        }
    }
}

// N <= 3 fp32 outputs whose rows hold whole 16-byte vectors: the pieces of two positions (one grid
// stride apart) are loaded before either is worked on, 2 * N loads per thread in flight instead of
// N.  Same statistics as screen_kernel; a kernel of its own so that its registers do not weigh on
// the general loop.
template <int N>
__global__ void __launch_bounds__(kScreenThreads, kScreenBlocksPerSm)
screen_few_kernel(const ScreenArgs A, ScreenHeader* __restrict__ header, ScreenPartial* __restrict__ partials) {
    constexpr int VEC = 4;
    __shared__ double s_pivot;
    __shared__ Acc s_acc[kScreenThreads / 32];
    const int tid = threadIdx.x;
    const double pivot = block_pivot<false>(A, &s_pivot);
    Acc a;
    acc_clear(a);
    const uint64_t nvec = A.n / VEC;
    const uint64_t stride = (uint64_t)gridDim.x * kScreenThreads;
    const uint32_t axes_wanted = (A.rows >= 2 ? 1u : 0u) | (A.cols >= 2 ? 2u : 0u);
    for (uint64_t v = (uint64_t)blockIdx.x * kScreenThreads + tid; v < nvec; v += 2 * stride) {
        const uint64_t v2 = v + stride;
        const bool two = v2 < nvec;
        uint4 qa[N], qb[N];
#pragma unroll
        for (int u = 0; u < N; ++u) qa[u] = __ldg(reinterpret_cast<const uint4*>(A.outs[u]) + v);
        if (two) {
#pragma unroll
            for (int u = 0; u < N; ++u) qb[u] = __ldg(reinterpret_cast<const uint4*>(A.outs[u]) + v2);
        }
        screen_position_loaded<N>(A, a, pivot, v, axes_wanted, qa);
        if (two) screen_position_loaded<N>(A, a, pivot, v2, axes_wanted, qb);
    }
    // (cols is a multiple of 4 here, so n is: no ragged end)
    block_end(a, axes_wanted, pivot, s_acc, header, partials);
}

__global__ void __launch_bounds__(kScreenThreads)
screen_finalize_kernel(const ScreenArgs A, const ScreenHeader* __restrict__ header,
                       const ScreenPartial* __restrict__ partials, int grid, float range_lim, double std_lim,
                       float spread_lim, rkv_screen_stats* __restrict__ out) {
    __shared__ Acc s_acc[kScreenThreads];
    const int tid = threadIdx.x;
    Acc a;
    a.sum = 0.0; a.sumsq = 0.0; a.n_fin = 0; a.n_nonfin = 0; a.arg = RKV_NO_INDEX;
    a.vmin = kInfF; a.vmax = -kInfF; a.spread = -1.0f; a.nonuniform = 0u;
    for (int p = tid; p < grid; p += kScreenThreads) {
        const ScreenPartial q = partials[p];
        Acc b;
        b.sum = q.sum; b.sumsq = q.sumsq; b.n_fin = q.n_fin; b.n_nonfin = q.n_nonfin; b.arg = q.arg;
        b.vmin = q.vmin; b.vmax = q.vmax; b.spread = q.spread; b.nonuniform = q.nonuniform;
        merge_acc(a, b);
    }
    s_acc[tid] = a;
    __syncthreads();
    for (int w = kScreenThreads / 2; w > 0; w >>= 1) {
        if (tid < w) { Acc t = s_acc[tid]; merge_acc(t, s_acc[tid + w]); s_acc[tid] = t; }
        __syncthreads();
    }
    if (tid == 0) {
        const Acc t = s_acc[0];
        rkv_screen_stats r;
        r.reserved = 0; r.reserved2 = 0;
        r.n_values = (uint64_t)A.S * A.n;
        r.n_nonfinite = t.n_nonfin;
        r.argmax_seed_spread = t.arg;
        double mean = 0.0, sd = 0.0;
        if (t.n_fin) {
            const double m1 = t.sum / (double)t.n_fin;
            double var = t.sumsq / (double)t.n_fin - m1 * m1;
            if (var < 0.0) var = 0.0;
            mean = header->pivot + m1;
            sd = sqrt(var);
        }
        r.mean = mean;
        r.std = sd;
        r.vmin = t.vmin;
        r.vmax = t.vmax;
        r.max_seed_spread = t.spread;
        uint32_t f = 0;
        if (t.n_fin && t.vmin >= -range_lim && t.vmax <= range_lim) f |= RKV_SCREEN_NARROW_RANGE;
        if (t.n_fin && sd < std_lim) f |= RKV_SCREEN_LOW_STD;
        if (A.S >= 2 && t.arg != RKV_NO_INDEX && t.spread < spread_lim) f |= RKV_SCREEN_LOW_SEED_VARIATION;
        if (A.rows >= 2 && !(t.nonuniform & 1u)) f |= RKV_SCREEN_UNIFORM_AXIS0;
        if (A.cols >= 2 && !(t.nonuniform & 2u)) f |= RKV_SCREEN_UNIFORM_AXIS1;
        if (t.n_nonfin) f |= RKV_SCREEN_NONFINITE;
        r.flags = f;
        *out = r;
    }
}

}  // namespace

}  // namespace rkv

using namespace rkv;

extern "C" {

size_t rkv_screen_workspace_bytes(void) {
    int sms = 0;
    if (current_num_sms(&sms) != RKV_OK) return 0;
    return sizeof(ScreenHeader) + (size_t)sms * kScreenBlocksPerSm * sizeof(ScreenPartial);
}

int rkv_screen_outputs(const void* const* outs, int S, uint64_t rows, uint64_t cols, int dtype, float range_lim,
                       double std_lim, float spread_lim, rkv_screen_stats* stats_out, void* workspace,
                       size_t workspace_bytes, void* cuda_stream) {
    if (!outs || !stats_out || S < 1 || rows < 1 || cols < 1) return RKV_ERR_INVALID_ARG;
    if (dtype != RKV_F32 && dtype != RKV_BF16) return RKV_ERR_INVALID_ARG;
    if (S > kScreenMaxSeeds) return RKV_ERR_UNSUPPORTED;
    if (rows >= kMaxN || cols >= kMaxN || rows * cols >= kMaxN) return RKV_ERR_UNSUPPORTED;
    if (!(range_lim >= 0.0f) || !(std_lim >= 0.0) || !(spread_lim >= 0.0f)) return RKV_ERR_INVALID_ARG;
    ScreenArgs A;
    memset(&A, 0, sizeof A);
    for (int s = 0; s < S; ++s) {
        if (!outs[s]) return RKV_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(outs[s]) & 15u) return RKV_ERR_ALIGNMENT;
        A.outs[s] = outs[s];
    }
    A.rows = rows; A.cols = cols; A.n = rows * cols; A.S = S;
    if (!workspace) return RKV_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return RKV_ERR_ALIGNMENT;
    int sms = 0;
    const int rc = current_num_sms(&sms);
    if (rc != RKV_OK) return rc;
    if (workspace_bytes < sizeof(ScreenHeader) + (size_t)sms * kScreenBlocksPerSm * sizeof(ScreenPartial))
        return RKV_ERR_WORKSPACE;
    const int grid_max = sms * (dtype == RKV_BF16 ? kScreenBlocksPerSmB16 : kScreenBlocksPerSm);
    // no more blocks than there are strides of work
    const int vec = dtype == RKV_BF16 ? 8 : 4;
    const uint64_t units = (A.cols % vec) == 0 ? (A.n + vec - 1) / vec : A.n;
    uint64_t want = (units + kScreenThreads - 1) / kScreenThreads;
    if (want < 1) want = 1;
    const int grid = want < (uint64_t)grid_max ? (int)want : grid_max;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    ScreenHeader* header = reinterpret_cast<ScreenHeader*>(workspace);
    ScreenPartial* partials = reinterpret_cast<ScreenPartial*>(header + 1);
    if (dtype == RKV_BF16) screen_kernel<true><<<grid, kScreenThreads, 0, stream>>>(A, header, partials);
    else if (S <= 3 && (A.cols % 4) == 0) {
        // (four outputs, eight loads in flight, spill at three blocks per SM and measure no faster)
        if (S == 1) screen_few_kernel<1><<<grid, kScreenThreads, 0, stream>>>(A, header, partials);
        else if (S == 2) screen_few_kernel<2><<<grid, kScreenThreads, 0, stream>>>(A, header, partials);
        else screen_few_kernel<3><<<grid, kScreenThreads, 0, stream>>>(A, header, partials);
    } else screen_kernel<false><<<grid, kScreenThreads, 0, stream>>>(A, header, partials);
    screen_finalize_kernel<<<1, kScreenThreads, 0, stream>>>(A, header, partials, grid, range_lim, std_lim,
                                                            spread_lim, stats_out);
    if (cudaGetLastError() != cudaSuccess) return RKV_ERR_CUDA;
    return RKV_OK;
}

}  // extern "C"
