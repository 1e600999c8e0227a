// rkv_gen_inputs: counter-based multi-distribution input generator (sm_100a).
//
// One thread produces whole Philox blocks (four consecutive elements each), two a
// step so that their dependent chains overlap: for bf16 the two blocks of one 16-byte
// store, for fp32 the blocks of two 16-byte stores a grid stride apart.
// Consecutive threads write consecutive 16-byte units, so a warp stores 512
// contiguous bytes.  The kernel is ALU-bound (about 50 integer + fp32
// instructions per element against 4 bytes written).
#include "rkv_internal.h"
#include "rkv_philox.cuh"

namespace rkv {

namespace {

template <int DIST, bool BF16>
__global__ void __launch_bounds__(256)
gen_kernel(uint64_t seed, uint64_t stream_id, uint64_t first_block, uint64_t n, void* __restrict__ out) {
    const PhiloxKey key = philox_key(seed);
    constexpr int kUnitElems = BF16 ? 8 : 4;
    const uint64_t n_units = (n + kUnitElems - 1) / kUnitElems;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t u = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; u < n_units; u += stride) {
        const uint64_t e0 = u * kUnitElems;
        const bool full = e0 + kUnitElems <= n;
        if (!BF16) {
            // two Philox blocks a step where the thread has two left (their dependent chains overlap)
            const uint64_t u2 = u + stride;
            const bool pair = u2 < n_units && (u2 + 1) * 4 <= n;
            float v[4], v2[4];
            gen_block<DIST>(first_block + u, stream_id, key, v);
            gen_block<DIST>(first_block + (pair ? u2 : u), stream_id, key, v2);    // (unconditional: one basic block)
            float* o = reinterpret_cast<float*>(out) + e0;
            if (full) {
                *reinterpret_cast<float4*>(o) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (e0 + q < n) o[q] = v[q];
            }
            if (pair) {
                *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + u2 * 4) = make_float4(v2[0], v2[1], v2[2], v2[3]);
                u += stride;
            }
        } else {
            float v[8];
            gen_block<DIST>(first_block + 2 * u, stream_id, key, v);
            gen_block<DIST>(first_block + 2 * u + 1, stream_id, key, v + 4);
            uint32_t h[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) h[q] = bf16_rne_bits(v[q]);
            uint16_t* o = reinterpret_cast<uint16_t*>(out) + e0;
            if (full) {
                *reinterpret_cast<uint4*>(o) = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16),
                                                          h[4] | (h[5] << 16), h[6] | (h[7] << 16));
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (e0 + q < n) o[q] = (uint16_t)h[q];
            }
        }
    }
}

template <int DIST>
int launch_dist(uint64_t seed, uint64_t stream_id, uint64_t first_block, uint64_t n, int dtype,
                void* out, int grid, cudaStream_t stream) {
    if (dtype == RKV_BF16)
        gen_kernel<DIST, true><<<grid, 256, 0, stream>>>(seed, stream_id, first_block, n, out);
    else
        gen_kernel<DIST, false><<<grid, 256, 0, stream>>>(seed, stream_id, first_block, n, out);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

}  // namespace

int launch_gen(uint64_t seed, uint64_t stream_id, int dist, uint64_t n, uint64_t first_elem,
               int dtype, void* out, int num_sms, cudaStream_t stream) {
    const int unit = dtype == RKV_BF16 ? 8 : 4;
    const uint64_t n_units = (n + unit - 1) / unit;
    uint64_t want = (n_units + 255) / 256;
    const uint64_t cap = (uint64_t)num_sms * 8;
    const int grid = (int)(want < cap ? (want ? want : 1) : cap);
    const uint64_t fb = first_elem >> 2;
    switch (dist) {
        case RKV_DIST_NORMAL: return launch_dist<0>(seed, stream_id, fb, n, dtype, out, grid, stream);
        case RKV_DIST_UNIFORM_PM1: return launch_dist<1>(seed, stream_id, fb, n, dtype, out, grid, stream);
        case RKV_DIST_STUDENT_T2: return launch_dist<2>(seed, stream_id, fb, n, dtype, out, grid, stream);
        case RKV_DIST_SPARSE90: return launch_dist<3>(seed, stream_id, fb, n, dtype, out, grid, stream);
        case RKV_DIST_NORMAL_1E4: return launch_dist<4>(seed, stream_id, fb, n, dtype, out, grid, stream);
        default: return RKV_ERR_INVALID_ARG;
    }
}

}  // namespace rkv
