// Philox4x32-10 and the five distribution transforms, device side.
//
// Every floating-point step is an explicit round-to-nearest intrinsic
// (__fmul_rn, __fadd_rn, __fmaf_rn, __fdiv_rn, __fsqrt_rn): the compiler can
// neither contract a multiply-add nor swap in an approximate divide or square
// root, and subnormals are kept.  The generator has to reproduce, bit for bit,
// the values a scalar IEEE-754 binary32 implementation of the same formulas
// gives.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace rkv {

// Ten round keys of one Philox key (Weyl sequence), computed once per thread.
struct PhiloxKey {
    uint32_t k0[10];
    uint32_t k1[10];
};

__device__ __forceinline__ PhiloxKey philox_key(uint64_t seed) {
    PhiloxKey k;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = a;
        k.k1[r] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return k;
}

// One block: counter (c0..c3) -> four words (Salmon et al., SC'11).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKey& key) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;   // mul.wide.u32
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ key.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ key.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Block j of stream `stream_id`: counter = (j lo, j hi, stream lo, stream hi).
__device__ __forceinline__ uint4 philox_block(uint64_t j, uint64_t stream_id, const PhiloxKey& key) {
    return philox4x32_10((uint32_t)j, (uint32_t)(j >> 32), (uint32_t)stream_id,
                         (uint32_t)(stream_id >> 32), key);
}

// log(k24 * 2^-24), k24 in [1, 2^24]: mantissa folded into [sqrt(1/2), sqrt(2)],
// log m = 2 atanh((m-1)/(m+1)) by its odd series up to s^9.
__device__ __forceinline__ float log_unit(uint32_t k24) {
    const float u = __fmul_rn(__uint2float_rn(k24), 0x1p-24f);
    const uint32_t b = __float_as_uint(u);
    int e = (int)(b >> 23) - 127;
    float m = __uint_as_float((b & 0x007FFFFFu) | 0x3F800000u);
    if (m > 0x1.6a09e6p+0f) {
        m = __fmul_rn(m, 0.5f);
        e += 1;
    }
    const float s = __fdiv_rn(__fadd_rn(m, -1.0f), __fadd_rn(m, 1.0f));
    const float s2 = __fmul_rn(s, s);
    float p = 0x1.c71c72p-3f;
    p = __fmaf_rn(s2, p, 0x1.24924ap-2f);
    p = __fmaf_rn(s2, p, 0x1.99999ap-2f);
    p = __fmaf_rn(s2, p, 0x1.555556p-1f);
    p = __fmaf_rn(s2, p, 2.0f);
    const float logm = __fmul_rn(s, p);
    return __fmaf_rn(__int2float_rn(e), 0x1.62e430p-1f, logm);
}

// sin, cos of the turn fraction k24 * 2^-24: exact octant split, Taylor
// polynomials on [0, pi/4].
__device__ __forceinline__ void sincos_turn(uint32_t k24, float& sn, float& cs) {
    const uint32_t oct = (k24 >> 21) & 7u;
    uint32_t rem = k24 & 0x1FFFFFu;
    if (oct & 1u) rem = 0x200000u - rem;
    const float t = __fmul_rn(__uint2float_rn(rem), 0x1p-21f);
    const float th = __fmul_rn(t, 0x1.921fb6p-1f);
    const float x2 = __fmul_rn(th, th);

    float ps = 0x1.71de3ap-19f;
    ps = __fmaf_rn(x2, ps, -0x1.a01a02p-13f);
    ps = __fmaf_rn(x2, ps, 0x1.111112p-7f);
    ps = __fmaf_rn(x2, ps, -0x1.555556p-3f);
    const float sv = __fmaf_rn(__fmul_rn(th, x2), ps, th);

    float pc = -0x1.27e4fcp-22f;
    pc = __fmaf_rn(x2, pc, 0x1.a01a02p-16f);
    pc = __fmaf_rn(x2, pc, -0x1.6c16c2p-10f);
    pc = __fmaf_rn(x2, pc, 0x1.555556p-5f);
    pc = __fmaf_rn(x2, pc, -0.5f);
    const float cv = __fmaf_rn(x2, pc, 1.0f);

    const bool swap = ((oct + 1u) & 2u) != 0u;
    float s = swap ? cv : sv;
    float c = swap ? sv : cv;
    if (oct & 4u) s = -s;
    if ((oct + 2u) & 4u) c = -c;
    sn = s;
    cs = c;
}

__device__ __forceinline__ void box_muller(uint32_t w0, uint32_t w1, float& z_even, float& z_odd) {
    const float lg = log_unit((w0 >> 8) + 1u);
    const float rad = __fsqrt_rn(__fmul_rn(-2.0f, lg));
    float sn, cs;
    sincos_turn(w1 >> 8, sn, cs);
    z_even = __fmul_rn(rad, cs);
    z_odd = __fmul_rn(rad, sn);
}

__device__ __forceinline__ float uniform_pm1(uint32_t w) {
    return __fadd_rn(__fmul_rn(__uint2float_rn(w >> 8), 0x1p-23f), -1.0f);
}

__device__ __forceinline__ float student_t2(uint32_t w) {
    const float u = __fmul_rn(__uint2float_rn(2u * (w >> 9) + 1u), 0x1p-24f);
    const float a = __fadd_rn(__fmul_rn(2.0f, u), -1.0f);
    const float b = __fmul_rn(u, __fadd_rn(1.0f, -u));
    return __fdiv_rn(a, __fsqrt_rn(__fmul_rn(2.0f, b)));
}

// fp32 -> bf16 bits, round to nearest even (generated values are never NaN).
__device__ __forceinline__ uint32_t bf16_rne_bits(float x) {
    uint32_t b = __float_as_uint(x);
    b += 0x7FFFu + ((b >> 16) & 1u);
    return b >> 16;
}

// The four fp32 values of block j of the tensor (seed key, stream_id, dist).
template <int DIST>
__device__ __forceinline__ void gen_block(uint64_t j, uint64_t stream_id, const PhiloxKey& key,
                                          float v[4]) {
    const uint4 w = philox_block(j, stream_id, key);
    if (DIST == 1) {
        v[0] = uniform_pm1(w.x); v[1] = uniform_pm1(w.y);
        v[2] = uniform_pm1(w.z); v[3] = uniform_pm1(w.w);
    } else if (DIST == 2) {
        v[0] = student_t2(w.x); v[1] = student_t2(w.y);
        v[2] = student_t2(w.z); v[3] = student_t2(w.w);
    } else {
        box_muller(w.x, w.y, v[0], v[1]);
        box_muller(w.z, w.w, v[2], v[3]);
        if (DIST == 4) {
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = __fmul_rn(v[q], 0x1.388p+13f);
        }
        if (DIST == 3) {
            const uint4 m = philox_block(j, stream_id + 1u, key);
            if (m.x < 0xE6666666u) v[0] = 0.0f;
            if (m.y < 0xE6666666u) v[1] = 0.0f;
            if (m.z < 0xE6666666u) v[2] = 0.0f;
            if (m.w < 0xE6666666u) v[3] = 0.0f;
        }
    }
}

__device__ __forceinline__ void gen_block_dyn(int dist, uint64_t j, uint64_t stream_id,
                                              const PhiloxKey& key, float v[4]) {
    switch (dist) {
        case 0: gen_block<0>(j, stream_id, key, v); break;
        case 1: gen_block<1>(j, stream_id, key, v); break;
        case 2: gen_block<2>(j, stream_id, key, v); break;
        case 3: gen_block<3>(j, stream_id, key, v); break;
        default: gen_block<4>(j, stream_id, key, v); break;
    }
}

}  // namespace rkv
