// Dense baseline: DiLoCo's outer step (Eq. 1).
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"

// ================================================================================================
// Dense baseline: DiLoCo's outer step (Eq. 1), for comparison on the same buffers.
//   Dbar = (1/R) sum_r (theta - theta_r);  m = beta m + Dbar;  theta = theta - alpha (Dbar + beta m)
// One CTA per chunk of the table (so exactly the table's elements are touched), 16 elements per
// thread, all R + 2 streams of a thread's vector in flight together.  fp32: differences and their
// sum in ascending r, one division by R, two fused multiply-adds.
// ================================================================================================
namespace {

struct LocalPtrs {
    const float* p[kMaxR];
};

__device__ __forceinline__ float diloco_elem(float th, float acc, float inv_r_num, float beta, float alpha, float& m) {
    const float dbar = __fdiv_rn(acc, inv_r_num);
    m = __fmaf_rn(beta, m, dbar);
    return __fmaf_rn(-alpha, __fmaf_rn(beta, m, dbar), th);
}

__global__ void __launch_bounds__(kThreads)
diloco_step_kernel(const ChunkDesc* __restrict__ chunks, int n_workers, float beta, float alpha,
                   float* __restrict__ theta, LocalPtrs loc, float* __restrict__ mom) {
    const ChunkDesc cd = chunks[blockIdx.x];
    const int tid = threadIdx.x;
    const float fr = (float)n_workers;
    if (cd.len == kChunk) {
        const int rs = cd.row_stride ? cd.row_stride : kTile;
        const long long off0 = cd.base + (long long)(tid >> 4) * rs + (4 * tid & 63), step = 16ll * rs;
#pragma unroll 1
        for (int i = 0; i < 4; ++i) {
            const long long off = off0 + i * step;
            const float4 th = *reinterpret_cast<const float4*>(theta + off);
            float4 m = *reinterpret_cast<const float4*>(mom + off);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
            for (int r = 0; r < n_workers; ++r) {
                const float4 l = __ldcs(reinterpret_cast<const float4*>(loc.p[r] + off));
                acc.x = __fadd_rn(acc.x, __fsub_rn(th.x, l.x));
                acc.y = __fadd_rn(acc.y, __fsub_rn(th.y, l.y));
                acc.z = __fadd_rn(acc.z, __fsub_rn(th.z, l.z));
                acc.w = __fadd_rn(acc.w, __fsub_rn(th.w, l.w));
            }
            float4 o;
            o.x = diloco_elem(th.x, acc.x, fr, beta, alpha, m.x);
            o.y = diloco_elem(th.y, acc.y, fr, beta, alpha, m.y);
            o.z = diloco_elem(th.z, acc.z, fr, beta, alpha, m.z);
            o.w = diloco_elem(th.w, acc.w, fr, beta, alpha, m.w);
            *reinterpret_cast<float4*>(theta + off) = o;
            *reinterpret_cast<float4*>(mom + off) = m;
        }
    } else {
        for (int p = tid; p < cd.len; p += kThreads) {
            const long long off = cd.base + p;
            const float th = theta[off];
            float acc = 0.f;
            for (int r = 0; r < n_workers; ++r) acc = __fadd_rn(acc, __fsub_rn(th, loc.p[r][off]));
            float m = mom[off];
            theta[off] = diloco_elem(th, acc, fr, beta, alpha, m);
            mom[off] = m;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Local outer momentum (Sec. 3.2; Alg. 2 and the first lines of Alg. 4 in the appendix on DiLoCo
// variants).  Per worker r and element, all fp32, single-rounded, in the algorithm's order:
//     d = theta - theta_r;   m_r = fma(mu, m_r, d);   nd_r = fma(mu, m_r, d)      (local Nesterov direction)
// STEP:  theta = fma(-alpha, (sum_r nd_r) / R, theta), the sum in ascending r (DiLoCo-LOM).
// !STEP: theta stays; nd_r replaces theta_r in its buffer, to be compressed next (DiLoCo-LOM + Top-k).
// One CTA per chunk of the table, 16 elements per thread.
// ------------------------------------------------------------------------------------------------
struct MomentumPtrs {
    float* p[kMaxR];
};
struct MutableLocalPtrs {
    float* p[kMaxR];
};

template <bool STEP>
__global__ void __launch_bounds__(kThreads)
lom_kernel(const ChunkDesc* __restrict__ chunks, int n_workers, float mu, float alpha, float* __restrict__ theta,
           MutableLocalPtrs loc, MomentumPtrs mom) {
    const ChunkDesc cd = chunks[blockIdx.x];
    const int tid = threadIdx.x;
    const float fr = (float)n_workers;
    if (cd.len == kChunk) {
        const int rs = cd.row_stride ? cd.row_stride : kTile;
        const long long off0 = cd.base + (long long)(tid >> 4) * rs + (4 * tid & 63), step = 16ll * rs;
#pragma unroll 1
        for (int i = 0; i < 4; ++i) {
            const long long off = off0 + i * step;
            const float4 th = *reinterpret_cast<const float4*>(theta + off);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
            for (int r = 0; r < n_workers; ++r) {
                const float4 l = *reinterpret_cast<const float4*>(loc.p[r] + off);
                float4 m = *reinterpret_cast<const float4*>(mom.p[r] + off);
                float4 d, nd;
                d.x = __fsub_rn(th.x, l.x); d.y = __fsub_rn(th.y, l.y); d.z = __fsub_rn(th.z, l.z); d.w = __fsub_rn(th.w, l.w);
                m.x = __fmaf_rn(mu, m.x, d.x); m.y = __fmaf_rn(mu, m.y, d.y); m.z = __fmaf_rn(mu, m.z, d.z); m.w = __fmaf_rn(mu, m.w, d.w);
                nd.x = __fmaf_rn(mu, m.x, d.x); nd.y = __fmaf_rn(mu, m.y, d.y); nd.z = __fmaf_rn(mu, m.z, d.z); nd.w = __fmaf_rn(mu, m.w, d.w);
                *reinterpret_cast<float4*>(mom.p[r] + off) = m;
                if (STEP) {
                    acc.x = __fadd_rn(acc.x, nd.x); acc.y = __fadd_rn(acc.y, nd.y);
                    acc.z = __fadd_rn(acc.z, nd.z); acc.w = __fadd_rn(acc.w, nd.w);
                } else {
                    *reinterpret_cast<float4*>(loc.p[r] + off) = nd;
                }
            }
            if (STEP) {
                float4 o;
                o.x = __fmaf_rn(-alpha, __fdiv_rn(acc.x, fr), th.x);
                o.y = __fmaf_rn(-alpha, __fdiv_rn(acc.y, fr), th.y);
                o.z = __fmaf_rn(-alpha, __fdiv_rn(acc.z, fr), th.z);
                o.w = __fmaf_rn(-alpha, __fdiv_rn(acc.w, fr), th.w);
                *reinterpret_cast<float4*>(theta + off) = o;
            }
        }
    } else {
        for (int p = tid; p < cd.len; p += kThreads) {
            const long long off = cd.base + p;
            const float th = theta[off];
            float acc = 0.f;
            for (int r = 0; r < n_workers; ++r) {
                const float d = __fsub_rn(th, loc.p[r][off]);
                const float m = __fmaf_rn(mu, mom.p[r][off], d);
                const float nd = __fmaf_rn(mu, m, d);
                mom.p[r][off] = m;
                if (STEP) acc = __fadd_rn(acc, nd);
                else loc.p[r][off] = nd;
            }
            if (STEP) theta[off] = __fmaf_rn(-alpha, __fdiv_rn(acc, fr), th);
        }
    }
}

}  // namespace
