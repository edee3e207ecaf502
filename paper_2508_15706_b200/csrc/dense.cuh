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

}  // namespace
