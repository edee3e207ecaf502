// Quantiser statistics: ordered fp64 sums per chunk and per (worker, tensor).
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// Quantiser statistics (Sec. 4).  The summation order is part of the definition of the payload
// bits: fp64, in three levels, each left to right: the slots of a chunk, the chunks of a group of 64
// consecutive chunks of the tensor, the groups.
// ------------------------------------------------------------------------------------------------

// (worker, chunk) of work item i; chunks x workers < 2^31 (checked on the host)
__device__ __forceinline__ void split_unit(long long i, long long n_chunks, int& r, int& g) {
    const unsigned ui = (unsigned)i, nc = (unsigned)n_chunks;
    r = (int)(ui / nc);
    g = (int)(ui - (unsigned)r * nc);
}

// The per-unit passes below give one lane the ordered fp64 chain of one (worker, chunk) unit, but a
// lane reading its own 256-byte run makes every load instruction of the warp touch 32 different
// lines.  Instead a warp takes 32 consecutive units -- contiguous in the staging array -- loads them
// together with fully coalesced 128-bit loads, 64 slots at a time, into a shared tile (row stride 65:
// conflict-free both ways) and every lane then walks its own row in slot order.
constexpr int kStatWarps = 4;      // per CTA
constexpr int kStatSlots = 64;     // slots per round
struct StatTile {
    float v[32][kStatSlots + 1];
};

// f(x) is called for the staged values of unit i0 + lane in slot order (keff of them; none when the
// unit does not exist).  Warp-collective.
template <typename F>
__device__ __forceinline__ void for_each_staged(const float* __restrict__ val, long long i0, long long n_units, int kp,
                                                int keff, StatTile& tile, F f) {
    const int lane = threadIdx.x & 31;
    for (int sb = 0; sb < kp; sb += kStatSlots) {
#pragma unroll 4
        for (int j = 0; j < 16; ++j) {
            const int row = 2 * j + (lane >> 4), c = 4 * (lane & 15);
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i0 + row < n_units && sb + c < kp)
                x = __ldcs(reinterpret_cast<const float4*>(val + (i0 + row) * kp + sb + c));
            tile.v[row][c + 0] = x.x;
            tile.v[row][c + 1] = x.y;
            tile.v[row][c + 2] = x.z;
            tile.v[row][c + 3] = x.w;
        }
        __syncwarp();
        const int n = min(kStatSlots, keff - sb);
        for (int s0 = 0; s0 < n; ++s0) f(tile.v[lane][s0]);
        __syncwarp();
    }
}

// mode 0: sum of values; mode 1: sum of squared fp32-centred values.  One lane per (worker, chunk).
template <int MODE>
__global__ void __launch_bounds__(32 * kStatWarps)
chunk_sum_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors,
                 int k, int kp, Workspace ws) {
    __shared__ StatTile tiles[kStatWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long total = n_chunks * n_workers;
    const long long i0 = ((long long)blockIdx.x * kStatWarps + warp) * 32, i = i0 + lane;
    if (i0 >= total) return;
    int r = 0, g = 0, keff = 0;
    float mu = 0.0f;
    if (i < total) {
        split_unit(i, n_chunks, r, g);
        keff = min(k, chunks[g].len);
        if (MODE == 1) mu = ws.tstat[(long long)r * n_tensors + chunks[g].tensor].mu;
    }
    double acc = 0.0;
    for_each_staged(ws.val, i0, total, kp, keff, tiles[warp], [&](float x) {
        if (MODE == 0) {
            acc += (double)x;
        } else {
            const double d = (double)__fsub_rn(x, mu);
            acc += d * d;  // d*d is exact in fp64, so fusing or not gives the same sum
        }
    });
    if (i < total) ws.psum[i] = acc;
}

// Per-bin sums and counts of one chunk.  codes: (cen >= -t) + (cen >= 0) + (cen >= t).
__device__ __forceinline__ int quant_code(float v, float mu, float t3) {
    const float cen = __fsub_rn(v, mu);
    return (cen >= -t3 ? 1 : 0) + (cen >= 0.0f ? 1 : 0) + (cen >= t3 ? 1 : 0);
}

// Visits the keff staged values of one unit in slot order, read by the thread itself: four 128-bit
// loads in flight at a time.  (The per-bin pass does more arithmetic per value and runs best at full
// occupancy, which the shared tiles of the cooperative form would halve.)
template <typename F>
__device__ __forceinline__ void for_each_staged_own(const float* __restrict__ v, int keff, F f) {
    int s0 = 0;
    for (; s0 + 16 <= keff; s0 += 16) {
        float4 x[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) x[q] = __ldcs(reinterpret_cast<const float4*>(v + s0) + q);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            f(x[q].x);
            f(x[q].y);
            f(x[q].z);
            f(x[q].w);
        }
    }
    for (; s0 < keff; ++s0) f(v[s0]);
}

__global__ void __launch_bounds__(128)
chunk_bins_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors,
                  int k, int kp, Workspace ws) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks * n_workers) return;
    int r, g;
    split_unit(i, n_chunks, r, g);
    const int keff = min(k, chunks[g].len);
    const float* __restrict__ v = ws.val + i * kp;
    const TStat st = ws.tstat[(long long)r * n_tensors + chunks[g].tensor];
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    unsigned n0 = 0, n1 = 0, n2 = 0, n3 = 0;
    for_each_staged_own(v, keff, [&](float x) {
        const int c = quant_code(x, st.mu, st.t3);
        const double d = (double)x;
        // add only to the value's own bin (adding +0 elsewhere could flip a -0 sum); nearly all
        // selected values sit in the two inner bins, so the branches diverge two ways at most
        if (c == 1) { s1 += d; ++n1; }
        else if (c == 2) { s2 += d; ++n2; }
        else if (c == 0) { s0 += d; ++n0; }
        else { s3 += d; ++n3; }
    });
    double2* pb = reinterpret_cast<double2*>(ws.pbin + i * 4);
    pb[0] = make_double2(s0, s1);
    pb[1] = make_double2(s2, s3);
    *reinterpret_cast<uint4*>(ws.pcnt + i * 4) = make_uint4(n0, n1, n2, n3);
}

// One CTA of four warps per (worker, tensor): the chunk partials are added group by group (64 consecutive
// chunks per group, left to right inside the group: one thread per group, 128 groups at a time, group sums
// parked in shared memory), then the group sums are added left to right by the first warp.
// STAGE 0: psum -> mu.  STAGE 1: psum -> sigma, 3 sigma.  STAGE 2: pbin/pcnt -> table (+ payload header).
constexpr int kSumGroup = 64;

template <int STAGE>
__global__ void __launch_bounds__(128)
tensor_reduce_kernel(const TensorInfo* __restrict__ tinfo, long long n_chunks, int n_workers, int n_tensors,
                     Workspace ws, WorkerPtrs ptrs) {
    constexpr int NV = STAGE < 2 ? 1 : 4;  // running sums
    __shared__ double gsum[128][NV];
    __shared__ unsigned long long cnt_s[4][4];
    const int tid = threadIdx.x, wib = tid >> 5, lane = tid & 31;
    const long long w = blockIdx.x;
    if (w >= (long long)n_workers * n_tensors) return;  // (whole CTA)
    const int r = (int)(w / n_tensors), t = (int)(w - (long long)r * n_tensors);
    const TensorInfo ti = tinfo[t];
    const long long first = (long long)r * n_chunks + ti.first_chunk;
    TStat* st = ws.tstat + (long long)r * n_tensors + t;
    const double n = (double)ti.n_slots;
    const long long n_groups = (ti.n_chunks + kSumGroup - 1) / kSumGroup;

    double acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = 0.0;
    unsigned long long cn[4] = {0, 0, 0, 0};
    for (long long g0 = 0; g0 < n_groups; g0 += 128) {
        // this thread's group
        double gs[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) gs[v] = 0.0;
        const long long c0 = (g0 + tid) * kSumGroup;
        const int cnt = (int)max(0ll, min((long long)kSumGroup, ti.n_chunks - c0));
        if (STAGE < 2) {
            const double* __restrict__ src = ws.psum + first + c0;
            int c = 0;
            for (; c + 16 <= cnt; c += 16) {  // sixteen loads in flight, additions in chunk order
                double x[16];
#pragma unroll
                for (int q = 0; q < 16; ++q) x[q] = src[c + q];
#pragma unroll
                for (int q = 0; q < 16; ++q) gs[0] += x[q];
            }
            for (; c < cnt; ++c) gs[0] += src[c];
        } else {
            const double2* __restrict__ src = reinterpret_cast<const double2*>(ws.pbin + (first + c0) * 4);
            const uint4* __restrict__ csrc = reinterpret_cast<const uint4*>(ws.pcnt + (first + c0) * 4);
            int c = 0;
            for (; c + 8 <= cnt; c += 8) {  // loads of eight chunks in flight, additions in chunk order
                double2 lo[8], hi[8];
                uint4 pc[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    lo[q] = src[2 * (c + q)];
                    hi[q] = src[2 * (c + q) + 1];
                    pc[q] = csrc[c + q];
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    gs[0] += lo[q].x; gs[1 % NV] += lo[q].y; gs[2 % NV] += hi[q].x; gs[3 % NV] += hi[q].y;
                    cn[0] += pc[q].x; cn[1] += pc[q].y; cn[2] += pc[q].z; cn[3] += pc[q].w;
                }
            }
            for (; c < cnt; ++c) {
                const double2 lo = src[2 * c], hi = src[2 * c + 1];
                gs[0] += lo.x; gs[1 % NV] += lo.y; gs[2 % NV] += hi.x; gs[3 % NV] += hi.y;
                const uint4 pc = csrc[c];
                cn[0] += pc.x; cn[1] += pc.y; cn[2] += pc.z; cn[3] += pc.w;
            }
        }
#pragma unroll
        for (int v = 0; v < NV; ++v) gsum[tid][v] = gs[v];
        __syncthreads();
        // the group sums of these 128 groups, in group order (every lane of the first warp runs the same chain)
        if (wib == 0) {
            const int ng = (int)min(128ll, n_groups - g0);
            for (int l = 0; l < ng; ++l) {
#pragma unroll
                for (int v = 0; v < NV; ++v) acc[v] += gsum[l][v];
            }
        }
        __syncthreads();
    }
    if (STAGE == 2) {  // the counts: integers, any order
#pragma unroll
        for (int bb = 0; bb < 4; ++bb) {
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) cn[bb] += __shfl_xor_sync(kFull, cn[bb], d);
            if (lane == 0) cnt_s[wib][bb] = cn[bb];
        }
        __syncthreads();
#pragma unroll
        for (int bb = 0; bb < 4; ++bb) cn[bb] = cnt_s[0][bb] + cnt_s[1][bb] + cnt_s[2][bb] + cnt_s[3][bb];
    }
    if (wib != 0) return;

    if (STAGE < 2) {
        if (lane == 0) {
            if (STAGE == 0) {
                st->mu = (float)(acc[0] / n);
            } else {
                const float sigma = (float)sqrt(acc[0] / n);
                st->sigma = sigma;
                st->t3 = __fmul_rn(3.0f, sigma);
            }
        }
    } else {
        if (lane == 0) {
            float lut[4];
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) lut[bb] = cn[bb] ? (float)(acc[bb % NV] / (double)cn[bb]) : 0.0f;
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) st->lut[bb] = lut[bb];
            st->pad = 0.0f;
            float4* hdr = reinterpret_cast<float4*>(ptrs.payload[r] + 16ll * t);
            *hdr = make_float4(lut[0], lut[1], lut[2], lut[3]);
        }
    }
}

}  // namespace
