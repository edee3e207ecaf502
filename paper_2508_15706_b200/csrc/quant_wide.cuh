// The quantiser, packing and decoding at 1, 3 and 4 bits per value (the paper's quantisation ablation).
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"
#include "quantiser.cuh"
#include <cuda_bf16.h>

// ================================================================================================
// Sec. 4 describes the quantiser for any width: values centred by the tensor's mean, [-6 sigma, 6 sigma]
// in 2^bits uniform bins, every bin stores the centroid of the raw values that fell into it; the paper
// trains with 2 bits and ablates 1, 3 and 4.  The 2-bit path has kernels of its own (quantiser.cuh,
// pack.cuh, the fused apply kernel); the kernels here serve the other widths with the same
// definitions and the same summation order, plainly: they are not on the benchmark's path.
//   inner edges   c_j sigma, c_j = -6 + 12 j / 2^bits (exact in fp32), one fp32 product each,
//                 code = number of edges the centred value reaches (lower edge inclusive)
//   payload       per tensor max(16, 4 * 2^bits) bytes of table; records of ceil(12 k / 8) index bytes,
//                 ceil(bits k / 8) code bytes (code of slot s at bits [bits s, bits s + bits)), padded to 16
// ================================================================================================
namespace {

struct TStatQ {  // per (worker, tensor), general width
    float lut[16];
};

__host__ __device__ constexpr int record_stride_q(int k, int bits) {
    return (record_index_bytes(k) + (bits * k + 7) / 8 + 15) / 16 * 16;
}
__host__ __device__ constexpr int header_bytes_q(int bits) { return (4 << bits) < 16 ? 16 : (4 << bits); }

template <int BITS>
__device__ __forceinline__ int quant_code_q(float v, float mu, float sigma) {
    constexpr int NB = 1 << BITS;
    const float cen = __fsub_rn(v, mu);
    int c = 0;
#pragma unroll
    for (int j = 1; j < NB; ++j) c += cen >= __fmul_rn(-6.0f + 12.0f * (float)j / (float)NB, sigma) ? 1 : 0;
    return c;
}

// Per-bin sums and counts of one unit, slot order.  One thread per (worker, chunk).
template <int BITS>
__global__ void __launch_bounds__(128)
chunk_bins_q_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors, int k, int kp,
                    Workspace ws, double* __restrict__ pbin, unsigned* __restrict__ pcnt) {
    constexpr int NB = 1 << BITS;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks * n_workers) return;
    int r, g;
    split_unit(i, n_chunks, r, g);
    const int keff = min(k, chunks[g].len);
    const float* __restrict__ v = ws.val + i * kp;
    const TStat st = ws.tstat[(long long)r * n_tensors + chunks[g].tensor];
    double sb[NB];
    unsigned nb[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        sb[b] = 0.0;
        nb[b] = 0;
    }
    for_each_staged_own(v, keff, [&](float x) {
        const int c = quant_code_q<BITS>(x, st.mu, st.sigma);
#pragma unroll
        for (int b = 0; b < NB; ++b)  // only the value's own bin (adding +0 elsewhere could flip a -0 sum)
            if (c == b) {
                sb[b] += (double)x;
                ++nb[b];
            }
    });
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        pbin[i * NB + b] = sb[b];
        pcnt[i * NB + b] = nb[b];
    }
}

// One warp per (worker, tensor): per bin, the chunk partials are added in groups of 64 consecutive
// chunks (left to right inside the group, one lane per group, 32 groups at a time), then the group
// sums left to right: the order of tensor_reduce_kernel.  Writes the table and the payload header.
template <int BITS>
__global__ void __launch_bounds__(128)
tensor_table_q_kernel(const TensorInfo* __restrict__ tinfo, long long n_chunks, int n_workers, int n_tensors,
                      const double* __restrict__ pbin, const unsigned* __restrict__ pcnt, TStatQ* __restrict__ tq,
                      WorkerPtrs ptrs) {
    constexpr int NB = 1 << BITS;
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * 4 + wib;
    if (w >= (long long)n_workers * n_tensors) return;
    const int r = (int)(w / n_tensors), t = (int)(w - (long long)r * n_tensors);
    const TensorInfo ti = tinfo[t];
    const long long first = (long long)r * n_chunks + ti.first_chunk;
    const long long n_groups = (ti.n_chunks + kSumGroup - 1) / kSumGroup;
    float* hdr = reinterpret_cast<float*>(ptrs.payload[r] + (long long)header_bytes_q(BITS) * t);
    double acc[NB];              // all bins in one walk over the chunk partials (each bin keeps its own order)
    unsigned long long cn[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        acc[b] = 0.0;
        cn[b] = 0;
    }
    for (long long g0 = 0; g0 < n_groups; g0 += 32) {
        double gs[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) gs[b] = 0.0;
        const long long c0 = (g0 + lane) * kSumGroup;
        const int cnt = (int)max(0ll, min((long long)kSumGroup, ti.n_chunks - c0));
        for (int c = 0; c < cnt; ++c) {
            const double* pb = pbin + (first + c0 + c) * NB;
            const unsigned* pc = pcnt + (first + c0 + c) * NB;
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                gs[b] += pb[b];
                cn[b] += pc[b];
            }
        }
        const int ng = (int)min(32ll, n_groups - g0);
        for (int l = 0; l < ng; ++l) {
#pragma unroll
            for (int b = 0; b < NB; ++b) acc[b] += __shfl_sync(kFull, gs[b], l);
        }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        unsigned long long n = cn[b];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) n += __shfl_xor_sync(kFull, n, d);
        if (lane == 0) {
            const float v = n ? (float)(acc[b] / (double)n) : 0.0f;
            tq[(long long)r * n_tensors + t].lut[b] = v;
            hdr[b] = v;
        }
    }
    if (lane == 0)  // a 1-bit table is 8 bytes of a 16-byte header
        for (int b = NB; b < header_bytes_q(BITS) / 4; ++b) hdr[b] = 0.0f;
}

// Codes, record, and (FIX) e[index] = value - table[code].  One warp per (worker, chunk).
// HALF: the error buffers are bfloat16 arrays and the corrected value is rounded to nearest-even on the store.
template <int BITS, bool FIX, bool HALF = false>
__global__ void __launch_bounds__(128)
pack_q_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors, int k, int kp,
              Workspace ws, const TStatQ* __restrict__ tq, long long rec_base, WorkerPtrs ptrs) {
    __shared__ __align__(16) unsigned rec[4][(record_stride_q(kMaxK, 4) / 4) + 4];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long i = (long long)blockIdx.x * 4 + warp;
    if (i >= n_chunks * n_workers) return;
    int r, g;
    split_unit(i, n_chunks, r, g);
    const ChunkDesc cd = chunks[g];
    const int keff = min(k, cd.len);
    const int stride = record_stride_q(k, BITS), words = stride / 4;
    const int code_bit0 = record_index_bytes(k) * 8;
    const long long slot_base = ((long long)r * n_chunks + g) * kp;
    const TStat st = ws.tstat[(long long)r * n_tensors + cd.tensor];
    const TStatQ* lut = tq + (long long)r * n_tensors + cd.tensor;
    for (int w = lane; w < words; w += 32) rec[warp][w] = 0;
    __syncwarp();
    for (int s = lane; s < keff; s += 32) {
        const unsigned p = ws.idx[slot_base + s];
        const float v = ws.val[slot_base + s];
        const int c = quant_code_q<BITS>(v, st.mu, st.sigma);
        const int bit = 12 * s;
        atomicOr(&rec[warp][bit >> 5], p << (bit & 31));
        if ((bit & 31) > 20) atomicOr(&rec[warp][(bit >> 5) + 1], p >> (32 - (bit & 31)));
        const int cbit = code_bit0 + BITS * s;
        atomicOr(&rec[warp][cbit >> 5], (unsigned)c << (cbit & 31));
        if ((cbit & 31) + BITS > 32) atomicOr(&rec[warp][(cbit >> 5) + 1], (unsigned)c >> (32 - (cbit & 31)));
        if (FIX && p < (unsigned)cd.len) {
            const long long at = cd.base + chunk_elem_offset(cd.row_stride, (int)p);
            const float fix = __fsub_rn(v, lut->lut[c]);
            if (HALF) reinterpret_cast<__nv_bfloat16*>(ptrs.e[r])[at] = __float2bfloat16_rn(fix);
            else ptrs.e[r][at] = fix;
        }
    }
    __syncwarp();
    uint4* dst = reinterpret_cast<uint4*>(ptrs.payload[r] + rec_base + (long long)stride * g);
    const uint4* src = reinterpret_cast<const uint4*>(rec[warp]);
    for (int w = lane; w < stride / 16; w += 32) dst[w] = src[w];
}

// Decode + average + outer update from payloads of general width.  One CTA of 256 threads per chunk;
// the workers are taken one after the other (a CTA barrier in between), so every position receives
// its values in ascending worker order, as in decode_avg_apply_kernel.
// HALF: theta is a bfloat16 array, widened for the update and rounded to nearest-even on the store.
template <int BITS, bool HALF = false>
__global__ void __launch_bounds__(kThreads)
apply_q_kernel(const ChunkDesc* __restrict__ chunks, int n_workers, int k, float scale, PayloadPtrs pl, long long rec_base,
               float* __restrict__ theta_sync) {
    __shared__ float acc[kChunk];
    __shared__ float lut[16];
    const int tid = threadIdx.x;
    const ChunkDesc cd = chunks[blockIdx.x];
    const int keff = min(k, cd.len), stride = record_stride_q(k, BITS), code_bit0 = record_index_bytes(k) * 8;
    for (int p = tid; p < kChunk; p += kThreads) acc[p] = 0.0f;
    for (int r = 0; r < n_workers; ++r) {
        __syncthreads();
        const uint8_t* src = pl.p[r];
        if (!src) continue;  // uniform
        if (tid < (1 << BITS)) lut[tid] = reinterpret_cast<const float*>(src + (long long)header_bytes_q(BITS) * cd.tensor)[tid];
        __syncthreads();
        const uint8_t* rec = src + rec_base + (long long)stride * blockIdx.x;
        for (int s = tid; s < keff; s += kThreads) {
            const int bit = 12 * s, by = bit >> 3;
            const unsigned two = rec[by] | ((unsigned)rec[by + 1] << 8);
            const unsigned p = (two >> (bit & 7)) & 0xFFFu;
            const int cbit = code_bit0 + BITS * s, cby = cbit >> 3;
            unsigned ctwo = rec[cby];
            if ((cbit & 7) + BITS > 8) ctwo |= (unsigned)rec[cby + 1] << 8;  // (only a code that straddles two bytes reads the second)
            const unsigned c = (ctwo >> (cbit & 7)) & ((1u << BITS) - 1u);
            if (p < (unsigned)cd.len) acc[p] = __fadd_rn(acc[p], lut[c]);
        }
    }
    __syncthreads();
    if (HALF) {
        __nv_bfloat16* __restrict__ th = reinterpret_cast<__nv_bfloat16*>(theta_sync) + cd.base;
        for (int p = tid; p < cd.len; p += kThreads) {
            const float a = acc[p];
            const long long at = chunk_elem_offset(cd.row_stride, p);
            if (!(scale < 0.0f && __float_as_uint(a) == 0u)) th[at] = __float2bfloat16_rn(__fmaf_rn(scale, a, __bfloat162float(th[at])));
        }
        return;
    }
    float* __restrict__ th = theta_sync + cd.base;
    for (int p = tid; p < cd.len; p += kThreads) {
        const float a = acc[p];
        if (!(scale < 0.0f && __float_as_uint(a) == 0u))
            th[chunk_elem_offset(cd.row_stride, p)] = __fmaf_rn(scale, a, th[chunk_elem_offset(cd.row_stride, p)]);
    }
}

}  // namespace
