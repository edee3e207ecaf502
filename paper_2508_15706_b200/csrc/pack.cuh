// Packing (12-bit indices, 2-bit codes), error-feedback subtract, flush of deferred values.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"
#include "quantiser.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// Pack + error-feedback subtract.  One warp per (worker, chunk): codes from (mu, 3 sigma), 12-bit
// indices and 2-bit codes OR-ed into a shared-memory record, record written as 16-byte vectors,
// e[index] = value - table[code] at the selected positions (Eq. 2 line 2).
// ------------------------------------------------------------------------------------------------
// MODE 0: records only (error feedback frozen).  MODE 1: e[index] = value - table[code].
// MODE 2: the corrected value replaces the staged value instead (deferred subtraction).
// HALF: the error buffers are bfloat16 arrays (MODE 1 rounds the corrected value to nearest-even on the store).
template <int MODE, bool HALF = false>
__global__ void __launch_bounds__(128)
pack_fix_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors,
                int k, int kp, Workspace ws, WorkerPtrs ptrs) {
    __shared__ __align__(16) unsigned rec[4][(record_stride(kFastMaxK) / 4) + 4];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long i = (long long)blockIdx.x * 4 + warp;
    if (i >= n_chunks * n_workers) return;
    int r, g;  // worker-major: neighbouring warps handle neighbouring blocks of one buffer
    split_unit(i, n_chunks, r, g);
    const ChunkDesc cd = chunks[g];
    const int keff = min(k, cd.len);
    const int stride = record_stride(k), words = stride / 4;
    const int code_word0 = record_index_bytes(k);  // byte offset of the code block
    const long long slot_base = ((long long)r * n_chunks + g) * kp;
    const TStat st = ws.tstat[(long long)r * n_tensors + cd.tensor];

    for (int w = lane; w < words; w += 32) rec[warp][w] = 0;
    __syncwarp();
    for (int s = lane; s < keff; s += 32) {
        const unsigned p = ws.idx[slot_base + s];
        const float v = ws.val[slot_base + s];
        const int c = quant_code(v, st.mu, st.t3);
        const int bit = 12 * s;
        atomicOr(&rec[warp][bit >> 5], p << (bit & 31));
        if ((bit & 31) > 20) atomicOr(&rec[warp][(bit >> 5) + 1], p >> (32 - (bit & 31)));
        const int cbit = code_word0 * 8 + 2 * s;
        atomicOr(&rec[warp][cbit >> 5], (unsigned)c << (cbit & 31));
        if (MODE == 1 && p < (unsigned)cd.len) {
            const long long at = cd.base + chunk_elem_offset(cd.row_stride, (int)p);
            const float fix = __fsub_rn(v, st.lut[c]);
            if (HALF) reinterpret_cast<bf16_bits*>(ptrs.e[r])[at] = (bf16_bits)bf16_narrow(fix);
            else ptrs.e[r][at] = fix;
        }
        if (MODE == 2) ws.val[slot_base + s] = __fsub_rn(v, st.lut[c]);
    }
    __syncwarp();
    uint4* dst = reinterpret_cast<uint4*>(ptrs.payload[r] + cd.rec_off);
    const uint4* src = reinterpret_cast<const uint4*>(rec[warp]);
    for (int w = lane; w < stride / 16; w += 32) dst[w] = src[w];
}

// Writes the corrected values waiting in the staging arrays into the error buffers (deferred
// subtraction made good).  One warp per (worker, chunk).  ZERO: writes +0 at the staged positions
// instead (Top-k without a quantiser sends the selected values exactly, so what stays behind there,
// u - Top-k(u), is zero: Alg. 2-4 of the appendix on DiLoCo variants).
template <bool ZERO, bool HALF = false>
__global__ void __launch_bounds__(128)
ef_flush_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int k, int kp, Workspace ws,
                WorkerPtrs ptrs) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long i = (long long)blockIdx.x * 4 + warp;
    if (i >= n_chunks * n_workers) return;
    int r, g;
    split_unit(i, n_chunks, r, g);
    if (!ptrs.e[r]) return;  // this worker was left out of the flush
    const ChunkDesc cd = chunks[g];
    const int keff = min(k, cd.len);
    const long long slot_base = ((long long)r * n_chunks + g) * kp;
    for (int s = lane; s < keff; s += 32) {
        const unsigned p = ws.idx[slot_base + s];
        if (p < (unsigned)cd.len) {
            const long long at = cd.base + chunk_elem_offset(cd.row_stride, (int)p);
            const float v = ZERO ? 0.0f : ws.val[slot_base + s];
            if (HALF) reinterpret_cast<bf16_bits*>(ptrs.e[r])[at] = (bf16_bits)bf16_narrow(v);
            else ptrs.e[r][at] = v;
        }
    }
}

}  // namespace
