// Payload validation and small utility kernels.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// Payload validation: never traps, reports through a device status word.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
validate_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_tensors, int k,
                const uint8_t* __restrict__ payload, int* __restrict__ status) {
    const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    bool bad = false;
    if (g < n_tensors) {
        const float* lut = reinterpret_cast<const float*>(payload + 16 * g);
        for (int b = 0; b < 4; ++b) bad |= !isfinite(lut[b]);
    }
    if (g < n_chunks) {
        const ChunkDesc cd = chunks[g];
        const int keff = min(k, cd.len), stride = record_stride(k), ib = record_index_bytes(k);
        const uint8_t* rec = payload + cd.rec_off;
        int prev = -1;
        for (int s = 0; s < k; ++s) {
            const int bit = 12 * s, by = bit >> 3;
            const unsigned two = rec[by] | ((unsigned)rec[by + 1] << 8);
            const int p = (two >> (bit & 7)) & 0xFFF;
            const int cbit = 2 * s;
            const int c = (rec[ib + (cbit >> 3)] >> (cbit & 7)) & 3;
            if (s < keff) {
                bad |= p >= cd.len || p <= prev;
                prev = p;
            } else {
                bad |= p != 0 || c != 0;
            }
        }
        // padding: bits after the last index, bits after the last code
        if ((12 * k) & 7) bad |= (rec[ib - 1] >> ((12 * k) & 7)) != 0;
        const int code_bits = 2 * k, cb_full = code_bits >> 3;
        if (code_bits & 7) bad |= (rec[ib + cb_full] >> (code_bits & 7)) != 0;
        for (int by = ib + ((code_bits + 7) >> 3); by < stride; ++by) bad |= rec[by] != 0;
    }
    if (bad) atomicExch(status, (int)SL_ERR_BAD_PAYLOAD);
}

__global__ void set_status_kernel(int* status, int v) { *status = v; }

__global__ void copy_stats_kernel(const TStat* __restrict__ src, int n, float* __restrict__ dst) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n * 8) dst[i] = reinterpret_cast<const float*>(src)[i];
}

}  // namespace
