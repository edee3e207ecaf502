// Payload validation and small utility kernels.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// Payload validation: never traps, reports through a device status word.
// ------------------------------------------------------------------------------------------------
// `bits` = bits per code (1..4), `hdr` = bytes of a tensor's table in the payload, records of `stride` bytes from
// `rec_base` on (the layout of every quantiser width: 12-bit indices, then the codes).
__global__ void __launch_bounds__(128)
validate_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_tensors, int k, int bits, int hdr,
                long long rec_base, int stride, const uint8_t* __restrict__ payload, int* __restrict__ status) {
    const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    bool bad = false;
    if (g < n_tensors) {
        const float* lut = reinterpret_cast<const float*>(payload + (long long)hdr * g);
        for (int b = 0; b < hdr / 4; ++b)  // the table's entries are finite, what follows them in the header is zero
            bad |= b < (1 << bits) ? !isfinite(lut[b]) : __float_as_uint(lut[b]) != 0u;
    }
    if (g < n_chunks) {
        const ChunkDesc cd = chunks[g];
        const int keff = min(k, cd.len), ib = record_index_bytes(k);
        const uint8_t* rec = payload + rec_base + (long long)stride * g;
        int prev = -1;
        for (int s = 0; s < k; ++s) {
            const int bit = 12 * s, by = bit >> 3;
            const unsigned two = rec[by] | ((unsigned)rec[by + 1] << 8);
            const int p = (two >> (bit & 7)) & 0xFFF;
            const int cbit = bits * s, cby = ib + (cbit >> 3);
            unsigned ctwo = rec[cby];
            if ((cbit & 7) + bits > 8) ctwo |= (unsigned)rec[cby + 1] << 8;  // (only a code that straddles two bytes)
            const int c = (ctwo >> (cbit & 7)) & ((1 << bits) - 1);
            if (s < keff) {
                bad |= p >= cd.len || p <= prev;
                prev = p;
            } else {
                bad |= p != 0 || c != 0;
            }
        }
        // padding: bits after the last index, bits after the last code, the bytes up to the stride
        if ((12 * k) & 7) bad |= (rec[ib - 1] >> ((12 * k) & 7)) != 0;
        const int code_bits = bits * k, cb_full = code_bits >> 3;
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
