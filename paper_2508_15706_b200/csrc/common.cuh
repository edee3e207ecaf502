// Constants, the chunk table and workspace layouts, small helpers shared by all kernels.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include <cuda_bf16.h>

namespace {

constexpr int kChunk = 4096;
constexpr int kTile = 64;
constexpr int kThreads = 256;          // threads per CTA of the chunk kernels
constexpr int kPerThread = kChunk / kThreads;  // 16 elements = 4 x float4
constexpr int kMaxR = 64;
constexpr int kMaxK = 2048;      // half a chunk: the densest setting of the paper's sweeps
constexpr int kFastMaxK = 256;   // largest k of the fused 2-bit kernels, the waiting lists and the wire codec
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kProfSlots = 9;     // kernels of one outer step
constexpr int kProfMaxSeq = 256;  // recorded sequences kept between two reads

thread_local char g_cuda_err[256] = "";

// One chunk of one tensor: where its elements live in the flat buffers.
struct ChunkDesc {
    long long base;    // element offset of in-chunk index 0
    int row_stride;    // elements between block rows (2-D blocks), 0 for flat runs
    int len;           // elements in the chunk (4096, or the short tail of a flat tensor)
    int tensor;        // owning tensor
    int chunk_in_tensor;
    long long rec_off; // byte offset of this chunk's record inside a payload
};
static_assert(sizeof(ChunkDesc) == 32, "ChunkDesc layout");

struct TensorInfo {
    long long first_chunk;
    long long n_chunks;
    long long n_slots;  // sum over chunks of min(k, len)
};

struct TStat {  // per (worker, tensor)
    float mu, sigma, t3;
    float lut[4];
    float pad;
};
static_assert(sizeof(TStat) == 32, "TStat layout");

struct WorkerPtrs {
    const float* theta_local[kMaxR];
    float* e[kMaxR];
    uint8_t* payload[kMaxR];
};

struct PayloadPtrs {
    const uint8_t* p[kMaxR];
};

struct Workspace {  // device arrays, dimensioned [workers][chunks]...
    float* val;          // [W][G][kp]
    uint16_t* idx;       // [W][G][kp]
    double* psum;        // [W][G]
    double* pbin;        // [W][G][4]
    unsigned* pcnt;      // [W][G][4]
    TStat* tstat;        // [W][T]
};

__host__ __device__ constexpr int record_index_bytes(int k) { return (12 * k + 7) / 8; }
__host__ __device__ constexpr int record_stride(int k) {
    return (record_index_bytes(k) + (2 * k + 7) / 8 + 15) / 16 * 16;
}

// bfloat16 storage (the upper half of an fp32): widening is exact, narrowing rounds to nearest-even.
typedef unsigned short bf16_bits;
__device__ __forceinline__ float bf16_widen(unsigned b) { return __uint_as_float(b << 16); }
__device__ __forceinline__ unsigned bf16_narrow(float x) { return (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ float4 bf16_widen4(const uint2& w) {
    return make_float4(bf16_widen(w.x & 0xFFFFu), bf16_widen(w.x >> 16), bf16_widen(w.y & 0xFFFFu), bf16_widen(w.y >> 16));
}
__device__ __forceinline__ uint2 bf16_narrow4(const float4& x) {
    uint2 w;
    w.x = bf16_narrow(x.x) | (bf16_narrow(x.y) << 16);
    w.y = bf16_narrow(x.z) | (bf16_narrow(x.w) << 16);
    return w;
}
__device__ __forceinline__ float4 bf16_load4(const bf16_bits* p) { return bf16_widen4(*reinterpret_cast<const uint2*>(p)); }
__device__ __forceinline__ void bf16_store4(bf16_bits* p, const float4& x) { *reinterpret_cast<uint2*>(p) = bf16_narrow4(x); }

// Element offset (relative to ChunkDesc::base) of in-chunk index p.
__device__ __forceinline__ long long chunk_elem_offset(int row_stride, int p) {
    return row_stride ? (long long)(p >> 6) * row_stride + (p & 63) : (long long)p;
}

}  // namespace
