// bfloat16 storage of theta, theta_r and e: the selection kernel and the store helpers of that mode.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"
#include "ef_select.cuh"

// ================================================================================================
// The paper trains and communicates in a setting it describes only at the level of the algorithm
// (Alg. 1, Eq. 2) and says nothing about the storage type of the outer-step state.  This mode halves
// that state: theta, theta_r and e are bfloat16 arrays.  The arithmetic is the fp32 arithmetic of the
// fp32 mode on the widened values -- Delta = theta - theta_r, u = fma(beta, e, Delta), selection and
// quantiser on the unrounded u -- and only what is stored is rounded, once, to nearest-even:
// e = bf16(u) where nothing was selected, bf16(u - table[code]) where something was,
// theta = bf16(fma(-alpha / D, sum, theta)).
//
// The selection kernel keeps the unrounded u of a unit in shared memory (one 16 KB block per warp), so
// the candidate read-back of select_unit works on exact values although the error buffer now holds
// rounded ones.  Plain 64-bit loads (four bfloat16), no tile copies: a chunk is 8 KB per array here.
// ================================================================================================
namespace {

constexpr int kHalfSelWarps = 12;  // what shared memory (16 KB of u per warp) and the register file allow
constexpr int kHalfSelThreads = 32 * kHalfSelWarps;
struct HalfSelSmem {
    __align__(16) float u[kHalfSelWarps][kChunk];
    __align__(16) unsigned bitmap[kHalfSelWarps][128];
    uint16_t cand[kHalfSelWarps][kCandCap];
};

// One warp per (chunk, worker) unit, units taken chunk-major so that the workers of a chunk follow one
// another (theta's block is re-read from L2).  The WorkerPtrs / theta pointers address bfloat16 arrays.
// PENDING: the corrected values of the previous step still wait in the staging arrays (deferred subtraction):
// they are rounded into the error buffer at their positions before the unit's e is read.
template <bool EF, int WIDE, bool PENDING = false>
__global__ void __launch_bounds__(kHalfSelThreads, 1)
ef_select_bf16_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int k, int kp, float beta,
                      const bf16_bits* __restrict__ theta_sync, WorkerPtrs ptrs, Workspace ws) {
    extern __shared__ __align__(16) unsigned char dyn_half[];
    HalfSelSmem& sm = *reinterpret_cast<HalfSelSmem*>(dyn_half);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* const scratch = sm.u[warp];
    unsigned* const bitmap = sm.bitmap[warp];
    const long long n_units = n_chunks * n_workers, step = (long long)gridDim.x * kHalfSelWarps;
    for (long long n = (long long)blockIdx.x * kHalfSelWarps + warp; n < n_units; n += step) {
        const long long g = n / n_workers;
        const int r = (int)(n - g * n_workers);
        const ChunkGeo cd = load_geo(chunks + g);
        const int keff = min(k, cd.len);
        const bf16_bits* __restrict__ tsp = theta_sync + cd.base;
        const bf16_bits* __restrict__ tlp = reinterpret_cast<const bf16_bits*>(ptrs.theta_local[r]) + cd.base;
        bf16_bits* __restrict__ er = EF ? reinterpret_cast<bf16_bits*>(ptrs.e[r]) + cd.base : nullptr;
        *reinterpret_cast<uint4*>(&bitmap[4 * lane]) = make_uint4(0u, 0u, 0u, 0u);
        const long long slot_base = ((long long)r * n_chunks + g) * kp;
        if (PENDING && EF) {  // (the lanes' plain loads below read what is patched here)
            for (int j = lane; j < keff; j += 32) {
                const unsigned p = ws.idx[slot_base + j];
                if (p < (unsigned)cd.len) er[chunk_elem_offset(cd.row_stride, (int)p)] = (bf16_bits)bf16_narrow(ws.val[slot_base + j]);
            }
            __syncwarp();
        }
        float u[128];
        if (cd.len == kChunk) {
            // a full chunk: the loads of 8 vectors per array are issued before any of them is used (the stores
            // into e would otherwise order every later load of e behind them)
#pragma unroll
            for (int i0 = 0; i0 < 32; i0 += 8) {
                uint2 wa[8], wl[8], we[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const long long off = chunk_elem_offset(cd.row_stride, 128 * (i0 + j) + 4 * lane);
                    wa[j] = __ldg(reinterpret_cast<const uint2*>(tsp + off));
                    wl[j] = __ldcs(reinterpret_cast<const uint2*>(tlp + off));
                    if (EF) we[j] = __ldcs(reinterpret_cast<const uint2*>(er + off));
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int i = i0 + j, p0 = 128 * i + 4 * lane;
                    float4 x;
                    x.x = __fsub_rn(bf16_widen(wa[j].x & 0xFFFFu), bf16_widen(wl[j].x & 0xFFFFu));
                    x.y = __fsub_rn(bf16_widen(wa[j].x >> 16), bf16_widen(wl[j].x >> 16));
                    x.z = __fsub_rn(bf16_widen(wa[j].y & 0xFFFFu), bf16_widen(wl[j].y & 0xFFFFu));
                    x.w = __fsub_rn(bf16_widen(wa[j].y >> 16), bf16_widen(wl[j].y >> 16));
                    if (EF) {
                        x.x = __fmaf_rn(beta, bf16_widen(we[j].x & 0xFFFFu), x.x);
                        x.y = __fmaf_rn(beta, bf16_widen(we[j].x >> 16), x.y);
                        x.z = __fmaf_rn(beta, bf16_widen(we[j].y & 0xFFFFu), x.z);
                        x.w = __fmaf_rn(beta, bf16_widen(we[j].y >> 16), x.w);
                        bf16_store4(er + chunk_elem_offset(cd.row_stride, p0), x);
                    }
                    *reinterpret_cast<float4*>(&scratch[p0]) = x;
                    u[4 * i + 0] = x.x;
                    u[4 * i + 1] = x.y;
                    u[4 * i + 2] = x.z;
                    u[4 * i + 3] = x.w;
                }
            }
        } else
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int p0 = 128 * i + 4 * lane;
            const long long off = chunk_elem_offset(cd.row_stride, p0);
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (p0 + 4 <= cd.len) {
                const float4 a = bf16_load4(tsp + off), l = bf16_load4(tlp + off);
                x.x = __fsub_rn(a.x, l.x);
                x.y = __fsub_rn(a.y, l.y);
                x.z = __fsub_rn(a.z, l.z);
                x.w = __fsub_rn(a.w, l.w);
                if (EF) {
                    const float4 ev = bf16_load4(er + off);
                    x.x = __fmaf_rn(beta, ev.x, x.x);
                    x.y = __fmaf_rn(beta, ev.y, x.y);
                    x.z = __fmaf_rn(beta, ev.z, x.z);
                    x.w = __fmaf_rn(beta, ev.w, x.w);
                    bf16_store4(er + off, x);
                }
            } else if (p0 < cd.len) {  // the vector that holds the end of a short chunk
                float t[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (p0 + j < cd.len) {
                        t[j] = __fsub_rn(bf16_widen(tsp[off + j]), bf16_widen(tlp[off + j]));
                        if (EF) {
                            t[j] = __fmaf_rn(beta, bf16_widen(er[off + j]), t[j]);
                            er[off + j] = (bf16_bits)bf16_narrow(t[j]);
                        }
                    }
                }
                x = make_float4(t[0], t[1], t[2], t[3]);
            }
            *reinterpret_cast<float4*>(&scratch[p0]) = x;
            u[4 * i + 0] = x.x;
            u[4 * i + 1] = x.y;
            u[4 * i + 2] = x.z;
            u[4 * i + 3] = x.w;
        }
        __syncwarp();
        USource src;
        src.ptr = reinterpret_cast<const unsigned*>(scratch);
        src.rs = kTile;
        select_unit<false, WIDE>(u, src, cd.len, keff, bitmap, sm.cand[warp], ws.idx + slot_base, ws.val + slot_base);
        __syncwarp();  // the block, the map and the list are free again
    }
}

}  // namespace
