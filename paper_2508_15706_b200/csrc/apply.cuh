// Decode + average + outer update (optionally fused with the packing step).
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"
#include "quantiser.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// Decode + average + outer update.  One CTA per chunk.  Every (worker, slot) entry of the chunk is
// decoded by its own thread and ORs its worker's bit into a per-position mask in shared memory.
// The mask gives the entry its rank among the workers that selected the same position (bits
// below its own), and the entries are added into a 4096-float shared tile in rounds: rank 0
// first, then rank 1, ... with a barrier in between.  Every position thus receives its values in
// ascending worker order (reproducible bits), one writer per position and round, and the number
// of rounds is the largest number of workers that meet at one position (3 or 4 at R = 16).  Then
// every thread applies theta = fma(-alpha/D, sum, theta) to its own 16 positions.
// Workers are taken in batches of at most 32 (one mask bit each, 8 entries per thread).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned get12(const unsigned* rec, int s) {
    const int bit = 12 * s;
    return __funnelshift_r(rec[bit >> 5], rec[(bit >> 5) + 1], bit & 31) & 0xFFFu;
}
__device__ __forceinline__ unsigned get2(const unsigned* rec, int code_byte0, int s) {
    const int bit = code_byte0 * 8 + 2 * s;
    return (rec[bit >> 5] >> (bit & 31)) & 3u;
}

constexpr int kApplyEntries = 8;  // most entries per thread and batch

// FUSE 0: the entries come from the payload records (sl_aggregate_apply).  FUSE 1 / 2: the whole outer
// step is running and the records do not exist yet: the entries come from the staging arrays, get
// their codes here, and the kernel also writes the records and the error correction, i.e. it does
// what pack_fix_kernel<1> / <2> does, saving that kernel's pass and the re-read of the records.
struct FuseArgs {
    Workspace ws;
    long long n_chunks;
    int n_tensors, kp;
};

// SPL = slots per lane: ceil(k / 32) rounded up to 1, 2, 4 or 8; WPW = workers per warp and batch (1, 2 or
// 4, SPL * WPW <= 8): a thread holds SPL * WPW entries and a batch is 8 * WPW workers
template <int SPL, int WPW, int FUSE>
__global__ void __launch_bounds__(kThreads, 4)
decode_avg_apply_kernel(const ChunkDesc* __restrict__ chunks, int n_workers, int k, float scale,
                        PayloadPtrs pl, float* __restrict__ theta_sync, FuseArgs fa, WorkerPtrs ptrs) {
    extern __shared__ __align__(16) unsigned char dyn[];
    float* acc = reinterpret_cast<float*>(dyn);                            // 4096 sums
    unsigned* wmask = reinterpret_cast<unsigned*>(acc + kChunk);           // 4096 worker masks
    float* luts = reinterpret_cast<float*>(wmask + kChunk);                // 32 x 4
    float* mu_t3 = luts + 4 * 32;                                          // 32 x 2 (FUSE: mean, 3 sigma)
    unsigned* recs = reinterpret_cast<unsigned*>(mu_t3 + 2 * 32);          // batch x (stride + 16) bytes
    const int stride = record_stride(k), rwords = stride / 4 + 4;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kEnt = SPL * WPW;  // entries per thread and batch
    static_assert(kEnt <= kApplyEntries && WPW <= 4, "entry budget");
    constexpr int batch = 8 * WPW;
    // FUSE: the staged (index, value) pairs of this thread's entries in the first batch.  They need
    // nothing from the chunk table (slots up to k exist for every chunk; those beyond the chunk's
    // own count are ignored later), so they start before anything else.
    unsigned pre_p[kEnt];
    float pre_v[kEnt];
#pragma unroll
    for (int e = 0; e < kEnt; ++e) {
        pre_p[e] = 0u;
        pre_v[e] = 0.f;
    }
    if (FUSE) {
#pragma unroll
        for (int wi = 0; wi < WPW; ++wi) {
            const int rb = warp + 8 * wi;
            const long long slot_base = ((long long)rb * fa.n_chunks + blockIdx.x) * fa.kp;
#pragma unroll
            for (int si = 0; si < SPL; ++si) {
                const int sl = lane + 32 * si;
                if (rb < n_workers && sl < k) {
                    pre_p[wi * SPL + si] = fa.ws.idx[slot_base + sl];
                    pre_v[wi * SPL + si] = fa.ws.val[slot_base + sl];
                }
            }
        }
    }
    const ChunkDesc cd = chunks[blockIdx.x];
    const int keff = min(k, cd.len);
    const int code_byte0 = record_index_bytes(k);
    float* __restrict__ th = theta_sync + cd.base;

    // theta loads first (in flight while the records are decoded);
    // vector i of this thread (in-chunk indices 1024 i + 4 tid ..+3) sits at th_vec + i * vec_step
    float4 a[4];
    const int rs = cd.row_stride ? cd.row_stride : kTile;
    float* __restrict__ th_vec = th + (long long)(tid >> 4) * rs + (4 * tid & 63);
    const long long vec_step = 16ll * rs;
    const bool full = cd.len == kChunk;
    if (full) {
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4*>(th_vec + i * vec_step);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<float4*>(acc + 1024 * i + 4 * tid) = make_float4(0.f, 0.f, 0.f, 0.f);

    // entry e of a thread: worker warp + 8 (e / SPL), slot lane + 32 (e % SPL)
    const int vec_per_rec = stride / 16;

    for (int r0 = 0; r0 < n_workers; r0 += batch) {
        const int nb = min(batch, n_workers - r0);
        // clear the masks, stage this batch's records and tables (the last barrier of the
        // previous batch's rounds has released both)
#pragma unroll
        for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(wmask + 1024 * i + 4 * tid) = make_uint4(0u, 0u, 0u, 0u);
        if (FUSE == 0) {
            for (int v = tid; v < nb * vec_per_rec; v += kThreads) {
                const int rb = v / vec_per_rec, w = v - rb * vec_per_rec;
                const uint8_t* src = pl.p[r0 + rb];
                if (src) {
                    const uint4 x = __ldg(reinterpret_cast<const uint4*>(src + cd.rec_off) + w);
                    *reinterpret_cast<uint4*>(recs + rb * rwords + 4 * w) = x;
                }
            }
            if (tid < nb) {
                const uint8_t* src = pl.p[r0 + tid];
                if (src) *reinterpret_cast<float4*>(luts + 4 * tid) = __ldg(reinterpret_cast<const float4*>(src + 16ll * cd.tensor));
                recs[tid * rwords + stride / 4] = 0;  // word read past the index block by get12
            }
        } else {
            // staged pairs of the later batches (the first batch's are already on their way)
#pragma unroll
            for (int wi = 0; wi < WPW; ++wi) {
                const int rb = warp + 8 * wi;
                const long long slot_base = ((long long)(r0 + rb) * fa.n_chunks + blockIdx.x) * fa.kp;
#pragma unroll
                for (int si = 0; si < SPL; ++si) {
                    const int sl = lane + 32 * si;
                    if (r0 > 0 && rb < nb && sl < keff) {
                        pre_p[wi * SPL + si] = fa.ws.idx[slot_base + sl];
                        pre_v[wi * SPL + si] = fa.ws.val[slot_base + sl];
                    }
                }
            }
            for (int w = tid; w < nb * rwords; w += kThreads) recs[w] = 0;  // the records are assembled here
            if (tid < nb) {
                const TStat st = fa.ws.tstat[(long long)(r0 + tid) * fa.n_tensors + cd.tensor];
                *reinterpret_cast<float4*>(luts + 4 * tid) = make_float4(st.lut[0], st.lut[1], st.lut[2], st.lut[3]);
                mu_t3[2 * tid] = st.mu;
                mu_t3[2 * tid + 1] = st.t3;
            }
        }
        __syncthreads();

        unsigned ent_p[kEnt];  // position | worker bit number << 12; 0xFFFFFFFF = no entry
        float ent_v[kEnt];
#pragma unroll
        for (int e = 0; e < kEnt; ++e) {
            ent_p[e] = 0xFFFFFFFFu;
            ent_v[e] = 0.f;
        }
#pragma unroll
        for (int wi = 0; wi < WPW; ++wi) {
            const int rb = warp + 8 * wi;
            if (rb < nb && pl.p[r0 + rb]) {  // uniform over the warp
                unsigned* rec = recs + rb * rwords;
                const long long slot_base = FUSE ? ((long long)(r0 + rb) * fa.n_chunks + blockIdx.x) * fa.kp : 0;
#pragma unroll
                for (int si = 0; si < SPL; ++si) {
                    const int sl = lane + 32 * si;
                    if (sl < keff) {
                        unsigned p, code;
                        if (FUSE == 0) {
                            p = get12(rec, sl);
                            code = get2(rec, code_byte0, sl);
                        } else {
                            p = pre_p[wi * SPL + si];
                            const float v = pre_v[wi * SPL + si];
                            code = (unsigned)quant_code(v, mu_t3[2 * rb], mu_t3[2 * rb + 1]);
                            const int bit = 12 * sl;
                            atomicOr(&rec[bit >> 5], p << (bit & 31));
                            if ((bit & 31) > 20) atomicOr(&rec[(bit >> 5) + 1], p >> (32 - (bit & 31)));
                            const int cbit = code_byte0 * 8 + 2 * sl;
                            atomicOr(&rec[cbit >> 5], code << (cbit & 31));
                            const float fixed = __fsub_rn(v, luts[4 * rb + code]);
                            if (FUSE == 1 && p < (unsigned)cd.len)
                                ptrs.e[r0 + rb][cd.base + chunk_elem_offset(cd.row_stride, (int)p)] = fixed;
                            if (FUSE == 2) fa.ws.val[slot_base + sl] = fixed;
                        }
                        if (p < (unsigned)cd.len) {
                            ent_v[wi * SPL + si] = luts[4 * rb + code];
                            ent_p[wi * SPL + si] = p | ((unsigned)rb << 12);
                            atomicOr(&wmask[p], 1u << rb);
                        }
                    }
                }
            }
        }
        __syncthreads();
        if (FUSE) {  // the records are complete: out they go
            for (int v = tid; v < nb * vec_per_rec; v += kThreads) {
                const int rb = v / vec_per_rec, w = v - rb * vec_per_rec;
                reinterpret_cast<uint4*>(ptrs.payload[r0 + rb] + cd.rec_off)[w] =
                    *reinterpret_cast<const uint4*>(recs + rb * rwords + 4 * w);
            }
        }
        // rank of every entry among the workers at its position; round 0
        int my_max = 0;
#pragma unroll
        for (int e = 0; e < kEnt; ++e) {
            if (ent_p[e] != 0xFFFFFFFFu) {
                const unsigned p = ent_p[e] & 0xFFFu, rb = ent_p[e] >> 12;
                const unsigned wm = wmask[p];
                const int rank = __popc(wm & ((1u << rb) - 1u));
                my_max = max(my_max, __popc(wm));
                if (rank == 0) {
                    acc[p] = __fadd_rn(acc[p], ent_v[e]);
                    ent_p[e] = 0xFFFFFFFFu;
                } else {
                    ent_p[e] = p | ((unsigned)rank << 12);  // from here on: position | rank << 12
                }
            }
        }
        for (int t = 1; __syncthreads_or(my_max > t); ++t) {
#pragma unroll
            for (int e = 0; e < kEnt; ++e) {
                if (ent_p[e] != 0xFFFFFFFFu && (int)(ent_p[e] >> 12) == t) {
                    const unsigned p = ent_p[e] & 0xFFFu;
                    acc[p] = __fadd_rn(acc[p], ent_v[e]);
                }
            }
        }
    }

    if (full) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 sv = *reinterpret_cast<const float4*>(acc + 1024 * i + 4 * tid);
            float4 o;
            o.x = __fmaf_rn(scale, sv.x, a[i].x);
            o.y = __fmaf_rn(scale, sv.y, a[i].y);
            o.z = __fmaf_rn(scale, sv.z, a[i].z);
            o.w = __fmaf_rn(scale, sv.w, a[i].w);
            *reinterpret_cast<float4*>(th_vec + i * vec_step) = o;
        }
    } else {
        for (int p = tid; p < cd.len; p += kThreads) th[p] = __fmaf_rn(scale, acc[p], th[p]);
    }
}

}  // namespace
