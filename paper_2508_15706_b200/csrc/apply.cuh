// Decode + average + outer update (optionally fused with the packing step, or with the decoding of coded payloads).
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"
#include "quantiser.cuh"
#include "index_codec.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// Decode + average + outer update (Eq. 2 lines 3-4).  Persistent CTAs of four warps, up to six per SM;
// a CTA takes whole chunks (b, b + grid, ...) and owns a 4096-float sum tile in shared memory.  For a
// chunk it
//   1. takes the chunk's theta (8 x 128 bits per thread, in registers until step 4) from the CTA's staging
//      block, where asynchronous copies issued one chunk earlier have put it, and starts the copies of
//      the next chunk's theta: a thread copies exactly the vectors it will own, so it waits for its own
//      copies only and no barrier is involved; the copies of chunk g + grid fly while chunk g is decoded,
//   2. decodes the workers in batches of 16, warp w the workers 4 w .. 4 w + 3 of the batch: a lane holds
//      the slot pairs (2 m, 2 m + 1), m = lane + 32 j, of a worker and turns them into (index, table value),
//   3. adds them into the tile in ascending worker order: the warps take turns (a CTA barrier between
//      two warps, a warp barrier between two workers of a warp).  A worker's indices are distinct, so
//      every position receives its values in worker order (reproducible bits) without atomics,
//   4. applies theta = fma(-alpha/D, sum, theta) to its 32 positions, clears the tile on the way and
//      stores the vectors that received anything.
//
// FUSE 3 / 4 serve the paper's Top-k baselines, which have no quantiser (appendix on DiLoCo variants):
// the staged values are added as they are and nothing is packed; FUSE 3 applies theta = fma(-alpha/R,
// sum, theta) (Alg. 4), FUSE 4 the Nesterov outer step on the average, m = fma(mu, m, avg), theta =
// fma(-alpha, fma(mu, m, avg), theta), for every element (Alg. 3: the momentum moves everywhere).
//
// FUSE 0: the entries come from the payload records (sl_aggregate_apply).  FUSE 1 / 2: the whole outer
// step is running and the records do not exist yet: the entries come from the staging arrays, get
// their codes here, and the kernel also writes the records and the error correction (e[index] =
// value - table[code] for FUSE 1; the same value back into the staging array for FUSE 2, the deferred
// form), i.e. it does what pack_fix_kernel<1> / <2> does, saving that kernel's pass.
//
// FUSE 5: the payloads are in the entropy-coded wire form (index_codec.cuh) and are decoded here instead of
// being expanded to records first.  A chunk's position in a worker's index stream is known only after
// the chunks before it in its group of 16 (one directory entry per group), so a CTA takes whole groups
// and walks their chunks in order.  The CTA has two extra warps for this: decoder thread r keeps worker r's
// read position and decodes the chunk's gaps through a 64-bit register window over the stream into one of
// two shared index lists, one chunk ahead of the four warps that run the update proper, which read the
// list and the code blocks.  The two groups meet through two counters in shared memory (chunks decoded,
// chunks whose list has been read) with bounded polls -- SL_ERR_TIMEOUT and an orderly exit of both groups if
// one ever runs out -- and each group keeps to a named barrier of its own size.  Reads of a
// stream are confined to the size its buffer is said to have; a stream that runs out reads as zeros
// and is recorded as SL_ERR_BAD_PAYLOAD.
//
// A slot pair is 24 bits of the index block (bytes 3 m .. 3 m + 2) and one nibble of the code block, so
// a lane assembles its part of a record with byte stores into the CTA's record buffer and the finished
// records leave as 16-byte vectors.
// ------------------------------------------------------------------------------------------------
struct FuseArgs {
    Workspace ws;
    long long n_chunks;
    int n_tensors, kp;
    // FUSE 4 only: the global outer momentum and its coefficient, alpha and the divisor
    float* momentum;
    float mu, alpha, divisor;
    // FUSE 5 only: layout of a coded payload, bits of index stream each worker's buffer holds
    unsigned long long dir_off, stream_off;
    unsigned long long stream_bits[kMaxR];
    int* status;
};

constexpr int kApplyWarps = 4;
constexpr int kApplyThreads = 32 * kApplyWarps;
constexpr int kApplyCtasPerSm = 6;   // what the shared memory of a CTA (tile, records, staging block) lets an SM hold
constexpr int kApplyBatch = 16;                  // workers decoded between two rounds of ordered additions
constexpr int kApplyPerWarp = kApplyBatch / kApplyWarps;
constexpr int kApplyDecoders = 64;                  // FUSE 5: two more warps, one thread per worker, decode one chunk ahead
constexpr int kApplyTile = kChunk + kApplyThreads;  // the sum tile + one dump slot per thread for entries that do not count

__host__ __device__ constexpr size_t apply_smem_bytes(int k) {
    return (size_t)kApplyTile * sizeof(float) + (size_t)kApplyBatch * (record_stride(k) + 32) + (size_t)kChunk * sizeof(float);
}

// 16-byte asynchronous copy global -> shared (L2 only), and the wait for all of this thread's copies
__device__ __forceinline__ void async_copy16(void* smem_dst, const void* gmem_src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void async_copy8(void* smem_dst, const void* gmem_src) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void async_copy_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

// PPL = slot pairs per lane: ceil(k / 64) rounded up to 1, 2 or 4
// HALF (FUSE 0-2): theta and the error buffers are bfloat16 arrays; they are widened on the way in and what is
// stored is rounded once to nearest-even, the arithmetic in between is the fp32 arithmetic of the fp32 form.
template <int PPL, int FUSE, bool HALF = false>
__global__ void __launch_bounds__(FUSE == 5 ? kApplyThreads + kApplyDecoders : kApplyThreads, kApplyCtasPerSm)
decode_avg_apply_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int k, float scale,
                        PayloadPtrs pl, float* __restrict__ theta_sync, FuseArgs fa, WorkerPtrs ptrs) {
    extern __shared__ __align__(16) unsigned char dyn[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int stride = record_stride(k), ib = record_index_bytes(k);
    float* acc = reinterpret_cast<float*>(dyn);
    uint8_t* recs = dyn + (size_t)kApplyTile * sizeof(float);
    // per worker of the batch: mean, 3 sigma, 0, present | the four table entries
    float4* tabs = reinterpret_cast<float4*>(recs + (size_t)kApplyBatch * stride);
    float4* stage = tabs + 2 * kApplyBatch;  // theta of the chunk to come: vector i of thread t at [128 i + t]
    constexpr int WB = kApplyPerWarp;
    constexpr bool PACK = FUSE == 1 || FUSE == 2;  // quantise, write records and the error correction
    constexpr bool RAW = FUSE == 3 || FUSE == 4;   // staged values travel unquantised
    constexpr bool STAGED = FUSE >= 1 && FUSE <= 4;  // the entries come from the staging arrays
    constexpr bool CODED = FUSE == 5;              // the entries come from entropy-coded payloads
    const unsigned dump = (unsigned)(kChunk + tid);  // where an entry that does not count adds its 0
    // per-worker strides of the staging arrays, in index pairs / value pairs (kp is a multiple of 8)
    const long long wstride = STAGED ? fa.n_chunks * (long long)fa.kp / 2 : 0;
    // CODED: two lists of kp decoded indices per worker, then the two counters and the abort flag
    uint16_t* sidx_all = reinterpret_cast<uint16_t*>(stage + kChunk / 4);
    const size_t sidx_len = CODED ? (size_t)n_workers * fa.kp : 0;
    // [0] chunks decoded, [1] chunks whose lists have been read, [2] abort (set by whoever's wait ran out),
    // [3] / [4] what the decoders / the update warps decided at their last meeting point (written by one thread
    // before the group's barrier and read by all after it, so that a whole group stops at the same place)
    int* sync_words = reinterpret_cast<int*>(sidx_all + 2 * ((sidx_len + 7) / 8 * 8));
    const int cb = (2 * k + 7) / 8;  // bytes of a chunk's code block in a coded payload
    // the 128 threads of the update meet at a barrier of their own when decoder warps share the CTA
    auto cta_sync = [&]() {
        if (CODED) asm volatile("bar.sync 1, 128;" ::: "memory");
        else __syncthreads();
    };
    // the CTA's walk: chunk after chunk inside a group of kIxcGroup when CODED, else every gridDim-th chunk
    auto next_of = [&](long long g) -> long long {
        if (!CODED) return g + gridDim.x;
        if ((g + 1) % kIxcGroup != 0 && g + 1 < n_chunks) return g + 1;
        return (g / kIxcGroup + gridDim.x) * kIxcGroup;
    };
    const long long g_first = CODED ? (long long)blockIdx.x * kIxcGroup : (long long)blockIdx.x;

    if (CODED) {
        if (tid == 0) sync_words[0] = sync_words[1] = sync_words[2] = sync_words[3] = sync_words[4] = 0;
        __syncthreads();  // (all 192 threads, once: the counters start at zero for both groups)
    }
    if (CODED && tid >= kApplyThreads) {
        // ------------------------------------------------------------ decoder warps: one chunk ahead
        const int d = tid - kApplyThreads;  // worker
        const bool mine = d < n_workers && pl.p[d] != nullptr;
        const unsigned long long sbits = mine ? fa.stream_bits[d] : 0ull;
        unsigned long long my_pos = 0;  // worker d's read position in its index stream
        bool my_bad = false;
        int i = 0;
        for (long long g = g_first; g < n_chunks; g = next_of(g), ++i) {
            if (d == 0) {  // the list that chunk i goes into was last used by chunk i - 2
                bool ok = false;
                for (unsigned it = 0; it < (1u << 22); ++it) {
                    int done;
                    asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(done) : "r"((unsigned)__cvta_generic_to_shared(&sync_words[1])) : "memory");
                    if (done >= i - 1) {
                        ok = true;
                        break;
                    }
                    if (*reinterpret_cast<volatile int*>(&sync_words[2])) break;
                    __nanosleep(64);
                }
                if (!ok) {
                    if (!*reinterpret_cast<volatile int*>(&sync_words[2])) atomicExch(fa.status, (int)SL_ERR_TIMEOUT);
                    *reinterpret_cast<volatile int*>(&sync_words[2]) = 1;
                    *reinterpret_cast<volatile int*>(&sync_words[3]) = 1;
                }
            }
            asm volatile("bar.sync 2, 64;" ::: "memory");
            if (*reinterpret_cast<volatile int*>(&sync_words[3])) break;  // (written by one thread before the barrier)
            if (mine) {
                const ChunkDesc dcd = chunks[g];
                const int dk = min(k, dcd.len);
                if (g % kIxcGroup == 0) {  // a new group: its directory entry
                    my_pos = reinterpret_cast<const unsigned*>(pl.p[d] + fa.dir_off)[g / kIxcGroup];
                    if (my_pos > sbits) {
                        my_bad = true;
                        my_pos = sbits;
                    }
                }
                IxcReader rd;
                ixc_reader_open(rd, reinterpret_cast<const unsigned*>(pl.p[d] + fa.stream_off), sbits, my_pos);
                uint16_t* out = sidx_all + (size_t)(i & 1) * ((sidx_len + 7) / 8 * 8) + (size_t)d * fa.kp;
                my_pos += ixc_decode_chunk(rd, ixc_code(dcd.len, dk), dk, [&](int s, unsigned idx) { out[s] = (uint16_t)idx; });
                if (my_pos > sbits) {
                    my_bad = true;
                    my_pos = sbits;
                }
            }
            asm volatile("bar.sync 2, 64;" ::: "memory");  // every worker's list of chunk i is written
            if (d == 0)
                asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"((unsigned)__cvta_generic_to_shared(&sync_words[0])), "r"(i + 1) : "memory");
        }
        if (my_bad) atomicExch(fa.status, (int)SL_ERR_BAD_PAYLOAD);
        return;
    }

    for (int i = tid; i < kApplyTile / 4; i += kApplyThreads) reinterpret_cast<float4*>(acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    cta_sync();

    // thread t owns in-chunk indices 512 i + 4 t + j: block row 8 i + t / 16, column 4 (t % 16)
    bf16_bits* const theta_h = reinterpret_cast<bf16_bits*>(theta_sync);  // HALF: the same array seen as bfloat16
    uint2* const stage_h = reinterpret_cast<uint2*>(stage);                 // HALF: four bfloat16 per vector
    auto prefetch_theta = [&](const ChunkDesc& d) {
        const int prs = d.row_stride ? d.row_stride : kTile;
        if (HALF) {
            const bf16_bits* src = theta_h + d.base + (long long)(tid >> 4) * prs + 4 * (tid & 15);
#pragma unroll
            for (int i = 0; i < 8; ++i) async_copy8(&stage_h[128 * i + tid], src + (long long)i * 8 * prs);
        } else {
            const float* src = theta_sync + d.base + (long long)(tid >> 4) * prs + 4 * (tid & 15);
#pragma unroll
            for (int i = 0; i < 8; ++i) async_copy16(&stage[128 * i + tid], src + (long long)i * 8 * prs);
        }
    };
    ChunkDesc cd_next;
    if (g_first < n_chunks) {
        cd_next = chunks[g_first];
        if (cd_next.len == kChunk) prefetch_theta(cd_next);
    }

    int seq = 0;  // position of the chunk in this CTA's walk
    for (long long g = g_first; g < n_chunks; g = next_of(g), ++seq) {
        const ChunkDesc cd = cd_next;
        const int keff = min(k, cd.len);
        const bool full = cd.len == kChunk;
        const int rs = cd.row_stride ? cd.row_stride : kTile;
        float* __restrict__ th = theta_sync + cd.base;
        float* __restrict__ th_vec = th + (long long)(tid >> 4) * rs + 4 * (tid & 15);
        const long long vec_step = 8ll * rs;
        float4 a[8];
        async_copy_wait_all();  // (this thread's copies; nothing is outstanding after a short chunk)
        if (full) {
#pragma unroll
            for (int i = 0; i < 8; ++i) a[i] = HALF ? bf16_widen4(stage_h[128 * i + tid]) : stage[128 * i + tid];
        }
        if (next_of(g) < n_chunks) {  // the block is free again (this thread's part of it): the next chunk's theta
            cd_next = chunks[next_of(g)];
            if (cd_next.len == kChunk) prefetch_theta(cd_next);
        }
        if (CODED) {
            if (tid == 0) {  // the decoders have finished this chunk's lists
                bool ok = false;
                for (unsigned it = 0; it < (1u << 22); ++it) {
                    int made;
                    asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(made) : "r"((unsigned)__cvta_generic_to_shared(&sync_words[0])) : "memory");
                    if (made > seq) {
                        ok = true;
                        break;
                    }
                    if (*reinterpret_cast<volatile int*>(&sync_words[2])) break;
                    __nanosleep(64);
                }
                if (!ok) {
                    if (!*reinterpret_cast<volatile int*>(&sync_words[2])) atomicExch(fa.status, (int)SL_ERR_TIMEOUT);
                    *reinterpret_cast<volatile int*>(&sync_words[2]) = 1;
                    *reinterpret_cast<volatile int*>(&sync_words[4]) = 1;
                }
            }
            cta_sync();
            if (*reinterpret_cast<volatile int*>(&sync_words[4])) break;  // (written by one thread before the barrier)
        }
        const uint16_t* sidx = sidx_all + (size_t)(seq & 1) * ((sidx_len + 7) / 8 * 8);
        // which of this lane's slots exist in this chunk (the same for every worker)
        bool in0[PPL], in1[PPL];
#pragma unroll
        for (int j = 0; j < PPL; ++j) {
            const int m = lane + 32 * j;
            in0[j] = 2 * m < keff;
            in1[j] = 2 * m + 1 < keff;
        }
        const unsigned* idx_pairs = STAGED ? reinterpret_cast<const unsigned*>(fa.ws.idx + g * fa.kp) : nullptr;
        float2* val_pairs = STAGED ? reinterpret_cast<float2*>(fa.ws.val + g * fa.kp) : nullptr;
        const TStat* tstat = STAGED ? fa.ws.tstat + cd.tensor : nullptr;

        for (int r0 = 0; r0 < n_workers; r0 += kApplyBatch) {
            const int nb = min(kApplyBatch, n_workers - r0);
            if (PACK) {  // the records of this batch start as zeros (unused slots and padding stay zero)
                for (int v = tid; v < nb * (stride / 16); v += kApplyThreads) reinterpret_cast<uint4*>(recs)[v] = make_uint4(0u, 0u, 0u, 0u);
            }
            if (tid < kApplyBatch) {  // what decodes worker r0 + tid: one load per thread, read back by all below
                float4 h = make_float4(0.f, 0.f, 0.f, 0.f), t = h;
                if (tid < nb) {
                    const int r = r0 + tid;
                    if (RAW) {
                        h.w = 1.f;
                    } else if (STAGED) {
                        const float4* st = reinterpret_cast<const float4*>(tstat + (long long)r * fa.n_tensors);
                        const float4 s0 = st[0], s1 = st[1];  // mu, sigma, 3 sigma, table[0] | table[1..3], pad
                        h = make_float4(s0.x, s0.z, 0.f, 1.f);
                        t = make_float4(s0.w, s1.x, s1.y, s1.z);
                    } else if (pl.p[r]) {
                        h.w = 1.f;
                        t = __ldg(reinterpret_cast<const float4*>(pl.p[r] + 16ll * cd.tensor));
                    }
                }
                tabs[2 * tid] = h;
                tabs[2 * tid + 1] = t;
            }
            // ---- A. this warp's workers of the batch (any order): pos = index pair, val = value pair / codes
            const int w0 = WB * warp;
            unsigned pos[WB][PPL];
            float2 val[WB][PPL];
#pragma unroll
            for (int q = 0; q < WB; ++q) {
                const int r = r0 + w0 + q;
#pragma unroll
                for (int j = 0; j < PPL; ++j) {
                    const int m = lane + 32 * j;
                    pos[q][j] = 0u;
                    val[q][j] = make_float2(0.f, 0.f);
                    if (w0 + q < nb && in0[j]) {
                        if (STAGED) {
                            pos[q][j] = idx_pairs[r * wstride + m];
                            val[q][j] = val_pairs[r * wstride + m];
                        } else if (CODED) {
                            if (pl.p[r]) {  // the decoded index pair and the pair's nibble of the chunk's code block
                                const unsigned x = reinterpret_cast<const unsigned*>(sidx + (size_t)r * fa.kp)[m];
                                const unsigned nib = (__ldg(pl.p[r] + 16ll * fa.n_tensors + (long long)cb * g + (m >> 1)) >> ((m & 1) * 4)) & 0xFu;
                                pos[q][j] = x;
                                val[q][j] = make_float2(__uint_as_float(nib & 3u), __uint_as_float(nib >> 2));
                            }
                        } else if (pl.p[r]) {
                            // 24 bits at byte 3 m of the record, from the aligned words around it (the second
                            // word may belong to the code block or the padding: inside the record either way)
                            const uint8_t* rec = pl.p[r] + cd.rec_off;
                            const int w = (3 * m) >> 2, sh = ((3 * m) & 3) * 8;
                            const unsigned lo = __ldg(reinterpret_cast<const unsigned*>(rec) + w);
                            const unsigned hi = sh > 8 ? __ldg(reinterpret_cast<const unsigned*>(rec) + w + 1) : 0u;
                            const unsigned x = __funnelshift_r(lo, hi, sh) & 0xFFFFFFu;
                            const unsigned nib = (__ldg(rec + ib + (m >> 1)) >> ((m & 1) * 4)) & 0xFu;
                            pos[q][j] = (x & 0xFFFu) | ((x >> 12) << 16);
                            val[q][j] = make_float2(__uint_as_float(nib & 3u), __uint_as_float(nib >> 2));  // the codes
                        }
                    }
                }
            }
            cta_sync();  // tables and zeroed records are in place
            if (CODED && r0 + kApplyBatch >= n_workers && tid == 0)  // the lists of this chunk have been read (last batch)
                asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"((unsigned)__cvta_generic_to_shared(&sync_words[1])), "r"(seq + 1) : "memory");
#pragma unroll
            for (int q = 0; q < WB; ++q) {
                const int r = r0 + w0 + q;
                const float4 hd = tabs[2 * (w0 + q)], lut = tabs[2 * (w0 + q) + 1];
                const bool have = hd.w != 0.f;  // false beyond the batch and for an absent worker
                const float mu = hd.x, t3 = hd.y;
                uint8_t* rec = recs + (size_t)(w0 + q) * stride;
#pragma unroll
                for (int j = 0; j < PPL; ++j) {
                    const int m = lane + 32 * j;
                    unsigned p0 = pos[q][j] & 0xFFFFu, p1 = pos[q][j] >> 16;
                    const bool ok0 = have && in0[j], ok1 = have && in1[j];
                    unsigned c0 = 0, c1 = 0;
                    if (PACK) {
                        c0 = (unsigned)quant_code(val[q][j].x, mu, t3);
                        c1 = (unsigned)quant_code(val[q][j].y, mu, t3);
                    } else if (!RAW) {
                        c0 = __float_as_uint(val[q][j].x);
                        c1 = __float_as_uint(val[q][j].y);
                    }
                    const float l0 = RAW ? val[q][j].x : c0 == 0 ? lut.x : c0 == 1 ? lut.y : c0 == 2 ? lut.z : lut.w;
                    const float l1 = RAW ? val[q][j].y : c1 == 0 ? lut.x : c1 == 1 ? lut.y : c1 == 2 ? lut.z : lut.w;
                    if (PACK) {
                        const float f0 = __fsub_rn(val[q][j].x, l0), f1 = __fsub_rn(val[q][j].y, l1);
                        if (FUSE == 1 && HALF) {
                            bf16_bits* eh = reinterpret_cast<bf16_bits*>(ptrs.e[r]) + cd.base;
                            if (ok0 && p0 < (unsigned)cd.len) eh[chunk_elem_offset(cd.row_stride, (int)p0)] = (bf16_bits)bf16_narrow(f0);
                            if (ok1 && p1 < (unsigned)cd.len) eh[chunk_elem_offset(cd.row_stride, (int)p1)] = (bf16_bits)bf16_narrow(f1);
                        } else if (FUSE == 1) {
                            if (ok0 && p0 < (unsigned)cd.len) ptrs.e[r][cd.base + chunk_elem_offset(cd.row_stride, (int)p0)] = f0;
                            if (ok1 && p1 < (unsigned)cd.len) ptrs.e[r][cd.base + chunk_elem_offset(cd.row_stride, (int)p1)] = f1;
                        } else if (ok0) {
                            // (slot 2 m + 1 exists in the array even when it is beyond keff: kp is even)
                            val_pairs[r * wstride + m] = make_float2(f0, f1);
                        }
                        // this lane's three bytes of the index block and its nibble of the code block
                        const unsigned x = (ok0 ? p0 : 0u) | ((ok1 ? p1 : 0u) << 12);
                        const unsigned nib = (ok0 ? c0 : 0u) | ((ok1 ? c1 : 0u) << 2);
                        const unsigned other = __shfl_xor_sync(kFull, nib, 1);
                        if (ok0) {
#pragma unroll
                            for (int bb = 0; bb < 3; ++bb)
                                if (3 * m + bb < ib) rec[3 * m + bb] = (uint8_t)(x >> (8 * bb));
                            if (!(lane & 1)) rec[ib + (m >> 1)] = (uint8_t)(nib | (other << 4));
                        }
                    }
                    // what step B adds where: entries that do not count add 0 to the thread's dump slot
                    const bool use0 = ok0 && p0 < (unsigned)cd.len, use1 = ok1 && p1 < (unsigned)cd.len;
                    p0 = use0 ? p0 : dump;
                    p1 = use1 ? p1 : dump;
                    pos[q][j] = p0 | (p1 << 16);
                    val[q][j] = make_float2(use0 ? l0 : 0.0f, use1 ? l1 : 0.0f);
                }
            }
            // ---- B. ascending worker order: the warps take turns, a warp's workers go one after the other
            // (a worker's positions are distinct; the barriers separate workers)
            for (int turn = 0; turn * WB < nb; ++turn) {
                if (warp == turn) {
#pragma unroll
                    for (int q = 0; q < WB; ++q) {
#pragma unroll
                        for (int j = 0; j < PPL; ++j) {
                            const unsigned p0 = pos[q][j] & 0xFFFFu, p1 = pos[q][j] >> 16;
                            acc[p0] = __fadd_rn(acc[p0], val[q][j].x);
                            acc[p1] = __fadd_rn(acc[p1], val[q][j].y);
                        }
                        __syncwarp();
                    }
                }
                cta_sync();
            }
            if (PACK) {  // the records of the batch are complete (written before the barriers above): out they go
                const int vpr = stride / 16;
                for (int v = tid; v < nb * vpr; v += kApplyThreads) {
                    const int rb = v / vpr, w = v - rb * vpr;
                    reinterpret_cast<uint4*>(ptrs.payload[r0 + rb] + cd.rec_off)[w] = reinterpret_cast<const uint4*>(recs)[v];
                }
            }
        }

        if (FUSE == 4) {  // Nesterov outer step on the average: every element moves
            float* __restrict__ mo = fa.momentum + cd.base;
            if (full) {
                float* __restrict__ mo_vec = mo + (long long)(tid >> 4) * rs + 4 * (tid & 15);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float* av = acc + 512 * i + 4 * tid;
                    const float4 sv = *reinterpret_cast<const float4*>(av);
                    float4 m = *reinterpret_cast<const float4*>(mo_vec + i * vec_step), o;
                    const float dx = __fdiv_rn(sv.x, fa.divisor), dy = __fdiv_rn(sv.y, fa.divisor);
                    const float dz = __fdiv_rn(sv.z, fa.divisor), dw = __fdiv_rn(sv.w, fa.divisor);
                    m.x = __fmaf_rn(fa.mu, m.x, dx); m.y = __fmaf_rn(fa.mu, m.y, dy);
                    m.z = __fmaf_rn(fa.mu, m.z, dz); m.w = __fmaf_rn(fa.mu, m.w, dw);
                    o.x = __fmaf_rn(-fa.alpha, __fmaf_rn(fa.mu, m.x, dx), a[i].x);
                    o.y = __fmaf_rn(-fa.alpha, __fmaf_rn(fa.mu, m.y, dy), a[i].y);
                    o.z = __fmaf_rn(-fa.alpha, __fmaf_rn(fa.mu, m.z, dz), a[i].z);
                    o.w = __fmaf_rn(-fa.alpha, __fmaf_rn(fa.mu, m.w, dw), a[i].w);
                    *reinterpret_cast<float4*>(th_vec + i * vec_step) = o;
                    *reinterpret_cast<float4*>(mo_vec + i * vec_step) = m;
                    *reinterpret_cast<float4*>(av) = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            } else {
                for (int p = tid; p < cd.len; p += kApplyThreads) {
                    const float d = __fdiv_rn(acc[p], fa.divisor);
                    const float m = __fmaf_rn(fa.mu, mo[p], d);
                    th[p] = __fmaf_rn(-fa.alpha, __fmaf_rn(fa.mu, m, d), th[p]);
                    mo[p] = m;
                    acc[p] = 0.0f;
                }
            }
        } else if (full) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float* av = acc + 512 * i + 4 * tid;
                const float4 sv = *reinterpret_cast<const float4*>(av);
                // a vector that received nothing keeps its bits; with scale < 0 so does one whose sums are
                // all +0 (fma(scale, +0, x) = x + -0 = x), and neither needs its store
                const bool untouched = scale < 0.0f && (__float_as_uint(sv.x) | __float_as_uint(sv.y) |
                                                        __float_as_uint(sv.z) | __float_as_uint(sv.w)) == 0u;
                if (!untouched) {
                    float4 o;
                    o.x = __fmaf_rn(scale, sv.x, a[i].x);
                    o.y = __fmaf_rn(scale, sv.y, a[i].y);
                    o.z = __fmaf_rn(scale, sv.z, a[i].z);
                    o.w = __fmaf_rn(scale, sv.w, a[i].w);
                    if (HALF)  // (an element that received nothing keeps its bits: fma(scale, +0, x) = x, and x is a bfloat16)
                        bf16_store4(theta_h + cd.base + (long long)(tid >> 4) * rs + 4 * (tid & 15) + i * vec_step, o);
                    else
                        *reinterpret_cast<float4*>(th_vec + i * vec_step) = o;
                    *reinterpret_cast<float4*>(av) = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        } else {
            for (int p = tid; p < cd.len; p += kApplyThreads) {  // (nothing was added at or beyond the chunk's length)
                if (HALF) {
                    bf16_bits* thh = theta_h + cd.base;
                    thh[p] = (bf16_bits)bf16_narrow(__fmaf_rn(scale, acc[p], bf16_widen(thh[p])));
                } else {
                    th[p] = __fmaf_rn(scale, acc[p], th[p]);
                }
                acc[p] = 0.0f;
            }
        }
        // (the next chunk's first additions come after several CTA barriers: the cleared tile is seen by all)
    }
    async_copy_wait_all();  // (an early exit leaves the copies of the chunk to come in flight)
}

}  // namespace
