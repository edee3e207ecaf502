// Kernel 1: pseudo-gradient + error feedback + chunk-wise Top-k (TMA and cp.async variants).
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"
#include "selection.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// Kernel 1: u = beta e + (theta - theta_r) written into e, chunk-wise Top-k of u into staging.
//
// Persistent CTAs (three or four per SM).  CTA b takes chunks b, b + grid, ... and, for each, the R
// workers in turn ("units"), so the chunk of theta_sync is fetched once per chunk and kept in
// registers.  theta_r and e of a unit travel global -> shared ahead of their use:
//   TMA variant      one tensor-map block copy per 64x64 block, issued by one thread, completion on
//                    shared-memory barriers with bounded waits; theta_r has one buffer (refilled from
//                    the unit's first barrier for the next unit), e two stages (filled two units
//                    ahead); u goes back to e as one block store from its stage;
//   cp.async variant 16-byte copies issued two units ahead by every thread for exactly the vectors it
//                    will consume itself, so no barrier guards their arrival; u is stored with
//                    128-bit stores.
// u is formed in registers and kept in the e stage for the selection.  Short tail chunks take plain
// loads and stores.
//
// PENDING: the error buffers hold u of the previous step and the corrected values (u - Dhat) of the
// selected entries wait in the staging arrays (deferred error-feedback subtraction).  The lists of
// the next units ride along three units ahead; before u is formed every warp substitutes the
// entries that fall into its 512 indices (the lists are sorted, so they form one run).
// ------------------------------------------------------------------------------------------------
// Shared memory of one CTA.  The cp.async variant keeps two theta_r stages (every thread refills its
// own slots two units ahead); the TMA variant needs one (it is free again at the unit's first
// barrier and refilled for the next unit from there).  With the four-class selection (k <= 64) the
// TMA variant also takes smaller candidate lists and pending-list slots: 54 KB in all, four CTAs
// per SM instead of three.
template <bool TMA, bool WIDE>
struct PipeSmemT {
    static constexpr bool kCompact = TMA && !WIDE;
    static constexpr int kLBuf = TMA ? 1 : 2;
    static constexpr int kPend = kCompact ? 64 : kMaxK;  // slots of a pending list (k rounded up to 8)
    static constexpr int kCtasPerSm = kCompact ? 4 : 3;
    float theta_l[kLBuf][kChunk];
    float e[2][kChunk];  // e on arrival, u after the update
    SelectSmemT<kCompact ? kSmallClassCap : kClassCap> sel;
    __align__(16) float pend_val[3][kPend];
    __align__(16) uint16_t pend_idx[3][kPend];
    unsigned long long l_bar;     // TMA variant: the theta_r block has landed
    unsigned long long e_bar[2];  // TMA variant: the e block of the stage has landed
    int abort;                    // TMA variant: a bounded wait ran out
};

// ---- TMA variant: tile copies through tensor maps, completion on shared-memory barriers ----------
// Every flat buffer is described, per distinct row length rs of the tensor table, as a 3-D array
// [rows][rs / 64][64] (element address = x0 + 64 x1 + rs x2); a 64x64 block is the box {64, 1, 64} at
// (0, x1, x2) and one copy instruction moves it.  The maps live in global memory, written by the
// host before the launch.  Waits poll a bounded number of times; when one runs out the kernel
// records SL_ERR_TIMEOUT and leaves.
constexpr unsigned kSpinLimit = 1u << 22;
constexpr int kMaxTmaClasses = 8;
constexpr int kTmaThread = 32 * 6;  // issues the tile copies (a warp other than the fetch warp, also lightly loaded)

struct TmaArgs {
    const CUtensorMap* maps;  // [slot][n_classes]
    int n_classes;
    int class_rs[kMaxTmaClasses];
    int slot_l[kMaxR], slot_e[kMaxR];  // map slot of theta_local[r], e[r]
    int* status;
};

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// true once the phase of this parity has completed; false after kSpinLimit polls
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity) {
    const unsigned addr = smem_u32(bar);
    for (unsigned it = 0; it < kSpinLimit; ++it) {
        unsigned done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}
// one 64x64 fp32 block, global -> shared, counted on `bar`
__device__ __forceinline__ void tma_load_block(void* dst_smem, const CUtensorMap* map, int x1, int x2,
                                               unsigned long long* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
            smem_u32(dst_smem)),
        "l"(map), "r"(0), "r"(x1), "r"(x2), "r"(smem_u32(bar))
        : "memory");
}
// one 64x64 fp32 block, shared -> global; joins the calling thread's open bulk group
__device__ __forceinline__ void tma_store_block(const CUtensorMap* map, int x1, int x2, const void* src_smem) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(map), "r"(0),
                 "r"(x1), "r"(x2), "r"(smem_u32(src_smem))
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// orders this thread's shared-memory writes before later asynchronous-copy reads of them
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// The part of a ChunkDesc the compression kernel needs (its first 16 bytes).
struct ChunkGeo {
    long long base;
    int row_stride;
    int len;
    int cls, x1, x2;  // TMA variant: row-length class and block coordinates (set by the kernel)
};
__device__ __forceinline__ ChunkGeo load_geo(const ChunkDesc* d) {
    const int4 v = __ldg(reinterpret_cast<const int4*>(d));
    ChunkGeo g;
    g.base = ((long long)v.y << 32) | (unsigned)v.x;
    g.row_stride = v.z;
    g.len = v.w;
    g.cls = g.x1 = g.x2 = 0;
    return g;
}

template <bool EF, bool PENDING, bool TMA, bool WIDE>
__global__ void __launch_bounds__(kThreads, (PipeSmemT<TMA, WIDE>::kCtasPerSm))
ef_topk_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int k, int kp, float beta,
               const float* __restrict__ theta_sync, WorkerPtrs ptrs, Workspace ws, TmaArgs tma) {
    extern __shared__ __align__(1024) unsigned char dyn_smem[];
    using Smem = PipeSmemT<TMA, WIDE>;
    Smem& sm = *reinterpret_cast<Smem*>(dyn_smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // 32-bit counters: chunks x workers < 2^31 is checked on the host
    const int grid = (int)gridDim.x, first = (int)blockIdx.x;
    const int my_chunks = ((int)n_chunks - first + grid - 1) / grid;  // >= 1: the grid never exceeds n_chunks
    const int n_units = my_chunks * n_workers;

    if (tid < 128) {
        sm.sel.bitmap[0][tid] = 0;
        sm.sel.bitmap[1][tid] = 0;
    }
    if (TMA && tid == kTmaThread) {
        mbar_init(&sm.l_bar, 1);
        mbar_init(&sm.e_bar[0], 1);
        mbar_init(&sm.e_bar[1], 1);
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }

    // This thread's i-th vector (in-chunk indices 512 warp + 128 i + 4 lane ..+3) lies in block row
    // 8 warp + 2 i + lane / 16 at column 4 (lane % 16): element offset off0 + 2 i rs from
    // ChunkDesc::base, rs = the block's row stride (64 for a flat run).
    const int sub_row = 8 * warp + (lane >> 4), sub_col = 4 * (lane & 15);
    const int slot0 = 512 * warp + 4 * lane;  // shared-tile index of the first vector; +128 per vector
    auto row_elems = [](const ChunkGeo& d) { return d.row_stride ? d.row_stride : kTile; };
    auto first_off = [&](const ChunkGeo& d) { return (long long)sub_row * row_elems(d) + sub_col; };
    // asynchronous loads of one unit into stage s (nothing for short chunks)
    auto issue_unit = [&](int s, const ChunkGeo& d, int r) {
        if (d.len == kChunk) {
            const long long off0 = d.base + first_off(d), step = 2ll * row_elems(d);
            const float* __restrict__ tl = ptrs.theta_local[r] + off0;
            const float* __restrict__ er = EF ? ptrs.e[r] + off0 : nullptr;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                cp_async16(&sm.theta_l[s][slot0 + 128 * i], tl + i * step);
                if (EF) cp_async16(&sm.e[s][slot0 + 128 * i], er + i * step);
            }
        }
    };
    // TMA variant: block coordinates in the 3-D view of row length rs, once per chunk
    auto with_coords = [&](ChunkGeo d) {
        if (TMA) {
            const int rs = row_elems(d);
            d.cls = 0;
            for (int q = 1; q < tma.n_classes; ++q) d.cls = tma.class_rs[q] == rs ? q : d.cls;
            d.x2 = (int)(d.base / rs);
            d.x1 = (int)(d.base - (long long)d.x2 * rs) >> 6;
        }
        return d;
    };
    // theta_r block of a unit into the single buffer (a short chunk moves nothing: the phase just ends)
    auto tma_load_l = [&](const ChunkGeo& d, int r) {
        if (d.len != kChunk) {
            mbar_arrive(&sm.l_bar);
            return;
        }
        mbar_arrive_expect_tx(&sm.l_bar, kChunk * (unsigned)sizeof(float));
        tma_load_block(sm.theta_l[0], tma.maps + tma.slot_l[r] * tma.n_classes + d.cls, d.x1, d.x2, &sm.l_bar);
    };
    // e block of a unit into stage s
    auto tma_load_e = [&](int s, const ChunkGeo& d, int r) {
        if (!EF) return;
        if (d.len != kChunk) {
            mbar_arrive(&sm.e_bar[s]);
            return;
        }
        mbar_arrive_expect_tx(&sm.e_bar[s], kChunk * (unsigned)sizeof(float));
        tma_load_block(sm.e[s], tma.maps + tma.slot_e[r] * tma.n_classes + d.cls, d.x1, d.x2, &sm.e_bar[s]);
    };
    // the fetch warp: the pending list of unit (chunk g, worker r) into ring slot `ring`
    auto issue_pending = [&](int ring, int g, int r) {
        const long long slot_base = ((long long)r * n_chunks + g) * kp;  // kp is a multiple of 8
        if (lane < (kp >> 3)) cp_async16(&sm.pend_idx[ring][8 * lane], ws.idx + slot_base + 8 * lane);
        for (int v = lane; v < (kp >> 2); v += 32) cp_async16(&sm.pend_val[ring][4 * v], ws.val + slot_base + 4 * v);
    };
    auto load_theta_s = [&](float4 (&ts)[4], const ChunkGeo& d) {
        if (d.len == kChunk) {
            const float* __restrict__ src = theta_sync + d.base + first_off(d);
            const long long step = 2ll * row_elems(d);
#pragma unroll
            for (int i = 0; i < 4; ++i) ts[i] = __ldg(reinterpret_cast<const float4*>(src + i * step));
        }
    };
    // (chunk ordinal, worker) of the unit `by` units after (c, r)
    auto ahead = [&](int c, int r, int by, int& c2, int& r2) {
        r2 = r + by;
        c2 = c;
        while (r2 >= n_workers) {
            r2 -= n_workers;
            ++c2;
        }
    };

    // descriptors of this CTA's current chunk and the two after it
    ChunkGeo cd = with_coords(load_geo(chunks + first)), cd1 = cd, cd2 = cd;
    if (my_chunks > 1) cd1 = with_coords(load_geo(chunks + first + grid));
    if (my_chunks > 2) cd2 = with_coords(load_geo(chunks + first + 2 * grid));

    // prologue: pending lists of units 0..2 (published by the barrier), then units 0 and 1
    if (PENDING) {
        if (warp == kFetchWarp) {
            for (int j = 0; j < 3 && j < n_units; ++j) {
                int c2, r2;
                ahead(0, 0, j, c2, r2);
                issue_pending(j, first + c2 * grid, r2);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
    }
    __syncthreads();
    if (TMA) {
        if (tid == kTmaThread) {
            tma_load_l(cd, 0);
            tma_load_e(0, cd, 0);
            if (n_units > 1) tma_load_e(1, n_workers > 1 ? cd : cd1, n_workers > 1 ? 1 : 0);
        }
    } else {
        issue_unit(0, cd, 0);
    }
    cp_async_commit();
    if (!TMA && n_units > 1) issue_unit(1, n_workers > 1 ? cd : cd1, n_workers > 1 ? 1 : 0);
    cp_async_commit();

    float4 ts[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) ts[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    load_theta_s(ts, cd);

    int c = 0, r = 0;  // chunk ordinal within this CTA, worker
    int n = 0;
    for (; n < n_units; ++n) {
        const int s = n & 1;
        const bool full = cd.len == kChunk;
        const int keff = min(k, cd.len);
        float* __restrict__ er = EF ? ptrs.e[r] + cd.base : nullptr;
        float* __restrict__ er_vec = EF ? er + first_off(cd) : nullptr;  // this thread's first vector (full chunks)
        const long long er_step = 2ll * row_elems(cd);
        float* tile = sm.e[s];

        cp_async_wait<1>();  // this unit's copies have landed (only the next unit's may be in flight)
        if (TMA) {
            if (!mbar_wait(&sm.l_bar, (unsigned)(n & 1))) sm.abort = 1;
            if (EF && !mbar_wait(&sm.e_bar[s], (unsigned)((n >> 1) & 1))) sm.abort = 1;
        }

        if (PENDING && EF) {  // substitute the corrected values of the previous step
            const int ring = n % 3;
            if (full) {
                __syncwarp();  // the whole warp's copies have landed
                for (int j = lane; j < keff; j += 32) {
                    const unsigned p = sm.pend_idx[ring][j];
                    if ((p >> 9) == (unsigned)warp) tile[p] = sm.pend_val[ring][j];
                }
                __syncwarp();
            } else {  // short chunk: patch global memory, which the plain loads below read
                for (int j = tid; j < keff; j += kThreads) {
                    const unsigned p = sm.pend_idx[ring][j];
                    if (p < (unsigned)cd.len) er[p] = sm.pend_val[ring][j];
                }
                __syncthreads();
            }
        }

        unsigned ub[kPerThread];
        if (full) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int v = slot0 + 128 * i;
                const float4 a = ts[i];
                const float4 l = *reinterpret_cast<const float4*>(&sm.theta_l[TMA ? 0 : s][v]);
                float4 u;
                u.x = __fsub_rn(a.x, l.x);
                u.y = __fsub_rn(a.y, l.y);
                u.z = __fsub_rn(a.z, l.z);
                u.w = __fsub_rn(a.w, l.w);
                if (EF) {
                    const float4 ev = *reinterpret_cast<const float4*>(&tile[v]);
                    u.x = __fmaf_rn(beta, ev.x, u.x);
                    u.y = __fmaf_rn(beta, ev.y, u.y);
                    u.z = __fmaf_rn(beta, ev.z, u.z);
                    u.w = __fmaf_rn(beta, ev.w, u.w);
                    if (!TMA) *reinterpret_cast<float4*>(er_vec + i * er_step) = u;
                }
                *reinterpret_cast<float4*>(&tile[v]) = u;
                ub[4 * i + 0] = __float_as_uint(u.x);
                ub[4 * i + 1] = __float_as_uint(u.y);
                ub[4 * i + 2] = __float_as_uint(u.z);
                ub[4 * i + 3] = __float_as_uint(u.w);
            }
            if (TMA && EF) fence_async_smem();  // the tile is about to be read by a block store
        } else {  // short tail of a flat tensor: element-wise with bounds
            const float* __restrict__ tsp = theta_sync + cd.base;
            const float* __restrict__ tl = ptrs.theta_local[r] + cd.base;
#pragma unroll
            for (int q = 0; q < kPerThread; ++q) {
                const int p = owned_index(tid, q);
                float u = 0.0f;
                if (p < cd.len) {
                    u = __fsub_rn(tsp[p], tl[p]);
                    if (EF) {
                        u = __fmaf_rn(beta, er[p], u);
                        er[p] = u;
                    }
                }
                tile[p] = u;
                ub[q] = __float_as_uint(u);
            }
        }
        // theta_sync of the next chunk, once the last worker of this one has used the registers
        if (r == n_workers - 1 && c + 1 < my_chunks) load_theta_s(ts, cd1);

        unsigned* bitmap = sm.sel.bitmap[s];
        Picked pk;
        pk.p0 = pk.v0 = pk.p1 = pk.v1 = 0u;
        bool exact = select_topk<WIDE>(ub, reinterpret_cast<const unsigned*>(tile), cd.len, keff, sm.sel, pk);
        if (tid < 128) sm.sel.bitmap[s ^ 1][tid] = 0;  // the other map: its readers passed the barrier above

        // refill for unit n + 2.  cp.async variant: the whole stage is consumed (nothing below reads
        // the tile).  TMA variant: one thread stores u, re-arms the stage and starts theta_r; e follows
        // once the selection and the store are done with the tile.  The fetch warp also fetches the
        // pending list of unit n + 3 (its ring slot was last read before the barrier above).
        if (TMA && *reinterpret_cast<volatile int*>(&sm.abort)) break;  // uniform: written before the barrier above
        int c2, r2;  // unit n + 2 and its chunk
        ahead(c, r, 2, c2, r2);
        const bool have2 = c2 < my_chunks;
        ChunkGeo d2;  // picked field by field: keeps the three descriptors in registers
        {
            const int dc = c2 - c;
            d2.base = dc == 0 ? cd.base : (dc == 1 ? cd1.base : cd2.base);
            d2.row_stride = dc == 0 ? cd.row_stride : (dc == 1 ? cd1.row_stride : cd2.row_stride);
            d2.len = dc == 0 ? cd.len : (dc == 1 ? cd1.len : cd2.len);
            d2.cls = dc == 0 ? cd.cls : (dc == 1 ? cd1.cls : cd2.cls);
            d2.x1 = dc == 0 ? cd.x1 : (dc == 1 ? cd1.x1 : cd2.x1);
            d2.x2 = dc == 0 ? cd.x2 : (dc == 1 ? cd1.x2 : cd2.x2);
        }
        if (TMA) {
            if (tid == kTmaThread) {
                if (EF && full) {  // u back into e: every thread fenced its writes before the barrier above
                    tma_store_block(tma.maps + tma.slot_e[r] * tma.n_classes + cd.cls, cd.x1, cd.x2, tile);
                    bulk_commit();
                }
                if (n + 1 < n_units) {  // the theta_r buffer was last read before that barrier: next unit's block
                    int c1n, r1n;
                    ahead(c, r, 1, c1n, r1n);
                    tma_load_l(c1n == c ? cd : cd1, r1n);
                }
            }
        } else if (have2) {
            issue_unit(s, d2, r2);
        }
        if (PENDING && warp == kFetchWarp) {
            int c3, r3;
            ahead(c, r, 3, c3, r3);
            if (c3 < my_chunks) issue_pending(n % 3, first + c3 * grid, r3);
        }
        cp_async_commit();

        bool e_started = false;  // TMA variant: the e block of unit n + 2 is on its way
        if (!exact) {
            __syncthreads();  // class lists complete: nobody reads the tile any more except the block store
            if (TMA && EF && tid == kTmaThread) {
                if (full) bulk_wait_read_all();  // once the store has read the tile, refill it
                if (have2) tma_load_e(s, d2, r2);
            }
            e_started = true;
            exact = select_rank<WIDE>(keff, sm.sel, bitmap, pk);
        }
        if (exact) {
            unsigned tmp[kPerThread];
            bool nonzero = false;
#pragma unroll
            for (int q = 0; q < kPerThread; ++q) {
                tmp[q] = ub[q];
                nonzero |= (ub[q] & 0x7FFFFFFFu) != 0;
            }
            select_exact_search(tmp, nonzero, cd.len, keff, sm.sel, bitmap);
        }
        __syncthreads();  // the map is complete
        if (TMA && EF && !e_started && tid == kTmaThread) {  // the exact search came straight from the threshold
            if (full) bulk_wait_read_all();
            if (have2) tma_load_e(s, d2, r2);
        }
        if (exact) {
            pk.mask = 0;
            if (tid < (int)sm.sel.n_exact) {
                pk.p0 = (&sm.sel.lpos[0][0])[tid];
                pk.v0 = (&sm.sel.lkey[0][0])[tid] | ((pk.p0 >> 12) << 31);
                pk.p0 &= 0xFFFu;
                pk.mask = 1u;
            }
        }

        const long long slot_base = ((long long)r * n_chunks + (first + c * grid)) * kp;
        emit_picked(pk, bitmap, keff, ws.idx + slot_base, ws.val + slot_base);

        if (++r == n_workers) {
            r = 0;
            ++c;
            cd = cd1;
            cd1 = cd2;
            if (c + 2 < my_chunks) cd2 = with_coords(load_geo(chunks + first + (c + 2) * grid));
        }
    }
    cp_async_wait<0>();
    if (TMA) {
        if (n < n_units) {
            // A wait ran out.  Report it, then give the copies still in flight a bounded time to
            // land before the shared memory they target is released.
            if (tid == 0) atomicExch(tma.status, (int)SL_ERR_TIMEOUT);
            mbar_wait(&sm.l_bar, (unsigned)(n & 1));
            if (EF)
                for (int u = n; u < n + 2 && u < n_units; ++u) mbar_wait(&sm.e_bar[u & 1], (unsigned)((u >> 1) & 1));
        }
        if (tid == kTmaThread) bulk_wait_all();
    }
}

}  // namespace
