// Kernel 1: pseudo-gradient + error feedback + chunk-wise Top-k, one warp per (chunk, worker) unit.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"

namespace {

// ------------------------------------------------------------------------------------------------
// u = beta e + (theta - theta_r) written into e, chunk-wise Top-k of u into the staging arrays
// (Eq. 2 line 1; Sec. 3.3).
//
// One persistent CTA per SM: eight consumer warps and one producer warp.  CTA b takes chunks b,
// b + grid, ... and, for each, the R workers in turn; (chunk, worker) = a "unit", numbered in that
// order.  The producer thread moves every unit's 64x64 blocks of theta_r and e into a ring of
// shared-memory slots with one tensor-map (TMA) copy each, and the chunk's block of theta once per
// chunk into a second, smaller ring; completion is counted on shared-memory barriers, a slot is
// handed back by its consumer through a second barrier.  A consumer warp claims the next unit,
// waits for its blocks, forms u for all 4096 elements in registers (128 per lane), stores u to e
// with 128-bit stores, hands the slot back and selects on its registers alone: no CTA-wide barrier
// exists, and the blocks in flight (up to five units, 160 KB) are decoupled from the selection.
//
// Lane l of a warp owns in-chunk indices p = 128 i + 4 l + j (i = 0..31, j = 0..3), register 4 i + j.
//
// Selection (exact: magnitude = float bits without the sign, ties to the lower index):
//  A. 8 group maxima per lane (16 values each; 32 of 4 values each for k > 128); M = the largest.
//  B. a threshold T by bisection over the group maxima: at least keff groups, hence at least keff
//     elements, reach T, and only a few more do (about 1.15 keff elements).
//  C. every element with key >= T is a candidate; the lanes list the candidates' positions in shared
//     memory.
//  D. the candidates are dealt out evenly (lane t takes entries t, t + 32, ...), their values read
//     back from where u was just stored.
//  E. bisection over the candidates' keys finds the keff-th largest; equal keys at the cut are
//     resolved by a second bisection over positions.
//  F. selected candidates set their bit in a 4096-bit map; its prefix popcount is the slot of each
//     (ascending in-chunk index) and the holder writes (index, value) to the staging arrays.
// All-zero chunks, thresholds of zero and more candidates than the list holds take an exact bitwise
// search over all 4096 keys instead (select_slow).  Beyond keff = 256 (instantiation WIDE = 2) a threshold
// over group maxima no longer thins the field and select_dense takes over: a key interval around the cut
// narrowed on the registers, everything above it marked directly, the elements inside it listed and ranked.
//
// Chunks that cannot travel as tensor-map blocks (short tails, tables whose blocks do not start on a
// 64-element boundary, tile copies switched off) are read and written with plain loads and stores by
// the consumer warp ("direct" units); the producer then only keeps the barrier phases in step.
//
// PENDING: the error buffers hold u of the previous step and the corrected values (u - Dhat) of the
// selected entries wait in the staging arrays (deferred error-feedback subtraction); the producer
// fetches each unit's list with its blocks and the consumer substitutes it before forming u.
// ------------------------------------------------------------------------------------------------

// ---- shared-memory barriers and tensor-map copies (inline PTX) ------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

constexpr unsigned kSpinLimit = 1u << 22;  // polls of a bounded wait
constexpr int kMaxTmaClasses = 8;

struct TmaArgs {
    const CUtensorMap* maps;  // [slot][n_classes]
    int n_classes;
    int class_rs[kMaxTmaClasses];
    int slot_l[kMaxR], slot_e[kMaxR];  // map slot of theta_local[r], e[r]
    int slot_s;                        // map slot of theta_sync
    int fresh;                         // maps were written since the last launch: fence before first use
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
// `bytes` (a multiple of 16, both addresses 16-byte aligned) global -> shared, counted on `bar`
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, unsigned bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// a tensor map in global memory that the host rewrote: make this thread's later copies see it
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* map) {
    asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(map) : "memory");
}
// orders this thread's shared-memory accesses before later asynchronous-copy writes to the same bytes
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- layout of the CTA's shared memory ------------------------------------------------------------
constexpr int kSelWarps = 8;                         // consumer warps
constexpr int kSelThreads = 32 * (kSelWarps + 1);    // + the producer warp
constexpr int kThetaRing = 3;                        // blocks of theta in flight or in use
constexpr int kUnitSlots = 5;                        // units in flight or in use
constexpr int kCandCap = 384;                        // candidate positions a warp can list
constexpr int kSelNarrowMaxK = 128;                  // largest k served by the groups-of-16 kernel

struct SelSmem {
    float theta_s[kThetaRing][kChunk];
    float theta_l[kUnitSlots][kChunk];
    float e[kUnitSlots][kChunk];
    __align__(16) float pend_val[kUnitSlots][kFastMaxK];
    __align__(16) uint16_t pend_idx[kUnitSlots][kFastMaxK];
    __align__(16) unsigned bitmap[kSelWarps][128];
    uint16_t cand[kSelWarps][kCandCap];
    unsigned long long full_s[kThetaRing], empty_s[kThetaRing];  // theta block landed / all R units done with it
    unsigned long long full_u[kUnitSlots], empty_u[kUnitSlots];  // unit's blocks landed / consumer done with them
    int next_unit;  // next unit a consumer warp may claim
    int issued;     // units whose barriers the producer has armed
    int abort;      // a bounded wait ran out
};
static_assert(sizeof(SelSmem) <= 227 * 1024, "shared memory of one CTA");

// The first 16 bytes of a ChunkDesc.
struct ChunkGeo {
    long long base;
    int row_stride;
    int len;
};
__device__ __forceinline__ ChunkGeo load_geo(const ChunkDesc* d) {
    const int4 v = __ldg(reinterpret_cast<const int4*>(d));
    ChunkGeo g;
    g.base = ((long long)v.y << 32) | (unsigned)v.x;
    g.row_stride = v.z;
    g.len = v.w;
    return g;
}

// Where the selection finds u again after it was stored: element p sits at ptr[(p >> 6) * rs + (p & 63)].
struct USource {
    const unsigned* ptr;  // global (the error buffer) or shared (a slot, when error feedback is frozen)
    int rs;
};
template <bool GLOBAL>
__device__ __forceinline__ unsigned usrc_load(const USource& s, unsigned p) {
    const unsigned* a = s.ptr + (long long)(p >> 6) * s.rs + (p & 63u);
    // global: u was stored by other lanes of this warp a moment ago; read it where the stores went (L2)
    return GLOBAL ? __ldcg(a) : *a;
}

__device__ __forceinline__ unsigned lane_pos(int lane, int q) { return 128u * (q >> 2) + 4u * lane + (q & 3); }

// Writes (index, value) of the entries marked in the warp's 4096-bit map to their slots, in ascending
// index order, reading the values back through `src`.  Word w of the map covers indices 32 w ..; lane l
// owns words 4 l .. 4 l + 3.
// BATCH > 1: the values of BATCH entries are fetched before any of them is stored (with many entries per lane
// the fetches, L2 reads when `src` is global, would otherwise wait for one another).
template <bool GLOBAL, int BATCH = 1>
__device__ __forceinline__ void emit_from_map(const unsigned* bitmap, const USource& src, int keff,
                                              uint16_t* __restrict__ out_idx, float* __restrict__ out_val) {
    const int lane = threadIdx.x & 31;
    const uint4 w = *reinterpret_cast<const uint4*>(&bitmap[4 * lane]);
    const unsigned words[4] = {w.x, w.y, w.z, w.w};
    const unsigned tot = __popc(w.x) + __popc(w.y) + __popc(w.z) + __popc(w.w);
    unsigned inc = tot;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned o = __shfl_up_sync(kFull, inc, d);
        if (lane >= d) inc += o;
    }
    unsigned slot = inc - tot;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        unsigned mm = words[q];
        while (mm) {
            unsigned p[BATCH], v[BATCH];
#pragma unroll
            for (int t = 0; t < BATCH; ++t) {
                p[t] = 0xFFFFu;
                if (mm) {
                    p[t] = 128u * lane + 32u * q + (__ffs(mm) - 1);
                    mm &= mm - 1;
                }
            }
#pragma unroll
            for (int t = 0; t < BATCH; ++t) v[t] = p[t] != 0xFFFFu ? usrc_load<GLOBAL>(src, p[t]) : 0u;
#pragma unroll
            for (int t = 0; t < BATCH; ++t) {
                if (p[t] != 0xFFFFu) {
                    if (slot < (unsigned)keff) {
                        out_idx[slot] = (uint16_t)p[t];
                        out_val[slot] = __uint_as_float(v[t]);
                    }
                    ++slot;
                }
            }
        }
    }
}

// Exact fallback for one unit: bitwise search for the keff-th largest key over all 4096 elements
// (re-read through `src`; indices >= len count as key 0 and cannot be selected because keff <= len),
// ties at the cut to the lower index.  Marks the map and writes the staging entries.  Warp-collective.
template <bool GLOBAL>
__device__ __noinline__ void select_slow(USource src, int len, int keff, unsigned* bitmap,
                                         uint16_t* __restrict__ out_idx, float* __restrict__ out_val) {
    const int lane = threadIdx.x & 31;
    unsigned key[128];
    unsigned any = 0;
#pragma unroll
    for (int q = 0; q < 128; ++q) {
        const unsigned p = lane_pos(lane, q);
        key[q] = (int)p < len ? (usrc_load<GLOBAL>(src, p) & 0x7FFFFFFFu) : 0u;
        any |= key[q];
    }
    any = __reduce_or_sync(kFull, any);
    // K = the keff-th largest key: the largest x with count(key >= x) >= keff
    unsigned lo = 0, hi = 0x80000000u, c_hi = 0;  // count(>= lo) >= keff > count(>= hi) = c_hi
    bool clean = false;                           // count(>= lo) == keff: no tie straddles the cut
    if (any) {
        while (hi - lo > 1) {
            const unsigned mid = lo + ((hi - lo) >> 1);
            unsigned c = 0;
#pragma unroll
            for (int q = 0; q < 128; ++q) c += key[q] >= mid ? 1u : 0u;
            c = __reduce_add_sync(kFull, c);
            if (c >= (unsigned)keff) {
                lo = mid;
                if (c == (unsigned)keff) {
                    clean = true;
                    break;
                }
            } else {
                hi = mid;
                c_hi = c;
            }
        }
    }
    // entries with key == lo fill the remaining places in index order: the largest index P taken
    unsigned P = 4095u;
    if (!clean) {
        const unsigned need = (unsigned)keff - c_hi;  // >= 1
        int plo = -1, phi = 4095;                     // count(key == lo, p <= plo) < need <= count(.., p <= phi)
        while (phi - plo > 1) {
            const int mid = plo + ((phi - plo) >> 1);
            unsigned c = 0;
#pragma unroll
            for (int q = 0; q < 128; ++q) c += (key[q] == lo && (int)lane_pos(lane, q) <= mid) ? 1u : 0u;
            c = __reduce_add_sync(kFull, c);
            if (c >= need) phi = mid;
            else plo = mid;
        }
        P = (unsigned)phi;
    }
#pragma unroll
    for (int q = 0; q < 128; ++q) {
        const unsigned p = lane_pos(lane, q);
        const bool sel = clean ? key[q] >= lo : (key[q] > lo || (key[q] == lo && p <= P));
        if (sel && (int)p < len) atomicOr(&bitmap[p >> 5], 1u << (p & 31));
    }
    __syncwarp();
    emit_from_map<GLOBAL>(bitmap, src, keff, out_idx, out_val);
}

// Selection for large keff (beyond 256 of 4096: the dense settings of the paper's sweeps), on the warp's
// registers.  A bitwise search narrows a key interval [lo, hi) around the cut until it holds at most
// kCandCap elements (about ten rounds over the 128 registers instead of the 31 + 12 of the exact
// fallback); the elements inside the interval are listed and a search over that short list finds the
// cut (key, and index among equal keys); everything at or above hi was marked in the map straight from the
// registers, the winners of the list are added, and the entries are written from the map.  Falls back to
// select_slow when the interval cannot be narrowed (a run of more than kCandCap equal keys at the cut).
// Warp-collective.
template <bool GLOBAL>
__device__ __forceinline__ void select_dense(const float (&u)[128], USource src, int len, int keff, unsigned* bitmap,
                                          uint16_t* cand, uint16_t* __restrict__ out_idx, float* __restrict__ out_val) {
    const int lane = threadIdx.x & 31;
    unsigned mx = 0;
#pragma unroll
    for (int q = 0; q < 128; ++q) mx = max(mx, __float_as_uint(u[q]) & 0x7FFFFFFFu);
    const unsigned M = __reduce_max_sync(kFull, mx);
    unsigned lo = 0, hi = M + 1u, c_lo = (unsigned)kChunk, c_hi = 0;  // count(>= lo) = c_lo >= keff > c_hi = count(>= hi)
    // first guesses: one and two binades below the largest key
    unsigned x = M > (1u << 23) ? M - (1u << 23) : (M >> 1);
    while (c_lo - c_hi > (unsigned)kCandCap && hi - lo > 1) {
        if (!(x > lo && x < hi)) x = lo + ((hi - lo) >> 1);
        unsigned c = 0;
#pragma unroll
        for (int q = 0; q < 128; ++q) c += (__float_as_uint(u[q]) & 0x7FFFFFFFu) >= x ? 1u : 0u;
        c = __reduce_add_sync(kFull, c);
        if (c >= (unsigned)keff) {
            lo = x;
            c_lo = c;
            x = hi;  // (out of range: the next guess is the midpoint)
        } else {
            hi = x;
            c_hi = c;
            x = x > (1u << 23) ? x - (1u << 23) : 0u;  // still too few: try a binade lower
        }
    }
    if (c_lo - c_hi > (unsigned)kCandCap) {  // more than a list's worth of equal keys at the cut
        select_slow<GLOBAL>(src, len, keff, bitmap, out_idx, out_val);
        return;
    }
    // elements at or above hi are selected: marked in the map straight from the registers (four consecutive
    // indices of a lane share a map word with seven other lanes); the ones inside the interval are listed.
    // (The registers are not needed after this: what follows works on the list and on the map.)
    unsigned hm[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        unsigned nib = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const unsigned key = __float_as_uint(u[4 * i + j]) & 0x7FFFFFFFu;
            nib |= key >= hi ? (1u << j) : 0u;
            hm[i >> 3] |= (key >= lo && key < hi) ? (1u << ((4 * i + j) & 31)) : 0u;
        }
        if (nib) atomicOr(&bitmap[4 * i + (lane >> 3)], nib << (4 * (lane & 7)));
    }
    // the list of the elements inside the interval
    const unsigned mine = __popc(hm[0]) + __popc(hm[1]) + __popc(hm[2]) + __popc(hm[3]);
    unsigned inc = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned o = __shfl_up_sync(kFull, inc, d);
        if (lane >= d) inc += o;
    }
    const unsigned n_b = __shfl_sync(kFull, inc, 31);  // = c_lo - c_hi
    {
        unsigned at = inc - mine;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            unsigned mm = hm[w];
            while (mm) {
                const unsigned b = __ffs(mm) - 1;
                mm &= mm - 1;
                cand[at++] = (uint16_t)lane_pos(lane, 32 * w + (int)b);
            }
        }
    }
    __syncwarp();
    // the `need` largest of the list, ties to the lower index
    constexpr int CPL = kCandCap / 32;
    const unsigned need = (unsigned)keff - c_hi;  // 1 .. n_b
    unsigned cp[CPL], ck[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const unsigned t = lane + 32u * j;
        cp[j] = t < n_b ? cand[t] : 0u;
        // (indices at or beyond the chunk's length hold key 0 and are never fetched: nothing exists there)
        ck[j] = (t < n_b && (int)cp[j] < len) ? (usrc_load<GLOBAL>(src, cp[j]) & 0x7FFFFFFFu) : 0u;
    }
    // (an empty place has key 0; when lo = 0 it would count, so empty places are excluded by position)
    unsigned l2 = lo, h2 = hi, cl2 = n_b, ch2 = 0;  // count(>= l2) = cl2 >= need > ch2 = count(>= h2), within the list
    while (cl2 != need && h2 - l2 > 1) {
        const unsigned xm = l2 + ((h2 - l2) >> 1);
        unsigned c = 0;
#pragma unroll
        for (int j = 0; j < CPL; ++j) c += (lane + 32u * j < n_b && ck[j] >= xm) ? 1u : 0u;
        c = __reduce_add_sync(kFull, c);
        if (c >= need) {
            l2 = xm;
            cl2 = c;
        } else {
            h2 = xm;
            ch2 = c;
        }
    }
    unsigned P = 4095u;
    const bool clean = cl2 == need;
    if (!clean) {
        const unsigned want = need - ch2;
        int plo = -1, phi = 4095;
        while (phi - plo > 1) {
            const int mid = plo + ((phi - plo) >> 1);
            unsigned c = 0;
#pragma unroll
            for (int j = 0; j < CPL; ++j) c += (lane + 32u * j < n_b && ck[j] == l2 && (int)cp[j] <= mid) ? 1u : 0u;
            c = __reduce_add_sync(kFull, c);
            if (c >= want) phi = mid;
            else plo = mid;
        }
        P = (unsigned)phi;
    }
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const bool in = lane + 32u * j < n_b;
        const bool sel = in && (clean ? ck[j] >= l2 : (ck[j] > l2 || (ck[j] == l2 && cp[j] <= P)));
        if (sel) atomicOr(&bitmap[cp[j] >> 5], 1u << (cp[j] & 31));
    }
    __syncwarp();
    emit_from_map<GLOBAL, 8>(bitmap, src, keff, out_idx, out_val);
}

// Steps D-F for a candidate list of n_c <= 32 CPL entries.  Warp-collective.
template <int CPL, bool GLOBAL>
__device__ __forceinline__ void rank_and_emit(const uint16_t* __restrict__ cand, unsigned n_c, unsigned T, unsigned probe,
                                              const USource& src, int keff, unsigned* bitmap,
                                              uint16_t* __restrict__ out_idx, float* __restrict__ out_val) {
    const int lane = threadIdx.x & 31;
    unsigned cp[CPL], cu[CPL], ck[CPL];
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const unsigned t = lane + 32u * j;
        cp[j] = t < n_c ? cand[t] : 0u;
    }
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const unsigned t = lane + 32u * j;
        cu[j] = t < n_c ? usrc_load<GLOBAL>(src, cp[j]) : 0u;
        ck[j] = cu[j] & 0x7FFFFFFFu;  // an empty place has key 0 < T and is never counted
    }
    // E. the keff-th largest key among the candidates
    unsigned lo = T, c_lo = n_c, c_hi = 0, hi;  // count(>= lo) = c_lo >= keff > c_hi = count(>= hi)
    {
        unsigned mx = 0;
#pragma unroll
        for (int j = 0; j < CPL; ++j) mx = max(mx, ck[j]);
        hi = __reduce_max_sync(kFull, mx) + 1u;
    }
    unsigned x = probe;
    while (c_lo != (unsigned)keff && hi - lo > 1) {
        if (!(x > lo && x < hi)) x = lo + ((hi - lo) >> 1);
        unsigned c = 0;
#pragma unroll
        for (int j = 0; j < CPL; ++j) c += ck[j] >= x ? 1u : 0u;
        c = __reduce_add_sync(kFull, c);
        if (c >= (unsigned)keff) {
            lo = x;
            c_lo = c;
        } else {
            hi = x;
            c_hi = c;
        }
        x = lo + ((hi - lo) >> 1);
    }
    unsigned P = 4095u;
    const bool clean = c_lo == (unsigned)keff;
    if (!clean) {  // equal keys straddle the cut: the lowest indices among them fill the remaining places
        const unsigned need = (unsigned)keff - c_hi;
        int plo = -1, phi = 4095;
        while (phi - plo > 1) {
            const int mid = plo + ((phi - plo) >> 1);
            unsigned c = 0;
#pragma unroll
            for (int j = 0; j < CPL; ++j) c += (ck[j] == lo && (int)cp[j] <= mid) ? 1u : 0u;
            c = __reduce_add_sync(kFull, c);
            if (c >= need) phi = mid;
            else plo = mid;
        }
        P = (unsigned)phi;
    }
    // F. map, prefix, ordered emission
    unsigned sel = 0;
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const bool s = clean ? ck[j] >= lo : (ck[j] > lo || (ck[j] == lo && cp[j] <= P));
        if (s) {
            sel |= 1u << j;
            atomicOr(&bitmap[cp[j] >> 5], 1u << (cp[j] & 31));
        }
    }
    __syncwarp();
    unsigned pack;  // exclusive count before this lane's 4 words | popcounts of its first three words
    {
        const uint4 w = *reinterpret_cast<const uint4*>(&bitmap[4 * lane]);
        const unsigned c0 = __popc(w.x), c1 = __popc(w.y), c2 = __popc(w.z), c3 = __popc(w.w);
        const unsigned tot = c0 + c1 + c2 + c3;
        unsigned inc = tot;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned o = __shfl_up_sync(kFull, inc, d);
            if (lane >= d) inc += o;
        }
        pack = (inc - tot) | (c0 << 13) | (c1 << 19) | (c2 << 25);
    }
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
        const unsigned p = cp[j], w = p >> 5;
        const unsigned pq = __shfl_sync(kFull, pack, w >> 2);
        if (sel & (1u << j)) {
            const unsigned sub = w & 3u;
            unsigned before = pq & 0x1FFFu;
            if (sub > 0) before += (pq >> 13) & 0x3Fu;
            if (sub > 1) before += (pq >> 19) & 0x3Fu;
            if (sub > 2) before += (pq >> 25) & 0x3Fu;
            const unsigned slot = before + __popc(bitmap[w] & ((1u << (p & 31)) - 1u));
            if (slot < (unsigned)keff) {
                out_idx[slot] = (uint16_t)p;
                out_val[slot] = __uint_as_float(cu[j]);
            }
        }
    }
}

// Steps A and B: GN group maxima per lane (groups of 128 / GN of the lane's values, 32 GN per chunk) and a
// threshold T that at least keff of them reach, and not many more; T = 0 when there is none (all-zero
// or mostly-zero chunk, maxima that are all NaN, keff beyond the number of groups).  `probe` = a key
// that fewer than keff groups reach: a good first guess for the element-level cut.
template <int GN>
__device__ __forceinline__ void group_threshold(const float (&u)[128], int keff, unsigned& T, unsigned& probe) {
    constexpr int GS = 128 / GN;
    // A. group maxima (on floats: a NaN is skipped, which can only lower the threshold)
    unsigned kg[GN];
    float mall = 0.0f;
#pragma unroll
    for (int g = 0; g < GN; ++g) {
        float m = 0.0f;
#pragma unroll
        for (int q = GS * g; q < GS * g + GS; q += 2) m = fmaxf(m, fmaxf(fabsf(u[q]), fabsf(u[q + 1])));
        kg[g] = __float_as_uint(m);
        mall = fmaxf(mall, m);
    }
    const unsigned M = __reduce_max_sync(kFull, __float_as_uint(mall));
    // B. bisection over the keys of the group maxima
    T = 0;
    probe = 0;
    if (M == 0u || keff > 32 * GN) return;
    unsigned lo = 0, hi = M + 1u, c_lo = 32 * GN;  // count(>= lo) = c_lo >= keff > count(>= hi)
    const unsigned enough = (unsigned)keff + max(2u, (unsigned)keff >> 3);
    unsigned x = M > (2u << 23) ? M - (2u << 23) : (M >> 1);  // first guess: a quarter of the largest magnitude
    for (int it = 0; it < 40; ++it) {
        unsigned c = 0;
#pragma unroll
        for (int g = 0; g < GN; ++g) c += kg[g] >= x ? 1u : 0u;
        c = __reduce_add_sync(kFull, c);
        if (c >= (unsigned)keff) {
            lo = x;
            c_lo = c;
        } else {
            hi = x;
        }
        if ((lo != 0u && c_lo <= enough) || hi - lo <= 1) break;
        x = lo + ((hi - lo) >> 1);
    }
    T = lo;
    probe = hi;
}

// Steps A-F on the warp's registers.  `u` = this lane's 128 values (0 at indices >= len).
// WIDE: 0 = k <= 128, 1 = k <= 256, 2 = beyond (kernels of their own, so that the common case carries neither the
// code nor the registers of the others)
template <bool GLOBAL, int WIDE>
__device__ __forceinline__ void select_unit(const float (&u)[128], const USource& src, int len, int keff,
                                            unsigned* bitmap, uint16_t* cand, uint16_t* __restrict__ out_idx,
                                            float* __restrict__ out_val) {
    const int lane = threadIdx.x & 31;
    // groups of 16 values up to k = 128 (about 1.15 k candidates); beyond that a threshold taken from 256
    // group maxima lets too many elements through, and groups of 4 take over (WIDE: a kernel of its own,
    // so that the common case carries neither the code nor the registers of the other)
    if (WIDE == 2 && keff > kFastMaxK) {  // beyond 256 of 4096 a threshold over group maxima no longer thins the field
        select_dense<GLOBAL>(u, src, len, keff, bitmap, cand, out_idx, out_val);
        return;
    }
    unsigned T, probe;
    group_threshold<WIDE ? 32 : 8>(u, keff, T, probe);
    if (T == 0u) {  // no usable threshold: exact search over everything
        select_slow<GLOBAL>(src, len, keff, bitmap, out_idx, out_val);
        return;
    }

    // C. candidates: key >= T as "not (|x| < T)" on floats (a NaN, the largest keys, passes)
    const float Tf = __uint_as_float(T);
    unsigned hm[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int q = 0; q < 128; ++q) hm[q >> 5] |= !(fabsf(u[q]) < Tf) ? (1u << (q & 31)) : 0u;
    const unsigned mine = __popc(hm[0]) + __popc(hm[1]) + __popc(hm[2]) + __popc(hm[3]);
    unsigned inc = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned o = __shfl_up_sync(kFull, inc, d);
        if (lane >= d) inc += o;
    }
    const unsigned n_c = __shfl_sync(kFull, inc, 31);
    if (n_c > (unsigned)kCandCap) {
        select_slow<GLOBAL>(src, len, keff, bitmap, out_idx, out_val);
        return;
    }
    {
        unsigned at = inc - mine;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            unsigned mm = hm[w];
            while (mm) {
                const unsigned b = __ffs(mm) - 1;
                mm &= mm - 1;
                cand[at++] = (uint16_t)lane_pos(lane, 32 * w + (int)b);
            }
        }
    }
    __syncwarp();
    if (n_c <= 128u) rank_and_emit<4, GLOBAL>(cand, n_c, T, probe, src, keff, bitmap, out_idx, out_val);
    else rank_and_emit<kCandCap / 32, GLOBAL>(cand, n_c, T, probe, src, keff, bitmap, out_idx, out_val);
}

// DELTA: the "theta_r" buffers hold the vector to compress itself (a local Nesterov direction, a
// momentum: the Top-k baselines of Alg. 2 and 4) instead of parameters to subtract from theta.
template <bool EF, bool PENDING, int WIDE, bool DELTA = false>
__global__ void __launch_bounds__(kSelThreads, 1)
ef_select_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int k, int kp, float beta,
                 const float* __restrict__ theta_sync, WorkerPtrs ptrs, Workspace ws, TmaArgs tma, int use_tma) {
    extern __shared__ __align__(1024) unsigned char dyn_smem[];
    SelSmem& sm = *reinterpret_cast<SelSmem*>(dyn_smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // 32-bit counters: chunks x workers < 2^31 is checked on the host
    const int grid = (int)gridDim.x, first = (int)blockIdx.x;
    const int my_chunks = ((int)n_chunks - first + grid - 1) / grid;  // >= 1: the grid never exceeds n_chunks
    const int n_units = my_chunks * n_workers;
    const unsigned pend_bytes = PENDING ? (unsigned)kp * 6u : 0u;

    if (tid == 0) {
        for (int i = 0; i < kThetaRing; ++i) {
            mbar_init(&sm.full_s[i], 1);
            mbar_init(&sm.empty_s[i], (unsigned)n_workers);
        }
        for (int i = 0; i < kUnitSlots; ++i) {
            mbar_init(&sm.full_u[i], 1);
            mbar_init(&sm.empty_u[i], 1);
        }
        sm.next_unit = 0;
        sm.issued = 0;
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();  // the only CTA-wide barrier: from here on the warps meet through the barriers above
    volatile int* abort_flag = &sm.abort;

    if (warp == kSelWarps) {
        // ------------------------------------------------------------------ producer (one thread)
        if (lane != 0) return;
        if (use_tma && tma.fresh) {
            for (int q = 0; q < tma.n_classes; ++q) {
                tensormap_acquire(tma.maps + tma.slot_s * tma.n_classes + q);
                for (int r = 0; r < n_workers; ++r) {
                    tensormap_acquire(tma.maps + tma.slot_l[r] * tma.n_classes + q);
                    if (EF) tensormap_acquire(tma.maps + tma.slot_e[r] * tma.n_classes + q);
                }
            }
        }
        int c = -1, c_armed = -1, r = n_workers - 1, cls = 0, x1 = 0, x2 = 0;
        bool tile = false;
        long long g = 0;
        int n = 0;
        for (; n < n_units; ++n) {
            if (*abort_flag) break;
            if (++r == n_workers) {  // next chunk: its block of theta
                r = 0;
                ++c;
                g = first + (long long)c * grid;
                const ChunkGeo d = load_geo(chunks + g);
                tile = use_tma && d.len == kChunk;
                const int b = c % kThetaRing;
                if (c >= kThetaRing && !mbar_wait(&sm.empty_s[b], (unsigned)((c / kThetaRing - 1) & 1))) break;
                if (tile) {
                    const int rs = d.row_stride ? d.row_stride : kTile;
                    cls = 0;
                    for (int q = 1; q < tma.n_classes; ++q) cls = tma.class_rs[q] == rs ? q : cls;
                    x2 = (int)(d.base / rs);
                    x1 = (int)(d.base - (long long)x2 * rs) >> 6;
                    if (DELTA) {  // nothing is subtracted from theta: its block is not needed
                        mbar_arrive(&sm.full_s[b]);
                    } else {
                        mbar_arrive_expect_tx(&sm.full_s[b], kChunk * (unsigned)sizeof(float));
                        tma_load_block(sm.theta_s[b], tma.maps + tma.slot_s * tma.n_classes + cls, x1, x2, &sm.full_s[b]);
                    }
                } else {
                    mbar_arrive(&sm.full_s[b]);
                }
                c_armed = c;
            }
            const int s = n % kUnitSlots;
            if (n >= kUnitSlots && !mbar_wait(&sm.empty_u[s], (unsigned)((n / kUnitSlots - 1) & 1))) break;
            const unsigned bytes = (tile ? (EF ? 2u : 1u) * kChunk * (unsigned)sizeof(float) : 0u) + pend_bytes;
            if (bytes) mbar_arrive_expect_tx(&sm.full_u[s], bytes);
            else mbar_arrive(&sm.full_u[s]);
            if (tile) {
                tma_load_block(sm.theta_l[s], tma.maps + tma.slot_l[r] * tma.n_classes + cls, x1, x2, &sm.full_u[s]);
                if (EF) tma_load_block(sm.e[s], tma.maps + tma.slot_e[r] * tma.n_classes + cls, x1, x2, &sm.full_u[s]);
            }
            if (PENDING) {
                const long long slot_base = ((long long)r * n_chunks + g) * kp;  // kp is a multiple of 8
                bulk_load(sm.pend_val[s], ws.val + slot_base, (unsigned)kp * 4u, &sm.full_u[s]);
                bulk_load(sm.pend_idx[s], ws.idx + slot_base, (unsigned)kp * 2u, &sm.full_u[s]);
            }
            // unit n is armed: consumers may now wait on its barriers
            asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(&sm.issued)), "r"(n + 1) : "memory");
        }
        if (n < n_units && !*abort_flag) {  // one of this thread's own waits ran out
            *abort_flag = 1;
            atomicExch(tma.status, (int)SL_ERR_TIMEOUT);
        }
        // Copies still in flight must land before the CTA's shared memory is released: wait (bounded)
        // for the last phase armed on every barrier.  After a complete run these return at once.
        for (int s = 0; s < kUnitSlots && s < n; ++s) {
            const int last = ((n - 1 - s) / kUnitSlots) * kUnitSlots + s;  // last unit issued into slot s
            mbar_wait(&sm.full_u[s], (unsigned)((last / kUnitSlots) & 1));
        }
        for (int b = 0; b < kThetaRing && b <= c_armed; ++b) {
            const int last = ((c_armed - b) / kThetaRing) * kThetaRing + b;
            mbar_wait(&sm.full_s[b], (unsigned)((last / kThetaRing) & 1));
        }
        return;
    }

    // ---------------------------------------------------------------------- consumers
    unsigned* bitmap = sm.bitmap[warp];
    uint16_t* cand = sm.cand[warp];
    while (true) {
        int n = 0;
        if (lane == 0) n = atomicAdd(&sm.next_unit, 1);
        n = __shfl_sync(kFull, n, 0);
        if (n >= n_units || *abort_flag) break;
        const int c = n / n_workers, r = n - c * n_workers;
        const long long g = first + (long long)c * grid;
        const ChunkGeo cd = load_geo(chunks + g);
        const bool full = cd.len == kChunk, tile = use_tma && full;
        const int keff = min(k, cd.len);
        const int s = n % kUnitSlots, b = c % kThetaRing;
        const int rs = cd.row_stride ? cd.row_stride : kTile;
        float* __restrict__ er = EF ? ptrs.e[r] + cd.base : nullptr;

        *reinterpret_cast<uint4*>(&bitmap[4 * lane]) = make_uint4(0u, 0u, 0u, 0u);
        // A parity wait only tells a barrier's current phase from the one before it, and more units can
        // be claimed than slots exist, so a warp first waits until the producer has armed the barriers
        // for this very unit (it publishes the number of units issued); from then on the barriers of
        // the slot and of the theta block are in this unit's phase and the parity is unambiguous.
        bool ok = false;
        for (unsigned it = 0; it < kSpinLimit; ++it) {
            int issued;
            asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(issued) : "r"(smem_u32(&sm.issued)) : "memory");
            if (issued > n) {
                ok = true;
                break;
            }
            if (*abort_flag) break;
            __nanosleep(32);
        }
        if (!ok || !mbar_wait(&sm.full_s[b], (unsigned)((c / kThetaRing) & 1)) ||
            !mbar_wait(&sm.full_u[s], (unsigned)((n / kUnitSlots) & 1))) {
            *abort_flag = 1;
            if (lane == 0) atomicExch(tma.status, (int)SL_ERR_TIMEOUT);
            break;
        }

        if (PENDING && EF) {  // substitute the corrected values of the previous step
            if (tile) {
                for (int j = lane; j < keff; j += 32) {
                    const unsigned p = sm.pend_idx[s][j];
                    if (p < (unsigned)kChunk) sm.e[s][p] = sm.pend_val[s][j];
                }
            } else {  // patch global memory, which the plain loads below read
                for (int j = lane; j < keff; j += 32) {
                    const unsigned p = sm.pend_idx[s][j];
                    if (p < (unsigned)cd.len) er[chunk_elem_offset(cd.row_stride, (int)p)] = sm.pend_val[s][j];
                }
            }
            __syncwarp();
        }

        float u[128];
        // where u can be found again: the error buffer, or (error feedback frozen) this unit's slot
        float* const scratch = sm.theta_l[s];
        if (tile) {
            const float* __restrict__ tsm = sm.theta_s[b];
            const float* tlm = sm.theta_l[s];  // (frozen error feedback writes u back into this block)
            const float* __restrict__ em = sm.e[s];
            float* __restrict__ er_vec = EF ? er + (long long)(lane >> 4) * rs + 4 * (lane & 15) : nullptr;
            const long long er_step = 2ll * rs;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int v = 128 * i + 4 * lane;
                const float4 l = *reinterpret_cast<const float4*>(&tlm[v]);
                float4 x = l;
                if (!DELTA) {
                    const float4 a = *reinterpret_cast<const float4*>(&tsm[v]);
                    x.x = __fsub_rn(a.x, l.x);
                    x.y = __fsub_rn(a.y, l.y);
                    x.z = __fsub_rn(a.z, l.z);
                    x.w = __fsub_rn(a.w, l.w);
                }
                if (EF) {
                    const float4 ev = *reinterpret_cast<const float4*>(&em[v]);
                    x.x = __fmaf_rn(beta, ev.x, x.x);
                    x.y = __fmaf_rn(beta, ev.y, x.y);
                    x.z = __fmaf_rn(beta, ev.z, x.z);
                    x.w = __fmaf_rn(beta, ev.w, x.w);
                    *reinterpret_cast<float4*>(er_vec + i * er_step) = x;
                } else {
                    *reinterpret_cast<float4*>(&scratch[v]) = x;
                }
                u[4 * i + 0] = x.x;
                u[4 * i + 1] = x.y;
                u[4 * i + 2] = x.z;
                u[4 * i + 3] = x.w;
            }
        } else {  // direct unit: plain loads and stores with bounds
            const float* __restrict__ tsp = theta_sync + cd.base;
            const float* __restrict__ tlp = ptrs.theta_local[r] + cd.base;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int p0 = 128 * i + 4 * lane;
                const long long off = chunk_elem_offset(cd.row_stride, p0);
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (p0 + 4 <= cd.len) {
                    const float4 l = *reinterpret_cast<const float4*>(tlp + off);
                    x = l;
                    if (!DELTA) {
                        const float4 a = *reinterpret_cast<const float4*>(tsp + off);
                        x.x = __fsub_rn(a.x, l.x);
                        x.y = __fsub_rn(a.y, l.y);
                        x.z = __fsub_rn(a.z, l.z);
                        x.w = __fsub_rn(a.w, l.w);
                    }
                    if (EF) {
                        const float4 ev = *reinterpret_cast<const float4*>(er + off);
                        x.x = __fmaf_rn(beta, ev.x, x.x);
                        x.y = __fmaf_rn(beta, ev.y, x.y);
                        x.z = __fmaf_rn(beta, ev.z, x.z);
                        x.w = __fmaf_rn(beta, ev.w, x.w);
                        *reinterpret_cast<float4*>(er + off) = x;
                    }
                } else if (p0 < cd.len) {  // the vector that holds the end of a short chunk
                    float t[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (p0 + j < cd.len) {
                            t[j] = DELTA ? tlp[off + j] : __fsub_rn(tsp[off + j], tlp[off + j]);
                            if (EF) {
                                t[j] = __fmaf_rn(beta, er[off + j], t[j]);
                                er[off + j] = t[j];
                            }
                        }
                    }
                    x = make_float4(t[0], t[1], t[2], t[3]);
                }
                if (!EF) *reinterpret_cast<float4*>(&scratch[p0]) = x;
                u[4 * i + 0] = x.x;
                u[4 * i + 1] = x.y;
                u[4 * i + 2] = x.z;
                u[4 * i + 3] = x.w;
            }
        }
        // the blocks are consumed (the slot stays in use as the copy of u when error feedback is frozen)
        if ((PENDING && EF && tile) || !EF) fence_async_smem();  // this lane's writes into the slot
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(&sm.empty_s[b]);
            if (EF) mbar_arrive(&sm.empty_u[s]);
        }

        USource src;
        if (EF) {
            src.ptr = reinterpret_cast<const unsigned*>(er);
            src.rs = rs;
        } else {
            src.ptr = reinterpret_cast<const unsigned*>(scratch);
            src.rs = kTile;
        }
        const long long slot_base = ((long long)r * n_chunks + g) * kp;
        select_unit<EF, WIDE>(u, src, cd.len, keff, bitmap, cand, ws.idx + slot_base, ws.val + slot_base);
        __syncwarp();  // the map and the list are free again
        if (!EF && lane == 0) mbar_arrive(&sm.empty_u[s]);
    }
}

}  // namespace
