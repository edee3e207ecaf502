// SparseLoCo outer step for sm_100a: kernels and the C ABI declared in include/sparseloco.h.
//
// Kernel sequence of one outer step (all on the caller's stream, no host synchronisation):
//   ef_topk_kernel         pseudo-gradient + error feedback + chunk-wise Top-k     (Eq. 2 line 1, Sec. 3.3)
//   chunk_sum_kernel       per-chunk fp64 sum of the selected values               (Sec. 4 quantiser: mean)
//   tensor_reduce_kernel<0>  chunk-ordered fp64 sum per (worker, tensor) -> mu
//   chunk_sum_kernel<1>    per-chunk fp64 sum of squared centred values            (sigma)
//   tensor_reduce_kernel<1>  -> sigma, bin edge 3 sigma
//   chunk_bins_kernel      per-chunk per-bin sums and counts                       (centroids)
//   tensor_reduce_kernel<2>  -> 4-entry table, written to the payload header
//   pack_fix_kernel        codes, 12-bit index + 2-bit code packing, e = u - Dhat   (Eq. 2 line 2)
//   decode_avg_apply_kernel  decode R payloads, sum, theta -= alpha/D * sum         (Eq. 2 lines 3-4)
//
// Everything is HBM-bound streaming except the per-chunk selection, which works on registers and
// shared memory.  No tensor cores: nothing here is a dense contraction.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "sparseloco.h"

namespace {

constexpr int kChunk = 4096;
constexpr int kTile = 64;
constexpr int kThreads = 256;          // threads per CTA of the chunk kernels
constexpr int kPerThread = kChunk / kThreads;  // 16 elements = 4 x float4
constexpr int kMaxR = 64;
constexpr int kMaxK = 256;
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

// Element offset (relative to ChunkDesc::base) of in-chunk index p.
__device__ __forceinline__ long long chunk_elem_offset(int row_stride, int p) {
    return row_stride ? (long long)(p >> 6) * row_stride + (p & 63) : (long long)p;
}

// ------------------------------------------------------------------------------------------------
// Asynchronous 16-byte copies global -> shared (one per thread and vector), grouped per unit.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src_gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src_gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most N of this thread's committed groups are still in flight
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// ------------------------------------------------------------------------------------------------
// Selection: the keff largest of 4096 (magnitude, then lower index), exact.
//
// key = float bits without the sign (31 bits); the order is (key descending, index ascending), so
// every element has a distinct rank and "the keff first" is exactly Top-k with the lowest-index
// tie-break.  Warp w owns in-chunk indices 512 w .. 512 w + 511; lane l of it owns
// p = 512 w + 128 i + 4 l + j, i, j in 0..3.  The 16 values are in registers and, for indexing by a
// run-time position, in the thread's own slots of a shared tile.
//
// 1. every lane takes the maximum key of its 16 values; every warp takes the ceil(keff/8)-th
//    largest of its 32 lane maxima (low 5 bits replaced by the lane number, so that the maxima
//    are distinct and one reduction per round suffices); T = the minimum over the 8 warps,
//    rounded down to a multiple of 32.  At least keff values have key >= T.  (In a short chunk
//    only the ceil(len/512) warps that own elements take part, ceil(keff/that) rounds each.)
// 2. the 8 warp values cluster around the keff-th largest key, so three splitters between their
//    minimum and maximum cut the candidates (key >= T, about 2 keff of them) into four classes.
//    Every candidate is appended to its class list; the class counts say which class holds the
//    cut: classes above it are selected whole, and only that class (some tens of entries) is
//    ranked, by all-pairs counting on (key, index).
// 3. selected entries set their bit in a 4096-bit map; a prefix popcount over the map gives every
//    selected entry its slot in ascending index order, and its owner writes (index, value).
// If T is 0 or a class list overflows (constant chunks, heavy ties, large k) an exact bitwise
// search over all 4096 (key, index) composites finds the keff-th largest instead.
// ------------------------------------------------------------------------------------------------
constexpr int kFetchWarp = 7;    // fetches the pending lists: the warp with the least selection work
constexpr int kClassCap = 224;  // entries per class list (<= threads: one thread per entry suffices)

struct SelectSmem {
    unsigned lkey[4][kClassCap];  // candidates per class: key
    uint16_t lpos[4][kClassCap];  //                        in-chunk index | sign << 12
    unsigned bitmap[2][128];   // selected positions, double-buffered by unit parity
    unsigned warp_t[8];
    unsigned cnt[4];
    unsigned warp_cnt[2][8];
    unsigned n_exact;          // entries the exact search appended
};

__device__ __forceinline__ unsigned long long make_composite(unsigned key, int p) {
    return ((unsigned long long)key << 12) | (unsigned long long)(4095 - p);
}

__device__ __forceinline__ int owned_index(int tid, int q) {
    return 512 * (tid >> 5) + 128 * (q >> 2) + 4 * (tid & 31) + (q & 3);
}

__device__ __forceinline__ void set_bit(unsigned* bitmap, unsigned p) { atomicOr(&bitmap[p >> 5], 1u << (p & 31)); }

// Exact fallback: bitwise search for the keff-th largest composite over all elements; the keff
// elements at or above it are appended to the class lists taken as one array (count in n_exact)
// and marked in the map.
// Contains CTA barriers.  Rare path, kept out of line.
__device__ __noinline__ void select_exact_search(const unsigned* ub, bool nonzero, int len, int keff,
                                                 SelectSmem& sm, unsigned* bitmap) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long res = 0;
    if (tid == 0) sm.n_exact = 0;
    const bool any = __syncthreads_or(nonzero);
    if (any) {
        int buf = 0;
        for (int bit = 42; bit >= 0; --bit) {
            const unsigned long long trial = res | (1ull << bit);
            unsigned c = 0;
            for (int q = 0; q < kPerThread; ++q) {
                const int p = owned_index(tid, q);
                c += (p < len && make_composite(ub[q] & 0x7FFFFFFFu, p) >= trial) ? 1u : 0u;
            }
            c = __reduce_add_sync(kFull, c);
            if (lane == 0) sm.warp_cnt[buf][warp] = c;
            __syncthreads();
            unsigned tot = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w) tot += sm.warp_cnt[buf][w];
            if (tot >= (unsigned)keff) res = trial;
            buf ^= 1;
        }
    } else {
        // all magnitudes are zero: the first keff indices win every tie
        res = make_composite(0u, keff - 1);
    }
    for (int q = 0; q < kPerThread; ++q) {
        const int p = owned_index(tid, q);
        const unsigned key = ub[q] & 0x7FFFFFFFu;
        if (p < len && make_composite(key, p) >= res) {
            const unsigned pos = atomicAdd(&sm.n_exact, 1u);
            if (pos < (unsigned)kMaxK) {  // the four lists taken as one array: room for kMaxK entries
                (&sm.lkey[0][0])[pos] = key;
                (&sm.lpos[0][0])[pos] = (uint16_t)((unsigned)p | ((ub[q] >> 31) << 12));
            }
            set_bit(bitmap, (unsigned)p);
        }
    }
}

// A thread's selected entries: at most two.
struct Picked {
    unsigned p0, v0;  // in-chunk index and value bits: one entry of the cut class
    unsigned p1, v1;  // one entry of the classes above the cut
    unsigned mask;    // bit i: entry i is selected
};

// First half of the selection: threshold and class lists.  `ub` = the thread's 16 value bit patterns
// (0 at in-chunk indices >= the chunk length); `tile` = the shared tile holding the same values (only
// the thread's own slots are read).  Contains one CTA barrier: every thread of the CTA must call
// it, and must synchronise again before select_rank().  Returns true when the threshold is 0, in
// which case nothing was listed and the exact search has to run instead.
__device__ __forceinline__ bool select_topk(const unsigned (&ub)[kPerThread], const unsigned* __restrict__ tile,
                                            int len, int keff, SelectSmem& sm, Picked& out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    out.mask = 0;

    // -- 1. threshold.  The lane maximum is taken on floats (|x|; a NaN is skipped, which can only
    // lower T); keys of non-NaN values order like their magnitudes.
    float mf = 0.0f;
#pragma unroll
    for (int q = 0; q < kPerThread; q += 2)
        mf = fmaxf(mf, fmaxf(fabsf(__uint_as_float(ub[q])), fabsf(__uint_as_float(ub[q + 1]))));
    const unsigned m = __float_as_uint(mf);
    // warps whose 512 indices lie beyond a short chunk have nothing to offer: the others share keff
    const int n_warps = min(8, (len + 511) >> 9);
    {
        // more than 32 rounds cannot be served by 32 lanes: tw ends as 0 and the exact search takes over
        const int rounds = n_warps == 8 ? (keff + 7) >> 3 : min(33, (keff + n_warps - 1) / n_warps);
        unsigned cur = (m & ~31u) | (unsigned)lane, tw = 0;
        for (int i = 0; i < rounds; ++i) {
            tw = __reduce_max_sync(kFull, cur);
            cur = cur == tw ? 0u : cur;  // retire the holder (tagged values are distinct, or all 0)
        }
        if (lane == 0) sm.warp_t[warp] = warp < n_warps ? (tw & ~31u) : 0xFFFFFFFFu;
        if (tid < 4) sm.cnt[tid] = 0;
    }
    __syncthreads();
    unsigned T, s1, s2, s3;
    {
        const uint4 a = *reinterpret_cast<const uint4*>(&sm.warp_t[0]);
        const uint4 b = *reinterpret_cast<const uint4*>(&sm.warp_t[4]);
        const unsigned lo = min(min(min(a.x, a.y), min(a.z, a.w)), min(min(b.x, b.y), min(b.z, b.w)));
        unsigned hi, mean;
        if (n_warps == 8) {
            hi = max(max(max(a.x, a.y), max(a.z, a.w)), max(max(b.x, b.y), max(b.z, b.w)));
            mean = (a.x >> 3) + (a.y >> 3) + (a.z >> 3) + (a.w >> 3) + (b.x >> 3) + (b.y >> 3) + (b.z >> 3) +
                   (b.w >> 3);
        } else {  // short chunk: any splitters do; take them between the extremes of the warps that count
            hi = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w) hi = max(hi, w < n_warps ? sm.warp_t[w] : 0u);
            mean = (lo >> 1) + (hi >> 1);
        }
        T = lo;
        s2 = max(mean, lo);
        s1 = (lo >> 1) + (s2 >> 1);
        s3 = (s2 >> 1) + (hi >> 1);
    }

    bool exact = T == 0;  // uniform over the CTA
    if (!exact) {
        // -- 2. candidates into class lists.  key >= T as "not (|x| < T)" on floats: T is the bit
        // pattern of a non-negative non-NaN float and a NaN (the largest keys) passes the test.
        unsigned hits = 0;
        const float Tf = __uint_as_float(T);
#pragma unroll
        for (int q = 0; q < kPerThread; ++q) hits |= !(fabsf(__uint_as_float(ub[q])) < Tf) ? (1u << q) : 0u;
        while (hits) {
            const int b = 31 - __clz(hits);
            hits &= ~(1u << b);
            const int p = owned_index(tid, b);
            const unsigned bits = tile[p];
            const unsigned kq = bits & 0x7FFFFFFFu;
            const unsigned cls = (kq >= s1 ? 1u : 0u) + (kq >= s2 ? 1u : 0u) + (kq >= s3 ? 1u : 0u);
            const unsigned pos = atomicAdd(&sm.cnt[cls], 1u);
            if (pos < kClassCap) {
                sm.lkey[cls][pos] = kq;
                sm.lpos[cls][pos] = (uint16_t)((unsigned)p | ((bits >> 31) << 12));
            }
        }
    }
    return exact;
}

// Second half of the selection, after the barrier that completes the class lists.  Returns true
// when a list overflowed: nothing was marked and the exact search has to run instead.
__device__ __forceinline__ bool select_rank(int keff, SelectSmem& sm, unsigned* bitmap, Picked& out) {
    const int tid = threadIdx.x;
    const uint4 cn = *reinterpret_cast<const uint4*>(&sm.cnt[0]);
    // the class holding the cut: the highest class c with count(classes >= c) >= keff
    unsigned above = 0, cstar = 3, L = cn.w;
    if (cn.w < (unsigned)keff) {
        above = cn.w; cstar = 2; L = cn.z;
        if (above + cn.z < (unsigned)keff) {
            above += cn.z; cstar = 1; L = cn.y;
            if (above + cn.y < (unsigned)keff) { above += cn.y; cstar = 0; L = cn.x; }
        }
    }
    if (max(max(cn.x, cn.y), max(cn.z, cn.w)) > (unsigned)kClassCap) return true;  // overflow: exact search
    const unsigned want = (unsigned)keff - above;  // 1 <= want <= L
    // classes above the cut are selected whole: `above` (< keff <= 256) entries, one per thread
    if (tid < (int)above) {
        unsigned c = 3, j = tid;
        if (j >= cn.w) {
            j -= cn.w;
            c = 2;
            if (j >= cn.z) {
                j -= cn.z;
                c = 1;
            }
        }
        out.p1 = sm.lpos[c][j];
        out.v1 = sm.lkey[c][j] | ((out.p1 >> 12) << 31);
        out.p1 &= 0xFFFu;
        out.mask |= 2u;
        set_bit(bitmap, out.p1);
    }
    // the cut class: entry i = tid >> sh is ranked by 2^sh adjacent lanes, each over one segment
    const unsigned* __restrict__ lk = sm.lkey[cstar];
    const uint16_t* __restrict__ lp = sm.lpos[cstar];
    unsigned sh = 0;
    while (sh < 3 && (L << (sh + 1)) <= 32u) ++sh;
    const unsigned i = tid >> sh, seg = tid & ((1u << sh) - 1u);
    const unsigned seglen = (L + (1u << sh) - 1u) >> sh;
    unsigned beat = 0, mp = 0, mk = 0, msign = 0;
    if (i < L) {
        mk = lk[i];
        mp = lp[i];
        msign = mp >> 12;
        mp &= 0xFFFu;
        const unsigned j0 = seg * seglen, j1 = min(j0 + seglen, L);
        for (unsigned j = j0; j < j1; ++j) {
            const unsigned ok = lk[j], op = lp[j] & 0xFFFu;
            beat += (ok > mk || (ok == mk && op < mp)) ? 1u : 0u;
        }
    }
    for (unsigned d = 1; d < (1u << sh); d <<= 1) beat += __shfl_xor_sync(kFull, beat, d);
    if (i < L && seg == 0 && beat < want) {
        out.p0 = mp;
        out.v0 = mk | (msign << 31);
        out.mask |= 1u;
        set_bit(bitmap, mp);
    }
    return false;
}

// Writes the thread's selected entries to their slots (ascending in-chunk index).  Every lane of a
// warp must call this together.  Reads the completed map.
__device__ __forceinline__ void emit_picked(const Picked& pk, const unsigned* __restrict__ bitmap, int keff,
                                            uint16_t* __restrict__ out_idx, float* __restrict__ out_val) {
    const int lane = threadIdx.x & 31;
    if (!__any_sync(kFull, pk.mask != 0)) return;
    // this lane's packed prefix: exclusive count before its 4 words | popcounts of its first three words
    unsigned pack;
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
    auto write_one = [&](bool active, unsigned pos, unsigned bits) {
        if (!__any_sync(kFull, active)) return;
        const unsigned p = active ? pos : 0u, w = p >> 5;
        const unsigned pq = __shfl_sync(kFull, pack, w >> 2);
        if (active) {
            const unsigned sub = w & 3u;
            unsigned before = pq & 0x1FFFu;
            if (sub > 0) before += (pq >> 13) & 0x3Fu;
            if (sub > 1) before += (pq >> 19) & 0x3Fu;
            if (sub > 2) before += (pq >> 25) & 0x3Fu;
            const unsigned slot = before + __popc(bitmap[w] & ((1u << (p & 31)) - 1u));
            if (slot < (unsigned)keff) {
                out_idx[slot] = (uint16_t)p;
                out_val[slot] = __uint_as_float(bits);
            }
        }
    };
    write_one(pk.mask & 1u, pk.p0, pk.v0);
    write_one(pk.mask & 2u, pk.p1, pk.v1);
}

// ------------------------------------------------------------------------------------------------
// Kernel 1: u = beta e + (theta - theta_r) written into e, chunk-wise Top-k of u into staging.
//
// Persistent CTAs (three per SM).  CTA b takes chunks b, b + grid, ... and, for each, the R workers
// in turn ("units"), so the chunk of theta_sync is fetched once per chunk and kept in registers.
// theta_r and e of a unit travel global -> shared as asynchronous 16-byte copies issued two units
// ahead (two stages); every thread copies exactly the vectors it will consume itself, so no barrier
// guards their arrival.  u is formed in registers, stored to e with 128-bit stores and kept in the
// e stage for the selection.  Short tail chunks take plain loads.
//
// PENDING: the error buffers hold u of the previous step and the corrected values (u - Dhat) of the
// selected entries wait in the staging arrays (deferred error-feedback subtraction).  The lists of
// the next units ride along three units ahead; before u is formed every warp substitutes the
// entries that fall into its 512 indices (the lists are sorted, so they form one run).
// ------------------------------------------------------------------------------------------------
struct PipeSmem {
    float theta_l[2][kChunk];
    float e[2][kChunk];  // e on arrival, u after the update
    SelectSmem sel;
    __align__(16) float pend_val[3][kMaxK];
    __align__(16) uint16_t pend_idx[3][kMaxK];
    unsigned long long full_bar[2];  // TMA variant: the stage's tiles have landed
    int abort;                       // TMA variant: a bounded wait ran out
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

template <bool EF, bool PENDING, bool TMA>
__global__ void __launch_bounds__(kThreads, 3)
ef_topk_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int k, int kp, float beta,
               const float* __restrict__ theta_sync, WorkerPtrs ptrs, Workspace ws, TmaArgs tma) {
    extern __shared__ __align__(1024) unsigned char dyn_smem[];
    PipeSmem& sm = *reinterpret_cast<PipeSmem*>(dyn_smem);
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
        mbar_init(&sm.full_bar[0], 1);
        mbar_init(&sm.full_bar[1], 1);
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
    // arms the stage barrier for one unit and starts its theta_r block (a short chunk moves nothing)
    auto tma_begin_unit = [&](int s, const ChunkGeo& d, int r) {
        unsigned long long* bar = &sm.full_bar[s];
        if (d.len != kChunk) {
            mbar_arrive(bar);
            return;
        }
        mbar_arrive_expect_tx(bar, (EF ? 2u : 1u) * kChunk * (unsigned)sizeof(float));
        tma_load_block(sm.theta_l[s], tma.maps + tma.slot_l[r] * tma.n_classes + d.cls, d.x1, d.x2, bar);
    };
    // the e block of a unit begun earlier
    auto tma_load_e = [&](int s, const ChunkGeo& d, int r) {
        if (!EF || d.len != kChunk) return;
        tma_load_block(sm.e[s], tma.maps + tma.slot_e[r] * tma.n_classes + d.cls, d.x1, d.x2, &sm.full_bar[s]);
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
            tma_begin_unit(0, cd, 0);
            tma_load_e(0, cd, 0);
            if (n_units > 1) {
                tma_begin_unit(1, n_workers > 1 ? cd : cd1, n_workers > 1 ? 1 : 0);
                tma_load_e(1, n_workers > 1 ? cd : cd1, n_workers > 1 ? 1 : 0);
            }
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
        if (TMA && !mbar_wait(&sm.full_bar[s], (unsigned)((n >> 1) & 1))) sm.abort = 1;

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
                const float4 l = *reinterpret_cast<const float4*>(&sm.theta_l[s][v]);
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
        bool exact = select_topk(ub, reinterpret_cast<const unsigned*>(tile), cd.len, keff, sm.sel, pk);
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
                if (have2) tma_begin_unit(s, d2, r2);  // the theta_r stage was last read before that barrier
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
            exact = select_rank(keff, sm.sel, bitmap, pk);
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
            for (int u = n; u < n + 2 && u < n_units; ++u) mbar_wait(&sm.full_bar[u & 1], (unsigned)((u >> 1) & 1));
        }
        if (tid == kTmaThread) bulk_wait_all();
    }
}

// ------------------------------------------------------------------------------------------------
// Quantiser statistics (Sec. 4).  The summation order is part of the definition of the payload
// bits: fp64, in three levels, each left to right: the slots of a chunk, the chunks of a group of 64
// consecutive chunks of the tensor, the groups.
// ------------------------------------------------------------------------------------------------

// Visits the keff staged values of one unit in slot order: four 128-bit loads in flight at a time.
template <typename F>
__device__ __forceinline__ void for_each_staged(const float* __restrict__ v, int keff, F f) {
    int s0 = 0;
    for (; s0 + 16 <= keff; s0 += 16) {
        float4 x[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) x[q] = __ldcs(reinterpret_cast<const float4*>(v + s0) + q);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            f(x[q].x);
            f(x[q].y);
            f(x[q].z);
            f(x[q].w);
        }
    }
    for (; s0 < keff; ++s0) f(v[s0]);
}

// (worker, chunk) of work item i; chunks x workers < 2^31 (checked on the host)
__device__ __forceinline__ void split_unit(long long i, long long n_chunks, int& r, int& g) {
    const unsigned ui = (unsigned)i, nc = (unsigned)n_chunks;
    r = (int)(ui / nc);
    g = (int)(ui - (unsigned)r * nc);
}

// mode 0: sum of values; mode 1: sum of squared fp32-centred values.  One thread per (worker, chunk).
template <int MODE>
__global__ void __launch_bounds__(128)
chunk_sum_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors,
                 int k, int kp, Workspace ws) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks * n_workers) return;
    int r, g;
    split_unit(i, n_chunks, r, g);
    const int keff = min(k, chunks[g].len);
    const float* __restrict__ v = ws.val + i * kp;
    float mu = 0.0f;
    if (MODE == 1) mu = ws.tstat[(long long)r * n_tensors + chunks[g].tensor].mu;
    double acc = 0.0;
    for_each_staged(v, keff, [&](float x) {
        if (MODE == 0) {
            acc += (double)x;
        } else {
            const double d = (double)__fsub_rn(x, mu);
            acc += d * d;  // d*d is exact in fp64, so fusing or not gives the same sum
        }
    });
    ws.psum[i] = acc;
}

// Per-bin sums and counts of one chunk.  codes: (cen >= -t) + (cen >= 0) + (cen >= t).
__device__ __forceinline__ int quant_code(float v, float mu, float t3) {
    const float cen = __fsub_rn(v, mu);
    return (cen >= -t3 ? 1 : 0) + (cen >= 0.0f ? 1 : 0) + (cen >= t3 ? 1 : 0);
}

__global__ void __launch_bounds__(128)
chunk_bins_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors,
                  int k, int kp, Workspace ws) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks * n_workers) return;
    int r, g;
    split_unit(i, n_chunks, r, g);
    const int keff = min(k, chunks[g].len);
    const float* __restrict__ v = ws.val + i * kp;
    const TStat st = ws.tstat[(long long)r * n_tensors + chunks[g].tensor];
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    unsigned n0 = 0, n1 = 0, n2 = 0, n3 = 0;
    for_each_staged(v, keff, [&](float x) {
        const int c = quant_code(x, st.mu, st.t3);
        const double d = (double)x;
        // add only to the value's own bin (adding +0 elsewhere could flip a -0 sum); nearly all
        // selected values sit in the two inner bins, so the branches diverge two ways at most
        if (c == 1) { s1 += d; ++n1; }
        else if (c == 2) { s2 += d; ++n2; }
        else if (c == 0) { s0 += d; ++n0; }
        else { s3 += d; ++n3; }
    });
    double2* pb = reinterpret_cast<double2*>(ws.pbin + i * 4);
    pb[0] = make_double2(s0, s1);
    pb[1] = make_double2(s2, s3);
    *reinterpret_cast<uint4*>(ws.pcnt + i * 4) = make_uint4(n0, n1, n2, n3);
}

// One warp per (worker, tensor): the chunk partials are added group by group (64 consecutive chunks
// per group, left to right inside the group: one lane per group, 32 groups at a time), then the
// group sums are added left to right.
// STAGE 0: psum -> mu.  STAGE 1: psum -> sigma, 3 sigma.  STAGE 2: pbin/pcnt -> table (+ payload header).
constexpr int kSumGroup = 64;

template <int STAGE>
__global__ void __launch_bounds__(128)
tensor_reduce_kernel(const TensorInfo* __restrict__ tinfo, long long n_chunks, int n_workers, int n_tensors,
                     Workspace ws, WorkerPtrs ptrs) {
    constexpr int NV = STAGE < 2 ? 1 : 4;  // running sums
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * 4 + wib;
    if (w >= (long long)n_workers * n_tensors) return;
    const int r = (int)(w / n_tensors), t = (int)(w - (long long)r * n_tensors);
    const TensorInfo ti = tinfo[t];
    const long long first = (long long)r * n_chunks + ti.first_chunk;
    TStat* st = ws.tstat + (long long)r * n_tensors + t;
    const double n = (double)ti.n_slots;
    const long long n_groups = (ti.n_chunks + kSumGroup - 1) / kSumGroup;

    double acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = 0.0;
    unsigned long long cn[4] = {0, 0, 0, 0};
    for (long long g0 = 0; g0 < n_groups; g0 += 32) {
        // this lane's group
        double gs[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) gs[v] = 0.0;
        const long long c0 = (g0 + lane) * kSumGroup;
        const int cnt = (int)max(0ll, min((long long)kSumGroup, ti.n_chunks - c0));
        if (STAGE < 2) {
            const double* __restrict__ src = ws.psum + first + c0;
            int c = 0;
            for (; c + 8 <= cnt; c += 8) {
                double x[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) x[q] = src[c + q];
#pragma unroll
                for (int q = 0; q < 8; ++q) gs[0] += x[q];
            }
            for (; c < cnt; ++c) gs[0] += src[c];
        } else {
            const double2* __restrict__ src = reinterpret_cast<const double2*>(ws.pbin + (first + c0) * 4);
            const uint4* __restrict__ csrc = reinterpret_cast<const uint4*>(ws.pcnt + (first + c0) * 4);
            int c = 0;
            for (; c + 4 <= cnt; c += 4) {  // loads of four chunks in flight, additions in chunk order
                double2 lo[4], hi[4];
                uint4 pc[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    lo[q] = src[2 * (c + q)];
                    hi[q] = src[2 * (c + q) + 1];
                    pc[q] = csrc[c + q];
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    gs[0] += lo[q].x; gs[1 % NV] += lo[q].y; gs[2 % NV] += hi[q].x; gs[3 % NV] += hi[q].y;
                    cn[0] += pc[q].x; cn[1] += pc[q].y; cn[2] += pc[q].z; cn[3] += pc[q].w;
                }
            }
            for (; c < cnt; ++c) {
                const double2 lo = src[2 * c], hi = src[2 * c + 1];
                gs[0] += lo.x; gs[1 % NV] += lo.y; gs[2 % NV] += hi.x; gs[3 % NV] += hi.y;
                const uint4 pc = csrc[c];
                cn[0] += pc.x; cn[1] += pc.y; cn[2] += pc.z; cn[3] += pc.w;
            }
        }
        // the group sums of these 32 groups, in group order (every lane runs the same chain)
        const int ng = (int)min(32ll, n_groups - g0);
        for (int l = 0; l < ng; ++l) {
#pragma unroll
            for (int v = 0; v < NV; ++v) acc[v] += __shfl_sync(kFull, gs[v], l);
        }
    }

    if (STAGE < 2) {
        if (lane == 0) {
            if (STAGE == 0) {
                st->mu = (float)(acc[0] / n);
            } else {
                const float sigma = (float)sqrt(acc[0] / n);
                st->sigma = sigma;
                st->t3 = __fmul_rn(3.0f, sigma);
            }
        }
    } else {
#pragma unroll
        for (int bb = 0; bb < 4; ++bb) {
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) cn[bb] += __shfl_xor_sync(kFull, cn[bb], d);
        }
        if (lane == 0) {
            float lut[4];
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) lut[bb] = cn[bb] ? (float)(acc[bb % NV] / (double)cn[bb]) : 0.0f;
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) st->lut[bb] = lut[bb];
            st->pad = 0.0f;
            float4* hdr = reinterpret_cast<float4*>(ptrs.payload[r] + 16ll * t);
            *hdr = make_float4(lut[0], lut[1], lut[2], lut[3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Pack + error-feedback subtract.  One warp per (worker, chunk): codes from (mu, 3 sigma), 12-bit
// indices and 2-bit codes OR-ed into a shared-memory record, record written as 16-byte vectors,
// e[index] = value - table[code] at the selected positions (Eq. 2 line 2).
// ------------------------------------------------------------------------------------------------
// MODE 0: records only (error feedback frozen).  MODE 1: e[index] = value - table[code].
// MODE 2: the corrected value replaces the staged value instead (deferred subtraction).
template <int MODE>
__global__ void __launch_bounds__(128)
pack_fix_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_workers, int n_tensors,
                int k, int kp, Workspace ws, WorkerPtrs ptrs) {
    __shared__ __align__(16) unsigned rec[4][(record_stride(kMaxK) / 4) + 4];
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
            float* er = ptrs.e[r] + cd.base + chunk_elem_offset(cd.row_stride, (int)p);
            *er = __fsub_rn(v, st.lut[c]);
        }
        if (MODE == 2) ws.val[slot_base + s] = __fsub_rn(v, st.lut[c]);
    }
    __syncwarp();
    uint4* dst = reinterpret_cast<uint4*>(ptrs.payload[r] + cd.rec_off);
    const uint4* src = reinterpret_cast<const uint4*>(rec[warp]);
    for (int w = lane; w < stride / 16; w += 32) dst[w] = src[w];
}

// Writes the corrected values waiting in the staging arrays into the error buffers (deferred
// subtraction made good).  One warp per (worker, chunk).
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
        if (p < (unsigned)cd.len) ptrs.e[r][cd.base + chunk_elem_offset(cd.row_stride, (int)p)] = ws.val[slot_base + s];
    }
}

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
    constexpr int kEnt = SPL * WPW;  // entries per thread and batch
    static_assert(kEnt <= kApplyEntries && WPW <= 4, "entry budget");
    constexpr int batch = 8 * WPW;
    const int vec_per_rec = stride / 16;

    for (int r0 = 0; r0 < n_workers; r0 += batch) {
        const int nb = min(batch, n_workers - r0);
        unsigned pre_p[kEnt];
        float pre_v[kEnt];
#pragma unroll
        for (int e = 0; e < kEnt; ++e) {
            pre_p[e] = 0u;
            pre_v[e] = 0.f;
        }
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
            // staged (index, value) pairs of this thread's entries: loads in flight across the barrier
#pragma unroll
            for (int wi = 0; wi < WPW; ++wi) {
                const int rb = warp + 8 * wi;
                const long long slot_base = ((long long)(r0 + rb) * fa.n_chunks + blockIdx.x) * fa.kp;
#pragma unroll
                for (int si = 0; si < SPL; ++si) {
                    const int sl = lane + 32 * si;
                    if (rb < nb && sl < keff) {
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

// ================================================================================================
// Entropy-coded index format (sl_encode_payload / sl_decode_payload)
//
// App. "Compression of indices" prices the naive format at 12 bits per index and reports 8.9 / 6.6 /
// 5.6 bits from a scheme it does not describe.  This is the library's own: per chunk, the gaps
// between consecutive selected indices in Golomb codes (unary quotient, truncated-binary remainder,
// divisor 0.693 x the mean gap), chunk after chunk in one bit stream, with the bit offset of every
// 16th chunk in a directory so that decoding runs in parallel.  The exact layout is in the header.
// ================================================================================================
namespace {

constexpr int kIxcGroup = 16;  // chunks per directory entry

struct IxcCode {  // Golomb parameters of a chunk of length L with m selected entries
    unsigned M, b, cut;
};
__host__ __device__ inline IxcCode ixc_code(int L, int m) {
    IxcCode c;
    const long long M = (693ll * (L - m) + 500ll * (m + 1)) / (1000ll * (m + 1));
    c.M = M < 1 ? 1u : (unsigned)M;
    c.b = 0;
    while ((1u << c.b) < c.M) ++c.b;
    c.cut = (1u << c.b) - c.M;
    return c;
}
// bits of the code of gap g
__device__ __forceinline__ unsigned ixc_code_bits(unsigned g, const IxcCode& c) {
    const unsigned q = g / c.M, r = g - q * c.M;
    return q + 1u + (c.M > 1u ? (r < c.cut ? c.b - 1u : c.b) : 0u);
}
// worst case of a chunk: one zero-bit and at most b remainder bits per value; the quotients
// together cannot exceed (L - m) / M
__host__ __device__ inline long long ixc_worst_bits(int L, int m) {
    const IxcCode c = ixc_code(L, m);
    return (long long)m * (c.b + 1) + (L - m) / c.M;
}

// K1: bits of every chunk's codes.  One thread per chunk.
__global__ void __launch_bounds__(128)
ixc_len_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int k, const uint8_t* __restrict__ payload,
               unsigned* __restrict__ lens) {
    const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_chunks) return;
    const ChunkDesc cd = chunks[g];
    const int m = min(k, cd.len);
    const IxcCode c = ixc_code(cd.len, m);
    const unsigned* rec = reinterpret_cast<const unsigned*>(payload + cd.rec_off);
    unsigned bits = 0;
    int prev = -1;
    for (int s = 0; s < m; ++s) {
        const int bit = 12 * s;
        const unsigned lo = rec[bit >> 5], hi = (bit & 31) > 20 ? rec[(bit >> 5) + 1] : 0u;
        const int p = (int)(__funnelshift_r(lo, hi, bit & 31) & 0xFFFu);
        const int gap = p - prev - 1;
        prev = p;
        bits += ixc_code_bits(gap < 0 ? 0u : (unsigned)gap, c);  // a malformed record cannot run away
    }
    lens[g] = bits;
}

// K2: exclusive prefix sum of the lengths (one block walks the array), directory, total size.
__global__ void __launch_bounds__(1024)
ixc_scan_kernel(const unsigned* __restrict__ lens, long long n_chunks, unsigned* __restrict__ offs,
                unsigned* __restrict__ dir, unsigned long long stream_off, unsigned long long* coded_bytes) {
    __shared__ unsigned warp_sum[32];
    __shared__ unsigned long long carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (long long base = 0; base < n_chunks; base += 1024) {
        const long long g = base + tid;
        const unsigned x = g < n_chunks ? lens[g] : 0u;
        unsigned inc = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned o = __shfl_up_sync(kFull, inc, d);
            if (lane >= d) inc += o;
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            unsigned w = warp_sum[lane], winc = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned o = __shfl_up_sync(kFull, winc, d);
                if (lane >= d) winc += o;
            }
            warp_sum[lane] = winc - w;  // exclusive over warps
        }
        __syncthreads();
        const unsigned long long carry = carry_s;
        const unsigned long long off = carry + warp_sum[warp] + (inc - x);
        if (g < n_chunks) {
            offs[g] = (unsigned)off;
            if ((g % kIxcGroup) == 0) dir[g / kIxcGroup] = (unsigned)off;
        }
        __syncthreads();
        if (tid == 1023) carry_s = off + x;
        __syncthreads();
    }
    if (tid == 0) {
        const unsigned long long bytes = stream_off + (carry_s + 7) / 8;
        *coded_bytes = (bytes + 15) / 16 * 16;
    }
}

// K3: tables, code blocks and the index stream (which must be zero on entry: chunks share words).
// One thread per chunk.
__global__ void __launch_bounds__(128)
ixc_write_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_tensors, int k,
                 const uint8_t* __restrict__ payload, const unsigned* __restrict__ offs, uint8_t* __restrict__ coded,
                 unsigned long long stream_off) {
    const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (g < 4ll * n_tensors)  // the tables, one 32-bit word per thread
        reinterpret_cast<unsigned*>(coded)[g] = reinterpret_cast<const unsigned*>(payload)[g];
    if (g >= n_chunks) return;
    const ChunkDesc cd = chunks[g];
    const int m = min(k, cd.len);
    const IxcCode c = ixc_code(cd.len, m);
    const int cb = (2 * k + 7) / 8, ib = (12 * k + 7) / 8;
    const uint8_t* recb = payload + cd.rec_off;
    uint8_t* cdst = coded + 16ll * n_tensors + (long long)cb * g;
    for (int i = 0; i < cb; ++i) cdst[i] = recb[ib + i];

    const unsigned* rec = reinterpret_cast<const unsigned*>(recb);
    unsigned* stream = reinterpret_cast<unsigned*>(coded + stream_off);  // stream_off is a multiple of 4
    unsigned long long pos = offs[g];
    unsigned long long acc = 0;  // bits not yet written, lowest first; `fill` of them are valid
    unsigned fill = (unsigned)(pos & 31);
    unsigned long long word = pos >> 5;
    auto put = [&](unsigned bits, unsigned n) {  // n <= 32 bits, lowest first
        acc |= (unsigned long long)bits << fill;
        fill += n;
        if (fill >= 32) {
            atomicOr(&stream[word++], (unsigned)acc);
            acc >>= 32;
            fill -= 32;
        }
    };
    int prev = -1;
    for (int s = 0; s < m; ++s) {
        const int bit = 12 * s;
        const unsigned lo = rec[bit >> 5], hi = (bit & 31) > 20 ? rec[(bit >> 5) + 1] : 0u;
        const int p = (int)(__funnelshift_r(lo, hi, bit & 31) & 0xFFFu);
        const unsigned gap = p - prev - 1 < 0 ? 0u : (unsigned)(p - prev - 1);
        prev = p;
        unsigned q = gap / c.M;
        const unsigned r = gap - q * c.M;
        for (; q >= 32; q -= 32) put(0xFFFFFFFFu, 32);
        put((1u << q) - 1u, q + 1);  // q one-bits, then the zero-bit
        if (c.M > 1) {
            const unsigned nb = r < c.cut ? c.b - 1 : c.b, v = r < c.cut ? r : r + c.cut;
            if (nb) put(__brev(v) >> (32 - nb), nb);  // most significant bit first
        }
    }
    if (fill) atomicOr(&stream[word], (unsigned)acc);
}

// K4: coded payload -> 12-bit records.  One thread per group of 16 chunks (one directory entry).
__global__ void __launch_bounds__(128)
ixc_decode_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_tensors, int k,
                  const uint8_t* __restrict__ coded, unsigned long long dir_off, unsigned long long stream_off,
                  uint8_t* __restrict__ payload) {
    const long long grp = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (grp < 4ll * n_tensors)
        reinterpret_cast<unsigned*>(payload)[grp] = reinterpret_cast<const unsigned*>(coded)[grp];
    const long long g0 = grp * kIxcGroup;
    if (g0 >= n_chunks) return;
    const unsigned* stream = reinterpret_cast<const unsigned*>(coded + stream_off);
    unsigned long long pos = reinterpret_cast<const unsigned*>(coded + dir_off)[grp];
    const int cb = (2 * k + 7) / 8, ib = (12 * k + 7) / 8, stride = record_stride(k);
    auto get1 = [&]() -> unsigned {
        const unsigned bit = (stream[pos >> 5] >> (pos & 31)) & 1u;
        ++pos;
        return bit;
    };
    for (long long g = g0; g < g0 + kIxcGroup && g < n_chunks; ++g) {
        const ChunkDesc cd = chunks[g];
        const int m = min(k, cd.len);
        const IxcCode c = ixc_code(cd.len, m);
        uint8_t* recb = payload + cd.rec_off;
        unsigned* rec = reinterpret_cast<unsigned*>(recb);
        // the record is this thread's alone: index words are assembled in a register and stored
        unsigned long long acc = 0;
        unsigned fill = 0;
        int w = 0, prev = -1;
        for (int s = 0; s < m; ++s) {
            unsigned q = 0;
            while (get1() && q < 4096u) ++q;  // a corrupted stream cannot run away
            unsigned r = 0;
            if (c.M > 1) {
                for (unsigned i = 0; i + 1 < c.b; ++i) r = (r << 1) | get1();
                if (r >= c.cut) r = ((r << 1) | get1()) - c.cut;
            }
            prev = prev + 1 + (int)(q * c.M + r);
            acc |= (unsigned long long)((unsigned)prev & 0xFFFu) << fill;
            fill += 12;
            if (fill >= 32) {
                rec[w++] = (unsigned)acc;
                acc >>= 32;
                fill -= 32;
            }
        }
        // rest of the index block, the code block, the padding: byte-wise after the whole words
        int byte = 4 * w;
        for (; byte < ib; ++byte, acc >>= 8) recb[byte] = (uint8_t)(acc & 0xFFu);
        const uint8_t* csrc = coded + 16ll * n_tensors + (long long)cb * g;
        for (int i = 0; i < cb; ++i) recb[ib + i] = csrc[i];
        for (byte = ib + cb; byte < stride; ++byte) recb[byte] = 0;
    }
}

}  // namespace

// ================================================================================================
// Dense baseline: DiLoCo's outer step (Eq. 1), for comparison on the same buffers.
//   Dbar = (1/R) sum_r (theta - theta_r);  m = beta m + Dbar;  theta = theta - alpha (Dbar + beta m)
// One CTA per chunk of the table (so exactly the table's elements are touched), 16 elements per
// thread, all R + 2 streams of a thread's vector in flight together.  fp32: differences and their
// sum in ascending r, one division by R, two fused multiply-adds.
// ================================================================================================
namespace {

struct LocalPtrs {
    const float* p[kMaxR];
};

__device__ __forceinline__ float diloco_elem(float th, float acc, float inv_r_num, float beta, float alpha, float& m) {
    const float dbar = __fdiv_rn(acc, inv_r_num);
    m = __fmaf_rn(beta, m, dbar);
    return __fmaf_rn(-alpha, __fmaf_rn(beta, m, dbar), th);
}

__global__ void __launch_bounds__(kThreads)
diloco_step_kernel(const ChunkDesc* __restrict__ chunks, int n_workers, float beta, float alpha,
                   float* __restrict__ theta, LocalPtrs loc, float* __restrict__ mom) {
    const ChunkDesc cd = chunks[blockIdx.x];
    const int tid = threadIdx.x;
    const float fr = (float)n_workers;
    if (cd.len == kChunk) {
        const int rs = cd.row_stride ? cd.row_stride : kTile;
        const long long off0 = cd.base + (long long)(tid >> 4) * rs + (4 * tid & 63), step = 16ll * rs;
#pragma unroll 1
        for (int i = 0; i < 4; ++i) {
            const long long off = off0 + i * step;
            const float4 th = *reinterpret_cast<const float4*>(theta + off);
            float4 m = *reinterpret_cast<const float4*>(mom + off);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
            for (int r = 0; r < n_workers; ++r) {
                const float4 l = __ldcs(reinterpret_cast<const float4*>(loc.p[r] + off));
                acc.x = __fadd_rn(acc.x, __fsub_rn(th.x, l.x));
                acc.y = __fadd_rn(acc.y, __fsub_rn(th.y, l.y));
                acc.z = __fadd_rn(acc.z, __fsub_rn(th.z, l.z));
                acc.w = __fadd_rn(acc.w, __fsub_rn(th.w, l.w));
            }
            float4 o;
            o.x = diloco_elem(th.x, acc.x, fr, beta, alpha, m.x);
            o.y = diloco_elem(th.y, acc.y, fr, beta, alpha, m.y);
            o.z = diloco_elem(th.z, acc.z, fr, beta, alpha, m.z);
            o.w = diloco_elem(th.w, acc.w, fr, beta, alpha, m.w);
            *reinterpret_cast<float4*>(theta + off) = o;
            *reinterpret_cast<float4*>(mom + off) = m;
        }
    } else {
        for (int p = tid; p < cd.len; p += kThreads) {
            const long long off = cd.base + p;
            const float th = theta[off];
            float acc = 0.f;
            for (int r = 0; r < n_workers; ++r) acc = __fadd_rn(acc, __fsub_rn(th, loc.p[r][off]));
            float m = mom[off];
            theta[off] = diloco_elem(th, acc, fr, beta, alpha, m);
            mom[off] = m;
        }
    }
}

}  // namespace

// ================================================================================================
// Host side
// ================================================================================================

struct sl_ctx {
    sl_config cfg;
    int device;
    int n_tensors;
    long long n_chunks;
    long long n_slots;
    long long flat_elems;
    int kp;
    std::vector<sl_tensor_desc> tensors;
    ChunkDesc* d_chunks;
    TensorInfo* d_tinfo;
    int ef_ctas;  // resident CTAs of the persistent compression kernel on this device
    // tensor-map (TMA) block copies: usable when every full chunk starts on a 64-element boundary
    bool tma_ok, tma_on;
    int n_classes;
    int class_rs[kMaxTmaClasses];       // distinct row lengths of full chunks (64 for flat runs)
    CUtensorMap* d_maps;                // [kMapSlots][n_classes]
    std::vector<CUtensorMap> h_maps;    // host copy the device array is filled from
    std::vector<const void*> slot_ptr;  // buffer described by each slot
    bool slots_cleared;                 // the slot table was emptied during the current assignment
    int* d_status;                      // device status word (SL_OK or what a kernel recorded)
    // entropy-coded payload: byte offsets of the directory and the index stream, worst-case size
    size_t ixc_dir_off, ixc_stream_off, ixc_capacity;
    bool deferred;              // deferred error-feedback subtraction (sl_set_ef_deferred)
    bool pending;               // corrected values of the last step still wait in the workspace
    float* pending_e[kMaxR];    // the error buffers they belong to
    void* ws_ptr;
    size_t ws_bytes;
    int last_workers;  // worker count the workspace was last laid out for
    // optional per-kernel timing (sl_profile_*)
    bool prof_on;
    int prof_steps;                        // compress/apply sequences recorded since the last read
    std::vector<cudaEvent_t> prof_events;  // [kProfMaxSeq][kProfSlots + 1]
    // copy stream + events of sl_outer_step_host (created on first use)
    cudaStream_t copy_stream;
    cudaEvent_t ev_copied[2], ev_consumed[2];
    bool host_path_ready;
};

namespace {

constexpr int kMapSlots = 2 * kMaxR + 2;  // buffers with tensor maps at one time: theta_local and e of every worker

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda)
typedef CUresult (*TmaEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TmaEncodeFn tma_encode_fn() {
    static TmaEncodeFn fn = []() -> TmaEncodeFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<TmaEncodeFn>(p);
    }();
    return fn;
}

sl_status cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return SL_ERR_CUDA;
}
#define SL_CUDA(call)                                      \
    do {                                                   \
        cudaError_t e_ = (call);                           \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

size_t workspace_bytes_for(const sl_ctx* c, int workers) {
    const size_t WG = (size_t)workers * (size_t)c->n_chunks;
    return up256(WG * c->kp * sizeof(float)) + up256(WG * c->kp * sizeof(uint16_t)) +
           up256(WG * sizeof(double)) + up256(WG * 4 * sizeof(double)) + up256(WG * 4 * sizeof(unsigned)) +
           up256((size_t)workers * c->n_tensors * sizeof(TStat));
}

Workspace carve(const sl_ctx* c, int workers) {
    const size_t WG = (size_t)workers * (size_t)c->n_chunks;
    char* p = static_cast<char*>(c->ws_ptr);
    Workspace w;
    w.val = reinterpret_cast<float*>(p);        p += up256(WG * c->kp * sizeof(float));
    w.idx = reinterpret_cast<uint16_t*>(p);     p += up256(WG * c->kp * sizeof(uint16_t));
    w.psum = reinterpret_cast<double*>(p);      p += up256(WG * sizeof(double));
    w.pbin = reinterpret_cast<double*>(p);      p += up256(WG * 4 * sizeof(double));
    w.pcnt = reinterpret_cast<unsigned*>(p);    p += up256(WG * 4 * sizeof(unsigned));
    w.tstat = reinterpret_cast<TStat*>(p);
    return w;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

unsigned blocks_for(long long items, int per_block) { return (unsigned)((items + per_block - 1) / per_block); }

// Event after profile slot `slot` (slot -1 = start of the sequence) of the sequence being recorded.
inline void prof_mark(sl_ctx* c, int slot, cudaStream_t st) {
    if (!c->prof_on || c->prof_steps >= kProfMaxSeq) return;
    cudaEventRecord(c->prof_events[(size_t)c->prof_steps * (kProfSlots + 1) + (slot + 1)], st);
}

// Slot of the tensor maps that describe the flat buffer at `ptr` (one map per row-length class);
// encodes and uploads them (ordered on `st`) the first time the pointer is seen.  -1 on failure.
int tma_map_slot(sl_ctx* c, const void* ptr, cudaStream_t st) {
    for (size_t i = 0; i < c->slot_ptr.size(); ++i)
        if (c->slot_ptr[i] == ptr) return (int)i;
    if ((int)c->slot_ptr.size() == kMapSlots) {  // full: start over (uploads are ordered after earlier launches)
        c->slot_ptr.clear();
        c->slots_cleared = true;
    }
    const int slot = (int)c->slot_ptr.size();
    TmaEncodeFn enc = tma_encode_fn();
    for (int q = 0; q < c->n_classes; ++q) {
        const cuuint64_t rs = (cuuint64_t)c->class_rs[q];
        const cuuint64_t dims[3] = {(cuuint64_t)kTile, rs / kTile, ((cuuint64_t)c->flat_elems + rs - 1) / rs + 1};
        const cuuint64_t strides[2] = {kTile * sizeof(float), rs * sizeof(float)};  // bytes, dimensions 1 and 2
        const cuuint32_t box[3] = {(cuuint32_t)kTile, 1u, (cuuint32_t)kTile};
        const cuuint32_t estr[3] = {1u, 1u, 1u};
        CUtensorMap* m = &c->h_maps[(size_t)slot * c->n_classes + q];
        if (enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -1;
    }
    if (cudaMemcpyAsync(c->d_maps + (size_t)slot * c->n_classes, &c->h_maps[(size_t)slot * c->n_classes],
                        sizeof(CUtensorMap) * c->n_classes, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return -1;
    c->slot_ptr.push_back(ptr);
    return slot;
}

sl_status launch_flush(sl_ctx* c, const WorkerPtrs& ptrs, cudaStream_t st) {
    const int R = c->cfg.R;
    const Workspace ws = carve(c, R);
    ef_flush_kernel<<<blocks_for(c->n_chunks * R, 4), 128, 0, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, c->kp, ws,
                                                                    ptrs);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

// Compression of `workers` workers whose pointers are in `ptrs` (kernels 1-8).  `defer`: leave the
// corrected values in the workspace instead of writing them into e (only with all R workers).
// `skip_pack`: the caller runs the packing step fused into the apply kernel right after.
sl_status launch_compress(sl_ctx* c, int workers, const float* theta_sync, const WorkerPtrs& ptrs,
                          cudaStream_t st, bool defer, bool skip_pack = false) {
    if (!c->ws_ptr || c->ws_bytes < workspace_bytes_for(c, workers)) return SL_ERR_NOMEM;
    const Workspace ws = carve(c, workers);
    c->last_workers = workers;
    const long long G = c->n_chunks, WG = G * workers;
    const int k = c->cfg.k, kp = c->kp, T = c->n_tensors;
    if (WG > 0x7FFFFFFFll) return SL_ERR_TOO_LARGE;
    const bool ef = c->cfg.ef_enabled != 0;
    bool consume = false;  // this step substitutes the waiting values while it streams e
    if (c->pending) {
        if (ef && defer) {
            consume = true;
        } else {  // nothing will read them in flight (frozen step): write them out first
            WorkerPtrs fp;
            memset(&fp, 0, sizeof(fp));
            for (int r = 0; r < c->cfg.R; ++r) fp.e[r] = c->pending_e[r];
            sl_status s = launch_flush(c, fp, st);
            if (s != SL_OK) return s;
        }
        c->pending = false;
    }

    // tile copies through tensor maps when the table allows it and every buffer got its maps
    TmaArgs ta;
    memset(&ta, 0, sizeof(ta));
    bool use_tma = c->tma_on;
    if (use_tma) {
        ta.maps = c->d_maps;
        ta.n_classes = c->n_classes;
        ta.status = c->d_status;
        for (int q = 0; q < c->n_classes; ++q) ta.class_rs[q] = c->class_rs[q];
        for (int pass = 0; pass < 2 && use_tma; ++pass) {
            // if the slot table fills up half-way, it is emptied and the assignment starts over: one
            // call needs at most 2 R slots, which an empty table holds
            c->slots_cleared = false;
            for (int r = 0; r < workers && use_tma; ++r) {
                ta.slot_l[r] = tma_map_slot(c, ptrs.theta_local[r], st);
                ta.slot_e[r] = ef ? tma_map_slot(c, ptrs.e[r], st) : 0;
                use_tma = ta.slot_l[r] >= 0 && ta.slot_e[r] >= 0;
            }
            if (!c->slots_cleared) break;
        }
    }

    prof_mark(c, -1, st);
    const unsigned ef_grid = (unsigned)(G < c->ef_ctas ? G : c->ef_ctas);  // persistent CTAs
    const size_t smem = sizeof(PipeSmem);
#define SL_LAUNCH_EF(EFV, PENDV, TMAV)                                                                          \
    ef_topk_kernel<EFV, PENDV, TMAV><<<ef_grid, kThreads, smem, st>>>(c->d_chunks, G, workers, k, kp, c->cfg.beta, \
                                                                      theta_sync, ptrs, ws, ta)
    if (use_tma) {
        if (!ef) SL_LAUNCH_EF(false, false, true);
        else if (consume) SL_LAUNCH_EF(true, true, true);
        else SL_LAUNCH_EF(true, false, true);
    } else {
        if (!ef) SL_LAUNCH_EF(false, false, false);
        else if (consume) SL_LAUNCH_EF(true, true, false);
        else SL_LAUNCH_EF(true, false, false);
    }
#undef SL_LAUNCH_EF
    prof_mark(c, 0, st);
    const unsigned cb = blocks_for(WG, 128), tb = blocks_for((long long)workers * T, 4);
    chunk_sum_kernel<0><<<cb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws);
    prof_mark(c, 1, st);
    tensor_reduce_kernel<0><<<tb, 128, 0, st>>>(c->d_tinfo, G, workers, T, ws, ptrs);
    prof_mark(c, 2, st);
    chunk_sum_kernel<1><<<cb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws);
    prof_mark(c, 3, st);
    tensor_reduce_kernel<1><<<tb, 128, 0, st>>>(c->d_tinfo, G, workers, T, ws, ptrs);
    prof_mark(c, 4, st);
    chunk_bins_kernel<<<cb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws);
    prof_mark(c, 5, st);
    tensor_reduce_kernel<2><<<tb, 128, 0, st>>>(c->d_tinfo, G, workers, T, ws, ptrs);
    prof_mark(c, 6, st);
    const unsigned pb = blocks_for(WG, 4);
    if (skip_pack)
        ;  // records, error correction: done by decode_avg_apply_kernel<., 1 or 2>
    else if (!ef)
        pack_fix_kernel<0><<<pb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, ptrs);
    else if (defer)
        pack_fix_kernel<2><<<pb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, ptrs);
    else
        pack_fix_kernel<1><<<pb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, ptrs);
    prof_mark(c, 7, st);
    SL_CUDA(cudaGetLastError());
    if (ef && defer) {
        c->pending = true;
        for (int r = 0; r < workers; ++r) c->pending_e[r] = ptrs.e[r];
    }
    return SL_OK;
}

// fuse: 0 = payloads in, 1 / 2 = also do the packing step of a compression in flight (see the kernel)
sl_status launch_apply(sl_ctx* c, const PayloadPtrs& pl, int present, float* theta_sync, cudaStream_t st, int fuse = 0,
                       const WorkerPtrs* fuse_ptrs = nullptr) {
    if (present == 0) return SL_OK;
    const int R = c->cfg.R;
    const double D = c->cfg.divide_by_present ? (double)present : (double)R;
    const float scale = (float)(-(double)c->cfg.outer_lr / D);
    const int stride = record_stride(c->cfg.k);
    const int nb = R < 32 ? R : 32;  // the kernel never stages more than 32 records at once
    const size_t smem = (size_t)kChunk * 8 + 32 * 24 + (size_t)nb * (stride + 16);
    const int spl = (c->cfg.k + 31) / 32;
    FuseArgs fa;
    memset(&fa, 0, sizeof(fa));
    WorkerPtrs wp;
    memset(&wp, 0, sizeof(wp));
    if (fuse) {
        fa.ws = carve(c, R);
        fa.n_chunks = c->n_chunks;
        fa.n_tensors = c->n_tensors;
        fa.kp = c->kp;
        wp = *fuse_ptrs;
    }
#define SL_APPLY2(SPLV, WPWV)                                                                                   \
    do {                                                                                                        \
        auto kern = fuse == 0 ? decode_avg_apply_kernel<SPLV, WPWV, 0>                                          \
                  : fuse == 1 ? decode_avg_apply_kernel<SPLV, WPWV, 1> : decode_avg_apply_kernel<SPLV, WPWV, 2>; \
        if (smem > 48 * 1024)                                                                                   \
            SL_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));        \
        kern<<<(unsigned)c->n_chunks, kThreads, smem, st>>>(c->d_chunks, R, c->cfg.k, scale, pl, theta_sync, fa, wp); \
    } while (0)
    // workers per warp: as few as cover min(R, 32) workers in one batch, within 8 entries per thread
#define SL_APPLY(SPLV, MAXW)                                             \
    do {                                                                 \
        if (R <= 8 || MAXW == 1) SL_APPLY2(SPLV, 1);                      \
        else if (R <= 16 || MAXW == 2) SL_APPLY2(SPLV, (MAXW >= 2 ? 2 : 1)); \
        else SL_APPLY2(SPLV, (MAXW >= 4 ? 4 : MAXW));                     \
    } while (0)
    if (spl <= 1) SL_APPLY(1, 4);
    else if (spl <= 2) SL_APPLY(2, 4);
    else if (spl <= 4) SL_APPLY(4, 2);
    else SL_APPLY(8, 1);
#undef SL_APPLY
#undef SL_APPLY2
    prof_mark(c, 8, st);
    if (c->prof_on && c->prof_steps < kProfMaxSeq) c->prof_steps++;
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = prev == dev || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" {

const char* sl_strerror(sl_status s) {
    switch (s) {
        case SL_OK: return "ok";
        case SL_ERR_INVALID_ARG: return "invalid argument";
        case SL_ERR_ALIGNMENT: return "pointer or offset not 16-byte aligned";
        case SL_ERR_UNSUPPORTED: return "configuration not supported by this library";
        case SL_ERR_BAD_PAYLOAD: return "malformed payload";
        case SL_ERR_CUDA: return "CUDA error";
        case SL_ERR_NOMEM: return "workspace missing or too small";
        case SL_ERR_TOO_LARGE: return "problem exceeds a built-in capacity";
        case SL_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    }
    return "unknown status";
}

const char* sl_last_cuda_error(void) { return g_cuda_err; }

size_t sl_record_stride(int32_t k) { return k < 1 ? 0 : (size_t)record_stride(k); }

sl_status sl_create(const sl_config* cfg, const sl_tensor_desc* tensors, int32_t n_tensors, sl_ctx** out) {
    if (!cfg || !tensors || !out || n_tensors < 1) return SL_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->k < 1 || cfg->R < 1 || cfg->H < 1) return SL_ERR_INVALID_ARG;
    if (!(cfg->beta >= 0.0f && cfg->beta <= 1.0f) || !isfinite(cfg->outer_lr)) return SL_ERR_INVALID_ARG;
    if (cfg->chunk_elems != kChunk || cfg->tile_dim != kTile || cfg->quant_bits != 2) return SL_ERR_UNSUPPORTED;
    if (cfg->k > kMaxK || cfg->R > kMaxR) return SL_ERR_UNSUPPORTED;

    sl_ctx* c = new (std::nothrow) sl_ctx();
    if (!c) return SL_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->n_tensors = n_tensors;
    c->kp = (cfg->k + 7) / 8 * 8;
    c->d_chunks = nullptr;
    c->d_tinfo = nullptr;
    c->ef_ctas = 0;
    c->tma_ok = c->tma_on = false;
    c->slots_cleared = false;
    c->n_classes = 0;
    c->d_maps = nullptr;
    c->d_status = nullptr;
    c->deferred = false;
    c->pending = false;
    c->ws_ptr = nullptr;
    c->ws_bytes = 0;
    c->last_workers = cfg->R;
    c->prof_on = false;
    c->prof_steps = 0;
    c->copy_stream = nullptr;
    c->host_path_ready = false;
    c->tensors.assign(tensors, tensors + n_tensors);

    const int stride = record_stride(cfg->k);
    std::vector<ChunkDesc> chunks;
    std::vector<TensorInfo> tinfo((size_t)n_tensors);
    long long rec_off = 16ll * n_tensors, flat = 0, slots = 0;
    for (int j = 0; j < n_tensors; ++j) {
        const sl_tensor_desc& t = tensors[j];
        if (t.rows < 1 || t.cols < 1 || t.offset < 0) { delete c; return SL_ERR_INVALID_ARG; }
        if (t.offset % 4 != 0) { delete c; return SL_ERR_ALIGNMENT; }
        const long long n = t.rows * t.cols;
        if (t.offset + n > flat) flat = t.offset + n;
        tinfo[j].first_chunk = (long long)chunks.size();
        long long tslots = 0;
        const bool tiled = t.rows > 1 && t.rows % kTile == 0 && t.cols % kTile == 0;
        if (tiled) {
            if (t.cols > 0x7FFFFFFFll) { delete c; return SL_ERR_TOO_LARGE; }
            const long long tr = t.rows / kTile, tc = t.cols / kTile;
            for (long long a = 0; a < tr; ++a)
                for (long long b = 0; b < tc; ++b) {
                    ChunkDesc d;
                    d.base = t.offset + a * kTile * t.cols + b * kTile;
                    d.row_stride = (int)t.cols;
                    d.len = kChunk;
                    d.tensor = j;
                    d.chunk_in_tensor = (int)(a * tc + b);
                    d.rec_off = rec_off;
                    rec_off += stride;
                    tslots += cfg->k < kChunk ? cfg->k : kChunk;
                    chunks.push_back(d);
                }
        } else {
            const long long nc = (n + kChunk - 1) / kChunk;
            for (long long a = 0; a < nc; ++a) {
                ChunkDesc d;
                d.base = t.offset + a * kChunk;
                d.row_stride = 0;
                const long long rest = n - a * kChunk;
                d.len = (int)(rest < kChunk ? rest : kChunk);
                d.tensor = j;
                d.chunk_in_tensor = (int)a;
                d.rec_off = rec_off;
                rec_off += stride;
                tslots += cfg->k < d.len ? cfg->k : d.len;
                chunks.push_back(d);
            }
        }
        tinfo[j].n_chunks = (long long)chunks.size() - tinfo[j].first_chunk;
        tinfo[j].n_slots = tslots;
        slots += tslots;
    }
    c->n_chunks = (long long)chunks.size();
    c->n_slots = slots;
    {   // row-length classes of the full chunks; block copies need 64-element alignment of every block
        bool ok = true;
        int ncls = 0;
        for (const ChunkDesc& d : chunks) {
            if (d.len != kChunk) continue;
            if (d.base % kTile != 0) { ok = false; break; }
            const int rs = d.row_stride ? d.row_stride : kTile;
            int q = 0;
            while (q < ncls && c->class_rs[q] != rs) ++q;
            if (q == ncls) {
                if (ncls == kMaxTmaClasses) { ok = false; break; }
                c->class_rs[ncls++] = rs;
            }
        }
        c->n_classes = ncls;
        c->tma_ok = ok && ncls > 0 && tma_encode_fn() != nullptr;
        c->tma_on = c->tma_ok;
    }
    c->flat_elems = flat;
    {
        const size_t cb = (2 * (size_t)cfg->k + 7) / 8, G = chunks.size();
        c->ixc_dir_off = (16 * (size_t)n_tensors + cb * G + 3) / 4 * 4;
        c->ixc_stream_off = c->ixc_dir_off + 4 * ((G + kIxcGroup - 1) / kIxcGroup);
        unsigned long long bits = 0;
        for (const ChunkDesc& d : chunks) bits += (unsigned long long)ixc_worst_bits(d.len, cfg->k < d.len ? cfg->k : d.len);
        c->ixc_capacity = bits < (1ull << 32) ? (c->ixc_stream_off + (size_t)((bits + 7) / 8) + 15) / 16 * 16 : 0;
    }

    cudaError_t e = cudaGetDevice(&c->device);
    int n_sms = 0, per_sm = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, c->device);
    const int smem_bytes = (int)sizeof(PipeSmem);
#define SL_SMEM_ATTR(...)                                                                                      \
    if (e == cudaSuccess)                                                                                      \
        e = cudaFuncSetAttribute(ef_topk_kernel<__VA_ARGS__>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes)
    SL_SMEM_ATTR(true, false, false);
    SL_SMEM_ATTR(false, false, false);
    SL_SMEM_ATTR(true, true, false);
    SL_SMEM_ATTR(true, false, true);
    SL_SMEM_ATTR(false, false, true);
    SL_SMEM_ATTR(true, true, true);
#undef SL_SMEM_ATTR
    if (e == cudaSuccess)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ef_topk_kernel<true, true, true>, kThreads,
                                                          sizeof(PipeSmem));
    c->ef_ctas = n_sms * (per_sm > 0 ? per_sm : 1);
    if (e == cudaSuccess) e = cudaMalloc(&c->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, sizeof(int));
    if (c->tma_ok) {
        c->h_maps.resize((size_t)kMapSlots * c->n_classes);
        if (e == cudaSuccess) e = cudaMalloc(&c->d_maps, sizeof(CUtensorMap) * kMapSlots * c->n_classes);
    }
    if (e == cudaSuccess) e = cudaMalloc(&c->d_chunks, chunks.size() * sizeof(ChunkDesc));
    if (e == cudaSuccess) e = cudaMalloc(&c->d_tinfo, tinfo.size() * sizeof(TensorInfo));
    if (e == cudaSuccess)
        e = cudaMemcpy(c->d_chunks, chunks.data(), chunks.size() * sizeof(ChunkDesc), cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(c->d_tinfo, tinfo.data(), tinfo.size() * sizeof(TensorInfo), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        sl_status s = cuda_fail(e, "sl_create");
        if (c->d_chunks) cudaFree(c->d_chunks);
        if (c->d_tinfo) cudaFree(c->d_tinfo);
        if (c->d_status) cudaFree(c->d_status);
        if (c->d_maps) cudaFree(c->d_maps);
        delete c;
        return s;
    }
    *out = c;
    return SL_OK;
}

sl_status sl_destroy(sl_ctx* c) {
    if (!c) return SL_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    cudaFree(c->d_chunks);
    cudaFree(c->d_tinfo);
    cudaFree(c->d_status);
    cudaFree(c->d_maps);
    for (auto& ev : c->prof_events) cudaEventDestroy(ev);
    if (c->host_path_ready) {
        cudaStreamDestroy(c->copy_stream);
        for (int i = 0; i < 2; ++i) {
            cudaEventDestroy(c->ev_copied[i]);
            cudaEventDestroy(c->ev_consumed[i]);
        }
    }
    delete c;
    return SL_OK;
}

sl_status sl_set_hyper(sl_ctx* c, float beta, float outer_lr, int32_t ef_enabled, int32_t divide_by_present) {
    if (!c) return SL_ERR_INVALID_ARG;
    if (!(beta >= 0.0f && beta <= 1.0f) || !isfinite(outer_lr)) return SL_ERR_INVALID_ARG;
    c->cfg.beta = beta;
    c->cfg.outer_lr = outer_lr;
    c->cfg.ef_enabled = ef_enabled != 0;
    c->cfg.divide_by_present = divide_by_present != 0;
    return SL_OK;
}

sl_status sl_payload_bytes(const sl_ctx* c, size_t* bytes) {
    if (!c || !bytes) return SL_ERR_INVALID_ARG;
    *bytes = 16 * (size_t)c->n_tensors + (size_t)record_stride(c->cfg.k) * (size_t)c->n_chunks;
    return SL_OK;
}

sl_status sl_num_chunks(const sl_ctx* c, int64_t* chunks, int64_t* slots) {
    if (!c) return SL_ERR_INVALID_ARG;
    if (chunks) *chunks = c->n_chunks;
    if (slots) *slots = c->n_slots;
    return SL_OK;
}

sl_status sl_flat_elems(const sl_ctx* c, int64_t* elems) {
    if (!c || !elems) return SL_ERR_INVALID_ARG;
    *elems = c->flat_elems;
    return SL_OK;
}

sl_status sl_workspace_bytes(const sl_ctx* c, size_t* bytes) {
    if (!c || !bytes) return SL_ERR_INVALID_ARG;
    *bytes = workspace_bytes_for(c, c->cfg.R);
    return SL_OK;
}

sl_status sl_set_workspace(sl_ctx* c, void* dev_ptr, size_t bytes) {
    if (!c) return SL_ERR_INVALID_ARG;
    if (c->pending) return SL_ERR_INVALID_ARG;  // the workspace holds part of the error state: sl_ef_flush() first
    if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255u)) return SL_ERR_ALIGNMENT;
    c->ws_ptr = dev_ptr;
    c->ws_bytes = dev_ptr ? bytes : 0;
    return SL_OK;
}

sl_status sl_compress(sl_ctx* c, const float* theta_sync, const float* theta_local, float* e, uint8_t* payload,
                      void* stream) {
    if (!c || !theta_sync || !theta_local || !payload) return SL_ERR_INVALID_ARG;
    if (c->cfg.ef_enabled && !e) return SL_ERR_INVALID_ARG;
    if (misaligned(theta_sync) || misaligned(theta_local) || misaligned(e) || misaligned(payload))
        return SL_ERR_ALIGNMENT;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    WorkerPtrs ptrs;
    memset(&ptrs, 0, sizeof(ptrs));
    ptrs.theta_local[0] = theta_local;
    ptrs.e[0] = e;
    ptrs.payload[0] = payload;
    return launch_compress(c, 1, theta_sync, ptrs, static_cast<cudaStream_t>(stream), false);
}

sl_status sl_aggregate_apply(sl_ctx* c, const uint8_t* const* payloads, float* theta_sync, void* stream) {
    if (!c || !payloads || !theta_sync) return SL_ERR_INVALID_ARG;
    if (misaligned(theta_sync)) return SL_ERR_ALIGNMENT;
    PayloadPtrs pl;
    memset(&pl, 0, sizeof(pl));
    int present = 0;
    for (int r = 0; r < c->cfg.R; ++r) {
        if (misaligned(payloads[r])) return SL_ERR_ALIGNMENT;
        pl.p[r] = payloads[r];
        present += payloads[r] != nullptr;
    }
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    return launch_apply(c, pl, present, theta_sync, static_cast<cudaStream_t>(stream));
}

sl_status sl_outer_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* const* e,
                        uint8_t* const* payloads, void* stream) {
    if (!c || !theta_sync || !theta_local || !payloads) return SL_ERR_INVALID_ARG;
    if (c->cfg.ef_enabled && !e) return SL_ERR_INVALID_ARG;
    if (misaligned(theta_sync)) return SL_ERR_ALIGNMENT;
    const int R = c->cfg.R;
    WorkerPtrs ptrs;
    PayloadPtrs pl;
    memset(&ptrs, 0, sizeof(ptrs));
    memset(&pl, 0, sizeof(pl));
    for (int r = 0; r < R; ++r) {
        if (!theta_local[r] || !payloads[r] || (c->cfg.ef_enabled && !e[r])) return SL_ERR_INVALID_ARG;
        if (misaligned(theta_local[r]) || misaligned(payloads[r]) || (e && misaligned(e[r]))) return SL_ERR_ALIGNMENT;
        for (int q = 0; q < r; ++q) {
            if (payloads[q] == payloads[r]) return SL_ERR_INVALID_ARG;
            if (c->cfg.ef_enabled && e[q] == e[r]) return SL_ERR_INVALID_ARG;
        }
        ptrs.theta_local[r] = theta_local[r];
        ptrs.e[r] = e ? e[r] : nullptr;
        ptrs.payload[r] = payloads[r];
        pl.p[r] = payloads[r];
    }
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool defer = c->deferred && c->cfg.ef_enabled;
    if (c->pending && defer) {  // the waiting values can only be substituted into the buffers they came from
        for (int r = 0; r < R; ++r)
            if (e[r] != c->pending_e[r]) return SL_ERR_INVALID_ARG;
    }
    const int fuse = c->cfg.ef_enabled ? (defer ? 2 : 1) : 0;  // packing fused into the apply kernel
    sl_status s = launch_compress(c, R, theta_sync, ptrs, st, defer, fuse != 0);
    if (s != SL_OK) return s;
    return launch_apply(c, pl, R, theta_sync, st, fuse, &ptrs);
}

sl_status sl_outer_step_host(sl_ctx* c, float* theta_sync, const float* const* theta_local_host, float* dev_stage,
                             size_t stage_elems, float* const* e, uint8_t* const* payloads, float* theta_sync_host,
                             void* stream) {
    if (!c || !theta_sync || !theta_local_host || !dev_stage || !payloads) return SL_ERR_INVALID_ARG;
    if (c->cfg.ef_enabled && !e) return SL_ERR_INVALID_ARG;
    if (misaligned(theta_sync) || misaligned(dev_stage)) return SL_ERR_ALIGNMENT;
    const int R = c->cfg.R;
    const size_t flat = (size_t)((c->flat_elems + 3) / 4 * 4);
    if (stage_elems < flat) return SL_ERR_NOMEM;
    const int nbuf = stage_elems >= 2 * flat ? 2 : 1;
    for (int r = 0; r < R; ++r) {
        if (!theta_local_host[r] || !payloads[r] || (c->cfg.ef_enabled && !e[r])) return SL_ERR_INVALID_ARG;
        if (misaligned(payloads[r]) || (e && misaligned(e[r]))) return SL_ERR_ALIGNMENT;
    }
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!c->host_path_ready) {
        SL_CUDA(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            SL_CUDA(cudaEventCreateWithFlags(&c->ev_copied[i], cudaEventDisableTiming));
            SL_CUDA(cudaEventCreateWithFlags(&c->ev_consumed[i], cudaEventDisableTiming));
        }
        c->host_path_ready = true;
    }
    PayloadPtrs pl;
    memset(&pl, 0, sizeof(pl));
    const size_t bytes = (size_t)c->flat_elems * sizeof(float);
    // Worker r's parameters travel on the copy stream into staging buffer r % nbuf while worker
    // r - 1 is being compressed on the caller's stream.
    SL_CUDA(cudaEventRecord(c->ev_consumed[0], st));  // orders the first copies after prior work on `st`
    SL_CUDA(cudaEventRecord(c->ev_consumed[1], st));
    for (int r = 0; r < R; ++r) {
        const int bsel = r % nbuf;
        float* stage = dev_stage + (size_t)bsel * flat;
        SL_CUDA(cudaStreamWaitEvent(c->copy_stream, c->ev_consumed[bsel], 0));
        SL_CUDA(cudaMemcpyAsync(stage, theta_local_host[r], bytes, cudaMemcpyHostToDevice, c->copy_stream));
        SL_CUDA(cudaEventRecord(c->ev_copied[bsel], c->copy_stream));
        SL_CUDA(cudaStreamWaitEvent(st, c->ev_copied[bsel], 0));
        WorkerPtrs ptrs;
        memset(&ptrs, 0, sizeof(ptrs));
        ptrs.theta_local[0] = stage;
        ptrs.e[0] = e ? e[r] : nullptr;
        ptrs.payload[0] = payloads[r];
        sl_status s = launch_compress(c, 1, theta_sync, ptrs, st, false);
        if (s != SL_OK) return s;
        SL_CUDA(cudaEventRecord(c->ev_consumed[bsel], st));
        pl.p[r] = payloads[r];
    }
    sl_status s = launch_apply(c, pl, R, theta_sync, st);
    if (s != SL_OK) return s;
    if (theta_sync_host)
        SL_CUDA(cudaMemcpyAsync(theta_sync_host, theta_sync, bytes, cudaMemcpyDeviceToHost, st));
    SL_CUDA(cudaStreamSynchronize(st));
    return SL_OK;
}

sl_status sl_profile_enable(sl_ctx* c, int32_t enable) {
    if (!c) return SL_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    if (enable && c->prof_events.empty()) {
        c->prof_events.resize((size_t)kProfMaxSeq * (kProfSlots + 1));
        for (auto& ev : c->prof_events) SL_CUDA(cudaEventCreate(&ev));
    }
    c->prof_on = enable != 0;
    c->prof_steps = 0;
    return SL_OK;
}

sl_status sl_profile_read(sl_ctx* c, float* ms_total, int64_t* launches) {
    if (!c || !ms_total || !launches) return SL_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    for (int i = 0; i < kProfSlots; ++i) { ms_total[i] = 0.0f; launches[i] = 0; }
    for (int q = 0; q < c->prof_steps; ++q) {
        cudaEvent_t* ev = &c->prof_events[(size_t)q * (kProfSlots + 1)];
        SL_CUDA(cudaEventSynchronize(ev[kProfSlots]));
        for (int i = 0; i < kProfSlots; ++i) {
            float ms = 0.0f;
            SL_CUDA(cudaEventElapsedTime(&ms, ev[i], ev[i + 1]));
            ms_total[i] += ms;
            launches[i] += 1;
        }
    }
    c->prof_steps = 0;
    return SL_OK;
}

const char* sl_profile_name(int32_t slot) {
    static const char* names[kProfSlots] = {"ef_topk", "chunk_sum", "tensor_mean", "chunk_var", "tensor_sigma",
                                            "chunk_bins", "tensor_lut", "pack_fix", "decode_avg_apply"};
    return slot >= 0 && slot < kProfSlots ? names[slot] : "";
}

sl_status sl_diloco_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* momentum,
                         float beta_outer, void* stream) {
    if (!c || !theta_sync || !theta_local || !momentum) return SL_ERR_INVALID_ARG;
    if (!(beta_outer >= 0.0f && beta_outer <= 1.0f)) return SL_ERR_INVALID_ARG;
    if (misaligned(theta_sync) || misaligned(momentum)) return SL_ERR_ALIGNMENT;
    LocalPtrs lp;
    memset(&lp, 0, sizeof(lp));
    for (int r = 0; r < c->cfg.R; ++r) {
        if (!theta_local[r]) return SL_ERR_INVALID_ARG;
        if (misaligned(theta_local[r])) return SL_ERR_ALIGNMENT;
        lp.p[r] = theta_local[r];
    }
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    diloco_step_kernel<<<(unsigned)c->n_chunks, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        c->d_chunks, c->cfg.R, beta_outer, c->cfg.outer_lr, theta_sync, lp, momentum);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

sl_status sl_coded_payload_capacity(const sl_ctx* c, size_t* bytes) {
    if (!c || !bytes) return SL_ERR_INVALID_ARG;
    if (!c->ixc_capacity) return SL_ERR_TOO_LARGE;  // the stream's bit offsets are 32-bit
    *bytes = c->ixc_capacity;
    return SL_OK;
}

sl_status sl_encode_payload(sl_ctx* c, const uint8_t* payload, uint8_t* coded, uint64_t* dev_coded_bytes,
                            void* stream) {
    if (!c || !payload || !coded || !dev_coded_bytes) return SL_ERR_INVALID_ARG;
    if (misaligned(payload) || misaligned(coded) || (reinterpret_cast<uintptr_t>(dev_coded_bytes) & 7u))
        return SL_ERR_ALIGNMENT;
    if (!c->ixc_capacity) return SL_ERR_TOO_LARGE;
    if (!c->ws_ptr || c->ws_bytes < workspace_bytes_for(c, c->cfg.R)) return SL_ERR_NOMEM;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // scratch: two 32-bit words per chunk in the partial-sum area of the workspace (unused between
    // compressions; the values a deferred subtraction keeps waiting live elsewhere)
    unsigned* lens = reinterpret_cast<unsigned*>(carve(c, c->cfg.R).psum);
    unsigned* offs = lens + c->n_chunks;
    const long long G = c->n_chunks;
    SL_CUDA(cudaMemsetAsync(coded + c->ixc_dir_off, 0, c->ixc_capacity - c->ixc_dir_off, st));
    ixc_len_kernel<<<blocks_for(G, 128), 128, 0, st>>>(c->d_chunks, G, c->cfg.k, payload, lens);
    ixc_scan_kernel<<<1, 1024, 0, st>>>(lens, G, offs, reinterpret_cast<unsigned*>(coded + c->ixc_dir_off),
                                        c->ixc_stream_off, reinterpret_cast<unsigned long long*>(dev_coded_bytes));
    const long long items = G > 4ll * c->n_tensors ? G : 4ll * c->n_tensors;
    ixc_write_kernel<<<blocks_for(items, 128), 128, 0, st>>>(c->d_chunks, G, c->n_tensors, c->cfg.k, payload, offs, coded,
                                                             c->ixc_stream_off);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

sl_status sl_decode_payload(sl_ctx* c, const uint8_t* coded, uint8_t* payload, void* stream) {
    if (!c || !coded || !payload) return SL_ERR_INVALID_ARG;
    if (misaligned(coded) || misaligned(payload)) return SL_ERR_ALIGNMENT;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    const long long groups = (c->n_chunks + kIxcGroup - 1) / kIxcGroup;
    const long long items = groups > 4ll * c->n_tensors ? groups : 4ll * c->n_tensors;
    ixc_decode_kernel<<<blocks_for(items, 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        c->d_chunks, c->n_chunks, c->n_tensors, c->cfg.k, coded, c->ixc_dir_off, c->ixc_stream_off, payload);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

sl_status sl_set_tile_copies(sl_ctx* c, int32_t use_tensor_maps) {
    if (!c) return SL_ERR_INVALID_ARG;
    if (use_tensor_maps && !c->tma_ok) return SL_ERR_UNSUPPORTED;
    c->tma_on = use_tensor_maps != 0;
    return SL_OK;
}

sl_status sl_device_status(sl_ctx* c, void* stream) {
    if (!c) return SL_ERR_INVALID_ARG;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int v = 0;
    SL_CUDA(cudaMemcpyAsync(&v, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    SL_CUDA(cudaStreamSynchronize(st));
    if (v != (int)SL_OK) SL_CUDA(cudaMemsetAsync(c->d_status, 0, sizeof(int), st));
    return (sl_status)v;
}

sl_status sl_set_ef_deferred(sl_ctx* c, int32_t on) {
    if (!c) return SL_ERR_INVALID_ARG;
    c->deferred = on != 0;
    return SL_OK;
}

sl_status sl_ef_pending(const sl_ctx* c, int32_t* pending) {
    if (!c || !pending) return SL_ERR_INVALID_ARG;
    *pending = c->pending ? 1 : 0;
    return SL_OK;
}

sl_status sl_ef_flush(sl_ctx* c, float* const* e, int32_t keep_pending, void* stream) {
    if (!c) return SL_ERR_INVALID_ARG;
    if (!c->pending) return SL_OK;
    WorkerPtrs ptrs;
    memset(&ptrs, 0, sizeof(ptrs));
    for (int r = 0; r < c->cfg.R; ++r) {
        float* dst = e ? e[r] : c->pending_e[r];
        if (!dst && !keep_pending) return SL_ERR_INVALID_ARG;  // a worker may be skipped only if its values stay
        if (misaligned(dst)) return SL_ERR_ALIGNMENT;
        ptrs.e[r] = dst;
    }
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    sl_status s = launch_flush(c, ptrs, static_cast<cudaStream_t>(stream));
    if (s != SL_OK) return s;
    if (!keep_pending) c->pending = false;
    return SL_OK;
}

sl_status sl_validate_payload(sl_ctx* c, const uint8_t* payload, int32_t* dev_status, void* stream) {
    if (!c || !payload || !dev_status) return SL_ERR_INVALID_ARG;
    if (misaligned(payload)) return SL_ERR_ALIGNMENT;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    set_status_kernel<<<1, 1, 0, st>>>(dev_status, (int)SL_OK);
    const long long items = c->n_chunks > c->n_tensors ? c->n_chunks : c->n_tensors;
    validate_kernel<<<blocks_for(items, 128), 128, 0, st>>>(c->d_chunks, c->n_chunks, c->n_tensors, c->cfg.k, payload,
                                                            dev_status);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

sl_status sl_read_stats(sl_ctx* c, int32_t worker, float* dev_out, void* stream) {
    if (!c || !dev_out || worker < 0 || worker >= c->last_workers) return SL_ERR_INVALID_ARG;
    if (!c->ws_ptr) return SL_ERR_NOMEM;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    const Workspace ws = carve(c, c->last_workers);
    copy_stats_kernel<<<blocks_for((long long)c->n_tensors * 8, 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        ws.tstat + (long long)worker * c->n_tensors, c->n_tensors, dev_out);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

}  // extern "C"

// ================================================================================================
// Compression of one tensor without any allocation (sl_compress_tensor_static)
// ================================================================================================

namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;
// Scratch of sl_compress_tensor_static(): chunk table, staged (index, value) pairs, partial sums and
// tensor statistics of one call.  One copy per GPU that loads the library, held until the process
// exits; shared by every call on that GPU.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticSetup {  // per device: address of the array above, launch shape of the persistent kernel
    void* scratch;
    int ef_ctas;
    bool ready;
};
StaticSetup g_static_setup[64];

// Chunk table of a single tensor at element offset 0 (same rules as sl_create()).
__global__ void __launch_bounds__(128)
build_single_tensor_table_kernel(long long rows, long long cols, int k, long long n_chunks, ChunkDesc* chunks,
                                 TensorInfo* tinfo) {
    const long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n = rows * cols;
    const bool tiled = rows > 1 && rows % kTile == 0 && cols % kTile == 0;
    if (g == 0) {
        long long slots = 0;
        if (tiled) {
            slots = n_chunks * min((long long)k, (long long)kChunk);
        } else {
            const long long tail = n - (n_chunks - 1) * kChunk;
            slots = (n_chunks - 1) * min((long long)k, (long long)kChunk) + min((long long)k, tail);
        }
        tinfo->first_chunk = 0;
        tinfo->n_chunks = n_chunks;
        tinfo->n_slots = slots;
    }
    if (g >= n_chunks) return;
    ChunkDesc d;
    if (tiled) {
        const long long tc = cols / kTile, a = g / tc, b = g - a * tc;
        d.base = a * kTile * cols + b * kTile;
        d.row_stride = (int)cols;
        d.len = kChunk;
    } else {
        d.base = g * kChunk;
        d.row_stride = 0;
        const long long rest = n - g * kChunk;
        d.len = (int)(rest < kChunk ? rest : kChunk);
    }
    d.tensor = 0;
    d.chunk_in_tensor = (int)g;
    d.rec_off = 16 + (long long)record_stride(k) * g;
    chunks[g] = d;
}

}  // namespace

extern "C" {

size_t sl_static_scratch_bytes(void) { return kStaticScratchBytes; }

sl_status sl_compress_tensor_static(const float* theta_sync, const float* theta_local, float* e, uint8_t* payload,
                                    int64_t rows, int64_t cols, int32_t k, float beta, void* stream) {
    if (!theta_sync || !theta_local || !e || !payload) return SL_ERR_INVALID_ARG;
    if (rows < 1 || cols < 1 || k < 1 || !(beta >= 0.0f && beta <= 1.0f)) return SL_ERR_INVALID_ARG;
    if (k > kMaxK) return SL_ERR_UNSUPPORTED;
    if (misaligned(theta_sync) || misaligned(theta_local) || misaligned(e) || misaligned(payload)) return SL_ERR_ALIGNMENT;
    if (cols > 0x7FFFFFFFll || rows > (1ll << 40) / cols) return SL_ERR_TOO_LARGE;
    const long long n = rows * cols;
    const bool tiled = rows > 1 && rows % kTile == 0 && cols % kTile == 0;
    const long long G = tiled ? (rows / kTile) * (cols / kTile) : (n + kChunk - 1) / kChunk;
    const int kp = (k + 7) / 8 * 8;
    // layout of the scratch: chunk table | tensor info | the arrays of a one-worker workspace
    const size_t WG = (size_t)G;
    const size_t off_tinfo = up256(WG * sizeof(ChunkDesc));
    const size_t off_val = off_tinfo + up256(sizeof(TensorInfo));
    const size_t off_idx = off_val + up256(WG * kp * sizeof(float));
    const size_t off_psum = off_idx + up256(WG * kp * sizeof(uint16_t));
    const size_t off_pbin = off_psum + up256(WG * sizeof(double));
    const size_t off_pcnt = off_pbin + up256(WG * 4 * sizeof(double));
    const size_t off_tstat = off_pcnt + up256(WG * 4 * sizeof(unsigned));
    const size_t need = off_tstat + up256(sizeof(TStat));
    if (need > kStaticScratchBytes) return SL_ERR_TOO_LARGE;  // the fixed scratch cannot hold this tensor

    int dev = -1;
    SL_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SL_ERR_UNSUPPORTED;
    StaticSetup& su = g_static_setup[dev];
    if (!su.ready) {  // first call on this device: resolve the array's device address, size the launch
        void* ptr = nullptr;
        SL_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        int n_sms = 0, per_sm = 0;
        SL_CUDA(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
        SL_CUDA(cudaFuncSetAttribute(ef_topk_kernel<true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)sizeof(PipeSmem)));
        SL_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ef_topk_kernel<true, false, false>, kThreads,
                                                              sizeof(PipeSmem)));
        su.scratch = ptr;
        su.ef_ctas = n_sms * (per_sm > 0 ? per_sm : 1);
        su.ready = true;
    }
    char* base = static_cast<char*>(su.scratch);
    ChunkDesc* d_chunks = reinterpret_cast<ChunkDesc*>(base);
    TensorInfo* d_tinfo = reinterpret_cast<TensorInfo*>(base + off_tinfo);
    Workspace ws;
    ws.val = reinterpret_cast<float*>(base + off_val);
    ws.idx = reinterpret_cast<uint16_t*>(base + off_idx);
    ws.psum = reinterpret_cast<double*>(base + off_psum);
    ws.pbin = reinterpret_cast<double*>(base + off_pbin);
    ws.pcnt = reinterpret_cast<unsigned*>(base + off_pcnt);
    ws.tstat = reinterpret_cast<TStat*>(base + off_tstat);
    WorkerPtrs ptrs;
    memset(&ptrs, 0, sizeof(ptrs));
    ptrs.theta_local[0] = theta_local;
    ptrs.e[0] = e;
    ptrs.payload[0] = payload;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Every array is fully rewritten by the kernels below before it is read, so nothing left behind
    // by an earlier call (of any size) is ever consumed and nothing has to be cleared.
    build_single_tensor_table_kernel<<<blocks_for(G, 128), 128, 0, st>>>(rows, cols, k, G, d_chunks, d_tinfo);
    const unsigned ef_grid = (unsigned)(G < su.ef_ctas ? G : su.ef_ctas);
    TmaArgs no_tma;
    memset(&no_tma, 0, sizeof(no_tma));
    ef_topk_kernel<true, false, false><<<ef_grid, kThreads, sizeof(PipeSmem), st>>>(d_chunks, G, 1, k, kp, beta,
                                                                                   theta_sync, ptrs, ws, no_tma);
    const unsigned cb = blocks_for(G, 128);
    chunk_sum_kernel<0><<<cb, 128, 0, st>>>(d_chunks, G, 1, 1, k, kp, ws);
    tensor_reduce_kernel<0><<<1, 128, 0, st>>>(d_tinfo, G, 1, 1, ws, ptrs);
    chunk_sum_kernel<1><<<cb, 128, 0, st>>>(d_chunks, G, 1, 1, k, kp, ws);
    tensor_reduce_kernel<1><<<1, 128, 0, st>>>(d_tinfo, G, 1, 1, ws, ptrs);
    chunk_bins_kernel<<<cb, 128, 0, st>>>(d_chunks, G, 1, 1, k, kp, ws);
    tensor_reduce_kernel<2><<<1, 128, 0, st>>>(d_tinfo, G, 1, 1, ws, ptrs);
    pack_fix_kernel<1><<<blocks_for(G, 4), 128, 0, st>>>(d_chunks, G, 1, 1, k, kp, ws, ptrs);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

}  // extern "C"
