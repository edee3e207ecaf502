// Exact chunk-wise Top-k: thresholds, candidate classes, ranking, ordered emission.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"

namespace {

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
//    minimum and maximum cut the candidates (key >= T, about 2 keff of them) into four classes
//    (for k > 64: eight classes, seven equal steps between the extremes and one class above).
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
constexpr int kSmallClassCap = 112;  // ... of the compact variant for k <= 64 (about 110 candidates in all)
// For k > 64 the three splitters leave the class around the cut too large (130 entries at k = 123,
// ranked by all pairs), so larger k use eight classes: seven equal steps from the smallest to the
// largest warp value and a top class above it.  The same list storage, cut differently: seven
// lists of kWideLowCap entries and the top class (mostly certain winners, the largest) behind them.
constexpr int kWideClasses = 8;
constexpr int kWideLowCap = 88;
constexpr int kWideTopCap = 256;  // one thread per entry must suffice; 7 * 88 + 256 <= 4 * kClassCap
static_assert((kWideClasses - 1) * kWideLowCap + kWideTopCap <= 4 * kClassCap, "list storage");
inline bool wide_classes(int k) { return k > 64; }  // host: which instantiation to launch

template <int CAP>
struct SelectSmemT {
    static constexpr int kCap = CAP;  // entries per class list in the four-class scheme
    unsigned lkey[4][CAP];  // candidates per class: key
    uint16_t lpos[4][CAP];  //                        in-chunk index | sign << 12
    unsigned bitmap[2][128];   // selected positions, double-buffered by unit parity
    unsigned warp_t[8];
    __align__(16) unsigned cnt[8];
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
template <class SM>
__device__ __noinline__ void select_exact_search(const unsigned* ub, bool nonzero, int len, int keff,
                                                 SM& sm, unsigned* bitmap) {
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
template <bool WIDE, class SM>
__device__ __forceinline__ bool select_topk(const unsigned (&ub)[kPerThread], const unsigned* __restrict__ tile,
                                            int len, int keff, SM& sm, Picked& out) {
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
        if (rounds == 8) {  // k = 57..64 on full chunks, the common case: unrolled
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                tw = __reduce_max_sync(kFull, cur);
                cur = cur == tw ? 0u : cur;
            }
        } else {
            for (int i = 0; i < rounds; ++i) {
                tw = __reduce_max_sync(kFull, cur);
                cur = cur == tw ? 0u : cur;  // retire the holder (tagged values are distinct, or all 0)
            }
        }
        if (lane == 0) sm.warp_t[warp] = warp < n_warps ? (tw & ~31u) : 0xFFFFFFFFu;
        if (tid < 8) sm.cnt[tid] = 0;
    }
    __syncthreads();
    unsigned T, s1, s2, s3;
    float wide_scale;  // eight classes: class = min(7, (key - T) * wide_scale), non-decreasing in the key
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
        wide_scale = hi > lo ? (float)(kWideClasses - 1) / (float)(hi - lo) : 0.0f;
    }
    constexpr bool wide = WIDE;

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
            unsigned cls, off, cap;
            if (wide) {
                cls = min((unsigned)(kWideClasses - 1), (unsigned)((float)(kq - T) * wide_scale));
                off = cls * kWideLowCap;
                cap = cls == kWideClasses - 1 ? kWideTopCap : kWideLowCap;
            } else {
                cls = (kq >= s1 ? 1u : 0u) + (kq >= s2 ? 1u : 0u) + (kq >= s3 ? 1u : 0u);
                off = cls * SM::kCap;
                cap = SM::kCap;
            }
            const unsigned pos = atomicAdd(&sm.cnt[cls], 1u);
            if (pos < cap) {
                (&sm.lkey[0][0])[off + pos] = kq;
                (&sm.lpos[0][0])[off + pos] = (uint16_t)((unsigned)p | ((bits >> 31) << 12));
            }
        }
    }
    return exact;
}

// Second half of the selection, after the barrier that completes the class lists.  Returns true
// when a list overflowed: nothing was marked and the exact search has to run instead.
template <bool WIDE, class SM>
__device__ __forceinline__ bool select_rank(int keff, SM& sm, unsigned* bitmap, Picked& out) {
    const int tid = threadIdx.x;
    unsigned above = 0, cstar, L, list_off;
    const unsigned* __restrict__ lkf = &sm.lkey[0][0];
    const uint16_t* __restrict__ lpf = &sm.lpos[0][0];
    if (!WIDE) {
        const uint4 cn = *reinterpret_cast<const uint4*>(&sm.cnt[0]);
        // the class holding the cut: the highest class c with count(classes >= c) >= keff
        cstar = 3;
        L = cn.w;
        if (cn.w < (unsigned)keff) {
            above = cn.w; cstar = 2; L = cn.z;
            if (above + cn.z < (unsigned)keff) {
                above += cn.z; cstar = 1; L = cn.y;
                if (above + cn.y < (unsigned)keff) { above += cn.y; cstar = 0; L = cn.x; }
            }
        }
        if (max(max(cn.x, cn.y), max(cn.z, cn.w)) > (unsigned)SM::kCap) return true;  // overflow: exact search
        list_off = cstar * SM::kCap;
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
            out.p1 = lpf[c * SM::kCap + j];
            out.v1 = lkf[c * SM::kCap + j] | ((out.p1 >> 12) << 31);
            out.p1 &= 0xFFFu;
            out.mask |= 2u;
            set_bit(bitmap, out.p1);
        }
    } else {
        const uint4 c_lo = *reinterpret_cast<const uint4*>(&sm.cnt[0]), c_hi = *reinterpret_cast<const uint4*>(&sm.cnt[4]);
        const unsigned cn[kWideClasses] = {c_lo.x, c_lo.y, c_lo.z, c_lo.w, c_hi.x, c_hi.y, c_hi.z, c_hi.w};
        bool found = false, overflow = false;
        cstar = 0;
        L = 0;
#pragma unroll
        for (int c = kWideClasses - 1; c >= 0; --c) {
            overflow |= cn[c] > (unsigned)(c == kWideClasses - 1 ? kWideTopCap : kWideLowCap);
            if (!found) {
                if (above + cn[c] >= (unsigned)keff) {
                    found = true;
                    cstar = (unsigned)c;
                    L = cn[c];
                } else {
                    above += cn[c];
                }
            }
        }
        if (overflow || !found) return true;
        list_off = cstar * kWideLowCap;
        if (tid < (int)above) {
            unsigned c = kWideClasses - 1, j = tid;
            while (j >= sm.cnt[c]) {  // ends above the cut class because tid < above
                j -= sm.cnt[c];
                --c;
            }
            out.p1 = lpf[c * kWideLowCap + j];
            out.v1 = lkf[c * kWideLowCap + j] | ((out.p1 >> 12) << 31);
            out.p1 &= 0xFFFu;
            out.mask |= 2u;
            set_bit(bitmap, out.p1);
        }
    }
    const unsigned want = (unsigned)keff - above;  // 1 <= want <= L
    // the cut class: entry i = tid >> sh is ranked by 2^sh adjacent lanes, each over one segment
    const unsigned* __restrict__ lk = lkf + list_off;
    const uint16_t* __restrict__ lp = lpf + list_off;
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

}  // namespace
