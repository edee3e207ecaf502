// Entropy-coded index format: Golomb gap codes, encode and decode kernels.
// Part of libsparseloco (one translation unit: included by sparseloco.cu).
#pragma once
#include "common.cuh"

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

// Reading a worker's index stream: a 64-bit window over the 32-bit words, refilled a word at a time through
// the read-only path (consecutive words: mostly L1 hits).  `stream_bits` (a multiple of 32) = the bits the
// caller's buffer holds: words past it read as zeros, so no access ever leaves the buffer.
struct IxcReader {
    const unsigned* stream;
    unsigned long long wtot, wnext, win;
    int have;  // valid bits in `win`, lowest first
};
__device__ __forceinline__ void ixc_refill(IxcReader& rd) {  // at least 32 valid bits afterwards
    while (rd.have < 32) {
        const unsigned x = rd.wnext < rd.wtot ? __ldg(rd.stream + rd.wnext) : 0u;
        rd.win |= (unsigned long long)x << rd.have;
        rd.have += 32;
        ++rd.wnext;
    }
}
__device__ __forceinline__ void ixc_reader_open(IxcReader& rd, const unsigned* stream, unsigned long long stream_bits,
                                                unsigned long long bit_pos) {
    rd.stream = stream;
    rd.wtot = stream_bits >> 5;
    rd.wnext = bit_pos >> 5;
    rd.win = 0;
    rd.have = 0;
    ixc_refill(rd);
    const int skip = (int)(bit_pos & 31ull);
    rd.win >>= skip;
    rd.have -= skip;
}
// Decodes the m gap codes of one chunk; emit(s, index) receives the ascending indices (12 bits kept).
// Returns the bits consumed.  A damaged stream cannot run away: a run of one-bits is cut at 4096 and bits
// beyond the buffer are zeros, so every code ends.
template <typename Emit>
__device__ __forceinline__ unsigned ixc_decode_chunk(IxcReader& rd, const IxcCode code, int m, Emit emit) {
    const int nb = code.M > 1u ? (int)code.b - 1 : 0;  // remainder bits before the optional last one
    unsigned consumed = 0;
    int prev = -1;
    for (int s = 0; s < m; ++s) {
        if (rd.have < 32) {  // (at most 32 bits are taken per round below, so one word restores the 32)
            const unsigned x = rd.wnext < rd.wtot ? __ldg(rd.stream + rd.wnext) : 0u;
            rd.win |= (unsigned long long)x << rd.have;
            rd.have += 32;
            ++rd.wnext;
        }
        const unsigned lo32 = (unsigned)rd.win, inv = ~lo32;
        const int ones = __ffs(inv) - 1;  // -1 when all 32 bits are ones
        unsigned gap;
        int used;
        if (ones >= 0 && ones <= 19) {
            // the whole code lies in these 32 bits (at most 20 + 11 + 1): no branches from here on
            const unsigned w2 = lo32 >> (ones + 1);
            const unsigned r1 = nb ? __brev(w2) >> (32 - nb) : 0u;
            const bool longer = code.M > 1u && r1 >= code.cut;  // truncated binary: one more bit
            const unsigned r = longer ? ((r1 << 1) | ((w2 >> nb) & 1u)) - code.cut : r1;
            gap = (unsigned)ones * code.M + r;
            used = ones + 1 + nb + (longer ? 1 : 0);
            rd.win >>= used;
            rd.have -= used;
        } else {  // a long run of one-bits: through the window 32 bits at a time (rare; bounded)
            unsigned q = 0, iv = inv;
            used = 0;
            while (iv == 0u && q < 4096u) {
                q += 32;
                rd.win >>= 32;
                rd.have -= 32;
                used += 32;
                ixc_refill(rd);
                iv = ~(unsigned)rd.win;
            }
            const int o2 = iv ? __ffs(iv) - 1 : 0;
            q += o2;
            rd.win >>= o2 + 1;
            rd.have -= o2 + 1;
            used += o2 + 1;
            unsigned r = 0;
            if (code.M > 1u) {  // truncated binary, most significant bit first
                ixc_refill(rd);
                if (nb) r = __brev((unsigned)rd.win) >> (32 - nb);
                rd.win >>= nb;
                rd.have -= nb;
                used += nb;
                if (r >= code.cut) {
                    r = ((r << 1) | ((unsigned)rd.win & 1u)) - code.cut;
                    rd.win >>= 1;
                    rd.have -= 1;
                    used += 1;
                }
            }
            gap = q * code.M + r;
        }
        consumed += (unsigned)used;
        prev = prev + 1 + (int)gap;
        emit(s, (unsigned)prev & 0xFFFu);
    }
    return consumed;
}

// K4: coded payload -> 12-bit records.  One thread per group of 16 chunks (one directory entry).
// `stream_bits` = bits of the index stream that the caller's buffer holds: a read position taken from
// the directory is clamped to it and a bit past it reads as 0, so a corrupted directory or stream
// never makes the kernel touch memory outside the coded buffer; either case (and a directory that
// does not ascend) is recorded as SL_ERR_BAD_PAYLOAD in `status`.
__global__ void __launch_bounds__(128)
ixc_decode_kernel(const ChunkDesc* __restrict__ chunks, long long n_chunks, int n_tensors, int k,
                  const uint8_t* __restrict__ coded, unsigned long long dir_off, unsigned long long stream_off,
                  unsigned long long stream_bits, uint8_t* __restrict__ payload, int* __restrict__ status) {
    const long long grp = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (grp < 4ll * n_tensors)
        reinterpret_cast<unsigned*>(payload)[grp] = reinterpret_cast<const unsigned*>(coded)[grp];
    const long long g0 = grp * kIxcGroup;
    if (g0 >= n_chunks) return;
    const unsigned* dir = reinterpret_cast<const unsigned*>(coded + dir_off);
    unsigned long long pos = dir[grp];
    bool bad = pos > stream_bits;
    if (g0 + kIxcGroup < n_chunks) bad |= dir[grp + 1] < pos;
    if (pos > stream_bits) pos = stream_bits;
    const int cb = (2 * k + 7) / 8, ib = (12 * k + 7) / 8, stride = record_stride(k);
    IxcReader rd;
    ixc_reader_open(rd, reinterpret_cast<const unsigned*>(coded + stream_off), stream_bits, pos);
    for (long long g = g0; g < g0 + kIxcGroup && g < n_chunks; ++g) {
        const ChunkDesc cd = chunks[g];
        const int m = min(k, cd.len);
        uint8_t* recb = payload + cd.rec_off;
        unsigned* rec = reinterpret_cast<unsigned*>(recb);
        // the record is this thread's alone: index words are assembled in a register and stored
        unsigned long long acc = 0;
        unsigned fill = 0;
        int w = 0;
        pos += ixc_decode_chunk(rd, ixc_code(cd.len, m), m, [&](int, unsigned idx) {
            acc |= (unsigned long long)idx << fill;
            fill += 12;
            if (fill >= 32) {
                rec[w++] = (unsigned)acc;
                acc >>= 32;
                fill -= 32;
            }
        });
        // rest of the index block, the code block, the padding: byte-wise after the whole words
        int byte = 4 * w;
        for (; byte < ib; ++byte, acc >>= 8) recb[byte] = (uint8_t)(acc & 0xFFu);
        const uint8_t* csrc = coded + 16ll * n_tensors + (long long)cb * g;
        for (int i = 0; i < cb; ++i) recb[ib + i] = csrc[i];
        for (byte = ib + cb; byte < stride; ++byte) recb[byte] = 0;
    }
    if (pos > stream_bits) bad = true;  // the codes ran past what the buffer holds
    if (bad) atomicExch(status, (int)SL_ERR_BAD_PAYLOAD);
}

}  // namespace
