// SparseLoCo outer step for sm_100a: the C ABI declared in include/sparseloco.h (host side, this
// file) over the kernels in the .cuh files beside it (one translation unit).
//
// Kernel sequence of one outer step (all on the caller's stream, no host synchronisation):
//   ef_select.cuh    ef_select_kernel         pseudo-gradient + error feedback + chunk-wise Top-k
//                                             (Eq. 2 line 1, Sec. 3.3), one warp per (chunk, worker)
//   quantiser.cuh    chunk_sum_kernel<0>      per-chunk fp64 sum of the selected values   (Sec. 4: mean)
//                    tensor_reduce_kernel<0>  grouped fp64 sum per (worker, tensor) -> mu
//                    chunk_sum_kernel<1>      per-chunk fp64 sum of squared centred values
//                    tensor_reduce_kernel<1>  -> sigma, bin edge 3 sigma
//                    chunk_bins_kernel        per-chunk per-bin sums and counts           (centroids)
//                    tensor_reduce_kernel<2>  -> 4-entry table, written to the payload header
//   pack.cuh         pack_fix_kernel          codes, 12-bit index + 2-bit code packing, e = u - Dhat
//                                             (Eq. 2 line 2); in sl_outer_step this runs inside:
//   apply.cuh        decode_avg_apply_kernel  decode R payloads, sum, theta -= alpha/D * sum
//                                             (Eq. 2 lines 3-4)
// Beside the path: index_codec.cuh (entropy-coded indices for the wire), dense.cuh (DiLoCo's dense
// outer step, Eq. 1, and the local-momentum baselines), misc.cuh (payload validation), quant_wide.cuh
// (quantiser widths 1, 3, 4 and k beyond 256: plain kernels), bf16_storage.cuh (the selection kernel
// for bfloat16 arrays).
//
// Everything is HBM-bound streaming except the per-chunk selection, which works on registers and
// shared memory.  No tensor cores: nothing here is a dense contraction.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "sparseloco.h"

#include "common.cuh"
#include "ef_select.cuh"
#include "quantiser.cuh"
#include "pack.cuh"
#include "apply.cuh"
#include "quant_wide.cuh"
#include "bf16_storage.cuh"
#include "misc.cuh"
#include "index_codec.cuh"
#include "dense.cuh"

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
    int qbits;          // bits per code in the payload (2 also when quant_bits = 32: no payload is written then)
    int rec_stride;     // bytes of one chunk record
    long long rec_base; // byte offset of the first record in a payload (after the tensor tables)
    std::vector<sl_tensor_desc> tensors;
    ChunkDesc* d_chunks;
    TensorInfo* d_tinfo;
    int ef_ctas;  // resident CTAs of the compact compression kernel on this device (informational)
    int n_sms;
    // tensor-map (TMA) block copies: usable when every full chunk starts on a 64-element boundary
    bool tma_ok, tma_on;
    int n_classes;
    int class_rs[kMaxTmaClasses];       // distinct row lengths of full chunks (64 for flat runs)
    CUtensorMap* d_maps;                // [kMapSlots][n_classes]
    std::vector<CUtensorMap> h_maps;    // host copy the device array is filled from
    std::vector<const void*> slot_ptr;  // buffer described by each slot
    bool slots_cleared;                 // the slot table was emptied during the current assignment
    bool maps_fresh;                    // maps were (re)written since the last compression launch
    bool upload_pending;                // ... and that upload has no event yet
    cudaEvent_t upload_event;           // recorded after the last upload, on upload_stream
    cudaStream_t upload_stream;
    int* d_status;                      // device status word (SL_OK or what a kernel recorded)
    // entropy-coded payload: byte offsets of the directory and the index stream, worst-case size
    size_t ixc_dir_off, ixc_stream_off, ixc_capacity;
    bool deferred;              // deferred error-feedback subtraction (sl_set_ef_deferred)
    bool pending;               // corrected values of the last step still wait in the workspace
    float* pending_e[kMaxR];    // the error buffers they belong to
    int pending_workers;        // how many workers' values wait (R after sl_outer_step, 1 after sl_compress)
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

constexpr int kMapSlots = 2 * kMaxR + 2;  // buffers with tensor maps at one time: theta, theta_local and e of every worker

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

// general-width quantiser (quant_bits 1, 3, 4): its per-unit bin partials and per-tensor tables follow
// the arrays of the 2-bit path in the workspace
// (also the 2-bit quantiser at k > 256, which the fused kernels are not laid out for)
inline bool half_store(const sl_ctx* c) { return c->cfg.bf16_storage != 0; }
inline bool wide_quant(const sl_ctx* c) {
    return c->cfg.quant_bits != 32 && (c->cfg.quant_bits != 2 || c->cfg.k > kFastMaxK);
}
// the paper's setting (2 bits, k <= 256): the tuned kernels, the deferred subtraction, the wire codec; fp32 or bfloat16 arrays
inline bool fast_2bit(const sl_ctx* c) { return c->cfg.quant_bits == 2 && c->cfg.k <= kFastMaxK; }
size_t wide_bytes_for(const sl_ctx* c, int workers) {
    if (!wide_quant(c)) return 0;
    const size_t WG = (size_t)workers * (size_t)c->n_chunks, nb = (size_t)1 << c->qbits;
    return up256(WG * nb * sizeof(double)) + up256(WG * nb * sizeof(unsigned)) +
           up256((size_t)workers * c->n_tensors * sizeof(TStatQ));
}

size_t narrow_bytes_for(const sl_ctx* c, int workers) {
    const size_t WG = (size_t)workers * (size_t)c->n_chunks;
    return up256(WG * c->kp * sizeof(float)) + up256(WG * c->kp * sizeof(uint16_t)) +
           up256(WG * sizeof(double)) + up256(WG * 4 * sizeof(double)) + up256(WG * 4 * sizeof(unsigned)) +
           up256((size_t)workers * c->n_tensors * sizeof(TStat));
}

size_t workspace_bytes_for(const sl_ctx* c, int workers) { return narrow_bytes_for(c, workers) + wide_bytes_for(c, workers); }

struct WideSpace {
    double* pbin;
    unsigned* pcnt;
    TStatQ* tq;
};
WideSpace carve_wide(const sl_ctx* c, int workers) {
    const size_t WG = (size_t)workers * (size_t)c->n_chunks, nb = (size_t)1 << c->qbits;
    char* p = static_cast<char*>(c->ws_ptr) + narrow_bytes_for(c, workers);
    WideSpace w;
    w.pbin = reinterpret_cast<double*>(p);      p += up256(WG * nb * sizeof(double));
    w.pcnt = reinterpret_cast<unsigned*>(p);    p += up256(WG * nb * sizeof(unsigned));
    w.tq = reinterpret_cast<TStatQ*>(p);
    return w;
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
    c->maps_fresh = true;     // the next launch fences before its first copy through a rewritten map
    c->upload_pending = true; // ... and other streams must be ordered after this upload
    return slot;
}

// Tensor maps are uploaded on the stream of the call that first sees a buffer.  A later call on another
// stream finds the slot by pointer alone, so it is ordered after the last upload through an event.
sl_status order_after_map_uploads(sl_ctx* c, cudaStream_t st) {
    if (c->upload_pending) {
        if (!c->upload_event) SL_CUDA(cudaEventCreateWithFlags(&c->upload_event, cudaEventDisableTiming));
        SL_CUDA(cudaEventRecord(c->upload_event, st));
        c->upload_stream = st;
        c->upload_pending = false;
    } else if (c->upload_event && st != c->upload_stream) {
        // (not while `st` is being captured into a graph: the event belongs to no capture; the header
        // asks for one ordinary call with the same buffers before a capture, which is what orders it)
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        SL_CUDA(cudaStreamIsCapturing(st, &cap));
        if (cap == cudaStreamCaptureStatusNone) SL_CUDA(cudaStreamWaitEvent(st, c->upload_event, 0));
    }
    return SL_OK;
}

sl_status launch_flush(sl_ctx* c, const WorkerPtrs& ptrs, cudaStream_t st) {
    const int R = c->pending_workers;  // (the staging arrays are laid out for the call that left the values)
    const Workspace ws = carve(c, R);
    if (half_store(c))
        ef_flush_kernel<false, true><<<blocks_for(c->n_chunks * R, 4), 128, 0, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k,
                                                                                     c->kp, ws, ptrs);
    else
        ef_flush_kernel<false><<<blocks_for(c->n_chunks * R, 4), 128, 0, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, c->kp,
                                                                               ws, ptrs);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

// Writes +0 at the staged positions of every worker's buffer in `bufs` (what Top-k leaves behind there).
sl_status launch_zero_selected(sl_ctx* c, float* const* bufs, cudaStream_t st) {
    const int R = c->cfg.R;
    WorkerPtrs zp;
    memset(&zp, 0, sizeof(zp));
    for (int r = 0; r < R; ++r) zp.e[r] = bufs[r];
    ef_flush_kernel<true><<<blocks_for(c->n_chunks * R, 4), 128, 0, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, c->kp,
                                                                          carve(c, R), zp);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

// The waiting values of a deferred subtraction go into the buffers of the step that left them.
sl_status flush_pending(sl_ctx* c, cudaStream_t st) {
    if (!c->pending) return SL_OK;
    WorkerPtrs fp;
    memset(&fp, 0, sizeof(fp));
    for (int r = 0; r < c->pending_workers; ++r) fp.e[r] = c->pending_e[r];
    sl_status s = launch_flush(c, fp, st);
    if (s == SL_OK) c->pending = false;
    return s;
}

// Kernel 1 for `workers` workers: u (from theta - theta_r, or with `delta` from the vectors in the
// theta_local slots themselves), error feedback when `ef`, chunk-wise Top-k into the staging arrays.
// `consume`: substitute the waiting values of a deferred subtraction on the way.
sl_status launch_select(sl_ctx* c, int workers, const float* theta_sync, const WorkerPtrs& ptrs, cudaStream_t st,
                        bool ef, bool consume, bool delta) {
    const Workspace ws = carve(c, workers);
    const long long G = c->n_chunks;
    const int k = c->cfg.k, kp = c->kp;
    if (half_store(c)) {  // bfloat16 arrays: the warp-per-unit kernel with plain loads
        if (delta || (consume && k > kFastMaxK)) return SL_ERR_UNSUPPORTED;
        const long long units = G * workers;
        const long long want = (units + kHalfSelWarps - 1) / kHalfSelWarps;
        const unsigned grid = (unsigned)(want < c->n_sms ? (want < 1 ? 1 : want) : c->n_sms);
        const bf16_bits* ts = reinterpret_cast<const bf16_bits*>(theta_sync);
#define SL_LAUNCH_HALF(EFV)                                                                                        \
    do {                                                                                                           \
        if (k > kFastMaxK)                                                                                         \
            ef_select_bf16_kernel<EFV, 2><<<grid, kHalfSelThreads, sizeof(HalfSelSmem), st>>>(                     \
                c->d_chunks, G, workers, k, kp, c->cfg.beta, ts, ptrs, ws);                                        \
        else if (k > kSelNarrowMaxK)                                                                               \
            ef_select_bf16_kernel<EFV, 1><<<grid, kHalfSelThreads, sizeof(HalfSelSmem), st>>>(                     \
                c->d_chunks, G, workers, k, kp, c->cfg.beta, ts, ptrs, ws);                                        \
        else                                                                                                       \
            ef_select_bf16_kernel<EFV, 0><<<grid, kHalfSelThreads, sizeof(HalfSelSmem), st>>>(                     \
                c->d_chunks, G, workers, k, kp, c->cfg.beta, ts, ptrs, ws);                                        \
    } while (0)
        if (ef && consume) {
            if (k > kSelNarrowMaxK)
                ef_select_bf16_kernel<true, 1, true><<<grid, kHalfSelThreads, sizeof(HalfSelSmem), st>>>(
                    c->d_chunks, G, workers, k, kp, c->cfg.beta, ts, ptrs, ws);
            else
                ef_select_bf16_kernel<true, 0, true><<<grid, kHalfSelThreads, sizeof(HalfSelSmem), st>>>(
                    c->d_chunks, G, workers, k, kp, c->cfg.beta, ts, ptrs, ws);
        } else if (ef) SL_LAUNCH_HALF(true);
        else SL_LAUNCH_HALF(false);
#undef SL_LAUNCH_HALF
        SL_CUDA(cudaGetLastError());
        return SL_OK;
    }
    // tile copies through tensor maps when the table allows it and every buffer got its maps
    TmaArgs ta;
    memset(&ta, 0, sizeof(ta));
    ta.status = c->d_status;
    bool use_tma = c->tma_on;
    if (use_tma) {
        ta.maps = c->d_maps;
        ta.n_classes = c->n_classes;
        for (int q = 0; q < c->n_classes; ++q) ta.class_rs[q] = c->class_rs[q];
        for (int pass = 0; pass < 2 && use_tma; ++pass) {
            // if the slot table fills up half-way, it is emptied and the assignment starts over: one
            // call needs at most 2 R + 1 slots, which an empty table holds
            c->slots_cleared = false;
            ta.slot_s = delta ? 0 : tma_map_slot(c, theta_sync, st);
            use_tma = ta.slot_s >= 0;
            for (int r = 0; r < workers && use_tma; ++r) {
                ta.slot_l[r] = tma_map_slot(c, ptrs.theta_local[r], st);
                ta.slot_e[r] = ef ? tma_map_slot(c, ptrs.e[r], st) : 0;
                use_tma = ta.slot_l[r] >= 0 && ta.slot_e[r] >= 0;
            }
            if (!c->slots_cleared) break;
        }
        if (use_tma) {
            sl_status s = order_after_map_uploads(c, st);
            if (s != SL_OK) return s;
            ta.fresh = c->maps_fresh ? 1 : 0;
            c->maps_fresh = false;
        }
    }
    // one persistent CTA per SM
    const unsigned grid = (unsigned)(G < c->n_sms ? G : c->n_sms);
    const int tm = use_tma ? 1 : 0;
#define SL_LAUNCH_SELECT(EFV, PENDV, DELTAV)                                                                         \
    do {                                                                                                             \
        if (k > kSelNarrowMaxK)                                                                                      \
            ef_select_kernel<EFV, PENDV, 1, DELTAV><<<grid, kSelThreads, sizeof(SelSmem), st>>>(                     \
                c->d_chunks, G, workers, k, kp, c->cfg.beta, theta_sync, ptrs, ws, ta, tm);                          \
        else                                                                                                         \
            ef_select_kernel<EFV, PENDV, 0, DELTAV><<<grid, kSelThreads, sizeof(SelSmem), st>>>(                     \
                c->d_chunks, G, workers, k, kp, c->cfg.beta, theta_sync, ptrs, ws, ta, tm);                          \
    } while (0)
    if (k > kFastMaxK) {  // the dense settings: no waiting lists, no baselines (refused before this point)
        if (consume || delta) return SL_ERR_UNSUPPORTED;
        if (ef)
            ef_select_kernel<true, false, 2><<<grid, kSelThreads, sizeof(SelSmem), st>>>(
                c->d_chunks, G, workers, k, kp, c->cfg.beta, theta_sync, ptrs, ws, ta, tm);
        else
            ef_select_kernel<false, false, 2><<<grid, kSelThreads, sizeof(SelSmem), st>>>(
                c->d_chunks, G, workers, k, kp, c->cfg.beta, theta_sync, ptrs, ws, ta, tm);
    } else if (delta) {
        if (ef) SL_LAUNCH_SELECT(true, false, true);
        else SL_LAUNCH_SELECT(false, false, true);
    } else if (!ef) {
        SL_LAUNCH_SELECT(false, false, false);
    } else if (consume) {
        SL_LAUNCH_SELECT(true, true, false);
    } else {
        SL_LAUNCH_SELECT(true, false, false);
    }
#undef SL_LAUNCH_SELECT
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
        bool same = c->pending_workers == workers;  // the values of exactly these buffers, in the same layout
        for (int r = 0; r < workers && same; ++r) same = ptrs.e[r] == c->pending_e[r];
        if (ef && defer && same) {
            consume = true;
            c->pending = false;
        } else {  // nothing will read them in flight (frozen step, other buffers): write them out first
            sl_status s = flush_pending(c, st);
            if (s != SL_OK) return s;
        }
    }

    prof_mark(c, -1, st);
    {
        sl_status s = launch_select(c, workers, theta_sync, ptrs, st, ef, consume, false);
        if (s != SL_OK) return s;
    }
    prof_mark(c, 0, st);
    const unsigned cb = blocks_for(WG, 128), tb = blocks_for((long long)workers * T, 4);
    const unsigned tr = (unsigned)((long long)workers * T);  // tensor_reduce_kernel: one CTA per (worker, tensor)
    chunk_sum_kernel<0><<<cb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws);
    prof_mark(c, 1, st);
    tensor_reduce_kernel<0><<<tr, 128, 0, st>>>(c->d_tinfo, G, workers, T, ws, ptrs);
    prof_mark(c, 2, st);
    chunk_sum_kernel<1><<<cb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws);
    prof_mark(c, 3, st);
    tensor_reduce_kernel<1><<<tr, 128, 0, st>>>(c->d_tinfo, G, workers, T, ws, ptrs);
    prof_mark(c, 4, st);
    if (wide_quant(c)) {  // 1, 3 or 4 bits: the general-width kernels, records and error correction in place
        const WideSpace wq = carve_wide(c, workers);
        const unsigned pbq = blocks_for(WG, 4);
#define SL_WIDE(BITSV)                                                                                              \
    do {                                                                                                            \
        chunk_bins_q_kernel<BITSV><<<cb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, wq.pbin, wq.pcnt);    \
        tensor_table_q_kernel<BITSV><<<tb, 128, 0, st>>>(c->d_tinfo, G, workers, T, wq.pbin, wq.pcnt, wq.tq, ptrs); \
        if (ef && half_store(c))                                                                                    \
            pack_q_kernel<BITSV, true, true><<<pbq, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, wq.tq, c->rec_base, ptrs); \
        else if (ef)                                                                                                \
            pack_q_kernel<BITSV, true><<<pbq, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, wq.tq, c->rec_base, ptrs); \
        else                                                                                                        \
            pack_q_kernel<BITSV, false><<<pbq, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, wq.tq, c->rec_base, ptrs); \
    } while (0)
        if (c->qbits == 1) SL_WIDE(1);
        else if (c->qbits == 2) SL_WIDE(2);
        else if (c->qbits == 3) SL_WIDE(3);
        else SL_WIDE(4);
#undef SL_WIDE
        prof_mark(c, 5, st);
        prof_mark(c, 6, st);
        prof_mark(c, 7, st);
        SL_CUDA(cudaGetLastError());
        return SL_OK;
    }
    chunk_bins_kernel<<<cb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws);
    prof_mark(c, 5, st);
    tensor_reduce_kernel<2><<<tr, 128, 0, st>>>(c->d_tinfo, G, workers, T, ws, ptrs);
    prof_mark(c, 6, st);
    const unsigned pb = blocks_for(WG, 4);
    if (skip_pack)
        ;  // records, error correction: done by decode_avg_apply_kernel<., 1 or 2>
    else if (!ef)
        pack_fix_kernel<0><<<pb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, ptrs);
    else if (defer)
        pack_fix_kernel<2><<<pb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, ptrs);
    else if (half_store(c))
        pack_fix_kernel<1, true><<<pb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, ptrs);
    else
        pack_fix_kernel<1><<<pb, 128, 0, st>>>(c->d_chunks, G, workers, T, k, kp, ws, ptrs);
    prof_mark(c, 7, st);
    SL_CUDA(cudaGetLastError());
    if (ef && defer) {
        c->pending = true;
        c->pending_workers = workers;
        for (int r = 0; r < workers; ++r) c->pending_e[r] = ptrs.e[r];
    }
    return SL_OK;
}

// fuse: 0 = payloads in, 1 / 2 = also do the packing step of a compression in flight (see the kernel)
// fuse 3 / 4: the Top-k baselines (raw staged values; 4 = Nesterov outer step with `momentum`, `mu`)
sl_status launch_apply(sl_ctx* c, const PayloadPtrs& pl, int present, float* theta_sync, cudaStream_t st, int fuse = 0,
                       const WorkerPtrs* fuse_ptrs = nullptr, float* momentum = nullptr, float mu = 0.0f) {
    if (present == 0) return SL_OK;
    const int R = c->cfg.R;
    const double D = c->cfg.divide_by_present ? (double)present : (double)R;
    const float scale = (float)(-(double)c->cfg.outer_lr / D);
    if (wide_quant(c) && fuse == 0) {  // payloads of 1, 3 or 4 bits per value
        const unsigned grid = (unsigned)c->n_chunks;
#define SL_APPLY_Q(BITSV)                                                                                          \
    do {                                                                                                           \
        if (half_store(c))                                                                                         \
            apply_q_kernel<BITSV, true><<<grid, kThreads, 0, st>>>(c->d_chunks, R, c->cfg.k, scale, pl, c->rec_base, theta_sync); \
        else                                                                                                       \
            apply_q_kernel<BITSV><<<grid, kThreads, 0, st>>>(c->d_chunks, R, c->cfg.k, scale, pl, c->rec_base, theta_sync); \
    } while (0)
        if (c->qbits == 1) SL_APPLY_Q(1);
        else if (c->qbits == 2) SL_APPLY_Q(2);
        else if (c->qbits == 3) SL_APPLY_Q(3);
        else SL_APPLY_Q(4);
#undef SL_APPLY_Q
        prof_mark(c, 8, st);
        if (c->prof_on && c->prof_steps < kProfMaxSeq) c->prof_steps++;
        SL_CUDA(cudaGetLastError());
        return SL_OK;
    }
    const size_t smem = apply_smem_bytes(c->cfg.k);
    const int ppl = (c->cfg.k + 63) / 64;
    FuseArgs fa;
    memset(&fa, 0, sizeof(fa));
    WorkerPtrs wp;
    memset(&wp, 0, sizeof(wp));
    if (fuse) {
        fa.ws = carve(c, R);
        fa.n_chunks = c->n_chunks;
        fa.n_tensors = c->n_tensors;
        fa.kp = c->kp;
        fa.momentum = momentum;
        fa.mu = mu;
        fa.alpha = c->cfg.outer_lr;
        fa.divisor = (float)D;
        if (fuse_ptrs) wp = *fuse_ptrs;
    }
    // persistent CTAs: as many as are resident at once
    // (a CTA's shared memory grows with k: 227 KB per SM, 1 KB reserved per CTA)
    const long long fit = (227ll * 1024) / ((long long)smem + 1024);
    const long long resident = (long long)c->n_sms * (fit < kApplyCtasPerSm ? (fit < 1 ? 1 : fit) : kApplyCtasPerSm);
    const unsigned grid = (unsigned)(c->n_chunks < resident ? c->n_chunks : resident);
#define SL_APPLY_H(PPLV)                                                                                        \
    do {                                                                                                        \
        auto kern = fuse == 0 ? decode_avg_apply_kernel<PPLV, 0, true>                                          \
                  : fuse == 1 ? decode_avg_apply_kernel<PPLV, 1, true> : decode_avg_apply_kernel<PPLV, 2, true>; \
        kern<<<grid, kApplyThreads, smem, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, scale, pl, theta_sync, fa, wp); \
    } while (0)
    if (half_store(c)) {
        if (fuse > 2) return SL_ERR_UNSUPPORTED;
        if (ppl <= 1) SL_APPLY_H(1);
        else if (ppl <= 2) SL_APPLY_H(2);
        else SL_APPLY_H(4);
        prof_mark(c, 8, st);
        if (c->prof_on && c->prof_steps < kProfMaxSeq) c->prof_steps++;
        SL_CUDA(cudaGetLastError());
        return SL_OK;
    }
#undef SL_APPLY_H
#define SL_APPLY(PPLV)                                                                                          \
    do {                                                                                                        \
        auto kern = fuse == 0 ? decode_avg_apply_kernel<PPLV, 0>                                                \
                  : fuse == 1 ? decode_avg_apply_kernel<PPLV, 1>                                                \
                  : fuse == 2 ? decode_avg_apply_kernel<PPLV, 2>                                                \
                  : fuse == 3 ? decode_avg_apply_kernel<PPLV, 3> : decode_avg_apply_kernel<PPLV, 4>;            \
        kern<<<grid, kApplyThreads, smem, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, scale, pl, theta_sync, fa, wp); \
    } while (0)
    if (ppl <= 1) SL_APPLY(1);
    else if (ppl <= 2) SL_APPLY(2);
    else SL_APPLY(4);
#undef SL_APPLY
    prof_mark(c, 8, st);
    if (c->prof_on && c->prof_steps < kProfMaxSeq) c->prof_steps++;
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

// Eq. 2 lines 3-4 straight from entropy-coded payloads (decode_avg_apply_kernel<., 5>).
sl_status launch_apply_coded(sl_ctx* c, const PayloadPtrs& pl, const size_t* coded_bytes, int present, float* theta_sync,
                             cudaStream_t st) {
    if (present == 0) return SL_OK;
    const int R = c->cfg.R;
    const double D = c->cfg.divide_by_present ? (double)present : (double)R;
    const float scale = (float)(-(double)c->cfg.outer_lr / D);
    FuseArgs fa;
    memset(&fa, 0, sizeof(fa));
    fa.n_chunks = c->n_chunks;
    fa.n_tensors = c->n_tensors;
    fa.kp = c->kp;
    fa.dir_off = c->ixc_dir_off;
    fa.stream_off = c->ixc_stream_off;
    fa.status = c->d_status;
    for (int r = 0; r < R; ++r) fa.stream_bits[r] = pl.p[r] ? (unsigned long long)((coded_bytes[r] - c->ixc_stream_off) / 4 * 4) * 8ull : 0ull;
    WorkerPtrs wp;
    memset(&wp, 0, sizeof(wp));
    // + two index lists per worker (each rounded up to 8 entries) and the words the two groups of warps meet through
    const size_t smem = apply_smem_bytes(c->cfg.k) + 2 * (((size_t)R * c->kp + 7) / 8 * 8) * sizeof(uint16_t) + 32;
    if (smem > 227u * 1024u) return SL_ERR_UNSUPPORTED;
    const long long groups = (c->n_chunks + kIxcGroup - 1) / kIxcGroup;
    const long long fit = (227ll * 1024) / ((long long)smem + 1024);
    const long long resident = (long long)c->n_sms * (fit < kApplyCtasPerSm ? (fit < 1 ? 1 : fit) : kApplyCtasPerSm);
    const unsigned grid = (unsigned)(groups < resident ? groups : resident);
    const int ppl = (c->cfg.k + 63) / 64;
    if (ppl <= 1)
        decode_avg_apply_kernel<1, 5><<<grid, kApplyThreads + kApplyDecoders, smem, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, scale, pl, theta_sync, fa, wp);
    else if (ppl <= 2)
        decode_avg_apply_kernel<2, 5><<<grid, kApplyThreads + kApplyDecoders, smem, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, scale, pl, theta_sync, fa, wp);
    else
        decode_avg_apply_kernel<4, 5><<<grid, kApplyThreads + kApplyDecoders, smem, st>>>(c->d_chunks, c->n_chunks, R, c->cfg.k, scale, pl, theta_sync, fa, wp);
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
    if (cfg->chunk_elems != kChunk || cfg->tile_dim != kTile) return SL_ERR_UNSUPPORTED;
    if (cfg->quant_bits != 32 && (cfg->quant_bits < 1 || cfg->quant_bits > 4)) return SL_ERR_UNSUPPORTED;
    if (cfg->k > kMaxK || cfg->R > kMaxR) return SL_ERR_UNSUPPORTED;
    if (cfg->k > kFastMaxK && cfg->quant_bits == 32) return SL_ERR_UNSUPPORTED;  // the unquantised kernels stop at 256
    if (cfg->bf16_storage != 0 && cfg->bf16_storage != 1) return SL_ERR_INVALID_ARG;
    if (cfg->bf16_storage && cfg->quant_bits == 32) return SL_ERR_UNSUPPORTED;

    {   // element ranges: no overflow, no two tensors sharing an element (kernels of different chunks would race)
        std::vector<std::pair<long long, long long>> span((size_t)n_tensors);
        for (int j = 0; j < n_tensors; ++j) {
            const sl_tensor_desc& t = tensors[j];
            if (t.rows < 1 || t.cols < 1 || t.offset < 0) return SL_ERR_INVALID_ARG;
            if (t.cols > 0x7FFFFFFFll || t.rows > (1ll << 40) / t.cols || t.offset > (1ll << 46)) return SL_ERR_TOO_LARGE;
            span[(size_t)j] = {(long long)t.offset, (long long)t.offset + t.rows * t.cols};
        }
        std::sort(span.begin(), span.end());
        for (int j = 1; j < n_tensors; ++j)
            if (span[(size_t)j].first < span[(size_t)j - 1].second) return SL_ERR_INVALID_ARG;
    }
    sl_ctx* c = new (std::nothrow) sl_ctx();
    if (!c) return SL_ERR_NOMEM;
    c->cfg = *cfg;
    c->n_tensors = n_tensors;
    c->kp = (cfg->k + 7) / 8 * 8;
    c->d_chunks = nullptr;
    c->d_tinfo = nullptr;
    c->ef_ctas = 0;
    c->tma_ok = c->tma_on = false;
    c->slots_cleared = false;
    c->maps_fresh = c->upload_pending = false;
    c->upload_event = nullptr;
    c->upload_stream = nullptr;
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

    c->qbits = cfg->quant_bits == 32 ? 2 : cfg->quant_bits;
    const int stride = record_stride_q(cfg->k, c->qbits);  // = record_stride(k) at 2 bits
    c->rec_stride = stride;
    c->rec_base = (long long)header_bytes_q(c->qbits) * n_tensors;
    std::vector<ChunkDesc> chunks;
    std::vector<TensorInfo> tinfo((size_t)n_tensors);
    long long rec_off = c->rec_base, flat = 0, slots = 0;
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
#define SL_SELECT_ATTR(EFV, PENDV, WIDEV)                                                                            \
    if (e == cudaSuccess)                                                                                            \
        e = cudaFuncSetAttribute(ef_select_kernel<EFV, PENDV, WIDEV>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                                 (int)sizeof(SelSmem))
    SL_SELECT_ATTR(true, false, 0); SL_SELECT_ATTR(true, true, 0); SL_SELECT_ATTR(false, false, 0);
    SL_SELECT_ATTR(true, false, 1); SL_SELECT_ATTR(true, true, 1); SL_SELECT_ATTR(false, false, 1);
    SL_SELECT_ATTR(true, false, 2); SL_SELECT_ATTR(false, false, 2);
#undef SL_SELECT_ATTR
#define SL_SELECT_ATTR_D(EFV, WIDEV)                                                                                 \
    if (e == cudaSuccess)                                                                                            \
        e = cudaFuncSetAttribute(ef_select_kernel<EFV, false, WIDEV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                 (int)sizeof(SelSmem))
    SL_SELECT_ATTR_D(true, 0); SL_SELECT_ATTR_D(false, 0); SL_SELECT_ATTR_D(true, 1); SL_SELECT_ATTR_D(false, 1);
#undef SL_SELECT_ATTR_D
#define SL_HALF_ATTR(EFV, WIDEV)                                                                                     \
    if (e == cudaSuccess)                                                                                            \
        e = cudaFuncSetAttribute(ef_select_bf16_kernel<EFV, WIDEV>, cudaFuncAttributeMaxDynamicSharedMemorySize,     \
                                 (int)sizeof(HalfSelSmem))
    SL_HALF_ATTR(true, 0); SL_HALF_ATTR(false, 0); SL_HALF_ATTR(true, 1); SL_HALF_ATTR(false, 1);
    SL_HALF_ATTR(true, 2); SL_HALF_ATTR(false, 2);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(ef_select_bf16_kernel<true, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(HalfSelSmem));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(ef_select_bf16_kernel<true, 1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)sizeof(HalfSelSmem));
#undef SL_HALF_ATTR
    per_sm = 1;
    {   // the apply kernel's shared memory grows with k (and, for coded payloads, with R): the limit is a property of
        // the function, shared by every context of the process, so it is set to the most any context can ask for
        const int asz = 227 * 1024;
#define SL_APPLY_ATTR(PPLV, FUSEV)                                                                                     \
    if (e == cudaSuccess)                                                                                              \
        e = cudaFuncSetAttribute(decode_avg_apply_kernel<PPLV, FUSEV>, cudaFuncAttributeMaxDynamicSharedMemorySize, asz)
        SL_APPLY_ATTR(1, 0); SL_APPLY_ATTR(1, 1); SL_APPLY_ATTR(1, 2); SL_APPLY_ATTR(1, 3); SL_APPLY_ATTR(1, 4);
        SL_APPLY_ATTR(2, 0); SL_APPLY_ATTR(2, 1); SL_APPLY_ATTR(2, 2); SL_APPLY_ATTR(2, 3); SL_APPLY_ATTR(2, 4);
        SL_APPLY_ATTR(4, 0); SL_APPLY_ATTR(4, 1); SL_APPLY_ATTR(4, 2); SL_APPLY_ATTR(4, 3); SL_APPLY_ATTR(4, 4);
        SL_APPLY_ATTR(1, 5); SL_APPLY_ATTR(2, 5); SL_APPLY_ATTR(4, 5);
#define SL_APPLY_ATTR_H(PPLV, FUSEV)                                                                                   \
    if (e == cudaSuccess)                                                                                              \
        e = cudaFuncSetAttribute(decode_avg_apply_kernel<PPLV, FUSEV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, asz)
        SL_APPLY_ATTR_H(1, 0); SL_APPLY_ATTR_H(1, 1); SL_APPLY_ATTR_H(1, 2);
        SL_APPLY_ATTR_H(2, 0); SL_APPLY_ATTR_H(2, 1); SL_APPLY_ATTR_H(2, 2);
        SL_APPLY_ATTR_H(4, 0); SL_APPLY_ATTR_H(4, 1); SL_APPLY_ATTR_H(4, 2);
#undef SL_APPLY_ATTR_H
#undef SL_APPLY_ATTR
    }
    c->n_sms = n_sms;
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
    if (c->upload_event) cudaEventDestroy(c->upload_event);
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
    *bytes = (size_t)c->rec_base + (size_t)c->rec_stride * (size_t)c->n_chunks;
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

namespace {
sl_status do_compress(sl_ctx* c, const float* theta_sync, const float* theta_local, float* e, uint8_t* payload,
                      void* stream);
sl_status do_aggregate_apply(sl_ctx* c, const uint8_t* const* payloads, float* theta_sync, void* stream);
sl_status do_outer_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* const* e,
                        uint8_t* const* payloads, void* stream);
sl_status do_ef_flush(sl_ctx* c, float* const* e, int32_t keep_pending, void* stream);
}  // namespace

// The fp32 entry points refuse a context made for bfloat16 storage and the other way round: the element
// type of the arrays is fixed when the context is created.
sl_status sl_compress(sl_ctx* c, const float* theta_sync, const float* theta_local, float* e, uint8_t* payload,
                      void* stream) {
    if (c && half_store(c)) return SL_ERR_UNSUPPORTED;
    return do_compress(c, theta_sync, theta_local, e, payload, stream);
}
sl_status sl_aggregate_apply(sl_ctx* c, const uint8_t* const* payloads, float* theta_sync, void* stream) {
    if (c && half_store(c)) return SL_ERR_UNSUPPORTED;
    return do_aggregate_apply(c, payloads, theta_sync, stream);
}
sl_status sl_outer_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* const* e,
                        uint8_t* const* payloads, void* stream) {
    if (c && half_store(c)) return SL_ERR_UNSUPPORTED;
    return do_outer_step(c, theta_sync, theta_local, e, payloads, stream);
}
sl_status sl_compress_bf16(sl_ctx* c, const uint16_t* theta_sync, const uint16_t* theta_local, uint16_t* e,
                           uint8_t* payload, void* stream) {
    if (c && !half_store(c)) return SL_ERR_UNSUPPORTED;
    return do_compress(c, reinterpret_cast<const float*>(theta_sync), reinterpret_cast<const float*>(theta_local),
                       reinterpret_cast<float*>(e), payload, stream);
}
sl_status sl_aggregate_apply_bf16(sl_ctx* c, const uint8_t* const* payloads, uint16_t* theta_sync, void* stream) {
    if (c && !half_store(c)) return SL_ERR_UNSUPPORTED;
    return do_aggregate_apply(c, payloads, reinterpret_cast<float*>(theta_sync), stream);
}
sl_status sl_outer_step_bf16(sl_ctx* c, uint16_t* theta_sync, const uint16_t* const* theta_local, uint16_t* const* e,
                             uint8_t* const* payloads, void* stream) {
    if (c && !half_store(c)) return SL_ERR_UNSUPPORTED;
    return do_outer_step(c, reinterpret_cast<float*>(theta_sync), reinterpret_cast<const float* const*>(theta_local),
                         reinterpret_cast<float* const*>(e), payloads, stream);
}

namespace {
sl_status do_compress(sl_ctx* c, const float* theta_sync, const float* theta_local, float* e, uint8_t* payload,
                      void* stream) {
    if (!c || !theta_sync || !theta_local || !payload) return SL_ERR_INVALID_ARG;
    if (c->cfg.quant_bits == 32) return SL_ERR_UNSUPPORTED;  // unquantised values have no payload format
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
    // with deferral on, this worker's corrected values wait in the workspace for its next sl_compress
    const bool defer = c->deferred && c->cfg.ef_enabled && fast_2bit(c);
    return launch_compress(c, 1, theta_sync, ptrs, static_cast<cudaStream_t>(stream), defer);
}

sl_status do_aggregate_apply(sl_ctx* c, const uint8_t* const* payloads, float* theta_sync, void* stream) {
    if (!c || !payloads || !theta_sync) return SL_ERR_INVALID_ARG;
    if (c->cfg.quant_bits == 32) return SL_ERR_UNSUPPORTED;
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


// The outer step without the quantiser (quant_bits = 32, the full-precision column of the paper's
// quantisation ablation): Top-k sends the selected values exactly, so nothing stays behind at the
// selected positions (e = u - u = +0 there) and the staged values are averaged as they are.
sl_status outer_step_unquantised(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* const* e,
                                 cudaStream_t st) {
    const int R = c->cfg.R;
    const bool ef = c->cfg.ef_enabled != 0;
    if (!c->ws_ptr || c->ws_bytes < workspace_bytes_for(c, R)) return SL_ERR_NOMEM;
    WorkerPtrs ptrs;
    memset(&ptrs, 0, sizeof(ptrs));
    for (int r = 0; r < R; ++r) {
        if (!theta_local[r] || (ef && !e[r])) return SL_ERR_INVALID_ARG;
        if (misaligned(theta_local[r]) || (ef && misaligned(e[r]))) return SL_ERR_ALIGNMENT;
        for (int q = 0; q < r; ++q)
            if (ef && e[q] == e[r]) return SL_ERR_INVALID_ARG;
        ptrs.theta_local[r] = theta_local[r];
        ptrs.e[r] = ef ? e[r] : nullptr;
    }
    sl_status s = flush_pending(c, st);
    if (s != SL_OK) return s;
    c->last_workers = R;
    if ((s = launch_select(c, R, theta_sync, ptrs, st, ef, false, false)) != SL_OK) return s;
    if (ef && (s = launch_zero_selected(c, e, st)) != SL_OK) return s;
    PayloadPtrs none;
    memset(&none, 0, sizeof(none));
    const int was = c->cfg.divide_by_present;
    c->cfg.divide_by_present = 0;
    s = launch_apply(c, none, R, theta_sync, st, 3);
    c->cfg.divide_by_present = was;
    return s;
}

sl_status do_outer_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* const* e,
                        uint8_t* const* payloads, void* stream) {
    if (c && c->cfg.quant_bits == 32) {
        if (!theta_sync || !theta_local || (c->cfg.ef_enabled && !e)) return SL_ERR_INVALID_ARG;
        if (misaligned(theta_sync)) return SL_ERR_ALIGNMENT;
        DeviceGuard g(c->device);
        if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
        return outer_step_unquantised(c, theta_sync, theta_local, e, static_cast<cudaStream_t>(stream));
    }
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
    if (wide_quant(c)) {  // general widths: the plain sequence, every worker's compression, then the aggregation
        sl_status s = launch_compress(c, R, theta_sync, ptrs, st, false);
        if (s != SL_OK) return s;
        return launch_apply(c, pl, R, theta_sync, st);
    }
    const bool defer = c->deferred && c->cfg.ef_enabled;
    if (c->pending && defer && c->pending_workers == R) {  // they can only be substituted into the buffers they came from
        for (int r = 0; r < R; ++r)
            if (e[r] != c->pending_e[r]) return SL_ERR_INVALID_ARG;
    }
    const int fuse = c->cfg.ef_enabled ? (defer ? 2 : 1) : 0;  // packing fused into the apply kernel
    sl_status s = launch_compress(c, R, theta_sync, ptrs, st, defer, fuse != 0);
    if (s != SL_OK) return s;
    return launch_apply(c, pl, R, theta_sync, st, fuse, &ptrs);
}
}  // namespace

sl_status sl_outer_step_host(sl_ctx* c, float* theta_sync, const float* const* theta_local_host, float* dev_stage,
                             size_t stage_elems, float* const* e, uint8_t* const* payloads, float* theta_sync_host,
                             void* stream) {
    if (!c || !theta_sync || !theta_local_host || !dev_stage || !payloads) return SL_ERR_INVALID_ARG;
    if (c->cfg.quant_bits == 32 || half_store(c)) return SL_ERR_UNSUPPORTED;  // (no payload format / fp32 arrays only)
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
    static const char* names[kProfSlots] = {"ef_select", "chunk_sum", "tensor_mean", "chunk_var", "tensor_sigma",
                                            "chunk_bins", "tensor_lut", "pack_fix", "decode_avg_apply"};
    return slot >= 0 && slot < kProfSlots ? names[slot] : "";
}

sl_status sl_diloco_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* momentum,
                         float beta_outer, void* stream) {
    if (!c || !theta_sync || !theta_local || !momentum) return SL_ERR_INVALID_ARG;
    if (half_store(c)) return SL_ERR_UNSUPPORTED;  // the baselines work on fp32 arrays
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

namespace {

// Common argument checks of the three baseline steps; fills the pointer tables.
sl_status variant_args(sl_ctx* c, const float* theta_sync, const float* const* theta_local, float* const* e,
                       float* const* m_r, float mu, WorkerPtrs& ptrs) {
    if (!c || !theta_sync || !theta_local) return SL_ERR_INVALID_ARG;
    if (half_store(c)) return SL_ERR_UNSUPPORTED;  // the baselines work on fp32 arrays
    if (!(mu >= 0.0f && mu <= 1.0f)) return SL_ERR_INVALID_ARG;
    if (misaligned(theta_sync)) return SL_ERR_ALIGNMENT;
    memset(&ptrs, 0, sizeof(ptrs));
    for (int r = 0; r < c->cfg.R; ++r) {
        if (!theta_local[r] || (e && !e[r]) || (m_r && !m_r[r])) return SL_ERR_INVALID_ARG;
        if (misaligned(theta_local[r]) || (e && misaligned(e[r])) || (m_r && misaligned(m_r[r]))) return SL_ERR_ALIGNMENT;
        for (int q = 0; q < r; ++q)
            if ((e && e[q] == e[r]) || (m_r && m_r[q] == m_r[r])) return SL_ERR_INVALID_ARG;
        ptrs.theta_local[r] = theta_local[r];
        ptrs.e[r] = e ? e[r] : nullptr;
    }
    return SL_OK;
}

}  // namespace

sl_status sl_lom_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* const* m_r, float mu,
                      int32_t sub_k, void* stream) {
    WorkerPtrs ptrs;
    if (!m_r) return SL_ERR_INVALID_ARG;
    sl_status s = variant_args(c, theta_sync, theta_local, nullptr, m_r, mu, ptrs);
    if (s != SL_OK) return s;
    if (sub_k && c->cfg.k > kFastMaxK) return SL_ERR_UNSUPPORTED;  // the unquantised kernels stop at 256
    if (sub_k && (!c->ws_ptr || c->ws_bytes < workspace_bytes_for(c, c->cfg.R))) return SL_ERR_NOMEM;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int R = c->cfg.R;
    MutableLocalPtrs lp;
    MomentumPtrs mp;
    memset(&lp, 0, sizeof(lp));
    memset(&mp, 0, sizeof(mp));
    for (int r = 0; r < R; ++r) {
        lp.p[r] = const_cast<float*>(theta_local[r]);  // the stepping kernel only reads them
        mp.p[r] = m_r[r];
    }
    lom_kernel<true><<<(unsigned)c->n_chunks, kThreads, 0, st>>>(c->d_chunks, R, mu, c->cfg.outer_lr, theta_sync, lp, mp);
    SL_CUDA(cudaGetLastError());
    if (sub_k) {  // m_r <- m_r - Top-k(m_r): select on the momenta themselves, zero what was selected
        if ((s = flush_pending(c, st)) != SL_OK) return s;
        WorkerPtrs sel;
        memset(&sel, 0, sizeof(sel));
        for (int r = 0; r < R; ++r) sel.theta_local[r] = m_r[r];
        if ((s = launch_select(c, R, theta_sync, sel, st, false, false, true)) != SL_OK) return s;
        return launch_zero_selected(c, m_r, st);
    }
    return SL_OK;
}

sl_status sl_diloco_topk_step(sl_ctx* c, float* theta_sync, const float* const* theta_local, float* const* e,
                              float* momentum, float mu, void* stream) {
    WorkerPtrs ptrs;
    if (!momentum) return SL_ERR_INVALID_ARG;
    sl_status s = variant_args(c, theta_sync, theta_local, e, nullptr, mu, ptrs);
    if (s != SL_OK) return s;
    if (c->cfg.k > kFastMaxK) return SL_ERR_UNSUPPORTED;  // the unquantised kernels stop at 256
    if (misaligned(momentum)) return SL_ERR_ALIGNMENT;
    if (!c->ws_ptr || c->ws_bytes < workspace_bytes_for(c, c->cfg.R)) return SL_ERR_NOMEM;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((s = flush_pending(c, st)) != SL_OK) return s;
    const int R = c->cfg.R;
    c->last_workers = R;
    if ((s = launch_select(c, R, theta_sync, ptrs, st, e != nullptr, false, false)) != SL_OK) return s;
    if (e && (s = launch_zero_selected(c, e, st)) != SL_OK) return s;  // e_r = u_r - Top-k(u_r)
    PayloadPtrs none;
    memset(&none, 0, sizeof(none));
    const int was = c->cfg.divide_by_present;
    c->cfg.divide_by_present = 0;  // Alg. 3 averages over all R workers
    s = launch_apply(c, none, R, theta_sync, st, 4, nullptr, momentum, mu);
    c->cfg.divide_by_present = was;
    return s;
}

sl_status sl_lom_topk_step(sl_ctx* c, float* theta_sync, float* const* theta_local, float* const* m_r, float* const* e,
                           float mu, void* stream) {
    WorkerPtrs ptrs;
    if (!m_r) return SL_ERR_INVALID_ARG;
    sl_status s = variant_args(c, theta_sync, theta_local, e, m_r, mu, ptrs);
    if (s != SL_OK) return s;
    if (c->cfg.k > kFastMaxK) return SL_ERR_UNSUPPORTED;  // the unquantised kernels stop at 256
    if (!c->ws_ptr || c->ws_bytes < workspace_bytes_for(c, c->cfg.R)) return SL_ERR_NOMEM;
    const int R = c->cfg.R;
    for (int r = 0; r < R; ++r)
        for (int q = 0; q < r; ++q)
            if (theta_local[q] == theta_local[r]) return SL_ERR_INVALID_ARG;  // they are written here
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((s = flush_pending(c, st)) != SL_OK) return s;
    c->last_workers = R;
    MutableLocalPtrs lp;
    MomentumPtrs mp;
    memset(&lp, 0, sizeof(lp));
    memset(&mp, 0, sizeof(mp));
    for (int r = 0; r < R; ++r) {
        lp.p[r] = theta_local[r];
        mp.p[r] = m_r[r];
    }
    // local momenta, and the local Nesterov directions in place of theta_r
    lom_kernel<false><<<(unsigned)c->n_chunks, kThreads, 0, st>>>(c->d_chunks, R, mu, c->cfg.outer_lr, theta_sync, lp, mp);
    SL_CUDA(cudaGetLastError());
    if ((s = launch_select(c, R, theta_sync, ptrs, st, e != nullptr, false, true)) != SL_OK) return s;
    if (e && (s = launch_zero_selected(c, e, st)) != SL_OK) return s;
    PayloadPtrs none;
    memset(&none, 0, sizeof(none));
    const int was = c->cfg.divide_by_present;
    c->cfg.divide_by_present = 0;
    s = launch_apply(c, none, R, theta_sync, st, 3);
    c->cfg.divide_by_present = was;
    return s;
}

sl_status sl_coded_payload_capacity(const sl_ctx* c, size_t* bytes) {
    if (!c || !bytes) return SL_ERR_INVALID_ARG;
    if (!fast_2bit(c)) return SL_ERR_UNSUPPORTED;  // a format of the 2-bit payload only
    if (!c->ixc_capacity) return SL_ERR_TOO_LARGE;  // the stream's bit offsets are 32-bit
    *bytes = c->ixc_capacity;
    return SL_OK;
}

sl_status sl_encode_payload(sl_ctx* c, const uint8_t* payload, uint8_t* coded, uint64_t* dev_coded_bytes,
                            void* stream) {
    if (!c || !payload || !coded || !dev_coded_bytes) return SL_ERR_INVALID_ARG;
    if (!fast_2bit(c)) return SL_ERR_UNSUPPORTED;  // a format of the 2-bit payload only
    if (misaligned(payload) || misaligned(coded) || (reinterpret_cast<uintptr_t>(dev_coded_bytes) & 7u))
        return SL_ERR_ALIGNMENT;
    if (!c->ixc_capacity) return SL_ERR_TOO_LARGE;
    if (!c->ws_ptr || c->ws_bytes < workspace_bytes_for(c, c->cfg.R)) return SL_ERR_NOMEM;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // scratch: two 32-bit words per chunk in the partial-sum area of the workspace as laid out for R workers
    // (unused between compressions).  The values a deferred subtraction keeps waiting live in the staging
    // arrays, which end before that area both in the layout for R workers and in the one sl_compress uses
    // for its single worker (R x G x kp x 6 bytes against G x kp x 6).
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

sl_status sl_decode_payload(sl_ctx* c, const uint8_t* coded, size_t coded_bytes, uint8_t* payload, void* stream) {
    if (!c || !coded || !payload) return SL_ERR_INVALID_ARG;
    if (!fast_2bit(c)) return SL_ERR_UNSUPPORTED;  // a format of the 2-bit payload only
    if (misaligned(coded) || misaligned(payload)) return SL_ERR_ALIGNMENT;
    if (!c->ixc_capacity) return SL_ERR_TOO_LARGE;
    // what the buffer is said to hold bounds every read; it must at least reach the index stream
    if (coded_bytes == 0 || coded_bytes > c->ixc_capacity) coded_bytes = c->ixc_capacity;
    if (coded_bytes < c->ixc_stream_off) return SL_ERR_INVALID_ARG;
    const unsigned long long stream_bits = (unsigned long long)((coded_bytes - c->ixc_stream_off) / 4 * 4) * 8ull;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    const long long groups = (c->n_chunks + kIxcGroup - 1) / kIxcGroup;
    const long long items = groups > 4ll * c->n_tensors ? groups : 4ll * c->n_tensors;
    ixc_decode_kernel<<<blocks_for(items, 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        c->d_chunks, c->n_chunks, c->n_tensors, c->cfg.k, coded, c->ixc_dir_off, c->ixc_stream_off, stream_bits,
        payload, c->d_status);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

sl_status sl_aggregate_apply_coded(sl_ctx* c, const uint8_t* const* coded, const size_t* coded_bytes, float* theta_sync,
                                   void* stream) {
    if (!c || !coded || !theta_sync) return SL_ERR_INVALID_ARG;
    if (!fast_2bit(c) || half_store(c)) return SL_ERR_UNSUPPORTED;  // the 2-bit payload, fp32 arrays
    if (!c->ixc_capacity) return SL_ERR_TOO_LARGE;
    if (misaligned(theta_sync)) return SL_ERR_ALIGNMENT;
    PayloadPtrs pl;
    memset(&pl, 0, sizeof(pl));
    size_t sizes[kMaxR];
    int present = 0;
    for (int r = 0; r < c->cfg.R; ++r) {
        if (misaligned(coded[r])) return SL_ERR_ALIGNMENT;
        pl.p[r] = coded[r];
        present += coded[r] != nullptr;
        size_t n = coded_bytes ? coded_bytes[r] : 0;
        if (n == 0 || n > c->ixc_capacity) n = c->ixc_capacity;
        if (coded[r] && n < c->ixc_stream_off) return SL_ERR_INVALID_ARG;
        sizes[r] = n;
    }
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    return launch_apply_coded(c, pl, sizes, present, theta_sync, static_cast<cudaStream_t>(stream));
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
    if (on && !fast_2bit(c)) return SL_ERR_UNSUPPORTED;  // only the 2-bit path defers
    c->deferred = on != 0;
    return SL_OK;
}

sl_status sl_ef_pending(const sl_ctx* c, int32_t* pending) {
    if (!c || !pending) return SL_ERR_INVALID_ARG;
    *pending = c->pending ? 1 : 0;
    return SL_OK;
}

sl_status sl_ef_flush_bf16(sl_ctx* c, uint16_t* const* e, int32_t keep_pending, void* stream) {
    if (c && !half_store(c)) return SL_ERR_UNSUPPORTED;
    return do_ef_flush(c, reinterpret_cast<float* const*>(e), keep_pending, stream);
}

sl_status sl_ef_flush(sl_ctx* c, float* const* e, int32_t keep_pending, void* stream) {
    if (c && half_store(c) && e) return SL_ERR_UNSUPPORTED;  // (with e = NULL the call is type-free)
    return do_ef_flush(c, e, keep_pending, stream);
}

namespace {
sl_status do_ef_flush(sl_ctx* c, float* const* e, int32_t keep_pending, void* stream) {
    if (!c) return SL_ERR_INVALID_ARG;
    if (!c->pending) return SL_OK;
    WorkerPtrs ptrs;
    memset(&ptrs, 0, sizeof(ptrs));
    for (int r = 0; r < c->pending_workers; ++r) {
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
}  // namespace

sl_status sl_streaming_due(int32_t H, int32_t P, int64_t inner_step, int32_t* fragment) {
    if (!fragment || H < 1 || P < 1 || P > H || inner_step < 1) return SL_ERR_INVALID_ARG;
    *fragment = -1;
    const int64_t t = inner_step % H;
    for (int32_t p = 0; p < P; ++p)
        if (t == (((int64_t)(p + 1) * H) / P) % H) {
            *fragment = p;
            break;
        }
    return SL_OK;
}

sl_status sl_validate_payload(sl_ctx* c, const uint8_t* payload, int32_t* dev_status, void* stream) {
    if (!c || !payload || !dev_status) return SL_ERR_INVALID_ARG;
    if (c->cfg.quant_bits == 32) return SL_ERR_UNSUPPORTED;  // unquantised values have no payload format
    if (misaligned(payload)) return SL_ERR_ALIGNMENT;
    DeviceGuard g(c->device);
    if (!g.ok) return cuda_fail(cudaErrorInvalidDevice, "set device");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    set_status_kernel<<<1, 1, 0, st>>>(dev_status, (int)SL_OK);
    const long long items = c->n_chunks > c->n_tensors ? c->n_chunks : c->n_tensors;
    validate_kernel<<<blocks_for(items, 128), 128, 0, st>>>(c->d_chunks, c->n_chunks, c->n_tensors, c->cfg.k, c->qbits,
                                                            header_bytes_q(c->qbits), c->rec_base, c->rec_stride, payload,
                                                            dev_status);
    SL_CUDA(cudaGetLastError());
    return SL_OK;
}

sl_status sl_read_stats(sl_ctx* c, int32_t worker, float* dev_out, void* stream) {
    if (!c || !dev_out || worker < 0 || worker >= c->last_workers) return SL_ERR_INVALID_ARG;
    if (!fast_2bit(c)) return SL_ERR_UNSUPPORTED;  // the 2-bit quantiser's table
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
    int* status;  // where the kernel would record a bounded wait that ran out: the array's last 256 bytes
    int ef_ctas;
    bool ready;
};
StaticSetup g_static_setup[64];
std::mutex g_static_setup_mutex;  // first calls from several host threads set a device up once

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
    if (k > kFastMaxK) return SL_ERR_UNSUPPORTED;
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
    if (need > kStaticScratchBytes - 256) return SL_ERR_TOO_LARGE;  // the fixed scratch cannot hold this tensor

    int dev = -1;
    SL_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SL_ERR_UNSUPPORTED;
    StaticSetup& su = g_static_setup[dev];
    std::lock_guard<std::mutex> lock(g_static_setup_mutex);  // (calls that overlap on the GPU race anyway: see the header)
    if (!su.ready) {  // first call on this device: resolve the array's device address, size the launch
        void* ptr = nullptr;
        SL_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        int n_sms = 0;
        SL_CUDA(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
        SL_CUDA(cudaFuncSetAttribute(ef_select_kernel<true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)sizeof(SelSmem)));
        SL_CUDA(cudaFuncSetAttribute(ef_select_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)sizeof(SelSmem)));
        su.scratch = ptr;
        su.status = reinterpret_cast<int*>(static_cast<char*>(ptr) + kStaticScratchBytes - 256);
        su.ef_ctas = n_sms;
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
    TmaArgs no_tma;  // plain loads and stores: nothing has to be encoded or uploaded for the caller's buffers
    memset(&no_tma, 0, sizeof(no_tma));
    no_tma.status = su.status;
    if (k > kSelNarrowMaxK)
        ef_select_kernel<true, false, 1><<<ef_grid, kSelThreads, sizeof(SelSmem), st>>>(d_chunks, G, 1, k, kp, beta, theta_sync,
                                                                                        ptrs, ws, no_tma, 0);
    else
        ef_select_kernel<true, false, 0><<<ef_grid, kSelThreads, sizeof(SelSmem), st>>>(d_chunks, G, 1, k, kp, beta, theta_sync,
                                                                                         ptrs, ws, no_tma, 0);
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
