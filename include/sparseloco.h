/*
 * libsparseloco -- the SparseLoCo outer step on one NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every buffer argument is a DEVICE pointer unless it says "host".  The caller owns all
 * device buffers it passes in (parameters, error buffers, payloads, workspace); the library owns
 * only the context object and the small device-side chunk table built by sl_create().  All work is
 * enqueued on the CUDA stream the caller passes (a cudaStream_t cast to void*; NULL = the default
 * stream) and no entry point synchronises the host, except sl_create()/sl_destroy() and
 * sl_outer_step_host().  There is no CPU implementation behind these calls.
 *
 * The method (paper: "SparseLoCo", Algorithm 1 and Eq. 2), per outer step, R workers:
 *     Delta_r   = theta - theta_r                          pseudo-gradient       (Sec. 3.1, Alg. 1)
 *     u_r       = beta * e_r + Delta_r                     error feedback        (Eq. 2 line 1)
 *     Dhat_r    = Q(TopK(u_r))                             chunk-wise Top-k, 2-bit quantiser
 *                                                          (Eq. 2 line 2; Sec. 3.3 chunking; Sec. 4 Q)
 *     e_r       = u_r - Dhat_r                             error update          (Eq. 2 line 2)
 *     theta     = theta - alpha * (1/R) sum_r Dhat_r       aggregate + outer SGD (Eq. 2 lines 3-4)
 *
 * Chunks (Sec. 3.3): a 2-D tensor whose sides are both multiples of 64 is cut into 64x64 blocks
 * (block-row-major; in-chunk index = 64 * row_in_block + col_in_block); every other tensor is cut
 * into row-major runs of 4096 elements with a short last run.  Top-k keeps, per chunk, the
 * min(k, chunk length) entries of largest magnitude (IEEE bit pattern without the sign, compared
 * as an integer; ties go to the lower in-chunk index), listed by ascending in-chunk index.
 *
 * Quantiser (Sec. 4): per (worker, tensor), over all selected values: mean mu, population sigma of
 * the centred values, bins (-inf,-3s) [-3s,0) [0,3s) [3s,inf) on centred values, table entry =
 * mean of the raw values in the bin (+0 when empty).  Sums are fp64, slot by slot inside a chunk,
 * then chunk by chunk inside a group of 64 consecutive chunks of the tensor, then group by group.
 *
 * Payload of one worker (little-endian; App. "Compression of indices": 12 bits per index):
 *     bytes [16 j, 16 j + 16)          table of tensor j: 4 x fp32
 *     then one record per chunk, in (tensor, chunk) order, each sl_record_stride(k) bytes:
 *         bits  [12 s, 12 s + 12)                   in-chunk index of slot s
 *         bytes from ceil(12 k / 8): bits [2 s, 2 s + 2)   code of slot s
 *     slots >= min(k, chunk length) and all padding are zero.
 * With quant_bits = b in {1, 3, 4} the same layout holds with b in place of 2: tables of 2^b fp32 entries
 * (max(16, 4 * 2^b) bytes per tensor; entry j = centroid of the bin between the edges (-6 + 12 j / 2^b) sigma
 * and (-6 + 12 (j + 1) / 2^b) sigma of the centred values, the outer bins open-ended), records of
 * roundup16(ceil(12 k / 8) + ceil(b k / 8)) bytes with the code of slot s at bits [b s, b s + b) of the code
 * block.  sl_payload_bytes() gives the size.
 */
#ifndef SPARSELOCO_H
#define SPARSELOCO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SL_OK = 0,
    SL_ERR_INVALID_ARG = 1, /* NULL pointer, size or hyper-parameter out of range */
    SL_ERR_ALIGNMENT = 2,   /* a device pointer or tensor offset is not 16-byte aligned */
    SL_ERR_UNSUPPORTED = 3, /* valid in the method, not built here (chunk != 4096, quant_bits not in 1..4 / 32,
                               an entry point that serves the 2-bit payload only, ...) */
    SL_ERR_BAD_PAYLOAD = 4, /* reported through the device status word of sl_validate_payload */
    SL_ERR_CUDA = 5,        /* a CUDA runtime call failed; see sl_last_cuda_error() */
    SL_ERR_NOMEM = 6,       /* workspace missing or too small; host allocation failed */
    SL_ERR_TOO_LARGE = 7,   /* problem exceeds a fixed built-in capacity */
    SL_ERR_TIMEOUT = 8      /* a bounded wait inside a kernel ran out; reported by sl_device_status() */
} sl_status;

/* One parameter tensor: rows x cols fp32, row-major, at element offset `offset` of every flat
 * buffer (theta, theta_r, e).  1-D tensors have rows == 1.  offset must be a multiple of 4. */
typedef struct {
    int64_t rows, cols;
    int64_t offset;
} sl_tensor_desc;

/* Hyper-parameters, named as in Algorithm 1's "Require" line and Sec. 4. */
typedef struct {
    int32_t chunk_elems;       /* C: must be 4096 */
    int32_t tile_dim;          /* must be 64 */
    int32_t k;                 /* entries kept per chunk, 1..2048 (the paper's density sweeps reach half a
                                  chunk).  The tuned kernels serve k <= 256; beyond that the selection is the exact
                                  bitwise search and packing / decoding run in the plain kernels of the
                                  quantiser ablation: no deferral, no wire codec, no quant_bits = 32,
                                  no Top-k baselines */
    int32_t R;                 /* workers, 1..64 */
    int32_t H;                 /* inner steps; carried for the caller, >= 1, unused by the math */
    float beta;                /* error-feedback decay, 0 <= beta <= 1 */
    float outer_lr;            /* alpha, finite */
    int32_t quant_bits;        /* 2 (the paper's setting; the fast path); 1, 3 or 4 (its ablation: 2^bits
                                  uniform bins over [-6 sigma, 6 sigma], plain kernels, no deferral, no wire
                                  codec); or 32 = no quantiser: the selected values are averaged
                                  as they are (sl_outer_step only: there is no payload format, payloads may be
                                  NULL) */
    int32_t ef_enabled;        /* 0 during the error-feedback freeze (App. "Freezing Error
                                  Feedback"): u = Delta and e is neither read nor written */
    int32_t divide_by_present; /* 0: average divides by R (Alg. 1); 1: by the payloads present */
    int32_t bf16_storage;      /* 0: theta, theta_r, e are fp32 arrays.  1: bfloat16 arrays, served by the
                                  sl_*_bf16 entry points only (see there); not with quant_bits = 32 */
} sl_config;

typedef struct sl_ctx sl_ctx;

/* Build a context for a tensor table on the current CUDA device.  Allocates the device chunk
 * table (32 bytes per chunk) -- the only allocation the library ever makes -- and synchronises.
 * `tensors` is a host array; the element ranges [offset, offset + rows * cols) must not overlap.
 * Errors: INVALID_ARG (also overlapping tensors), ALIGNMENT (offset % 4), UNSUPPORTED, TOO_LARGE
 * (cols >= 2^31, a tensor of more than 2^40 elements), NOMEM (host allocation failed), CUDA. */
sl_status sl_create(const sl_config* cfg, const sl_tensor_desc* tensors, int32_t n_tensors,
                    sl_ctx** out);
sl_status sl_destroy(sl_ctx* ctx);

/* Change beta / outer_lr / ef_enabled / divide_by_present / H between steps (k, R, chunking are
 * fixed at creation).  Host-side only. */
sl_status sl_set_hyper(sl_ctx* ctx, float beta, float outer_lr, int32_t ef_enabled,
                       int32_t divide_by_present);

/* Closed forms (host-side, no device work). */
size_t sl_record_stride(int32_t k);                                   /* bytes of one chunk record */
sl_status sl_payload_bytes(const sl_ctx* ctx, size_t* bytes_per_worker); /* 16 T + stride * chunks */
sl_status sl_num_chunks(const sl_ctx* ctx, int64_t* chunks, int64_t* slots_per_worker);
sl_status sl_flat_elems(const sl_ctx* ctx, int64_t* elems); /* max over tensors of offset + size */

/* Scratch memory: selected (index, value) pairs and per-chunk partial sums for R workers.
 * sl_workspace_bytes() gives the size sl_outer_step() needs (sl_compress() needs 1/R of it); the
 * caller allocates it (256-byte aligned) and lends it with sl_set_workspace().  Contents need not
 * be preserved between calls.  Calls that share a workspace must not overlap on the device. */
sl_status sl_workspace_bytes(const sl_ctx* ctx, size_t* bytes);
sl_status sl_set_workspace(sl_ctx* ctx, void* dev_ptr, size_t bytes);

/* One worker's compression + error feedback (Alg. 1, green block; Eq. 2 lines 1-2).
 *   theta_sync, theta_local : flat fp32, read only.
 *   e       : flat fp32, updated in place to u - Dhat (untouched when ef_enabled == 0).
 *   payload : sl_payload_bytes() bytes, fully overwritten.
 * Errors: INVALID_ARG (NULL), ALIGNMENT, NOMEM (workspace), CUDA (launch failure). */
sl_status sl_compress(sl_ctx* ctx, const float* theta_sync, const float* theta_local, float* e,
                      uint8_t* payload, void* cuda_stream);

/* Decode and average R payloads and apply the outer update (Alg. 1, orange block; Eq. 2 lines 3-4).
 *   payloads : HOST array of R DEVICE pointers; NULL = that worker is absent.
 *   theta_sync : updated in place: theta - alpha * (sum_r Dhat_r) / D, sum in fp32 with r
 *   ascending, D = R or the number present.  Elements no worker selected are bit-unchanged.
 * Payloads are trusted to be well formed (run sl_validate_payload on anything received from
 * outside); an index beyond the chunk is ignored rather than written. */
sl_status sl_aggregate_apply(sl_ctx* ctx, const uint8_t* const* payloads, float* theta_sync,
                             void* cuda_stream);

/* The whole outer step for R resident workers: sl_compress for r = 0..R-1, then
 * sl_aggregate_apply, with identical results, but free to share work between workers.
 *   theta_local, e, payloads : HOST arrays of R DEVICE pointers.  theta_local entries may alias
 *   each other; e and payload entries must not.
 * The call only enqueues work, so it can be captured in a CUDA graph and replayed -- after one
 * ordinary call with the same buffers (descriptors of a buffer are built and uploaded the first time
 * its pointer is seen) and with the deferred subtraction off (that mode keeps host-side state that a
 * replay would not advance). */
sl_status sl_outer_step(sl_ctx* ctx, float* theta_sync, const float* const* theta_local,
                        float* const* e, uint8_t* const* payloads, void* cuda_stream);

/* The same three calls for a context created with bf16_storage = 1: theta_sync, theta_local and e are
 * arrays of bfloat16 bit patterns (the upper halves of fp32 values), same element offsets, same
 * alignment rules (16-byte aligned pointers).  The paper states the method (Alg. 1, Eq. 2) without
 * naming a storage type; this mode halves the state the outer step streams.  Definition: all
 * arithmetic is that of the fp32 calls on the widened values -- Delta = theta - theta_r,
 * u = fma(beta, e, Delta), selection and quantiser on the unrounded u, so the payload is the one the
 * fp32 calls would write for these inputs -- and every store rounds once to the nearest bfloat16,
 * ties to even: e = bf16(u), or bf16(u - table[code]) at the selected positions;
 * theta = bf16(fma(-alpha / D, sum, theta)) where some worker selected the element, else unchanged.
 * At 2 bits and k <= 256 the quantiser statistics and the fused packing / update kernel are the tuned ones
 * of the fp32 path (with widening loads and rounding stores), the deferred subtraction is available
 * (sl_set_ef_deferred; the waiting values stay fp32 in the workspace and are rounded when they reach e;
 * sl_ef_flush_bf16 for explicit buffers) and so are the wire codec, sl_validate_payload and sl_read_stats;
 * the selection runs in a warp-per-unit kernel with plain loads (no tile copies).  Other widths and
 * larger k run in the plain kernels.  Not available: sl_outer_step_host, sl_aggregate_apply_coded, the
 * comparison methods, quant_bits = 32.
 * Errors as for the fp32 calls; UNSUPPORTED when the context is not a bf16_storage one (and the
 * fp32 calls return UNSUPPORTED for a context that is). */
sl_status sl_compress_bf16(sl_ctx* ctx, const uint16_t* theta_sync, const uint16_t* theta_local, uint16_t* e,
                           uint8_t* payload, void* cuda_stream);
sl_status sl_aggregate_apply_bf16(sl_ctx* ctx, const uint8_t* const* payloads, uint16_t* theta_sync,
                                  void* cuda_stream);
sl_status sl_outer_step_bf16(sl_ctx* ctx, uint16_t* theta_sync, const uint16_t* const* theta_local,
                             uint16_t* const* e, uint8_t* const* payloads, void* cuda_stream);
sl_status sl_ef_flush_bf16(sl_ctx* ctx, uint16_t* const* e, int32_t keep_pending, void* cuda_stream);

/* Dense baseline on the same buffers: DiLoCo's outer step with Nesterov outer momentum (Eq. 1),
 *     Dbar = (1/R) sum_r (theta - theta_r);  m = beta_outer m + Dbar;
 *     theta = theta - alpha (Dbar + beta_outer m),        alpha = the context's outer_lr.
 *   theta_sync, momentum : flat fp32, updated in place (only the elements of the tensor table);
 *   theta_local : HOST array of R DEVICE pointers, read only, may alias.
 * No compression, no workspace.  Errors: INVALID_ARG (NULL, beta_outer outside [0, 1]), ALIGNMENT, CUDA. */
sl_status sl_diloco_step(sl_ctx* ctx, float* theta_sync, const float* const* theta_local, float* momentum,
                         float beta_outer, void* cuda_stream);

/* The paper's Top-k and local-outer-momentum variants on the same buffers (Sec. 3.2; appendix "Exact
 * algorithmic description of DiLoCo variants", Alg. 2-4).  None of them quantises: Top-k keeps the
 * selected values as they are, chunk-wise with the chunking and tie rule above, k = the context's k.
 * alpha = the context's outer_lr, the error-feedback decay rho = the context's beta, mu = the outer
 * momentum coefficient (0 <= mu <= 1).  What a worker keeps (m_r, e_r) and what it selects on are fp32,
 * formed by single-rounded operations in the algorithm's order: d = theta - theta_r; m_r = fma(mu, m_r,
 * d); nd_r = fma(mu, m_r, d); u_r = fma(rho, e_r, .).  Averages are fp32 sums in ascending r divided by
 * R.  All pointer tables are HOST arrays of R DEVICE pointers; buffers are flat fp32 and only the
 * elements of the tensor table are touched.  The Top-k steps use the lent workspace (NOMEM without
 * one); waiting values of a deferred subtraction are written out first.
 *
 *   sl_lom_step         Alg. 2, DiLoCo-LOM: m_r and theta updated in place, theta = theta - alpha mean_r
 *                       nd_r.  sub_k != 0: DiLoCo-LOM-Sub-k, afterwards m_r = m_r - Top-k(m_r), i.e. the k
 *                       largest entries of every chunk of m_r become +0.
 *   sl_diloco_topk_step Alg. 3, DiLoCo + Top-k: u_r = theta - theta_r, or fma(rho, e_r, theta - theta_r)
 *                       when e is given (then e_r = u_r - Top-k(u_r) in place); D = mean_r Top-k(u_r);
 *                       momentum = fma(mu, momentum, D); theta = theta - alpha (D + mu momentum).
 *   sl_lom_topk_step    Alg. 4, DiLoCo-LOM + Top-k: m_r and nd_r as in Alg. 2, u_r = nd_r or fma(rho, e_r,
 *                       nd_r); theta = theta - alpha mean_r Top-k(u_r).  theta_local is CONSUMED: on return
 *                       buffer r holds nd_r (the entries must be distinct buffers).
 * Errors: INVALID_ARG (NULL, mu outside [0, 1], aliased state buffers), ALIGNMENT, NOMEM, CUDA. */
sl_status sl_lom_step(sl_ctx* ctx, float* theta_sync, const float* const* theta_local, float* const* m_r,
                      float mu, int32_t sub_k, void* cuda_stream);
sl_status sl_diloco_topk_step(sl_ctx* ctx, float* theta_sync, const float* const* theta_local, float* const* e,
                              float* momentum, float mu, void* cuda_stream);
sl_status sl_lom_topk_step(sl_ctx* ctx, float* theta_sync, float* const* theta_local, float* const* m_r,
                           float* const* e, float mu, void* cuda_stream);

/* Entropy-coded indices for the wire (App. "Compression of indices": 12 bits per index is the naive
 * cost, log2 C(4096, k) / k the bound, 8.9 / 6.6 / 5.6 bits at k = 32 / 128 / 256 what the paper
 * reports from a scheme it does not describe).  The coding below is this library's own and reaches
 * about 8.4 / 6.4 / 5.4 bits on uniformly drawn index sets.  sl_encode_payload() rewrites a 12-bit
 * payload (as written by sl_compress / sl_outer_step) into the coded form for transmission;
 * sl_decode_payload() restores the identical 12-bit payload, which sl_aggregate_apply() consumes.
 *
 * One chunk of length L with m = min(k, L) ascending indices p_0 < p_1 < ...: gaps g_0 = p_0,
 * g_i = p_i - p_(i-1) - 1; divisor M = max(1, (693 (L - m) + 500 (m + 1)) / (1000 (m + 1))) in integer
 * arithmetic; the code of g is g / M one-bits, a zero-bit, then g % M in truncated binary
 * (b = ceil(log2 M), cut = 2^b - M: values below cut in b - 1 bits, else value + cut in b bits, most
 * significant bit first; nothing when M = 1).  Bit i of a stream sits in byte i / 8 at bit i % 8.
 * Coded payload (little-endian), T tensors, G chunks, cb = ceil(2 k / 8):
 *     [0, 16 T)                 the tensor tables, unchanged
 *     [16 T, 16 T + cb G)       the chunks' code blocks, copied from the records
 *     next multiple of 4        ceil(G / 16) x uint32: bit offset in the index stream of the first
 *                               chunk of every group of 16 chunks
 *     then                      the index stream, chunk after chunk without padding,
 *                               zero-filled to a multiple of 16 bytes
 *   sl_coded_payload_capacity : bytes a coded payload can take at worst (size `coded` with it);
 *                               TOO_LARGE if the stream could exceed 2^32 bits.
 *   sl_encode_payload         : payload (12-bit form) -> coded; the coded size in bytes is written to
 *                               *dev_coded_bytes (DEVICE uint64, 8-byte aligned).  Uses the lent
 *                               workspace as scratch (NOMEM without one) and must not overlap a
 *                               compression on another stream.
 *   sl_decode_payload         : coded -> payload (sl_payload_bytes() bytes, fully overwritten).
 *                               coded_bytes (host value) = bytes of `coded` that may be read: the size
 *                               sl_encode_payload reported, or 0 for the full capacity; it must cover
 *                               the tables, code blocks and directory (else INVALID_ARG).  No read
 *                               goes past it: a directory entry beyond it is clamped and a stream
 *                               that runs out reads as zero bits, so a corrupted input yields a
 *                               wrong but well-formed-sized record, never an out-of-range access.
 *                               Such an input (also a directory that does not ascend) records
 *                               SL_ERR_BAD_PAYLOAD in the device status word (sl_device_status); run
 *                               sl_validate_payload on the result as well.
 *   sl_aggregate_apply_coded  : Eq. 2 lines 3-4 (decode, average, outer update) straight from R coded
 *                               payloads, the decoding fused into the update kernel: what
 *                               sl_decode_payload for every worker followed by sl_aggregate_apply does,
 *                               bit for bit, without the 12-bit payloads in between.  `coded` = HOST
 *                               array of R DEVICE pointers (NULL = absent worker), `coded_bytes` = HOST
 *                               array of the R sizes as for sl_decode_payload (NULL or 0 = full
 *                               capacity).  Reads stay inside the stated sizes; a damaged input gives
 *                               a wrong update of in-range elements and SL_ERR_BAD_PAYLOAD in the
 *                               device status word, so validate untrusted payloads first
 *                               (sl_decode_payload + sl_validate_payload).  UNSUPPORTED when the
 *                               per-CTA staging would not fit shared memory (R x k beyond about 64 x 256). */
sl_status sl_coded_payload_capacity(const sl_ctx* ctx, size_t* bytes);
sl_status sl_encode_payload(sl_ctx* ctx, const uint8_t* payload, uint8_t* coded, uint64_t* dev_coded_bytes,
                            void* cuda_stream);
sl_status sl_decode_payload(sl_ctx* ctx, const uint8_t* coded, size_t coded_bytes, uint8_t* payload,
                            void* cuda_stream);
sl_status sl_aggregate_apply_coded(sl_ctx* ctx, const uint8_t* const* coded, const size_t* coded_bytes,
                                   float* theta_sync, void* cuda_stream);

/* How the compression kernel moves the 64x64 blocks of theta, theta_r and e (no counterpart in the paper).
 * 1: one tensor-map (TMA) block copy per block, issued by a producer thread, completion on
 * shared-memory barriers -- the default whenever every full chunk starts on a 64-element boundary of
 * the flat buffers (tensor offsets that are multiples of 64) and the table has at most 8 distinct row
 * lengths; else UNSUPPORTED.  0: every chunk is read and written with plain 128-bit loads and stores by
 * the warp that processes it (works for any table; short tail chunks always go this way).  Results are
 * identical.  The tensor maps of a buffer are built the first time its pointer is passed in.
 *
 * The kernel waits for its copies with a bounded number of polls; if a wait ever runs out the kernel
 * records SL_ERR_TIMEOUT in a device status word and returns early, leaving e and the staged selection
 * of that call undefined.  sl_device_status() synchronises the stream, returns the recorded status
 * (SL_OK when nothing went wrong; SL_ERR_BAD_PAYLOAD after sl_decode_payload met a damaged input) and
 * clears it. */
sl_status sl_set_tile_copies(sl_ctx* ctx, int32_t use_tensor_maps);
sl_status sl_device_status(sl_ctx* ctx, void* cuda_stream);

/* Deferred error-feedback subtraction (a storage choice; the paper has no counterpart).  Writing
 * e = u - Dhat at the k selected positions of every chunk after the table is known costs a
 * scattered read-modify-write of one 32-byte sector per selected value.  With deferral on,
 * sl_outer_step() leaves e_r = u_r at those positions and keeps the corrected values (u - Dhat) in
 * the workspace; the next sl_outer_step() substitutes them while it streams e_r, with identical
 * arithmetic, so payloads, theta_sync and the true error are bit-for-bit those of the default mode.
 * While values wait (sl_ef_pending): the error state of worker r is its buffer e[r] with those
 * entries substituted; the workspace must be left untouched and stay lent; the next
 * sl_outer_step() must be given the same e pointers (else INVALID_ARG).
 *   sl_ef_flush(ctx, e, keep_pending, stream) writes the waiting values into e (HOST array of R
 *   DEVICE pointers; NULL = the buffers of the last step), which then hold the true error.  With
 *   keep_pending != 0 the values keep waiting (use it to materialise a copy, e.g. for a checkpoint),
 *   and NULL entries of e skip that worker (one spare buffer then serves all workers in turn).
 * sl_compress() defers in the same way for its one worker (the deployment with one worker per GPU: the
 * values of that worker wait for its next sl_compress(), which must be given the same e).
 * A step that cannot substitute them (error feedback frozen, deferral switched off, other buffers or
 * another number of workers than the call that left them, sl_outer_step_host()) writes them into the
 * buffers of the call that left them first.  sl_ef_flush()'s array then has as many entries as that
 * call had workers. */
sl_status sl_set_ef_deferred(sl_ctx* ctx, int32_t on);
sl_status sl_ef_pending(const sl_ctx* ctx, int32_t* pending);
sl_status sl_ef_flush(sl_ctx* ctx, float* const* e, int32_t keep_pending, void* cuda_stream);

/* Same step with the workers' parameters in HOST memory (pinned for full speed), the shape a
 * deployment has when the inner loop's result arrives over the host (Alg. 1: every worker's
 * Dhat_r is gathered before the update).  theta_local_host is a host array of R host pointers;
 * worker r is copied to the caller-owned device staging area `dev_stage` (stage_elems floats:
 * at least sl_flat_elems() rounded up to 4; with twice that, the copy of worker r + 1 overlaps
 * the compression of worker r on an internal copy stream) and compressed; then the payloads are
 * aggregated and, if theta_sync_host is not NULL, the updated theta_sync is copied back to it.
 * Synchronises the stream before returning.  e, payloads and theta_sync stay resident on the
 * device (Alg. 1 keeps e_r on its worker).  Errors as sl_outer_step, plus NOMEM (stage too small). */
sl_status sl_outer_step_host(sl_ctx* ctx, float* theta_sync, const float* const* theta_local_host,
                             float* dev_stage, size_t stage_elems, float* const* e,
                             uint8_t* const* payloads, float* theta_sync_host, void* cuda_stream);

/* Streaming SparseLoCo (App. "Streaming SparseLoCo": the model is cut into P fragments, each still
 * synchronised every H inner steps, but in turn, so that a P-th of the payload travels every H / P
 * steps).  A fragment is a context of its own whose tensor offsets point into the same flat buffers;
 * this host-side helper is the schedule: after `inner_step` inner steps (counted from 1) fragment
 *     p  is due  iff  inner_step mod H == ((p + 1) * H / P) mod H          (integer division),
 * i.e. fragment 0 first, after H / P steps, fragment P - 1 at every multiple of H.  Writes the due
 * fragment to *fragment, or -1 when none is.  Errors: INVALID_ARG (NULL, H < 1, P < 1, P > H,
 * inner_step < 1). */
sl_status sl_streaming_due(int32_t H, int32_t P, int64_t inner_step, int32_t* fragment);

/* Check one payload before trusting it: every index < chunk length and strictly ascending over
 * the used slots, unused slots and padding zero, table entries finite.  Writes SL_OK or
 * SL_ERR_BAD_PAYLOAD to *dev_status (device int32); never traps.  Serves every quantiser width and
 * every k (the record layout is the same: 12-bit indices, then the codes); UNSUPPORTED only with
 * quant_bits = 32, which has no payload. */
sl_status sl_validate_payload(sl_ctx* ctx, const uint8_t* payload, int32_t* dev_status,
                              void* cuda_stream);

/* Per-(worker, tensor) quantiser statistics of the most recent compression, for logging:
 * copies 8 floats per tensor (mu, sigma, 3 sigma, table[4], 0) for workspace worker slot
 * `worker` into dev_out (device, 8 * n_tensors floats). */
sl_status sl_read_stats(sl_ctx* ctx, int32_t worker, float* dev_out, void* cuda_stream);

/* Optional per-kernel timing for benchmarks (no counterpart in the paper, which reports no
 * kernel times).  While enabled, every outer step / compression records CUDA events between its
 * kernels on the caller's stream (up to 256 sequences between reads).  sl_profile_read()
 * waits for the recorded events, writes per-kernel total milliseconds and launch counts into
 * two host arrays of SL_PROFILE_SLOTS entries, and clears the record. */
#define SL_PROFILE_SLOTS 9
sl_status sl_profile_enable(sl_ctx* ctx, int32_t enable);
sl_status sl_profile_read(sl_ctx* ctx, float* ms_total, int64_t* launches);
const char* sl_profile_name(int32_t slot);

/* Compression of ONE tensor of ONE worker that allocates nothing (the paper has no counterpart:
 * this is sl_compress() for callers that cannot allocate device memory).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a training loop that has handed
 * all device memory to a caching allocator or a fixed arena, a latency-critical section that must
 * not take the allocator's device-wide synchronisation, a plug-in that is only given buffers.  Such
 * a caller cannot create a context (sl_create allocates the chunk table) nor lend a workspace.
 *
 * Instead, the chunk table, the staged (index, value) pairs, the partial sums and the tensor
 * statistics live in a fixed array of sl_static_scratch_bytes() = 4 MiB inside the library, one copy
 * per GPU that loads the library, held until the process exits.  The caller still passes inputs
 * and outputs:
 *   theta_sync, theta_local : the tensor, rows x cols fp32 row-major (rows == 1 for a vector), read only
 *   e       : same shape, updated in place to u - Dhat (error feedback always on, coefficient beta)
 *   payload : 16 + sl_record_stride(k) * chunks bytes, fully overwritten: the 16-byte table, then
 *             the records, i.e. the payload sl_compress() writes for a one-tensor table
 * Results are bit-identical to sl_compress() on a context holding this single tensor.
 *
 * Limits and rules:
 *   - the tensor must fit the scratch: about (88 + 6 roundup8(k)) bytes per chunk, i.e. about 8,800
 *     chunks (36 M elements) at k = 64; larger calls return SL_ERR_TOO_LARGE and do nothing.
 *   - the first call on a device looks up the array's device address and sizes the launch (no
 *     allocation, but host-side queries): make that first call before any stream capture.
 *   - every call on a GPU shares the one array: calls whose kernels overlap on the GPU (different
 *     streams, different threads) race; serialise them.  Nothing has to be cleared between calls:
 *     each call rewrites every scratch location before reading it, whatever the previous call left.
 *   - no cudaMalloc, cudaFree or other allocating routine is called; all work is enqueued on
 *     `cuda_stream` and the call does not synchronise.
 * Errors: INVALID_ARG (NULL, rows/cols/k < 1, beta outside [0,1]), ALIGNMENT (a pointer not 16-byte
 * aligned), UNSUPPORTED (k > 256), TOO_LARGE, CUDA. */
size_t sl_static_scratch_bytes(void);
sl_status sl_compress_tensor_static(const float* theta_sync, const float* theta_local, float* e,
                                    uint8_t* payload, int64_t rows, int64_t cols, int32_t k, float beta,
                                    void* cuda_stream);

const char* sl_strerror(sl_status s);
const char* sl_last_cuda_error(void); /* text of the last CUDA error seen by this thread */

#ifdef __cplusplus
}
#endif
#endif /* SPARSELOCO_H */
