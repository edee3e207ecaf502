/*
 * CPU oracle for the SparseLoCo outer step.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-definition implementation of what the outer step
 * computes, written from the paper's statement of the method.  It shares no
 * code with the CUDA library and is never called by it: only the tests, the
 * smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What follows what:
 *   pseudo-gradient  Delta_r = theta - theta_r         Sec. 3.1; Algorithm 1, pseudo-gradient line
 *   error feedback   u = beta e + Delta                Eq. 2 line 1; Algorithm 1, compression line
 *   chunked Top-k    64x64 blocks of 2-D tensors, runs of 4096 of 1-D tensors,
 *                    Top-k by magnitude inside each chunk       Sec. 3.3 (chunk-wise Top-k paragraph)
 *   quantiser Q      per tensor: centre by the mean, [-6 sigma, 6 sigma] in four
 *                    uniform bins, each bin's centroid as look-up table    Sec. 4 (experimental setup)
 *   index cost       12 bits per in-chunk index at C = 4096     App. "Compression of indices"
 *   EF subtract      e = u - Delta_hat                  Eq. 2 line 2; Algorithm 1, error line
 *   aggregate        Delta = (1/R) sum_r Delta_hat_r    Eq. 2 line 3; Algorithm 1, aggregation line
 *   outer update     theta = theta - alpha Delta        Eq. 2 line 4; Algorithm 1, last line
 *   EF freeze        e neither used nor accumulated     App. "Freezing Error Feedback"
 *
 * Readings taken where the paper is silent (each is also listed in the design
 * notes of the repository):
 *   - "magnitude" = the IEEE-754 bit pattern with the sign bit cleared, compared
 *     as an unsigned integer; ties go to the lowest in-chunk index.
 *   - in-chunk index of a 64x64 block is row-major inside the block; blocks are
 *     visited block-row-major; a 2-D tensor whose sides are not both multiples
 *     of the block side is treated as 1-D (row-major runs of 4096, short tail).
 *   - selected entries of a chunk are listed by ascending in-chunk index.
 *   - u = fmaf(beta, e, theta - theta_r): one fp32 subtraction, one fused
 *     multiply-add, round-to-nearest, denormals kept.
 *   - sigma is the population standard deviation (divide by n) of the fp32
 *     centred values; sums are fp64, taken slot by slot inside a chunk, then
 *     chunk by chunk inside a group of 64 consecutive chunks, then group by group.
 *     Bin edges on centred values are -3 sigma, 0, +3 sigma
 *     with the lower edge inclusive; values beyond +-6 sigma fall in the outer
 *     bins.  Centroids are means of the raw (uncentred) values; an empty bin
 *     stores +0.
 *   - the average divides by R even when a worker's payload is absent, unless
 *     divide_by_present is set.
 *   - bf16 storage (storage_bf16 = 1; the paper does not speak of storage types): theta,
 *     theta_r and e hold bfloat16 values (here: fp32 arrays whose entries are bf16-representable).
 *     All arithmetic is the fp32 / fp64 arithmetic above on the widened values, so the selection
 *     and the quantiser see the unrounded u; only what is stored is rounded, once, to nearest-even
 *     bfloat16: e = bf16(u) where nothing was selected, e = bf16(u - Delta_hat) where something
 *     was, theta = bf16(theta - alpha Delta) for the elements some worker selected.
 *
 * Every function here is pinned by tests/test_oracle_*.py against brute force,
 * hand-worked cases, closed forms and invariants (none of them produced by this
 * file or by the CUDA path).
 *
 * Arithmetic: fp32 where the method stores fp32 (u, e, centred values, sigma,
 * thresholds, table), fp64 for every accumulation.  Build with
 * -ffp-contract=off and without -ffast-math.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t rows, cols; /* 1-D tensor: rows == 1 */
    int64_t offset;     /* element offset into every flat buffer */
} orc_tensor;

typedef struct {
    int32_t chunk_elems; /* C; tile_dim * tile_dim */
    int32_t tile_dim;    /* side of a 2-D block */
    int32_t k;
    int32_t R, H;
    float beta, outer_lr;
    int32_t quant_bits;        /* 2 (the paper's setting), 1 / 3 / 4 (its ablation), or 32 = values sent unquantised */
    int32_t ef_enabled;        /* 0 during the error-feedback freeze */
    int32_t divide_by_present; /* 0: divide by R; 1: by the number of payloads present */
    int32_t storage_bf16;      /* 1: theta, theta_r and e are bfloat16 values; results are rounded on store */
} orc_config;

/* ---------------------------------------------------------------- bfloat16 rounding
 * bfloat16 = sign, 8 exponent bits, 7 fraction bits (the upper half of an fp32).  Round to nearest,
 * ties to even, in one step from the given value: |x| = f 2^ex with f in [0.5, 1) has its 8
 * significant bits down to 2^(ex - 8); subnormals (below 2^-126) share the spacing 2^-133. */
float orc_bf16_round_d(double x) {
    if (x == 0.0 || !isfinite(x)) return (float)x;
    int ex;
    (void)frexp(x, &ex);
    int lsb = ex - 8;
    if (lsb < -133) lsb = -133;
    double q = nearbyint(ldexp(x, -lsb)); /* exact scaling; nearbyint rounds half to even (default mode) */
    return (float)ldexp(q, lsb);
}
float orc_bf16_round(float x) { return orc_bf16_round_d((double)x); }

static int g_threads = 1;
void orc_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int orc_get_threads(void) { return g_threads; }

/* ---------------------------------------------------------------- chunk geometry (Sec. 3.3) */

static int is_tiled(const orc_config* c, const orc_tensor* t) {
    return t->rows > 1 && t->rows % c->tile_dim == 0 && t->cols % c->tile_dim == 0;
}

int64_t orc_num_chunks(const orc_config* c, const orc_tensor* t) {
    int64_t n = t->rows * t->cols;
    if (is_tiled(c, t)) return (t->rows / c->tile_dim) * (t->cols / c->tile_dim);
    return (n + c->chunk_elems - 1) / c->chunk_elems;
}

/* Length of chunk `ch` of tensor t. */
int64_t orc_chunk_len(const orc_config* c, const orc_tensor* t, int64_t ch) {
    if (is_tiled(c, t)) return c->chunk_elems;
    int64_t n = t->rows * t->cols;
    int64_t start = ch * c->chunk_elems;
    int64_t rest = n - start;
    return rest < c->chunk_elems ? rest : c->chunk_elems;
}

/* Element position (inside the tensor, row-major) of in-chunk index p of chunk ch. */
int64_t orc_chunk_pos(const orc_config* c, const orc_tensor* t, int64_t ch, int64_t p) {
    if (is_tiled(c, t)) {
        int64_t tiles_per_row = t->cols / c->tile_dim;
        int64_t tr = ch / tiles_per_row, tc = ch % tiles_per_row;
        int64_t row = tr * c->tile_dim + p / c->tile_dim;
        int64_t col = tc * c->tile_dim + p % c->tile_dim;
        return row * t->cols + col;
    }
    return ch * c->chunk_elems + p;
}

int64_t orc_total_chunks(const orc_config* c, const orc_tensor* ts, int32_t nt) {
    int64_t s = 0;
    for (int32_t j = 0; j < nt; ++j) s += orc_num_chunks(c, &ts[j]);
    return s;
}

/* Total number of selected entries of one worker: sum over chunks of min(k, chunk length). */
int64_t orc_total_slots(const orc_config* c, const orc_tensor* ts, int32_t nt) {
    int64_t s = 0;
    for (int32_t j = 0; j < nt; ++j) {
        int64_t nc = orc_num_chunks(c, &ts[j]);
        for (int64_t ch = 0; ch < nc; ++ch) {
            int64_t L = orc_chunk_len(c, &ts[j], ch);
            s += L < c->k ? L : c->k;
        }
    }
    return s;
}

/* ---------------------------------------------------------------- payload geometry (App. index cost) */

/* Bytes of one chunk record: k 12-bit indices, then k 2-bit codes, rounded up to 16. */
int64_t orc_record_stride(int32_t k) {
    int64_t idx_bytes = (12 * (int64_t)k + 7) / 8;
    int64_t code_bytes = (2 * (int64_t)k + 7) / 8;
    return (idx_bytes + code_bytes + 15) / 16 * 16;
}

/* The same for a quantiser of `bits` bits per value (1..4; the paper's ablation over quantisation
 * widths): k 12-bit indices, then k codes of `bits` bits, rounded up to 16. */
int64_t orc_record_stride_q(int32_t k, int32_t bits) {
    int64_t idx_bytes = (12 * (int64_t)k + 7) / 8;
    int64_t code_bytes = ((int64_t)bits * (int64_t)k + 7) / 8;
    return (idx_bytes + code_bytes + 15) / 16 * 16;
}

/* Bytes of a tensor's table in the payload: 2^bits fp32 entries, at least 16 bytes. */
int64_t orc_header_bytes(int32_t bits) {
    int64_t b = 4 * ((int64_t)1 << bits);
    return b < 16 ? 16 : b;
}

static int32_t payload_bits(const orc_config* c) { return c->quant_bits == 32 ? 2 : c->quant_bits; }

/* Bytes of one worker's payload: one table per tensor (16 bytes at 2 bits), then every chunk record. */
int64_t orc_payload_bytes(const orc_config* c, const orc_tensor* ts, int32_t nt) {
    const int32_t b = payload_bits(c);
    return orc_header_bytes(b) * (int64_t)nt + orc_record_stride_q(c->k, b) * orc_total_chunks(c, ts, nt);
}

/* ---------------------------------------------------------------- pseudo-gradient + error feedback */

/* u[i] = beta * e[i] + (theta[i] - theta_r[i]); with the freeze on, u = theta - theta_r.
 * Eq. 2 line 1 / Algorithm 1. */
void orc_ef_accumulate(const float* theta, const float* theta_r, const float* e, int64_t n,
                       float beta, int ef_enabled, float* u) {
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        float d = theta[i] - theta_r[i];
        u[i] = ef_enabled ? fmaf(beta, e[i], d) : d;
    }
}

/* ---------------------------------------------------------------- Top-k of one chunk */

typedef struct {
    uint32_t key; /* magnitude: bit pattern without the sign */
    int32_t p;    /* in-chunk index */
} keyed;

static uint32_t mag_key(float x) {
    uint32_t b;
    memcpy(&b, &x, 4);
    return b & 0x7FFFFFFFu;
}

static int cmp_mag_desc_index_asc(const void* a, const void* b) {
    const keyed* x = (const keyed*)a;
    const keyed* y = (const keyed*)b;
    if (x->key != y->key) return x->key > y->key ? -1 : 1;
    return x->p < y->p ? -1 : (x->p > y->p ? 1 : 0);
}

static int cmp_int32_asc(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}

/* The min(k, L) entries of u[0..L) of largest magnitude, ties to the lower index,
 * returned as ascending in-chunk indices.  Full sort, by definition.  Returns the count. */
int32_t orc_topk_chunk(const float* u, int32_t L, int32_t k, int32_t* idx_out) {
    keyed* a = (keyed*)malloc(sizeof(keyed) * (size_t)(L > 0 ? L : 1));
    for (int32_t p = 0; p < L; ++p) {
        a[p].key = mag_key(u[p]);
        a[p].p = p;
    }
    qsort(a, (size_t)L, sizeof(keyed), cmp_mag_desc_index_asc);
    int32_t m = k < L ? k : L;
    for (int32_t s = 0; s < m; ++s) idx_out[s] = a[s].p;
    qsort(idx_out, (size_t)m, sizeof(int32_t), cmp_int32_asc);
    free(a);
    return m;
}

/* ---------------------------------------------------------------- quantiser Q of one tensor */

#define ORC_SUM_GROUP 64 /* chunks per group in the three-level summation order */

/* v: the tensor's selected values, chunk after chunk, each chunk's `cnt[c]` values in slot order.
 * Outputs: mu, sigma, lut[4], code per value.  Sec. 4: centre by the mean, [-6 sigma, 6 sigma]
 * in four uniform bins (edges -3 sigma, 0, 3 sigma on centred values), centroid table. */
void orc_quantize_tensor(const float* v, const int32_t* cnt, int64_t n_chunks, float* mu_out,
                         float* sigma_out, float lut[4], uint8_t* code) {
    int64_t n = 0;
    for (int64_t c = 0; c < n_chunks; ++c) n += cnt[c];
    lut[0] = lut[1] = lut[2] = lut[3] = 0.0f;
    *mu_out = 0.0f;
    *sigma_out = 0.0f;
    if (n == 0) return;

    /* Every sum over the tensor is taken in three fixed levels, all fp64, each left to right:
     * the slots of a chunk, the chunks of a group of ORC_SUM_GROUP consecutive chunks, the groups. */
    double S = 0.0;
    {
        const float* q = v;
        for (int64_t c0 = 0; c0 < n_chunks; c0 += ORC_SUM_GROUP) {
            double sg = 0.0;
            for (int64_t c = c0; c < n_chunks && c < c0 + ORC_SUM_GROUP; ++c) {
                double sc = 0.0;
                for (int32_t s = 0; s < cnt[c]; ++s) sc += (double)q[s];
                sg += sc;
                q += cnt[c];
            }
            S += sg;
        }
    }
    float mu = (float)(S / (double)n);

    double V = 0.0;
    {
        const float* q = v;
        for (int64_t c0 = 0; c0 < n_chunks; c0 += ORC_SUM_GROUP) {
            double vg = 0.0;
            for (int64_t c = c0; c < n_chunks && c < c0 + ORC_SUM_GROUP; ++c) {
                double vc = 0.0;
                for (int32_t s = 0; s < cnt[c]; ++s) {
                    float cen = q[s] - mu;
                    double d = (double)cen;
                    vc += d * d;
                }
                vg += vc;
                q += cnt[c];
            }
            V += vg;
        }
    }
    float sigma = (float)sqrt(V / (double)n);
    float t = 3.0f * sigma;

    double Sb[4] = {0.0, 0.0, 0.0, 0.0};
    int64_t nb[4] = {0, 0, 0, 0};
    {
        const float* q = v;
        uint8_t* cq = code;
        for (int64_t c0 = 0; c0 < n_chunks; c0 += ORC_SUM_GROUP) {
            double sgb[4] = {0.0, 0.0, 0.0, 0.0};
            for (int64_t c = c0; c < n_chunks && c < c0 + ORC_SUM_GROUP; ++c) {
                double sb[4] = {0.0, 0.0, 0.0, 0.0};
                for (int32_t s = 0; s < cnt[c]; ++s) {
                    float cen = q[s] - mu;
                    int b = (cen >= -t) + (cen >= 0.0f) + (cen >= t);
                    cq[s] = (uint8_t)b;
                    sb[b] += (double)q[s];
                    nb[b] += 1;
                }
                for (int b = 0; b < 4; ++b) sgb[b] += sb[b];
                q += cnt[c];
                cq += cnt[c];
            }
            for (int b = 0; b < 4; ++b) Sb[b] += sgb[b];
        }
    }
    for (int b = 0; b < 4; ++b) lut[b] = nb[b] ? (float)(Sb[b] / (double)nb[b]) : 0.0f;
    *mu_out = mu;
    *sigma_out = sigma;
}

/* The quantiser of Sec. 4 at any width (the paper's ablation uses 1, 2, 3 and 4 bits): centred by
 * the mean, [-6 sigma, 6 sigma] in 2^bits uniform bins, every bin stores the centroid of the raw
 * values that fell into it.  Written like the 2-bit routine above, with the same fixed summation
 * order: the inner edges are c_j sigma with c_j = -6 + 12 j / 2^bits (j = 1 .. 2^bits - 1; multiples
 * of 0.75, exact in fp32), each the fp32 product of c_j and sigma, lower edge inclusive, so that
 * code = number of edges the centred value reaches; values beyond +-6 sigma fall in the outer bins.
 * At bits = 2 the edges are -3 sigma, 0, 3 sigma: the routine above. */
void orc_quantize_tensor_q(const float* v, const int32_t* cnt, int64_t n_chunks, int32_t bits,
                           float* mu_out, float* sigma_out, float* lut /* 2^bits */, uint8_t* code) {
    const int nbins = 1 << bits;
    int64_t n = 0;
    for (int64_t c = 0; c < n_chunks; ++c) n += cnt[c];
    for (int b = 0; b < nbins; ++b) lut[b] = 0.0f;
    *mu_out = 0.0f;
    *sigma_out = 0.0f;
    if (n == 0) return;

    double S = 0.0;
    {
        const float* q = v;
        for (int64_t c0 = 0; c0 < n_chunks; c0 += ORC_SUM_GROUP) {
            double sg = 0.0;
            for (int64_t c = c0; c < n_chunks && c < c0 + ORC_SUM_GROUP; ++c) {
                double sc = 0.0;
                for (int32_t s = 0; s < cnt[c]; ++s) sc += (double)q[s];
                sg += sc;
                q += cnt[c];
            }
            S += sg;
        }
    }
    const float mu = (float)(S / (double)n);

    double V = 0.0;
    {
        const float* q = v;
        for (int64_t c0 = 0; c0 < n_chunks; c0 += ORC_SUM_GROUP) {
            double vg = 0.0;
            for (int64_t c = c0; c < n_chunks && c < c0 + ORC_SUM_GROUP; ++c) {
                double vc = 0.0;
                for (int32_t s = 0; s < cnt[c]; ++s) {
                    const float cen = q[s] - mu;
                    vc += (double)cen * (double)cen;
                }
                vg += vc;
                q += cnt[c];
            }
            V += vg;
        }
    }
    const float sigma = (float)sqrt(V / (double)n);

    float edge[15];
    for (int j = 1; j < nbins; ++j) edge[j - 1] = (-6.0f + 12.0f * (float)j / (float)nbins) * sigma;

    double Sb[16];
    int64_t nb[16];
    for (int b = 0; b < 16; ++b) { Sb[b] = 0.0; nb[b] = 0; }
    {
        const float* q = v;
        uint8_t* cq = code;
        for (int64_t c0 = 0; c0 < n_chunks; c0 += ORC_SUM_GROUP) {
            double sgb[16];
            for (int b = 0; b < 16; ++b) sgb[b] = 0.0;
            for (int64_t c = c0; c < n_chunks && c < c0 + ORC_SUM_GROUP; ++c) {
                double sb[16];
                for (int b = 0; b < 16; ++b) sb[b] = 0.0;
                for (int32_t s = 0; s < cnt[c]; ++s) {
                    const float cen = q[s] - mu;
                    int b = 0;
                    for (int j = 0; j < nbins - 1; ++j) b += cen >= edge[j];
                    cq[s] = (uint8_t)b;
                    sb[b] += (double)q[s];
                    nb[b] += 1;
                }
                for (int b = 0; b < nbins; ++b) sgb[b] += sb[b];
                q += cnt[c];
                cq += cnt[c];
            }
            for (int b = 0; b < nbins; ++b) Sb[b] += sgb[b];
        }
    }
    for (int b = 0; b < nbins; ++b) lut[b] = nb[b] ? (float)(Sb[b] / (double)nb[b]) : 0.0f;
    *mu_out = mu;
    *sigma_out = sigma;
}

/* ---------------------------------------------------------------- packing (little-endian bit order) */

static void put_bits(uint8_t* base, int64_t bit, int nbits, uint32_t val) {
    for (int i = 0; i < nbits; ++i) {
        if ((val >> i) & 1u) base[(bit + i) >> 3] |= (uint8_t)(1u << ((bit + i) & 7));
    }
}

static uint32_t get_bits(const uint8_t* base, int64_t bit, int nbits) {
    uint32_t v = 0;
    for (int i = 0; i < nbits; ++i) {
        v |= (uint32_t)((base[(bit + i) >> 3] >> ((bit + i) & 7)) & 1u) << i;
    }
    return v;
}

/* One chunk record: index block (12 bits per slot), then code block (2 bits per slot) starting
 * at byte ceil(12k/8).  Slots >= m and all padding stay zero. */
void orc_pack_record(const int32_t* idx, const uint8_t* code, int32_t m, int32_t k, uint8_t* rec) {
    memset(rec, 0, (size_t)orc_record_stride(k));
    int64_t code_base = ((12 * (int64_t)k + 7) / 8) * 8;
    for (int32_t s = 0; s < m; ++s) {
        put_bits(rec, 12 * (int64_t)s, 12, (uint32_t)idx[s]);
        put_bits(rec, code_base + 2 * (int64_t)s, 2, code[s]);
    }
}

void orc_unpack_record(const uint8_t* rec, int32_t m, int32_t k, int32_t* idx, uint8_t* code) {
    int64_t code_base = ((12 * (int64_t)k + 7) / 8) * 8;
    for (int32_t s = 0; s < m; ++s) {
        idx[s] = (int32_t)get_bits(rec, 12 * (int64_t)s, 12);
        code[s] = (uint8_t)get_bits(rec, code_base + 2 * (int64_t)s, 2);
    }
}

/* The same with codes of `bits` bits (1..4). */
void orc_pack_record_q(const int32_t* idx, const uint8_t* code, int32_t m, int32_t k, int32_t bits, uint8_t* rec) {
    memset(rec, 0, (size_t)orc_record_stride_q(k, bits));
    int64_t code_base = ((12 * (int64_t)k + 7) / 8) * 8;
    for (int32_t s = 0; s < m; ++s) {
        put_bits(rec, 12 * (int64_t)s, 12, (uint32_t)idx[s]);
        put_bits(rec, code_base + (int64_t)bits * s, bits, code[s]);
    }
}

void orc_unpack_record_q(const uint8_t* rec, int32_t m, int32_t k, int32_t bits, int32_t* idx, uint8_t* code) {
    int64_t code_base = ((12 * (int64_t)k + 7) / 8) * 8;
    for (int32_t s = 0; s < m; ++s) {
        idx[s] = (int32_t)get_bits(rec, 12 * (int64_t)s, 12);
        code[s] = (uint8_t)get_bits(rec, code_base + (int64_t)bits * s, bits);
    }
}

/* ---------------------------------------------------------------- one worker's compression */

/*
 * Algorithm 1, compression + error feedback block, for one worker over all tensors.
 *   theta, theta_r, e : flat fp32 buffers (tensor j at ts[j].offset); e is updated in place
 *                       (left untouched when ef_enabled == 0).
 *   payload           : orc_payload_bytes() bytes, or NULL (also unused when quant_bits == 32).
 *   sel_idx, sel_val, sel_hat : optional (may be NULL) arrays of orc_total_slots() entries, in
 *                       (tensor, chunk, slot) order: in-chunk index, raw value u, decoded value.
 *   stats             : optional, 18 floats per tensor: mu, sigma, the table (2^bits entries, then zeros).
 */
void orc_compress(const orc_config* cfg, const orc_tensor* ts, int32_t nt, const float* theta,
                  const float* theta_r, float* e, uint8_t* payload, int32_t* sel_idx,
                  float* sel_val, float* sel_hat, float* stats) {
    const int32_t k = cfg->k, C = cfg->chunk_elems;
    const int32_t qb = cfg->quant_bits;            /* 1..4, or 32 = values travel unquantised */
    const int quantised = qb >= 1 && qb <= 4;
    const int64_t stride = orc_record_stride_q(k, payload_bits(cfg)), hdr = orc_header_bytes(payload_bits(cfg));
    int64_t rec_off = hdr * (int64_t)nt; /* records follow the per-tensor tables */
    int64_t slot_off = 0;
    if (payload && quantised) memset(payload, 0, (size_t)orc_payload_bytes(cfg, ts, nt));

    for (int32_t j = 0; j < nt; ++j) {
        const orc_tensor* t = &ts[j];
        const int64_t n = t->rows * t->cols, nc = orc_num_chunks(cfg, t);
        const float* th = theta + t->offset;
        const float* tr = theta_r + t->offset;
        float* ej = e + t->offset;

        float* u = (float*)malloc(sizeof(float) * (size_t)n);
        orc_ef_accumulate(th, tr, ej, n, cfg->beta, cfg->ef_enabled, u);

        int32_t* cnt = (int32_t*)malloc(sizeof(int32_t) * (size_t)nc);
        int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)(nc * k));
        float* val = (float*)malloc(sizeof(float) * (size_t)(nc * k));

        /* chunk-wise Top-k; chunks are independent */
#pragma omp parallel for num_threads(g_threads) schedule(dynamic, 4)
        for (int64_t ch = 0; ch < nc; ++ch) {
            int32_t L = (int32_t)orc_chunk_len(cfg, t, ch);
            float* cu = (float*)malloc(sizeof(float) * (size_t)C);
            for (int32_t p = 0; p < L; ++p) cu[p] = u[orc_chunk_pos(cfg, t, ch, p)];
            cnt[ch] = orc_topk_chunk(cu, L, k, idx + ch * k);
            for (int32_t s = 0; s < cnt[ch]; ++s) val[ch * k + s] = cu[idx[ch * k + s]];
            free(cu);
        }

        /* the tensor's selected values, chunk after chunk in slot order */
        int64_t m_total = 0;
        for (int64_t ch = 0; ch < nc; ++ch) m_total += cnt[ch];
        float* v = (float*)malloc(sizeof(float) * (size_t)(m_total ? m_total : 1));
        float* vhat = (float*)malloc(sizeof(float) * (size_t)(m_total ? m_total : 1));
        uint8_t* code = (uint8_t*)malloc((size_t)(m_total ? m_total : 1));
        {
            int64_t w = 0;
            for (int64_t ch = 0; ch < nc; ++ch)
                for (int32_t s = 0; s < cnt[ch]; ++s) v[w++] = val[ch * k + s];
        }

        float mu = 0.0f, sigma = 0.0f, lut[16];
        for (int b = 0; b < 16; ++b) lut[b] = 0.0f;
        if (qb == 2) {
            orc_quantize_tensor(v, cnt, nc, &mu, &sigma, lut, code);
            for (int64_t w = 0; w < m_total; ++w) vhat[w] = lut[code[w]];
        } else if (quantised) {
            orc_quantize_tensor_q(v, cnt, nc, qb, &mu, &sigma, lut, code);
            for (int64_t w = 0; w < m_total; ++w) vhat[w] = lut[code[w]];
        } else { /* 32: values travel unquantised */
            for (int64_t w = 0; w < m_total; ++w) vhat[w] = v[w];
        }
        if (stats) { /* 18 floats per tensor: mu, sigma, table (2^bits entries, the rest 0) */
            stats[18 * j + 0] = mu;
            stats[18 * j + 1] = sigma;
            for (int b = 0; b < 16; ++b) stats[18 * j + 2 + b] = lut[b];
        }

        /* payload: table, then records */
        if (payload && quantised) {
            memcpy(payload + hdr * (int64_t)j, lut, (size_t)(4 << qb));
            int64_t w = 0;
            for (int64_t ch = 0; ch < nc; ++ch) {
                if (qb == 2) orc_pack_record(idx + ch * k, code + w, cnt[ch], k, payload + rec_off + ch * stride);
                else orc_pack_record_q(idx + ch * k, code + w, cnt[ch], k, qb, payload + rec_off + ch * stride);
                w += cnt[ch];
            }
        }
        rec_off += nc * stride;

        /* error feedback: e = u - Delta_hat (Eq. 2 line 2) */
        if (cfg->ef_enabled) {
            for (int64_t i = 0; i < n; ++i) ej[i] = u[i];
            int64_t w = 0;
            for (int64_t ch = 0; ch < nc; ++ch)
                for (int32_t s = 0; s < cnt[ch]; ++s, ++w) {
                    int64_t pos = orc_chunk_pos(cfg, t, ch, idx[ch * k + s]);
                    ej[pos] = u[pos] - vhat[w];
                }
            if (cfg->storage_bf16) /* the stored error is the bfloat16 nearest to it */
                for (int64_t i = 0; i < n; ++i) ej[i] = orc_bf16_round(ej[i]);
        }

        {
            int64_t w = 0;
            for (int64_t ch = 0; ch < nc; ++ch)
                for (int32_t s = 0; s < cnt[ch]; ++s, ++w) {
                    if (sel_idx) sel_idx[slot_off + w] = idx[ch * k + s];
                    if (sel_val) sel_val[slot_off + w] = v[w];
                    if (sel_hat) sel_hat[slot_off + w] = vhat[w];
                }
        }
        slot_off += m_total;

        free(u); free(cnt); free(idx); free(val); free(v); free(vhat); free(code);
    }
}

/* ---------------------------------------------------------------- aggregate + outer update */

/*
 * Eq. 2 lines 3-4 from sparse lists.  For worker r (r < R), sel_idx[r] / sel_hat[r] hold its
 * selected in-chunk indices and decoded values in (tensor, chunk, slot) order, or are NULL when
 * that worker is absent.  theta[i] <- (float)(theta[i] - alpha * (sum_r hat_r[i]) / D) in fp64,
 * r ascending; elements no worker selected are left bit-unchanged.
 */
void orc_aggregate_apply_sparse(const orc_config* cfg, const orc_tensor* ts, int32_t nt,
                                const int32_t* const* sel_idx, const float* const* sel_hat,
                                float* theta) {
    const int32_t k = cfg->k, R = cfg->R;
    int present = 0;
    for (int32_t r = 0; r < R; ++r) present += sel_idx[r] != NULL;
    const double D = cfg->divide_by_present ? (double)present : (double)R;
    if (present == 0) return;

    int64_t slot_off = 0;
    for (int32_t j = 0; j < nt; ++j) {
        const orc_tensor* t = &ts[j];
        const int64_t n = t->rows * t->cols, nc = orc_num_chunks(cfg, t);
        double* acc = (double*)calloc((size_t)n, sizeof(double));
        uint8_t* hit = (uint8_t*)calloc((size_t)n, 1);
        int64_t m_tensor = 0; /* slots of this tensor in every worker's list */
        for (int64_t ch = 0; ch < nc; ++ch) {
            int64_t L = orc_chunk_len(cfg, t, ch);
            m_tensor += L < k ? L : k;
        }
        for (int32_t r = 0; r < R; ++r) {
            if (!sel_idx[r]) continue;
            int64_t w = slot_off;
            for (int64_t ch = 0; ch < nc; ++ch) {
                int64_t L = orc_chunk_len(cfg, t, ch);
                int64_t m = L < k ? L : k;
                for (int64_t s = 0; s < m; ++s, ++w) {
                    int64_t pos = orc_chunk_pos(cfg, t, ch, sel_idx[r][w]);
                    acc[pos] += (double)sel_hat[r][w];
                    hit[pos] = 1;
                }
            }
        }
        float* th = theta + t->offset;
        for (int64_t i = 0; i < n; ++i) {
            if (!hit[i]) continue;
            const double x = (double)th[i] - (double)cfg->outer_lr * acc[i] / D;
            th[i] = cfg->storage_bf16 ? orc_bf16_round_d(x) : (float)x;
        }
        slot_off += m_tensor;
        free(acc); free(hit);
    }
}

/* Decode one worker's payload (2-bit format) into sparse lists in (tensor, chunk, slot) order.
 * Sec. 4: values are dequantised through the table before aggregation. */
void orc_decode_payload(const orc_config* cfg, const orc_tensor* ts, int32_t nt,
                        const uint8_t* payload, int32_t* sel_idx, float* sel_hat) {
    const int32_t k = cfg->k, qb = payload_bits(cfg);
    const int64_t stride = orc_record_stride_q(k, qb), hdr = orc_header_bytes(qb);
    int64_t rec_off = hdr * (int64_t)nt, w = 0;
    uint8_t* code = (uint8_t*)malloc((size_t)k);
    for (int32_t j = 0; j < nt; ++j) {
        float lut[16];
        memcpy(lut, payload + hdr * (int64_t)j, (size_t)(4 << qb));
        int64_t nc = orc_num_chunks(cfg, &ts[j]);
        for (int64_t ch = 0; ch < nc; ++ch) {
            int64_t L = orc_chunk_len(cfg, &ts[j], ch);
            int32_t m = (int32_t)(L < k ? L : k);
            if (qb == 2) orc_unpack_record(payload + rec_off + ch * stride, m, k, sel_idx + w, code);
            else orc_unpack_record_q(payload + rec_off + ch * stride, m, k, qb, sel_idx + w, code);
            for (int32_t s = 0; s < m; ++s) sel_hat[w + s] = lut[code[s]];
            w += m;
        }
        rec_off += nc * stride;
    }
    free(code);
}

/* Eq. 2 lines 3-4 from R packed payloads (NULL = absent worker). */
void orc_aggregate_apply(const orc_config* cfg, const orc_tensor* ts, int32_t nt,
                         const uint8_t* const* payloads, float* theta) {
    const int32_t R = cfg->R;
    const int64_t slots = orc_total_slots(cfg, ts, nt);
    int32_t** idx = (int32_t**)calloc((size_t)R, sizeof(int32_t*));
    float** hat = (float**)calloc((size_t)R, sizeof(float*));
    for (int32_t r = 0; r < R; ++r) {
        if (!payloads[r]) continue;
        idx[r] = (int32_t*)malloc(sizeof(int32_t) * (size_t)(slots ? slots : 1));
        hat[r] = (float*)malloc(sizeof(float) * (size_t)(slots ? slots : 1));
        orc_decode_payload(cfg, ts, nt, payloads[r], idx[r], hat[r]);
    }
    orc_aggregate_apply_sparse(cfg, ts, nt, (const int32_t* const*)idx, (const float* const*)hat,
                               theta);
    for (int32_t r = 0; r < R; ++r) { free(idx[r]); free(hat[r]); }
    free(idx); free(hat);
}

/* One full outer step (Algorithm 1, lines after the inner loop): compress every worker, then
 * aggregate and update theta.  payloads[r] must each hold orc_payload_bytes() bytes. */
void orc_outer_step(const orc_config* cfg, const orc_tensor* ts, int32_t nt, float* theta,
                    const float* const* theta_r, float* const* e, uint8_t* const* payloads) {
    for (int32_t r = 0; r < cfg->R; ++r)
        orc_compress(cfg, ts, nt, theta, theta_r[r], e[r], payloads[r], NULL, NULL, NULL, NULL);
    orc_aggregate_apply(cfg, ts, nt, (const uint8_t* const*)payloads, theta);
}

/* ================================================================ entropy-coded indices
 *
 * App. "Compression of indices": 12 bits per index is the naive cost; the bound is
 * log2 C(C, k) / k bits (8.3 / 6.3 / 5.3 at k = 32 / 128 / 256) and the paper reports 8.9 / 6.6 /
 * 5.6 from a custom scheme of which it names only the ingredients.  The scheme below is this
 * library's own; what is pinned is round-trip exactness, the closed-form length, and that the
 * rate on uniformly drawn index sets lies between the bound and the paper's achieved numbers.
 *
 * One chunk, length L, m_sel = min(k, L) ascending indices p_0 < p_1 < ...:
 *   gaps        g_0 = p_0,  g_i = p_i - p_(i-1) - 1
 *   divisor     M = max(1, (693 (L - m_sel) + 500 (m_sel + 1)) / (1000 (m_sel + 1)))   (integers:
 *               0.693 x the mean gap, the Golomb optimum for geometric gaps)
 *   code of g   q = g / M one-bits, a zero-bit, then r = g % M in truncated binary:
 *               b = ceil(log2 M), cut = 2^b - M; r < cut -> r in b - 1 bits, else r + cut in b bits,
 *               most significant bit first (nothing when M = 1)
 * The chunk's codes follow one another; bit i of a stream sits in byte i / 8 at bit i % 8.
 *
 * Coded payload of one worker (all multi-byte fields little-endian):
 *   [0, 16 T)                      the T tensor tables, as in the 12-bit payload
 *   [16 T, 16 T + cb G)            the code blocks of the G chunks, cb = ceil(2 k / 8) bytes each,
 *                                  copied from the 12-bit records
 *   up to the next multiple of 4, then ceil(G / 16) x uint32: bit offset, within the index stream,
 *                                  of the first chunk of every group of 16 chunks
 *   the index stream: every chunk's codes in (tensor, chunk) order, no padding between chunks
 *   zero bytes up to a multiple of 16
 */

static int32_t ixc_divisor(int32_t L, int32_t m_sel) {
    int64_t M = (693 * (int64_t)(L - m_sel) + 500 * (int64_t)(m_sel + 1)) / (1000 * (int64_t)(m_sel + 1));
    return M < 1 ? 1 : (int32_t)M;
}

static int ixc_ceil_log2(int32_t M) {
    int b = 0;
    while ((1 << b) < M) ++b;
    return b;
}

static void ixc_put_bit(uint8_t* stream, int64_t* pos, int bit) {
    if (stream && bit) stream[*pos >> 3] |= (uint8_t)(1u << (*pos & 7));
    ++*pos;
}

/* Appends the codes of one chunk at bit position *pos (stream may be NULL: length only). */
void orc_ixc_encode_chunk(const int32_t* idx, int32_t m_sel, int32_t L, uint8_t* stream, int64_t* pos) {
    const int32_t M = ixc_divisor(L, m_sel);
    const int b = ixc_ceil_log2(M);
    const int32_t cut = (1 << b) - M;
    int32_t prev = -1;
    for (int32_t s = 0; s < m_sel; ++s) {
        const int32_t g = idx[s] - prev - 1;
        prev = idx[s];
        const int32_t q = g / M, r = g % M;
        for (int32_t i = 0; i < q; ++i) ixc_put_bit(stream, pos, 1);
        ixc_put_bit(stream, pos, 0);
        if (M > 1) {
            int nb = b;
            int32_t v = r + cut;
            if (r < cut) { nb = b - 1; v = r; }
            for (int i = nb - 1; i >= 0; --i) ixc_put_bit(stream, pos, (v >> i) & 1);
        }
    }
}

static int ixc_get_bit(const uint8_t* stream, int64_t* pos) {
    int bit = (stream[*pos >> 3] >> (*pos & 7)) & 1;
    ++*pos;
    return bit;
}

void orc_ixc_decode_chunk(const uint8_t* stream, int64_t* pos, int32_t m_sel, int32_t L, int32_t* idx) {
    const int32_t M = ixc_divisor(L, m_sel);
    const int b = ixc_ceil_log2(M);
    const int32_t cut = (1 << b) - M;
    int32_t prev = -1;
    for (int32_t s = 0; s < m_sel; ++s) {
        int32_t q = 0;
        while (ixc_get_bit(stream, pos)) ++q;
        int32_t r = 0;
        if (M > 1) {
            for (int i = 0; i < b - 1; ++i) r = (r << 1) | ixc_get_bit(stream, pos);
            if (r >= cut) r = ((r << 1) | ixc_get_bit(stream, pos)) - cut;
        }
        prev = prev + 1 + q * M + r;
        idx[s] = prev;
    }
}

static int64_t ixc_fixed_bytes(const orc_config* c, const orc_tensor* ts, int32_t nt, int64_t* dir_off) {
    const int64_t G = orc_total_chunks(c, ts, nt);
    const int64_t cb = (2 * (int64_t)c->k + 7) / 8;
    int64_t off = 16 * (int64_t)nt + cb * G;
    off = (off + 3) / 4 * 4;
    if (dir_off) *dir_off = off;
    return off + 4 * ((G + 15) / 16);
}

/* 12-bit payload -> coded payload.  out may be NULL (size only).  Returns the coded size in bytes. */
int64_t orc_ixc_encode_payload(const orc_config* c, const orc_tensor* ts, int32_t nt, const uint8_t* payload,
                               uint8_t* out) {
    const int32_t k = c->k;
    const int64_t stride = orc_record_stride(k), cb = (2 * (int64_t)k + 7) / 8, ib = (12 * (int64_t)k + 7) / 8;
    int64_t dir_off = 0;
    const int64_t stream_off = ixc_fixed_bytes(c, ts, nt, &dir_off);
    /* length first */
    int64_t pos = 0, g = 0;
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)k);
    uint8_t* code = (uint8_t*)malloc((size_t)k);
    for (int pass = 0; pass < 2; ++pass) {
        int64_t total = 0;
        if (pass == 1) {
            total = (stream_off + (pos + 7) / 8 + 15) / 16 * 16;
            if (!out) { free(idx); free(code); return total; }
            memset(out, 0, (size_t)total);
            memcpy(out, payload, (size_t)(16 * (int64_t)nt));
        }
        pos = 0;
        g = 0;
        const uint8_t* rec = payload + 16 * (int64_t)nt;
        for (int32_t j = 0; j < nt; ++j) {
            const int64_t nc = orc_num_chunks(c, &ts[j]);
            for (int64_t ch = 0; ch < nc; ++ch, ++g, rec += stride) {
                const int32_t L = (int32_t)orc_chunk_len(c, &ts[j], ch);
                const int32_t m_sel = L < k ? L : k;
                orc_unpack_record(rec, m_sel, k, idx, code);
                if (pass == 1) {
                    memcpy(out + 16 * (int64_t)nt + cb * g, rec + ib, (size_t)cb);
                    if (g % 16 == 0) {
                        uint32_t o = (uint32_t)pos;
                        memcpy(out + dir_off + 4 * (g / 16), &o, 4);
                    }
                }
                orc_ixc_encode_chunk(idx, m_sel, L, pass == 1 ? out + stream_off : NULL, &pos);
            }
        }
        if (pass == 1) { free(idx); free(code); return total; }
    }
    return 0;
}

/* coded payload -> 12-bit payload (orc_payload_bytes() bytes, fully written). */
void orc_ixc_decode_payload(const orc_config* c, const orc_tensor* ts, int32_t nt, const uint8_t* coded,
                            uint8_t* payload) {
    const int32_t k = c->k;
    const int64_t stride = orc_record_stride(k), cb = (2 * (int64_t)k + 7) / 8;
    const int64_t stream_off = ixc_fixed_bytes(c, ts, nt, NULL);
    memset(payload, 0, (size_t)orc_payload_bytes(c, ts, nt));
    memcpy(payload, coded, (size_t)(16 * (int64_t)nt));
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)k);
    uint8_t* code = (uint8_t*)malloc((size_t)k);
    int64_t pos = 0, g = 0;
    uint8_t* rec = payload + 16 * (int64_t)nt;
    for (int32_t j = 0; j < nt; ++j) {
        const int64_t nc = orc_num_chunks(c, &ts[j]);
        for (int64_t ch = 0; ch < nc; ++ch, ++g, rec += stride) {
            const int32_t L = (int32_t)orc_chunk_len(c, &ts[j], ch);
            const int32_t m_sel = L < k ? L : k;
            orc_ixc_decode_chunk(coded + stream_off, &pos, m_sel, L, idx);
            const uint8_t* cblk = coded + 16 * (int64_t)nt + cb * g;
            for (int32_t s = 0; s < m_sel; ++s) code[s] = (uint8_t)((cblk[(2 * s) >> 3] >> ((2 * s) & 7)) & 3);
            orc_pack_record(idx, code, m_sel, k, rec);
        }
    }
    free(idx);
    free(code);
}

/* ================================================================ dense baselines (Sec. 3.1, 3.2)
 *
 * DiLoCo's outer step, Eq. 1:  Dbar = (1/R) sum_r (theta - theta_r);  m = beta m + Dbar;
 * theta = theta - alpha (Dbar + beta m)   (Nesterov outer momentum, one global m).
 * DiLoCo-LOM (Sec. 3.2): every replica keeps its own momentum m_r = beta m_r + Delta_r, sends
 * Delta_r + beta m_r, and theta moves by alpha times their mean.  Proposition 1 states that the two
 * coincide when the m_r start equal; the tests use that as a pin.  fp64 throughout, results rounded
 * to fp32 once.  Only the elements of the tensor table are touched.
 */
void orc_diloco_step(const orc_tensor* ts, int32_t nt, int32_t R, float beta_outer, float alpha,
                     float* theta, const float* const* theta_r, float* m) {
    for (int32_t j = 0; j < nt; ++j) {
        const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
#pragma omp parallel for num_threads(g_threads) schedule(static)
        for (int64_t i = o; i < o + n; ++i) {
            double acc = 0.0;
            for (int32_t r = 0; r < R; ++r) acc += (double)theta[i] - (double)theta_r[r][i];
            const double dbar = acc / (double)R;
            const double mm = (double)beta_outer * (double)m[i] + dbar;
            theta[i] = (float)((double)theta[i] - (double)alpha * (dbar + (double)beta_outer * mm));
            m[i] = (float)mm;
        }
    }
}

void orc_diloco_lom_step(const orc_tensor* ts, int32_t nt, int32_t R, float beta_outer, float alpha,
                         float* theta, const float* const* theta_r, double* const* m_r) {
    for (int32_t j = 0; j < nt; ++j) {
        const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
        for (int64_t i = o; i < o + n; ++i) {
            double acc = 0.0;
            for (int32_t r = 0; r < R; ++r) {
                const double d = (double)theta[i] - (double)theta_r[r][i];
                m_r[r][i] = (double)beta_outer * m_r[r][i] + d;
                acc += d + (double)beta_outer * m_r[r][i];
            }
            theta[i] = (float)((double)theta[i] - (double)alpha * acc / (double)R);
        }
    }
}

/* ================================================================ the paper's Top-k / LOM variants
 *
 * App. "Exact algorithmic description of DiLoCo variants", Alg. 2-4 (Sec. 3.2 for LOM and Sub-k).
 * No quantiser: Top-k keeps the selected values as they are.  All Top-k operations are chunk-wise with
 * the chunking and tie rule of the main path.  Precision: what a worker keeps between steps (m_r, e_r)
 * and what its selection is taken on are fp32, formed by single-rounded operations in the algorithm's
 * order -- d = theta - theta_r; m_r = fma(mu, m_r, d); Nesterov direction nd = fma(mu, m_r, d);
 * u = fma(rho, e_r, .) -- because the selection depends on their bits; everything across workers (the
 * average, the global momentum, the parameter update) is evaluated in fp64 and rounded once.
 */

/* Chunk-wise Top-k of a flat buffer u (tensor j at ts[j].offset): for every chunk the selected
 * element positions (inside the flat buffer) and values, appended to pos / val; returns the count. */
static int64_t topk_of_flat(const orc_config* cfg, const orc_tensor* ts, int32_t nt, const float* u,
                            int64_t* pos, float* val) {
    const int32_t k = cfg->k, C = cfg->chunk_elems;
    int64_t w = 0;
    float* cu = (float*)malloc(sizeof(float) * (size_t)C);
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)(k > 0 ? k : 1));
    for (int32_t j = 0; j < nt; ++j) {
        const orc_tensor* t = &ts[j];
        const int64_t nc = orc_num_chunks(cfg, t);
        for (int64_t ch = 0; ch < nc; ++ch) {
            const int32_t L = (int32_t)orc_chunk_len(cfg, t, ch);
            for (int32_t p = 0; p < L; ++p) cu[p] = u[t->offset + orc_chunk_pos(cfg, t, ch, p)];
            const int32_t m = orc_topk_chunk(cu, L, k, idx);
            for (int32_t s = 0; s < m; ++s, ++w) {
                pos[w] = t->offset + orc_chunk_pos(cfg, t, ch, idx[s]);
                val[w] = cu[idx[s]];
            }
        }
    }
    free(cu);
    free(idx);
    return w;
}

/* Alg. 2: DiLoCo-LOM, and DiLoCo-LOM-Sub-k when sub_k != 0.  theta and the local momenta m_r (fp32)
 * are updated in place; alpha = cfg->outer_lr, k = cfg->k. */
void orc_lom_step(const orc_config* cfg, const orc_tensor* ts, int32_t nt, float mu, int32_t sub_k,
                  float* theta, const float* const* theta_r, float* const* m_r) {
    const int32_t R = cfg->R;
    for (int32_t j = 0; j < nt; ++j) {
        const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
        for (int64_t i = o; i < o + n; ++i) {
            double acc = 0.0;
            for (int32_t r = 0; r < R; ++r) {
                const float d = theta[i] - theta_r[r][i];
                const float m = fmaf(mu, m_r[r][i], d); /* local momentum */
                m_r[r][i] = m;
                acc += (double)fmaf(mu, m, d); /* local Nesterov direction */
            }
            theta[i] = (float)((double)theta[i] - (double)cfg->outer_lr * acc / (double)R);
        }
    }
    if (sub_k) { /* m_r <- m_r - Top-k(m_r): the selected entries become zero */
        const int64_t slots = orc_total_slots(cfg, ts, nt);
        int64_t* pos = (int64_t*)malloc(sizeof(int64_t) * (size_t)(slots ? slots : 1));
        float* val = (float*)malloc(sizeof(float) * (size_t)(slots ? slots : 1));
        for (int32_t r = 0; r < R; ++r) {
            const int64_t w = topk_of_flat(cfg, ts, nt, m_r[r], pos, val);
            for (int64_t s = 0; s < w; ++s) m_r[r][pos[s]] = m_r[r][pos[s]] - val[s];
        }
        free(pos);
        free(val);
    }
}

/* Alg. 3: DiLoCo + Top-k, with error feedback when e != NULL (decay rho = cfg->beta).  theta, the
 * global momentum m and the e_r are updated in place. */
void orc_diloco_topk_step(const orc_config* cfg, const orc_tensor* ts, int32_t nt, float mu,
                          float* theta, const float* const* theta_r, float* const* e, float* m) {
    const int32_t R = cfg->R;
    int64_t flat = 0;
    for (int32_t j = 0; j < nt; ++j) {
        const int64_t end = ts[j].offset + ts[j].rows * ts[j].cols;
        if (end > flat) flat = end;
    }
    const int64_t slots = orc_total_slots(cfg, ts, nt);
    double* acc = (double*)calloc((size_t)flat, sizeof(double));
    float* u = (float*)calloc((size_t)flat, sizeof(float));
    int64_t* pos = (int64_t*)malloc(sizeof(int64_t) * (size_t)(slots ? slots : 1));
    float* val = (float*)malloc(sizeof(float) * (size_t)(slots ? slots : 1));
    for (int32_t r = 0; r < R; ++r) {
        for (int32_t j = 0; j < nt; ++j) {
            const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
            for (int64_t i = o; i < o + n; ++i) {
                const float d = theta[i] - theta_r[r][i];
                u[i] = e ? fmaf(cfg->beta, e[r][i], d) : d;
            }
        }
        const int64_t w = topk_of_flat(cfg, ts, nt, u, pos, val);
        if (e) { /* e_r = u - Dhat */
            for (int32_t j = 0; j < nt; ++j) {
                const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
                for (int64_t i = o; i < o + n; ++i) e[r][i] = u[i];
            }
            for (int64_t s = 0; s < w; ++s) e[r][pos[s]] = u[pos[s]] - val[s];
        }
        for (int64_t s = 0; s < w; ++s) acc[pos[s]] += (double)val[s];
    }
    for (int32_t j = 0; j < nt; ++j) {
        const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
        for (int64_t i = o; i < o + n; ++i) {
            const double dbar = acc[i] / (double)R;
            const double mm = (double)mu * (double)m[i] + dbar;
            theta[i] = (float)((double)theta[i] - (double)cfg->outer_lr * (dbar + (double)mu * mm));
            m[i] = (float)mm;
        }
    }
    free(acc); free(u); free(pos); free(val);
}

/* Alg. 4: DiLoCo-LOM + Top-k, with error feedback when e != NULL.  theta, the local momenta m_r and
 * the e_r are updated in place. */
void orc_lom_topk_step(const orc_config* cfg, const orc_tensor* ts, int32_t nt, float mu,
                       float* theta, const float* const* theta_r, float* const* m_r, float* const* e) {
    const int32_t R = cfg->R;
    int64_t flat = 0;
    for (int32_t j = 0; j < nt; ++j) {
        const int64_t end = ts[j].offset + ts[j].rows * ts[j].cols;
        if (end > flat) flat = end;
    }
    const int64_t slots = orc_total_slots(cfg, ts, nt);
    double* acc = (double*)calloc((size_t)flat, sizeof(double));
    uint8_t* hit = (uint8_t*)calloc((size_t)flat, 1);
    float* u = (float*)calloc((size_t)flat, sizeof(float));
    int64_t* pos = (int64_t*)malloc(sizeof(int64_t) * (size_t)(slots ? slots : 1));
    float* val = (float*)malloc(sizeof(float) * (size_t)(slots ? slots : 1));
    for (int32_t r = 0; r < R; ++r) {
        for (int32_t j = 0; j < nt; ++j) {
            const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
            for (int64_t i = o; i < o + n; ++i) {
                const float d = theta[i] - theta_r[r][i];
                const float mm = fmaf(mu, m_r[r][i], d);
                m_r[r][i] = mm;
                const float nd = fmaf(mu, mm, d);
                u[i] = e ? fmaf(cfg->beta, e[r][i], nd) : nd;
            }
        }
        const int64_t w = topk_of_flat(cfg, ts, nt, u, pos, val);
        if (e) {
            for (int32_t j = 0; j < nt; ++j) {
                const int64_t n = ts[j].rows * ts[j].cols, o = ts[j].offset;
                for (int64_t i = o; i < o + n; ++i) e[r][i] = u[i];
            }
            for (int64_t s = 0; s < w; ++s) e[r][pos[s]] = u[pos[s]] - val[s];
        }
        for (int64_t s = 0; s < w; ++s) {
            acc[pos[s]] += (double)val[s];
            hit[pos[s]] = 1;
        }
    }
    for (int64_t i = 0; i < flat; ++i)
        if (hit[i]) theta[i] = (float)((double)theta[i] - (double)cfg->outer_lr * acc[i] / (double)R);
    free(acc); free(hit); free(u); free(pos); free(val);
}
