/*
 * CPU oracle for the MLA decode hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of what the CUDA library computes.  It shares
 * no code with the CUDA path and is only ever called from tests, from the smoke
 * check and from the benchmark's CPU-baseline leg.  Nothing here is blocked,
 * fused or reordered beyond the definition:
 *
 *   - the KV cache holds ONE latent row per token, with no head axis: all query
 *     heads read the same history (the premise of the paper's layouts, Sec. 1);
 *   - absorbed MLA: a query row and a cache row are d_q = d_c + d_r wide and the
 *     value read back per head is d_z = d_c wide (Sec. 3, "Cost" paragraph of
 *     DOP, Eq. "dop-traffic"); with the DeepSeek-V3 dimensions of App. A,
 *     d_c = 512 and d_r = 64;
 *   - decode presents one query row per request and every head attends over the
 *     request's complete history (Sec. 3 "Computation"; Sec. 4.1 "Handoff");
 *   - position-sharded CP partitions one request's token history (App. E); the
 *     partial results are combined through their log-sum-exp.
 *
 * The attention formula itself is the textbook softmax attention; the paper
 * does not print it; what the paper leaves open (row layout, LSE base, empty
 * ranges, fp8 format) is stated at each function.
 *
 * Pins (tests/test_oracle_pins.py): closed forms (n = 1, n = 2, identical
 * V rows, q = 0), invariants (key shift, permutation of tokens and of page
 * placement, head / request / KV-range concatenation), a dense library
 * attention on gathered rows, brute force in exact rational / high precision
 * arithmetic on tiny inputs, and the e4m3 code table against its definition.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* bf16 bit pattern -> double (exact: bf16 is the top half of an IEEE float). */
static double bf16_to_double(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* e4m3fn byte -> double: 1 sign, 4 exponent (bias 7), 3 mantissa bits; exponent
 * field 0 is subnormal (2^-6 * m/8); S.1111.111 is NaN; there is no infinity. */
double oracle_e4m3_to_double(uint8_t code) {
    int sign = code >> 7;
    int e = (code >> 3) & 0xF;
    int m = code & 0x7;
    double v;
    if (e == 0xF && m == 0x7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* Read element d of the cache row that holds token t of request i. */
static inline double kv_elem(const void *kv_pool, int kv_dtype, const float *kv_scales,
                             int64_t page, int slot, int d, int d_qk, int page_size) {
    int64_t row = page * page_size + slot;
    if (kv_dtype == 0) {
        return bf16_to_double(((const uint16_t *)kv_pool)[row * d_qk + d]);
    }
    return oracle_e4m3_to_double(((const uint8_t *)kv_pool)[row * d_qk + d]) * (double)kv_scales[row];
}

/*
 * Decode attention for the (request, head) pairs of one shard.
 *
 *   q            [B][H][d_qk] bf16 bit patterns, strides in elements
 *   kv_pool      [P][page_size][d_qk] bf16 bits (kv_dtype 0) or e4m3 bytes (1)
 *   kv_scales    [P][page_size] float, only for kv_dtype 1
 *   block_table  [B][table_stride] int32, page ids
 *   seq_lens     [B]
 *   kv_begin/end [B] or NULL: the token range, clipped to [0, seq_len)
 *   pairs        optional [n_pairs][2] (request, head) list; NULL = every request
 *                and every head in [head_begin, head_end)
 *   out          [B][H][d_v] double, lse [B][H] double; only the computed
 *                (request, head) entries are written.
 */
int oracle_mla_decode(int B, int H, int d_qk, int d_v, int page_size,
                      const uint16_t *q, int64_t q_stride_b, int64_t q_stride_h,
                      const void *kv_pool, int kv_dtype, const float *kv_scales,
                      const int32_t *block_table, int64_t table_stride,
                      const int32_t *seq_lens,
                      int head_begin, int head_end,
                      const int32_t *kv_begin, const int32_t *kv_end,
                      double softmax_scale,
                      const int32_t *pairs, int64_t n_pairs,
                      double *out, double *lse) {
    int h = head_end - head_begin;
    int64_t total = pairs ? n_pairs : (int64_t)B * (h > 0 ? h : 0);
    if (h < 0 || head_begin < 0 || head_end > H) return -1;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t job = 0; job < total; ++job) {
        int i, g;
        if (pairs) { i = pairs[2 * job]; g = pairs[2 * job + 1]; }
        else { i = (int)(job / h); g = head_begin + (int)(job % h); }

        int s = seq_lens[i];
        int lo = kv_begin ? kv_begin[i] : 0;
        int hi = kv_end ? kv_end[i] : s;
        if (lo < 0) lo = 0;
        if (hi > s) hi = s;
        int n = hi > lo ? hi - lo : 0;

        double *o = out + ((int64_t)i * H + g) * d_v;
        double *L = lse + (int64_t)i * H + g;
        for (int d = 0; d < d_v; ++d) o[d] = 0.0;
        if (n == 0) { *L = -INFINITY; continue; }

        const uint16_t *qrow = q + i * q_stride_b + g * q_stride_h;
        double *logit = (double *)malloc(sizeof(double) * (size_t)n);

        /* logits: l_t = scale * sum_d q[d] * row_t[d] over all d_qk columns */
        double m = -INFINITY;
        for (int t = lo; t < hi; ++t) {
            int64_t page = block_table[i * table_stride + t / page_size];
            int slot = t % page_size;
            double acc = 0.0;
            for (int d = 0; d < d_qk; ++d)
                acc += bf16_to_double(qrow[d]) *
                       kv_elem(kv_pool, kv_dtype, kv_scales, page, slot, d, d_qk, page_size);
            logit[t - lo] = softmax_scale * acc;
            if (logit[t - lo] > m) m = logit[t - lo];
        }
        /* softmax weights, normaliser, log-sum-exp (natural log) */
        double Z = 0.0;
        for (int t = 0; t < n; ++t) Z += exp(logit[t] - m);
        *L = m + log(Z);
        /* O = sum_t w_t * V_t, V_t = the first d_v columns of the same row */
        for (int t = lo; t < hi; ++t) {
            int64_t page = block_table[i * table_stride + t / page_size];
            int slot = t % page_size;
            double w = exp(logit[t - lo] - m) / Z;
            for (int d = 0; d < d_v; ++d)
                o[d] += w * kv_elem(kv_pool, kv_dtype, kv_scales, page, slot, d, d_qk, page_size);
        }
        free(logit);
    }
    return 0;
}

/*
 * Sparse decode in the cache format of the paper's runs.
 *
 * The serving stack of the evaluation runs a SPARSE absorbed-MLA backend (Sec. 5,
 * "Setup"): for every decode query an indexer has picked the tokens of the request's
 * history that the query attends over, and attention is the same softmax attention as
 * oracle_mla_decode restricted to that token list.  The cache row of that stack holds an
 * FP8 latent with its scales and a BF16 rope part (App. B, the per-token KV payload;
 * Sec. 5 "FP8 E4M3 KV").  The paper gives the contents, not the offsets; the byte layout
 * read here is, per token, 656 bytes:
 *     [0, 512)    e4m3 codes c_d of the latent, d = 0..511
 *     [512, 528)  four float scales s_b, one per block of 128 latent dims
 *     [528, 656)  64 bf16 rope values r_j
 * so that the row's 576 key columns are  k_d = c_d * s_{d / 128}  (d < 512),  k_{512+j} = r_j,
 * and the value read back is the latent, v_d = k_d (d < 512).
 *
 *   q           [B][H][576] bf16 bits, strides in elements
 *   kv_pool     [P][page_size][656] bytes
 *   sel         [B][sel_stride] int32: token positions within the request, in any order;
 *               request i uses its first sel_count[i] entries.  An entry outside
 *               [0, seq_lens[i]) is an argument error (returns -2, nothing defined).
 *   out         [B][H][512] double, lse [B][H] double, written for heads [head_begin, head_end)
 *
 * A request with sel_count = 0 gives out = 0, lse = -inf.  A token listed twice counts twice.
 */
enum { SPARSE_ROW_BYTES = 656, SPARSE_D_LATENT = 512, SPARSE_D_ROPE = 64, SPARSE_BLOCK = 128 };

static double sparse_row_elem(const uint8_t *row, int d) {
    if (d < SPARSE_D_LATENT) {
        float s;
        memcpy(&s, row + SPARSE_D_LATENT + 4 * (d / SPARSE_BLOCK), sizeof s);
        return oracle_e4m3_to_double(row[d]) * (double)s;
    }
    uint16_t bits;
    memcpy(&bits, row + SPARSE_D_LATENT + 16 + 2 * (d - SPARSE_D_LATENT), sizeof bits);
    return bf16_to_double(bits);
}

int oracle_mla_decode_sparse(int B, int H, int page_size,
                             const uint16_t *q, int64_t q_stride_b, int64_t q_stride_h,
                             const uint8_t *kv_pool,
                             const int32_t *block_table, int64_t table_stride,
                             const int32_t *seq_lens,
                             const int32_t *sel, int64_t sel_stride, const int32_t *sel_count,
                             int head_begin, int head_end, double softmax_scale,
                             double *out, double *lse) {
    const int d_qk = SPARSE_D_LATENT + SPARSE_D_ROPE, d_v = SPARSE_D_LATENT;
    int h = head_end - head_begin;
    if (h < 0 || head_begin < 0 || head_end > H) return -1;
    for (int i = 0; i < B; ++i)
        for (int j = 0; j < sel_count[i]; ++j) {
            int t = sel[i * sel_stride + j];
            if (t < 0 || t >= seq_lens[i]) return -2;
        }
    int64_t total = (int64_t)B * h;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t job = 0; job < total; ++job) {
        int i = (int)(job / h), g = head_begin + (int)(job % h);
        int n = sel_count[i];
        double *o = out + ((int64_t)i * H + g) * d_v;
        double *L = lse + (int64_t)i * H + g;
        for (int d = 0; d < d_v; ++d) o[d] = 0.0;
        if (n <= 0) { *L = -INFINITY; continue; }
        const uint16_t *qrow = q + i * q_stride_b + g * q_stride_h;
        double *logit = (double *)malloc(sizeof(double) * (size_t)n);
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) {
            int t = sel[i * sel_stride + j];
            int64_t page = block_table[i * table_stride + t / page_size];
            const uint8_t *row = kv_pool + (page * page_size + t % page_size) * SPARSE_ROW_BYTES;
            double acc = 0.0;
            for (int d = 0; d < d_qk; ++d) acc += bf16_to_double(qrow[d]) * sparse_row_elem(row, d);
            logit[j] = softmax_scale * acc;
            if (logit[j] > m) m = logit[j];
        }
        double Z = 0.0;
        for (int j = 0; j < n; ++j) Z += exp(logit[j] - m);
        *L = m + log(Z);
        for (int j = 0; j < n; ++j) {
            int t = sel[i * sel_stride + j];
            int64_t page = block_table[i * table_stride + t / page_size];
            const uint8_t *row = kv_pool + (page * page_size + t % page_size) * SPARSE_ROW_BYTES;
            double w = exp(logit[j] - m) / Z;
            for (int d = 0; d < d_v; ++d) o[d] += w * sparse_row_elem(row, d);
        }
        free(logit);
    }
    return 0;
}

/*
 * Attention for R query rows per request (a short prefill chunk or a multi-token
 * decode step: the batch entry of a request carries q_i > 1 rows, Sec. 4.1).  The R
 * rows are the request's R newest tokens, already in the cache; row r sits at position
 * seq_len - R + r and attends causally, i.e. over the tokens
 *     [max(0, kv_begin), min(kv_end, seq_len - (R - 1 - r))),
 * with the same formula as oracle_mla_decode for each row on its own:
 *     l_t = scale * q_r . row_t,  lse = ln sum_t exp(l_t),  out = sum_t exp(l_t - lse) row_t[0..d_v).
 * A row whose range is empty gives out = 0, lse = -inf.
 *
 *   q    [B][H][R][d_qk] bf16 bits: element (i, g, r, d) at i*q_stride_b + g*q_stride_h + r*d_qk + d
 *   out  [B][H][R][d_v] double, lse [B][H][R] double (dense)
 */
int oracle_mla_decode_rows(int B, int H, int R, int d_qk, int d_v, int page_size,
                           const uint16_t *q, int64_t q_stride_b, int64_t q_stride_h,
                           const void *kv_pool, int kv_dtype, const float *kv_scales,
                           const int32_t *block_table, int64_t table_stride,
                           const int32_t *seq_lens,
                           int head_begin, int head_end,
                           const int32_t *kv_begin, const int32_t *kv_end,
                           double softmax_scale,
                           double *out, double *lse) {
    int h = head_end - head_begin;
    if (h < 0 || head_begin < 0 || head_end > H || R < 1) return -1;
    int64_t total = (int64_t)B * h * R;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t job = 0; job < total; ++job) {
        int r = (int)(job % R);
        int g = head_begin + (int)((job / R) % h);
        int i = (int)(job / ((int64_t)R * h));

        int s = seq_lens[i];
        int lo = kv_begin ? kv_begin[i] : 0;
        int hi = kv_end ? kv_end[i] : s;
        int causal_end = s - (R - 1 - r);          /* one past the row's own position */
        if (lo < 0) lo = 0;
        if (hi > causal_end) hi = causal_end;
        int n = hi > lo ? hi - lo : 0;

        double *o = out + (((int64_t)i * H + g) * R + r) * d_v;
        double *L = lse + ((int64_t)i * H + g) * R + r;
        for (int d = 0; d < d_v; ++d) o[d] = 0.0;
        if (n == 0) { *L = -INFINITY; continue; }

        const uint16_t *qrow = q + i * q_stride_b + g * q_stride_h + (int64_t)r * d_qk;
        double *logit = (double *)malloc(sizeof(double) * (size_t)n);
        double m = -INFINITY;
        for (int t = lo; t < hi; ++t) {
            int64_t page = block_table[i * table_stride + t / page_size];
            int slot = t % page_size;
            double acc = 0.0;
            for (int d = 0; d < d_qk; ++d)
                acc += bf16_to_double(qrow[d]) *
                       kv_elem(kv_pool, kv_dtype, kv_scales, page, slot, d, d_qk, page_size);
            logit[t - lo] = softmax_scale * acc;
            if (logit[t - lo] > m) m = logit[t - lo];
        }
        double Z = 0.0;
        for (int t = 0; t < n; ++t) Z += exp(logit[t] - m);
        *L = m + log(Z);
        for (int t = lo; t < hi; ++t) {
            int64_t page = block_table[i * table_stride + t / page_size];
            int slot = t % page_size;
            double w = exp(logit[t - lo] - m) / Z;
            for (int d = 0; d < d_v; ++d)
                o[d] += w * kv_elem(kv_pool, kv_dtype, kv_scales, page, slot, d, d_qk, page_size);
        }
        free(logit);
    }
    return 0;
}

/*
 * Merge of partial attention results over disjoint KV ranges:
 *   L = ln sum_j exp(L_j),  O = sum_j exp(L_j - L) * O_j.
 * Parts with L_j = -inf contribute nothing; if every part is -inf, O = 0 and
 * L = -inf.  part_out [parts][rows][d_v], part_lse [parts][rows].
 */
int oracle_lse_merge(int parts, int64_t rows, int d_v,
                     const double *part_out, const double *part_lse,
                     double *out, double *lse) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double m = -INFINITY;
        for (int j = 0; j < parts; ++j)
            if (part_lse[j * rows + r] > m) m = part_lse[j * rows + r];
        double *o = out + r * d_v;
        for (int d = 0; d < d_v; ++d) o[d] = 0.0;
        if (m == -INFINITY) { lse[r] = -INFINITY; continue; }
        double Z = 0.0;
        for (int j = 0; j < parts; ++j)
            if (part_lse[j * rows + r] != -INFINITY) Z += exp(part_lse[j * rows + r] - m);
        double L = m + log(Z);
        lse[r] = L;
        for (int j = 0; j < parts; ++j) {
            double Lj = part_lse[j * rows + r];
            if (Lj == -INFINITY) continue;
            double w = exp(Lj - L);
            const double *pj = part_out + (j * rows + r) * d_v;
            for (int d = 0; d < d_v; ++d) o[d] += w * pj[d];
        }
    }
    return 0;
}

/*
 * Page migration: copy n listed pages (and their scale pages) from one pool to
 * another and rewrite every block-table entry that names a moved page.  Page
 * ids in the table are arena-global: a source page j has id src_id_base +
 * src_page_ids[j], its destination dst_id_base + dst_page_ids[j].  Every other
 * byte of both pools and every other table entry is left as it was.
 */
int oracle_kv_page_migrate(const uint8_t *src_pool, const float *src_scales,
                           uint8_t *dst_pool, float *dst_scales,
                           int64_t page_bytes, int page_size,
                           const int32_t *src_page_ids, const int32_t *dst_page_ids, int64_t n,
                           int32_t src_id_base, int32_t dst_id_base,
                           int32_t *block_table, int64_t num_table_entries) {
    for (int64_t j = 0; j < n; ++j) {
        memcpy(dst_pool + (int64_t)dst_page_ids[j] * page_bytes,
               src_pool + (int64_t)src_page_ids[j] * page_bytes, (size_t)page_bytes);
        if (src_scales && dst_scales)
            memcpy(dst_scales + (int64_t)dst_page_ids[j] * page_size,
                   src_scales + (int64_t)src_page_ids[j] * page_size,
                   sizeof(float) * (size_t)page_size);
    }
    for (int64_t e = 0; e < num_table_entries; ++e) {
        int32_t id = block_table[e];
        if (id < 0) continue;
        for (int64_t j = 0; j < n; ++j) {
            if (id == src_id_base + src_page_ids[j]) {
                block_table[e] = dst_id_base + dst_page_ids[j];
                break;
            }
        }
    }
    return 0;
}
