/*
 * TEST INFRASTRUCTURE -- the CPU oracle of the hooked paged-attention path.
 *
 * A plain, slow, fp64 evaluation of what the hooked attention forward returns, written
 * out from the definition: the analyzer of the paper's Section 2.2 recomputes the
 * selected heads' attention weights from queries and keys and aggregates them over
 * token ranges; the active mode of Section 2 / Section 3 (activation steering) adds a
 * steering vector to an internal activation.  Here both are evaluated for every
 * requested query row in the most direct way:
 *
 *   1. scores      x_t = scale * sum_d q[d] * K[t][d]          for every visible key t <= pos
 *   2. softmax     p_t = exp(x_t - max_t x) / sum_t exp(x_t - max_t x)   (two passes over a
 *                  materialised row -- no online softmax, no tiling, no key chunks)
 *   3. output      o[d] = sum_t p_t * V[t][d]  (+ alpha[h] * steer_vec[h][d] if alpha[h] != 0)
 *   4. span mass   mass_j = sum of p_t over keys t in [a_j, b_j) that are visible
 *
 * Nothing here is shared with the CUDA library: own bf16 widening, own page arithmetic,
 * own loops.  Only tests, the smoke check and the CPU-baseline leg of the bench may use
 * this file; the product path never calls it.
 *
 * Readings taken where the paper is silent: causal alignment is bottom-right (query row
 * i of a sequence with n rows and L visible keys sits at position L - n + i and sees keys
 * 0..pos); spans are absolute key positions, half-open, clipped to the visible range;
 * head indices are query-head indices and query head h reads KV head h / (Hq / Hkv);
 * steering is added per head after the softmax normalisation; span masses are reported
 * for every evaluated row (callers that probe only the last row of each sequence take
 * that row).
 *
 * Pins (tests/test_oracle_pins.py): brute force with a materialised probability matrix
 * on tiny contiguous inputs, closed forms (identical keys, first row, two keys,
 * dominating key), invariants (partition of the keys sums to one, additivity, alpha = 0,
 * GQA = replicated MHA, decode = last prefill row, page permutation), and the library
 * special case (hooks off, causal scaled-dot-product attention in fp64).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double widen_bf16(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int hook_attn_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * rows: global query-row indices to evaluate (NULL = all rows 0..total_q-1, num_rows = total_q).
 * out:  fp64 [num_rows][Hq][D]
 * mass: fp64 [num_rows][P][S], P = number of nonzero head_mask entries, slot = rank of the
 *       head among the probed heads in ascending order (may be NULL when nothing is probed).
 * returns 0, or a negative code for inconsistent arguments.
 */
int hook_attn_oracle(
    int num_seqs, int total_q, int num_q_heads, int num_kv_heads, int head_dim, int page_size,
    int max_blocks_per_seq, int num_spans, double scale,
    const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
    int64_t kv_block_stride, int64_t kv_token_stride, int64_t kv_head_stride,
    const int32_t *block_table, const int32_t *seq_lens, const int32_t *cu_q_lens,
    const int32_t *spans, const float *steer_vec, const uint8_t *head_mask, const float *alpha,
    const int32_t *rows, int num_rows, double *out, double *mass)
{
    if (num_q_heads <= 0 || num_kv_heads <= 0 || num_q_heads % num_kv_heads != 0) return -1;
    if (head_dim <= 0 || page_size <= 0) return -1;
    const int group = num_q_heads / num_kv_heads;

    /* slot of each probed head in the compact span_mass layout */
    int *slot = (int *)malloc(sizeof(int) * (size_t)num_q_heads);
    int num_probed = 0;
    for (int h = 0; h < num_q_heads; ++h)
        slot[h] = (head_mask && head_mask[h]) ? num_probed++ : -1;
    if (num_probed > 0 && num_spans > 0 && (!spans || !mass)) { free(slot); return -2; }

    int max_len = 0;
    for (int s = 0; s < num_seqs; ++s) {
        int n = cu_q_lens[s + 1] - cu_q_lens[s];
        if (n < 0 || n > seq_lens[s] || seq_lens[s] < 0) { free(slot); return -3; }
        if (seq_lens[s] > max_len) max_len = seq_lens[s];
        if ((int64_t)max_blocks_per_seq * page_size < seq_lens[s]) { free(slot); return -4; }
    }
    if (cu_q_lens[num_seqs] != total_q) { free(slot); return -3; }

    const long units = (long)num_rows * num_q_heads;
    int bad = 0;

#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)(max_len > 0 ? max_len : 1));
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            const int r = (int)(u / num_q_heads);
            const int h = (int)(u % num_q_heads);
            const int row = rows ? rows[r] : r;
            if (row < 0 || row >= total_q) {
#pragma omp atomic write
                bad = 1;
                continue;
            }

            /* which sequence owns this row */
            int s = 0;
            while (s + 1 < num_seqs && cu_q_lens[s + 1] <= row) ++s;
            const int n_s = cu_q_lens[s + 1] - cu_q_lens[s];
            const int i = row - cu_q_lens[s];
            const int pos = seq_lens[s] - n_s + i; /* absolute position; sees keys 0..pos */
            const int g = h / group;
            const uint16_t *qrow = q + ((int64_t)row * num_q_heads + h) * head_dim;

            /* 1. scores over every visible key, fetched through the block table */
            double mx = -INFINITY;
            for (int t = 0; t <= pos; ++t) {
                const int64_t page = block_table[(int64_t)s * max_blocks_per_seq + t / page_size];
                const uint16_t *krow = k_cache + page * kv_block_stride
                                       + (int64_t)(t % page_size) * kv_token_stride
                                       + (int64_t)g * kv_head_stride;
                double dot = 0.0;
                for (int d = 0; d < head_dim; ++d)
                    dot += widen_bf16(qrow[d]) * widen_bf16(krow[d]);
                p[t] = scale * dot;
                if (p[t] > mx) mx = p[t];
            }
            /* 2. softmax */
            double z = 0.0;
            for (int t = 0; t <= pos; ++t) { p[t] = exp(p[t] - mx); z += p[t]; }
            for (int t = 0; t <= pos; ++t) p[t] /= z;

            /* 3. weighted sum of the values, then the steering add */
            double *o = out + ((int64_t)r * num_q_heads + h) * head_dim;
            for (int d = 0; d < head_dim; ++d) o[d] = 0.0;
            for (int t = 0; t <= pos; ++t) {
                const int64_t page = block_table[(int64_t)s * max_blocks_per_seq + t / page_size];
                const uint16_t *vrow = v_cache + page * kv_block_stride
                                       + (int64_t)(t % page_size) * kv_token_stride
                                       + (int64_t)g * kv_head_stride;
                for (int d = 0; d < head_dim; ++d) o[d] += p[t] * widen_bf16(vrow[d]);
            }
            if (alpha && steer_vec && alpha[h] != 0.0f)
                for (int d = 0; d < head_dim; ++d)
                    o[d] += (double)alpha[h] * (double)steer_vec[(int64_t)h * head_dim + d];

            /* 4. attention mass on each configured key span */
            if (slot[h] >= 0 && num_spans > 0) {
                double *m = mass + ((int64_t)r * num_probed + slot[h]) * num_spans;
                for (int j = 0; j < num_spans; ++j) {
                    int lo = spans[((int64_t)s * num_spans + j) * 2 + 0];
                    int hi = spans[((int64_t)s * num_spans + j) * 2 + 1];
                    if (lo < 0) lo = 0;
                    if (hi > pos + 1) hi = pos + 1;
                    double acc = 0.0;
                    for (int t = lo; t < hi; ++t) acc += p[t];
                    m[j] = acc;
                }
            }
        }
        free(p);
    }
    free(slot);
    return bad ? -5 : 0;
}
