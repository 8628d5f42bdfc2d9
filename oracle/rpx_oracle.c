/*
 * fp64 CPU oracle for prefix+suffix scoring.  TEST INFRASTRUCTURE ONLY: it is called by the
 * tests, the smoke check and the benchmark's CPU-baseline leg, never by the product path, and
 * it shares no code with the CUDA library.
 *
 * The paper states (Section 2.3, "Observation and Opportunity"; Section 3.1, Phases 1 and 2;
 * Section 4.3) that splitting a model invocation at the first response position changes only
 * WHEN work runs: the retained prefix KV is exactly the state a serial pass would recompute and
 * prefix plus suffix log-probabilities are the full-sequence values.  The split is therefore a
 * re-ordering, not an approximation, so the oracle is the plain monolithic definition:
 *
 *   attention   for position i of one whole sequence (prompt and response concatenated) and
 *               query head h with KV head g = h / (H_q / H_kv):
 *                   s_j = scale * sum_c q[i,h,c] * k[j,g,c]            j = 0..i
 *                   m   = max_j s_j ;  p_j = exp(s_j - m) ;  l = sum_j p_j
 *                   O[i,h,:] = sum_j p_j * v[j,g,:] / l ;  LSE[i,h] = m + ln l
 *   log-prob    for row n:  z_v = sum_c hidden[n,c] * W[v,c]           v = 0..V-1
 *                   logprob[n] = z_target - (max_v z_v + ln sum_v exp(z_v - max_v z_v))
 *   slot map    slot(s,t) = block_table[s][t / block_size] * block_size + t % block_size
 *   entropy     (extension) H[n] = - sum_v p_v ln p_v with p = softmax(z[n,:])
 *
 * Every input element is promoted to double first; sums run in index order with no blocking.
 * Pins (tests/test_oracle_pins.py): brute force on tiny inputs in extended precision with a
 * structurally different evaluation, closed forms (Q = 0, row 0, W = 0, V = ones / one-hot),
 * the GQA -> replicated-MHA reduction, torch's fp64 CPU attention and log_softmax, and the
 * split == monolithic invariant.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1 };

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static inline double load_elem(const void* base, int dtype, int64_t idx) {
    if (dtype == ORACLE_BF16) return bf16_to_f64(((const uint16_t*)base)[idx]);
    return (double)((const float*)base)[idx];
}

/* float -> bf16 bits, round to nearest, ties to even (NaN kept quiet). */
static inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

int rpx_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Monolithic causal GQA attention for a list of rows.
 *   q [tokens][H_q][d], k/v [tokens][H_kv][d] with token strides in elements; sequences packed
 *   back to back, sequence s owning tokens cu_seqlens[s] .. cu_seqlens[s+1]-1.
 *   rows: n_rows triples (s, i, h): sequence, position inside it, query head.
 *   out [n_rows][d] and lse [n_rows] in double.
 * Returns 0, or -1 on an out-of-range row.
 */
int rpx_oracle_attn_rows(const void* q, const void* k, const void* v, int dtype,
                         int64_t q_tok_stride, int64_t k_tok_stride, int64_t v_tok_stride,
                         const int32_t* cu_seqlens, int32_t batch,
                         int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, double scale,
                         const int32_t* rows, int64_t n_rows, double* out, double* lse) {
    if (num_kv_heads <= 0 || num_q_heads % num_kv_heads != 0) return -1;
    const int group = num_q_heads / num_kv_heads;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int s = rows[3 * r + 0], i = rows[3 * r + 1], h = rows[3 * r + 2];
        if (s < 0 || s >= batch || h < 0 || h >= num_q_heads || i < 0 ||
            i >= cu_seqlens[s + 1] - cu_seqlens[s]) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        const int g = h / group;
        const int64_t tok0 = cu_seqlens[s];
        const int64_t qoff = (tok0 + i) * q_tok_stride + (int64_t)h * head_dim;
        double* sc = (double*)malloc(sizeof(double) * (size_t)(i + 1));
        double m = -INFINITY;
        for (int j = 0; j <= i; ++j) {
            const int64_t koff = (tok0 + j) * k_tok_stride + (int64_t)g * head_dim;
            double dot = 0.0;
            for (int c = 0; c < head_dim; ++c)
                dot += load_elem(q, dtype, qoff + c) * load_elem(k, dtype, koff + c);
            sc[j] = dot * scale;
            if (sc[j] > m) m = sc[j];
        }
        double l = 0.0;
        for (int j = 0; j <= i; ++j) {
            sc[j] = exp(sc[j] - m);
            l += sc[j];
        }
        double* o = out + r * head_dim;
        for (int c = 0; c < head_dim; ++c) o[c] = 0.0;
        for (int j = 0; j <= i; ++j) {
            const int64_t voff = (tok0 + j) * v_tok_stride + (int64_t)g * head_dim;
            for (int c = 0; c < head_dim; ++c) o[c] += sc[j] * load_elem(v, dtype, voff + c);
        }
        for (int c = 0; c < head_dim; ++c) o[c] /= l;
        if (lse) lse[r] = m + log(l);
        free(sc);
    }
    return bad ? -1 : 0;
}

/*
 * Monolithic log-softmax + gather for a list of rows.
 *   hidden [n][hidden_dim] (row stride in elements), w [vocab][hidden_dim] row-major,
 *   target_ids [n] indexed by the row number, rows: n_rows row numbers.
 *   logprob [n_rows], lse [n_rows] (nullable) in double.
 * A target outside [0, vocab) gives NaN for that row.
 */
int rpx_oracle_logprob_rows(const void* hidden, int64_t hidden_row_stride, const void* w, int dtype,
                            const int32_t* target_ids, const int64_t* rows, int64_t n_rows,
                            int32_t hidden_dim, int32_t vocab, double* logprob, double* lse) {
    double* z = (double*)malloc(sizeof(double) * (size_t)n_rows * (size_t)vocab);
    if (!z) return -2;
#pragma omp parallel for schedule(static)
    for (int32_t vv = 0; vv < vocab; ++vv) {
        const int64_t woff = (int64_t)vv * hidden_dim;
        for (int64_t r = 0; r < n_rows; ++r) {
            const int64_t hoff = rows[r] * hidden_row_stride;
            double dot = 0.0;
            for (int c = 0; c < hidden_dim; ++c)
                dot += load_elem(hidden, dtype, hoff + c) * load_elem(w, dtype, woff + c);
            z[r * (int64_t)vocab + vv] = dot;
        }
    }
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_rows; ++r) {
        const double* zr = z + r * (int64_t)vocab;
        double m = -INFINITY;
        for (int32_t vv = 0; vv < vocab; ++vv)
            if (zr[vv] > m) m = zr[vv];
        double l = 0.0;
        for (int32_t vv = 0; vv < vocab; ++vv) l += exp(zr[vv] - m);
        const double ls = m + log(l);
        const int32_t t = target_ids[rows[r]];
        logprob[r] = (t >= 0 && t < vocab) ? zr[t] - ls : NAN;
        if (lse) lse[r] = ls;
    }
    free(z);
    return 0;
}

/*
 * Entropy of the next-token distribution for a list of rows (an extension beyond the paper, which
 * only needs log-probs): with p_v = exp(z_v - lse),  H[n] = - sum_v p_v * ln p_v, written out as
 * that definition in double (terms with p_v == 0 contribute 0).
 */
int rpx_oracle_entropy_rows(const void* hidden, int64_t hidden_row_stride, const void* w, int dtype,
                            const int64_t* rows, int64_t n_rows, int32_t hidden_dim, int32_t vocab,
                            double* entropy) {
    double* z = (double*)malloc(sizeof(double) * (size_t)n_rows * (size_t)vocab);
    if (!z) return -2;
#pragma omp parallel for schedule(static)
    for (int32_t vv = 0; vv < vocab; ++vv) {
        const int64_t woff = (int64_t)vv * hidden_dim;
        for (int64_t r = 0; r < n_rows; ++r) {
            const int64_t hoff = rows[r] * hidden_row_stride;
            double dot = 0.0;
            for (int c = 0; c < hidden_dim; ++c)
                dot += load_elem(hidden, dtype, hoff + c) * load_elem(w, dtype, woff + c);
            z[r * (int64_t)vocab + vv] = dot;
        }
    }
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_rows; ++r) {
        const double* zr = z + r * (int64_t)vocab;
        double m = -INFINITY;
        for (int32_t vv = 0; vv < vocab; ++vv)
            if (zr[vv] > m) m = zr[vv];
        double l = 0.0;
        for (int32_t vv = 0; vv < vocab; ++vv) l += exp(zr[vv] - m);
        const double ls = m + log(l);
        double h = 0.0;
        for (int32_t vv = 0; vv < vocab; ++vv) {
            const double lp = zr[vv] - ls;
            const double pv = exp(lp);
            if (pv > 0.0) h -= pv * lp;
        }
        entropy[r] = h;
    }
    free(z);
    return 0;
}

/* slot(s,t) = block_table[s][t / block_size] * block_size + t % block_size */
int64_t rpx_oracle_slot(const int32_t* block_table, int32_t block_table_stride, int32_t s, int32_t t,
                        int32_t block_size) {
    return (int64_t)block_table[(int64_t)s * block_table_stride + t / block_size] * block_size +
           t % block_size;
}

/*
 * Expected boundary-KV cache image.  The caller pre-fills k_cache / v_cache (bf16 bits,
 * [num_blocks][H_kv][block_size][d]) with its sentinel; this writes
 *   cache[slot / block_size][g][slot % block_size][:] = bf16(K[cu_seqlens[s] + t, g, :])
 * for every prefix position t < cu_seqlens[s+1] - cu_seqlens[s] and leaves the rest alone.
 * fp32 inputs are rounded to nearest-even; bf16 inputs are copied bit for bit.
 */
int rpx_oracle_cache_image(const void* k, const void* v, int dtype, int64_t k_tok_stride,
                           int64_t v_tok_stride, const int32_t* cu_seqlens, int32_t batch,
                           int32_t num_kv_heads, int32_t head_dim, const int32_t* block_table,
                           int32_t block_table_stride, int32_t block_size, int64_t num_blocks,
                           uint16_t* k_cache, uint16_t* v_cache) {
    for (int32_t s = 0; s < batch; ++s) {
        const int32_t len = cu_seqlens[s + 1] - cu_seqlens[s];
        for (int32_t t = 0; t < len; ++t) {
            const int64_t slot = rpx_oracle_slot(block_table, block_table_stride, s, t, block_size);
            const int64_t blk = slot / block_size, off = slot % block_size;
            if (blk < 0 || blk >= num_blocks) return -1;
            const int64_t tok = (int64_t)cu_seqlens[s] + t;
            for (int32_t g = 0; g < num_kv_heads; ++g) {
                const int64_t dst = ((blk * num_kv_heads + g) * block_size + off) * head_dim;
                for (int32_t c = 0; c < head_dim; ++c) {
                    const int64_t ks = tok * k_tok_stride + (int64_t)g * head_dim + c;
                    const int64_t vs = tok * v_tok_stride + (int64_t)g * head_dim + c;
                    if (dtype == ORACLE_BF16) {
                        k_cache[dst + c] = ((const uint16_t*)k)[ks];
                        v_cache[dst + c] = ((const uint16_t*)v)[vs];
                    } else {
                        k_cache[dst + c] = f32_to_bf16_rne(((const float*)k)[ks]);
                        v_cache[dst + c] = f32_to_bf16_rne(((const float*)v)[vs]);
                    }
                }
            }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Backward through the boundary (Section 3.2, the autograd contract of the training actor's prefix; Table 4,
 * row on the boundary prefix KV of the training actor, which stays attached to the graph): gradients of the
 * suffix flow into the prefix through the retained K and V.  As in the forward direction the split is a
 * re-ordering, so the oracle is the gradient of the monolithic definitions above, written out term by term.
 *
 *   LM head     with p_v = exp(z_v - lse) and an upstream gradient g[n] = dL / d logprob[n]:
 *                   dL/dz_v      = g[n] * ([v == target] - p_v)
 *                   dhidden[n,:] = sum_v dL/dz_v * W[v,:]
 *                   dW[v,:]      = sum_n dL/dz_v(n) * hidden[n,:]
 *   attention   with P_ij the softmax weights of row (i,h) over keys j <= i, g = h / (H_q / H_kv), and an
 *               upstream gradient dO[i,h,:]:
 *                   dP_ij = sum_c dO[i,h,c] * V[j,g,c]
 *                   D_i   = sum_j P_ij * dP_ij
 *                   dS_ij = P_ij * (dP_ij - D_i)
 *                   dQ[i,h,:] = scale * sum_j dS_ij * K[j,g,:]
 *                   dK[j,g,:] = scale * sum_{h in g} sum_{i >= j} dS_ij * Q[i,h,:]
 *                   dV[j,g,:] =         sum_{h in g} sum_{i >= j} P_ij  * dO[i,h,:]
 *               A key j of the prompt receives contributions from prompt queries and from response queries
 *               alike: that sum over both is what "gradients flow from the suffix into the prefix" means.
 * Pins (tests/test_oracle_backward_pins.py): central finite differences of the forward routines above,
 * torch's fp64 autograd on CPU, closed forms (a one-key sequence, W = 0, uniform scores), the identity
 * sum_v dL/dz_v = 0, and a split evaluation (prefix queries and suffix queries accumulated separately) against
 * the monolithic sums.
 */

/*
 * LM-head backward for all n rows.
 *   upstream [n] (double), target_ids [n]; dhidden [n][hidden_dim] and dw [vocab][hidden_dim] (nullable) in double.
 * A target outside [0, vocab) has no one-hot term (its log-prob is NaN in the forward pass); callers keep such rows
 * out of the comparison.
 */
int rpx_oracle_logprob_backward(const void* hidden, int64_t hidden_row_stride, const void* w, int dtype,
                                const int32_t* target_ids, const double* upstream, int64_t n, int32_t hidden_dim,
                                int32_t vocab, double* dhidden, double* dw) {
    double* dz = (double*)malloc(sizeof(double) * (size_t)n * (size_t)vocab);
    if (!dz) return -2;
    /* logits */
#pragma omp parallel for schedule(static)
    for (int32_t vv = 0; vv < vocab; ++vv) {
        const int64_t woff = (int64_t)vv * hidden_dim;
        for (int64_t r = 0; r < n; ++r) {
            const int64_t hoff = r * hidden_row_stride;
            double dot = 0.0;
            for (int c = 0; c < hidden_dim; ++c)
                dot += load_elem(hidden, dtype, hoff + c) * load_elem(w, dtype, woff + c);
            dz[r * (int64_t)vocab + vv] = dot;
        }
    }
    /* dL/dz = g * (onehot - softmax) */
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n; ++r) {
        double* zr = dz + r * (int64_t)vocab;
        double m = -INFINITY;
        for (int32_t vv = 0; vv < vocab; ++vv)
            if (zr[vv] > m) m = zr[vv];
        double l = 0.0;
        for (int32_t vv = 0; vv < vocab; ++vv) l += exp(zr[vv] - m);
        const int32_t t = target_ids[r];
        for (int32_t vv = 0; vv < vocab; ++vv) {
            const double pv = exp(zr[vv] - m) / l;
            zr[vv] = upstream[r] * ((vv == t ? 1.0 : 0.0) - pv);
        }
    }
    /* dhidden = dz . W */
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n; ++r) {
        double* dh = dhidden + r * (int64_t)hidden_dim;
        for (int c = 0; c < hidden_dim; ++c) dh[c] = 0.0;
        for (int32_t vv = 0; vv < vocab; ++vv) {
            const double d = dz[r * (int64_t)vocab + vv];
            const int64_t woff = (int64_t)vv * hidden_dim;
            for (int c = 0; c < hidden_dim; ++c) dh[c] += d * load_elem(w, dtype, woff + c);
        }
    }
    /* dW = dz^T . hidden */
    if (dw) {
#pragma omp parallel for schedule(static)
        for (int32_t vv = 0; vv < vocab; ++vv) {
            double* dwr = dw + (int64_t)vv * hidden_dim;
            for (int c = 0; c < hidden_dim; ++c) dwr[c] = 0.0;
            for (int64_t r = 0; r < n; ++r) {
                const double d = dz[r * (int64_t)vocab + vv];
                const int64_t hoff = r * hidden_row_stride;
                for (int c = 0; c < hidden_dim; ++c) dwr[c] += d * load_elem(hidden, dtype, hoff + c);
            }
        }
    }
    free(dz);
    return 0;
}

/*
 * Monolithic causal GQA attention backward for whole sequences.
 *   q, dout [tokens][H_q][d]; k, v [tokens][H_kv][d] (token strides in elements; dout is double, contiguous
 *   [tokens][H_q][d]); dq [tokens][H_q][d], dk, dv [tokens][H_kv][d] in double, contiguous, written in full.
 * Loops are over (sequence, head, query row), each row adding its terms into dk and dv of the keys it sees;
 * rows of one KV head are taken by one thread, so no two threads add into the same element.
 */
int rpx_oracle_attn_backward(const void* q, const void* k, const void* v, int dtype, int64_t q_tok_stride,
                             int64_t k_tok_stride, int64_t v_tok_stride, const int32_t* cu_seqlens, int32_t batch,
                             int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, double scale,
                             const double* dout, double* dq, double* dk, double* dv) {
    if (num_kv_heads <= 0 || num_q_heads % num_kv_heads != 0) return -1;
    const int group = num_q_heads / num_kv_heads;
    const int64_t total = cu_seqlens[batch];
    for (int64_t i = 0; i < total * num_q_heads * head_dim; ++i) dq[i] = 0.0;
    for (int64_t i = 0; i < total * num_kv_heads * head_dim; ++i) dk[i] = dv[i] = 0.0;
    int failed = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t s = 0; s < batch; ++s) {
        for (int32_t g = 0; g < num_kv_heads; ++g) {
            const int64_t tok0 = cu_seqlens[s];
            const int32_t len = cu_seqlens[s + 1] - cu_seqlens[s];
            double* p = (double*)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
            double* dp = (double*)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
            if (!p || !dp) {
#pragma omp atomic write
                failed = 1;
                free(p);
                free(dp);
                continue;
            }
            for (int32_t h = g * group; h < (g + 1) * group; ++h) {
                for (int32_t i = 0; i < len; ++i) {
                    const int64_t qoff = (tok0 + i) * q_tok_stride + (int64_t)h * head_dim;
                    const double* dor = dout + ((tok0 + i) * num_q_heads + h) * head_dim;
                    /* forward: P_ij */
                    double m = -INFINITY;
                    for (int32_t j = 0; j <= i; ++j) {
                        const int64_t koff = (tok0 + j) * k_tok_stride + (int64_t)g * head_dim;
                        double dot = 0.0;
                        for (int c = 0; c < head_dim; ++c)
                            dot += load_elem(q, dtype, qoff + c) * load_elem(k, dtype, koff + c);
                        p[j] = dot * scale;
                        if (p[j] > m) m = p[j];
                    }
                    double l = 0.0;
                    for (int32_t j = 0; j <= i; ++j) {
                        p[j] = exp(p[j] - m);
                        l += p[j];
                    }
                    for (int32_t j = 0; j <= i; ++j) p[j] /= l;
                    /* dP_ij and D_i */
                    double big_d = 0.0;
                    for (int32_t j = 0; j <= i; ++j) {
                        const int64_t voff = (tok0 + j) * v_tok_stride + (int64_t)g * head_dim;
                        double dot = 0.0;
                        for (int c = 0; c < head_dim; ++c) dot += dor[c] * load_elem(v, dtype, voff + c);
                        dp[j] = dot;
                        big_d += p[j] * dot;
                    }
                    /* dS_ij, and the three gradients */
                    double* dqr = dq + ((tok0 + i) * num_q_heads + h) * head_dim;
                    for (int32_t j = 0; j <= i; ++j) {
                        const double ds = p[j] * (dp[j] - big_d);
                        const int64_t koff = (tok0 + j) * k_tok_stride + (int64_t)g * head_dim;
                        double* dkr = dk + ((tok0 + j) * num_kv_heads + g) * head_dim;
                        double* dvr = dv + ((tok0 + j) * num_kv_heads + g) * head_dim;
                        for (int c = 0; c < head_dim; ++c) {
                            dqr[c] += scale * ds * load_elem(k, dtype, koff + c);
                            dkr[c] += scale * ds * load_elem(q, dtype, qoff + c);
                            dvr[c] += p[j] * dor[c];
                        }
                    }
                }
            }
            free(p);
            free(dp);
        }
    }
    return failed ? -2 : 0;
}
