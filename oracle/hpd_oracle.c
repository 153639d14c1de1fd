/*
 * CPU oracle for the Hyper-Parallel Decoding (HPD) decode step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
 * path is checked against.  It shares no code, header, table or helper with the CUDA
 * library and must never be called from the product path; only the test-suite, the
 * smoke check and the benchmark's cpu-baseline leg execute it.
 *
 * What it computes (each function cites the passage it follows):
 *   - position IDs with K_max gaps                      Algorithm 2, Sec. 4.3.1
 *   - per-step bookkeeping tables for live branches      Sec. 4.3.2-4.3.6 (append order,
 *                                                        IDs = previous + 1, pruning, b*J*N rows)
 *   - rotary embedding at an assigned position ID        Sec. 4.3.1 ("position IDs define
 *                                                        positional embeddings"), Sec. 4.4
 *   - per-branch attention                               Eq. 5-6: a value token depends on the
 *                                                        prompt and on its own earlier tokens only
 *   - position-order attention (second mode)             Sec. 4.3.2 / Fig. 3 / Sec. 4.4: the mask the
 *                                                        paper runs, causal in position-ID order over
 *                                                        the whole stacked prompt, with K_max gaps
 *
 * Precision: inputs are fp32 values (the harness widens bf16 exactly); every product,
 * sum, exponential and trigonometric value is taken in fp64.  There is no blocking,
 * no online softmax, no fusion: the concatenated sequence of a branch is materialised
 * and ordinary causal attention is evaluated on it.
 *
 * Parity pins (tests marked "not gpu"): Algorithm 2 against the position numbers the
 * paper prints for its K_max = 7 figure; rope against closed forms and the relative-
 * position identity; attention against a full-matrix masked softmax in numpy, against
 * the library's causal SDPA, and against closed forms; the step against branch/document
 * permutation invariance; the position-order mode against ordinary causal attention on the
 * position-sorted sequence, against the fine-tuning mask of Sec. 4.4 written out in token
 * order, and against the branch-local mode for single-branch groups.  Nothing in the paper prints an attention output value, so
 * beyond those pins the numeric values themselves are parity unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------------------
 * Algorithm 2 (Appendix, "Position ID assignment"): pos_id = range(|s|); for attribute i
 * in order, the IDs of its tokens start(a_i)..end(a_i) (inclusive) are raised by the
 * running offset, which then grows by K_max.  Value token k of attribute n is later given
 * pos_id[end(a_n)] + k.
 * ---------------------------------------------------------------------------------- */
void hpdo_alg2_position_ids(int len_s, int n_attr, const int32_t* attr_start, const int32_t* attr_end,
                            int k_max, int32_t* pos_id)
{
    for (int t = 0; t < len_s; ++t) pos_id[t] = t;
    int offset = 0;
    for (int i = 0; i < n_attr; ++i) {
        for (int t = attr_start[i]; t <= attr_end[i]; ++t) pos_id[t] += offset;
        offset += k_max;
    }
}

/* Position ID of value token k (k = 1 is the first generated token) of attribute n. */
int32_t hpdo_alg2_value_position(const int32_t* pos_id, const int32_t* attr_end, int n, int k)
{
    return pos_id[attr_end[n]] + k;
}

/* ------------------------------------------------------------------------------------
 * Step bookkeeping.  Slots are all branches ever admitted, grouped by document in prompt
 * order.  The step's rows are the live slots in ascending slot id (Sec. 4.3.4: finished
 * values are pruned from the input; Sec. 4.3.6: b*J*N rows when nothing is pruned).
 *   branch_start = position ID of the branch's first token: the document prefix occupies
 *                  positions 0..L_d-1, so the branch starts at L_d; with pos_gap > 0 the
 *                  j-th branch of the document is shifted by Algorithm 2's running offset
 *                  j*pos_gap.
 *   pos_id       = branch_start + depth (Sec. 4.3.3: IDs are the previous step's plus one).
 *   suffix_off   = first row of the slot's slab in the branch cache (slot * cap);
 *   suffix_len   = depth, the number of this branch's tokens cached before the step.
 * Entries past n_active are set to -1.  Returns 0, or -1 for inconsistent arguments.
 * ---------------------------------------------------------------------------------- */
int hpdo_build_meta(int n_docs, int n_slots,
                    const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt,
                    const int32_t* slot_depth, const uint8_t* slot_alive,
                    int32_t suffix_cap, int32_t pos_gap,
                    int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                    int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                    int32_t* suffix_off, int32_t* suffix_len, int32_t* n_active)
{
    int kv = 0, sl = 0;
    for (int d = 0; d < n_docs; ++d) {
        if (doc_prefix_len[d] < 0 || doc_branch_cnt[d] < 0) return -1;
        doc_kv_start[d] = kv;   kv += doc_prefix_len[d];
        doc_slot_start[d] = sl; sl += doc_branch_cnt[d];
    }
    doc_kv_start[n_docs] = kv;
    doc_slot_start[n_docs] = sl;
    if (sl != n_slots) return -1;

    int r = 0;
    for (int d = 0; d < n_docs; ++d) {
        doc_active_start[d] = r;
        for (int j = 0; j < doc_branch_cnt[d]; ++j) {
            int s = doc_slot_start[d] + j;
            if (!slot_alive[s]) continue;
            active_slot[r]  = s;
            doc_id[r]       = d;
            branch_start[r] = doc_prefix_len[d] + j * pos_gap;
            pos_id[r]       = branch_start[r] + slot_depth[s];
            suffix_off[r]   = s * suffix_cap;
            suffix_len[r]   = slot_depth[s];
            ++r;
        }
    }
    doc_active_start[n_docs] = r;
    *n_active = r;
    for (int i = r; i < n_slots; ++i) {
        active_slot[i] = doc_id[i] = branch_start[i] = pos_id[i] = suffix_off[i] = suffix_len[i] = -1;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------
 * Rotary embedding at position `pos` for n_heads vectors of length D.  Half-split pairing:
 * element i is paired with i + D/2; inverse frequency theta^(-2i/D); the pair is rotated by
 * the angle pos * inv_freq:   out[i]       = x[i] cos - x[i+D/2] sin
 *                             out[i+D/2]   = x[i+D/2] cos + x[i] sin.
 * (The paper only says that the assigned position IDs define the positional embedding;
 * the pairing convention is the one of the decoder families it runs.)
 * ---------------------------------------------------------------------------------- */
void hpdo_rope(int n_heads, int D, double theta, int32_t pos, const float* x, double* out)
{
    int half = D / 2;
    for (int h = 0; h < n_heads; ++h) {
        const float* xv = x + (size_t)h * D;
        double* ov = out + (size_t)h * D;
        for (int i = 0; i < half; ++i) {
            double inv_freq = pow(theta, -2.0 * (double)i / (double)D);
            double ang = (double)pos * inv_freq;
            double c = cos(ang), s = sin(ang);
            double a = (double)xv[i], b = (double)xv[i + half];
            ov[i]        = a * c - b * s;
            ov[i + half] = b * c + a * s;
        }
    }
}

/* ------------------------------------------------------------------------------------
 * Ordinary causal scaled-dot-product attention, one query row.  The query sits at
 * sequence index `row` of a sequence whose keys/values are K,V[0..]; causality lets it see
 * indices 0..row (itself included).  Grouped-query attention: q head h uses kv head
 * h / (Hq/Hkv).  Softmax with the maximum subtracted; lse = max + log(sum).
 *   q [Hq, D], K,V [>= row+1, Hkv, D]  ->  o [Hq, D], lse [Hq]
 * ---------------------------------------------------------------------------------- */
void hpdo_causal_attention_row(int row, int Hq, int Hkv, int D, double scale,
                               const double* q, const double* K, const double* V,
                               double* o, double* lse, double* score_scratch /* [row+1] */)
{
    int G = Hq / Hkv;
    int n = row + 1;
    for (int h = 0; h < Hq; ++h) {
        int hk = h / G;
        const double* qv = q + (size_t)h * D;
        double mx = -INFINITY;
        for (int j = 0; j < n; ++j) {
            const double* kv = K + ((size_t)j * Hkv + hk) * D;
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += qv[d] * kv[d];
            score_scratch[j] = acc * scale;
            if (score_scratch[j] > mx) mx = score_scratch[j];
        }
        double den = 0.0;
        for (int j = 0; j < n; ++j) {
            score_scratch[j] = exp(score_scratch[j] - mx);
            den += score_scratch[j];
        }
        double* ov = o + (size_t)h * D;
        for (int d = 0; d < D; ++d) ov[d] = 0.0;
        for (int j = 0; j < n; ++j) {
            const double* vv = V + ((size_t)j * Hkv + hk) * D;
            double p = score_scratch[j] / den;
            for (int d = 0; d < D; ++d) ov[d] += p * vv[d];
        }
        if (lse) lse[h] = mx + log(den);
    }
}

/* ------------------------------------------------------------------------------------
 * One decode step for every live branch (Eq. 5-6; Sec. 4.3.3).  For row r (document d,
 * depth k, position pos_id[r]):
 *   q' = rope(q[r], pos), k' = rope(k_new[r], pos);
 *   sequence = the document's cached prefix rows, then the branch's k cached rows, then
 *              (k', v_new[r]); its length is L_d + k + 1 and the new token is its last index;
 *   o[r] = causal attention of q' at that last index.
 * Cached keys are used as stored (a KV cache holds keys already rotated).
 *   q [n_active,Hq,D], k_new,v_new [n_active,Hkv,D], prefix_k/v [sum L,Hkv,D],
 *   suffix_k/v [n_slots*cap,Hkv,D]  ->  o [n_active,Hq,D], lse [n_active,Hq],
 *   q_rot [n_active,Hq,D], k_rot [n_active,Hkv,D]   (outputs in fp32; lse/q_rot/k_rot may be NULL)
 * Returns the number of threads used, or -1 on allocation failure.
 * ---------------------------------------------------------------------------------- */
int hpdo_decode_step(int Hq, int Hkv, int D, double theta, double scale,
                     int n_active,
                     const int32_t* doc_id, const int32_t* pos_id,
                     const int32_t* suffix_off, const int32_t* suffix_len,
                     const int32_t* doc_kv_start, const int32_t* doc_prefix_len,
                     const float* q, const float* k_new, const float* v_new,
                     const float* prefix_k, const float* prefix_v,
                     const float* suffix_k, const float* suffix_v,
                     float* o, float* lse, float* q_rot, float* k_rot,
                     int n_threads)
{
    int used = 1, fail = 0;
    size_t kvw = (size_t)Hkv * D, qw = (size_t)Hq * D;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel
    {
#ifdef _OPENMP
#pragma omp single
        used = omp_get_num_threads();
#endif
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n_active; ++r) {
            int d = doc_id[r];
            int L = doc_prefix_len[d];
            int k = suffix_len[r];
            int n = L + k + 1;
            double* Kc = (double*)malloc(sizeof(double) * (size_t)n * kvw);
            double* Vc = (double*)malloc(sizeof(double) * (size_t)n * kvw);
            double* qr = (double*)malloc(sizeof(double) * qw);
            double* orow = (double*)malloc(sizeof(double) * qw);
            double* lrow = (double*)malloc(sizeof(double) * (size_t)Hq);
            double* sc = (double*)malloc(sizeof(double) * (size_t)n);
            if (!Kc || !Vc || !qr || !orow || !lrow || !sc) {
                fail = 1;
            } else {
                /* the concatenated sequence: prefix, own earlier tokens, the new token */
                const float* pk = prefix_k + (size_t)doc_kv_start[d] * kvw;
                const float* pv = prefix_v + (size_t)doc_kv_start[d] * kvw;
                for (size_t i = 0; i < (size_t)L * kvw; ++i) { Kc[i] = pk[i]; Vc[i] = pv[i]; }
                const float* sk = suffix_k + (size_t)suffix_off[r] * kvw;
                const float* sv = suffix_v + (size_t)suffix_off[r] * kvw;
                for (size_t i = 0; i < (size_t)k * kvw; ++i) {
                    Kc[(size_t)L * kvw + i] = sk[i];
                    Vc[(size_t)L * kvw + i] = sv[i];
                }
                hpdo_rope(Hkv, D, theta, pos_id[r], k_new + (size_t)r * kvw, Kc + (size_t)(L + k) * kvw);
                for (size_t i = 0; i < kvw; ++i) Vc[(size_t)(L + k) * kvw + i] = v_new[(size_t)r * kvw + i];
                hpdo_rope(Hq, D, theta, pos_id[r], q + (size_t)r * qw, qr);

                hpdo_causal_attention_row(n - 1, Hq, Hkv, D, scale, qr, Kc, Vc, orow, lrow, sc);

                for (size_t i = 0; i < qw; ++i) o[(size_t)r * qw + i] = (float)orow[i];
                if (lse) for (int h = 0; h < Hq; ++h) lse[(size_t)r * Hq + h] = (float)lrow[h];
                if (q_rot) for (size_t i = 0; i < qw; ++i) q_rot[(size_t)r * qw + i] = (float)qr[i];
                if (k_rot) for (size_t i = 0; i < kvw; ++i) k_rot[(size_t)r * kvw + i] = (float)Kc[(size_t)(L + k) * kvw + i];
            }
            free(Kc); free(Vc); free(qr); free(orow); free(lrow); free(sc);
        }
    }
    return fail ? -1 : used;
}

/* Append rule of Sec. 4.3.2 in the branch-slab layout: the step's rotated key and its value
 * go to row suffix_off + suffix_len of the branch cache, unless the slab is full (Sec. 4.3.4:
 * values that reach K_max are truncated).  overflow[r] = 1 marks a suppressed write. */
void hpdo_kv_append(int Hkv, int D, int n_active, int32_t suffix_cap,
                    const int32_t* suffix_off, const int32_t* suffix_len,
                    const float* k_rot, const float* v_new,
                    float* suffix_k, float* suffix_v, uint8_t* overflow)
{
    size_t kvw = (size_t)Hkv * D;
    for (int r = 0; r < n_active; ++r) {
        if (suffix_len[r] >= suffix_cap) { if (overflow) overflow[r] = 1; continue; }
        if (overflow) overflow[r] = 0;
        size_t dst = ((size_t)suffix_off[r] + (size_t)suffix_len[r]) * kvw;
        memcpy(suffix_k + dst, k_rot + (size_t)r * kvw, kvw * sizeof(float));
        memcpy(suffix_v + dst, v_new + (size_t)r * kvw, kvw * sizeof(float));
    }
}


/* ====================================================================================
 * Position-order mode: the mask the paper's implementation runs (Sec. 4.3.2 "the triangular
 * attention mask is computed using the position ID ordering"; Fig. 3 (a); Sec. 4.4).
 *
 * A group (one stacked prompt) is the model input s = cat(p, a_1..a_N): L tokens in memory, the
 * last ones being the attribute-key tokens of the skeleton, attribute j ending at memory index
 * vis[j] - 1.  Algorithm 2 leaves a gap of K_max position IDs after every attribute; with
 * start(a_j) = end(a_{j-1}) + 1 (structure tokens are ignored, Sec. 4.3.1) this gives
 *     position of prefix token t        = t + K_max * #{ j : vis[j] <= t }
 *     position of value token k of j    = vis[j] + j*K_max + k        (= pos_id[end(a_j)] + k + 1)
 * Value tokens are appended to the cache out of order; a new token sees every token of its group
 * -- prompt, skeleton, cached value tokens of ANY branch, this step's new tokens -- whose position
 * ID is not larger than its own.
 * ==================================================================================== */

/* Bookkeeping of the position-order mode: the tables of hpdo_build_meta with a per-slot anchor.
 * slot_vis[s] = number of the group's prefix tokens up to and including the slot's attribute key;
 * branch_start = slot_vis + j*pos_gap, prefix_vis[r] = slot_vis of the row's slot. */
int hpdo_build_meta_skeleton(int n_docs, int n_slots,
                             const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt,
                             const int32_t* slot_depth, const uint8_t* slot_alive, const int32_t* slot_vis,
                             int32_t suffix_cap, int32_t pos_gap,
                             int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                             int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                             int32_t* suffix_off, int32_t* suffix_len, int32_t* prefix_vis, int32_t* n_active)
{
    int kv = 0, sl = 0;
    for (int d = 0; d < n_docs; ++d) {
        doc_kv_start[d] = kv;   kv += doc_prefix_len[d];
        doc_slot_start[d] = sl; sl += doc_branch_cnt[d];
    }
    doc_kv_start[n_docs] = kv;
    doc_slot_start[n_docs] = sl;
    if (sl != n_slots) return -1;
    int r = 0;
    for (int d = 0; d < n_docs; ++d) {
        doc_active_start[d] = r;
        for (int j = 0; j < doc_branch_cnt[d]; ++j) {
            int s = doc_slot_start[d] + j;
            if (slot_vis[s] < 0 || slot_vis[s] > doc_prefix_len[d]) return -1;
            if (!slot_alive[s]) continue;
            active_slot[r]  = s;
            doc_id[r]       = d;
            branch_start[r] = slot_vis[s] + j * pos_gap;
            pos_id[r]       = branch_start[r] + slot_depth[s];
            suffix_off[r]   = s * suffix_cap;
            suffix_len[r]   = slot_depth[s];
            prefix_vis[r]   = slot_vis[s];
            ++r;
        }
    }
    doc_active_start[n_docs] = r;
    *n_active = r;
    for (int i = r; i < n_slots; ++i)
        active_slot[i] = doc_id[i] = branch_start[i] = pos_id[i] = suffix_off[i] = suffix_len[i] = prefix_vis[i] = -1;
    return 0;
}

/* One decode step in position-order mode.  For every live row the visible tokens of its group are
 * collected by comparing position IDs, one token at a time, and ordinary attention is taken over
 * them (the query's own token last).  Inputs as hpdo_decode_step plus the slot tables; k_max is
 * the position gap.  Returns the number of threads used, or -1. */
int hpdo_decode_step_posorder(int Hq, int Hkv, int D, double theta, double scale,
                              const int32_t* doc_prefix_len, const int32_t* doc_kv_start, const int32_t* doc_slot_start,
                              const int32_t* slot_depth, const uint8_t* slot_alive, const int32_t* slot_vis,
                              int32_t suffix_cap, int32_t k_max,
                              int n_active, const int32_t* active_slot, const int32_t* doc_id,
                              const float* q, const float* k_new, const float* v_new,
                              const float* prefix_k, const float* prefix_v,
                              const float* suffix_k, const float* suffix_v,
                              float* o, float* lse, float* q_rot, float* k_rot, int32_t* pos_out,
                              int n_threads)
{
    int used = 1, fail = 0;
    size_t kvw = (size_t)Hkv * D, qw = (size_t)Hq * D;
    /* position of every row's new token, and all rotated new keys (other rows may see them) */
    int32_t* pos = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n_active > 0 ? n_active : 1));
    double* kr = (double*)malloc(sizeof(double) * kvw * (size_t)(n_active > 0 ? n_active : 1));
    if (!pos || !kr) { free(pos); free(kr); return -1; }
    for (int r = 0; r < n_active; ++r) {
        int s = active_slot[r], d = doc_id[r];
        int j = s - doc_slot_start[d];
        pos[r] = slot_vis[s] + j * k_max + slot_depth[s];
        hpdo_rope(Hkv, D, theta, pos[r], k_new + (size_t)r * kvw, kr + (size_t)r * kvw);
        if (pos_out) pos_out[r] = pos[r];
        if (k_rot) for (size_t i = 0; i < kvw; ++i) k_rot[(size_t)r * kvw + i] = (float)kr[(size_t)r * kvw + i];
    }
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel
    {
#ifdef _OPENMP
#pragma omp single
        used = omp_get_num_threads();
#endif
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n_active; ++r) {
            int d = doc_id[r], L = doc_prefix_len[d];
            int s0 = doc_slot_start[d], s1 = doc_slot_start[d + 1];
            int P = pos[r];
            /* upper bound of visible tokens: the prefix, every cached token and every new token of the group */
            size_t cap_n = (size_t)L + 1;
            for (int s = s0; s < s1; ++s) cap_n += (size_t)slot_depth[s] + 1;
            double* Kc = (double*)malloc(sizeof(double) * cap_n * kvw);
            double* Vc = (double*)malloc(sizeof(double) * cap_n * kvw);
            double* qr = (double*)malloc(sizeof(double) * qw);
            double* orow = (double*)malloc(sizeof(double) * qw);
            double* lrow = (double*)malloc(sizeof(double) * (size_t)Hq);
            double* sc = (double*)malloc(sizeof(double) * cap_n);
            if (!Kc || !Vc || !qr || !orow || !lrow || !sc) {
                fail = 1;
            } else {
                size_t n = 0;
                /* prompt and skeleton tokens, in memory order, by their Algorithm 2 position */
                for (int t = 0; t < L; ++t) {
                    int before = 0;
                    for (int s = s0; s < s1; ++s) if (slot_vis[s] <= t) ++before;
                    int pt = t + k_max * before;
                    if (pt > P) continue;
                    const float* pk = prefix_k + ((size_t)doc_kv_start[d] + t) * kvw;
                    const float* pv = prefix_v + ((size_t)doc_kv_start[d] + t) * kvw;
                    for (size_t i = 0; i < kvw; ++i) { Kc[n * kvw + i] = pk[i]; Vc[n * kvw + i] = pv[i]; }
                    ++n;
                }
                /* cached value tokens of every branch of the group, alive or retired */
                for (int s = s0; s < s1; ++s) {
                    int j = s - s0;
                    for (int k = 0; k < slot_depth[s]; ++k) {
                        int pt = slot_vis[s] + j * k_max + k;
                        if (pt > P) continue;
                        const float* sk = suffix_k + ((size_t)s * suffix_cap + k) * kvw;
                        const float* sv = suffix_v + ((size_t)s * suffix_cap + k) * kvw;
                        for (size_t i = 0; i < kvw; ++i) { Kc[n * kvw + i] = sk[i]; Vc[n * kvw + i] = sv[i]; }
                        ++n;
                    }
                }
                /* this step's new tokens of the other live branches, then the row's own token last */
                for (int pass = 0; pass < 2; ++pass) {
                    for (int r2 = 0; r2 < n_active; ++r2) {
                        if (doc_id[r2] != d) continue;
                        if ((pass == 0) == (r2 == r)) continue;
                        if (pos[r2] > P) continue;
                        for (size_t i = 0; i < kvw; ++i) {
                            Kc[n * kvw + i] = kr[(size_t)r2 * kvw + i];
                            Vc[n * kvw + i] = v_new[(size_t)r2 * kvw + i];
                        }
                        ++n;
                    }
                }
                hpdo_rope(Hq, D, theta, P, q + (size_t)r * qw, qr);
                hpdo_causal_attention_row((int)n - 1, Hq, Hkv, D, scale, qr, Kc, Vc, orow, lrow, sc);
                for (size_t i = 0; i < qw; ++i) o[(size_t)r * qw + i] = (float)orow[i];
                if (lse) for (int h = 0; h < Hq; ++h) lse[(size_t)r * Hq + h] = (float)lrow[h];
                if (q_rot) for (size_t i = 0; i < qw; ++i) q_rot[(size_t)r * qw + i] = (float)qr[i];
            }
            free(Kc); free(Vc); free(qr); free(orow); free(lrow); free(sc);
        }
    }
    free(pos); free(kr);
    return fail ? -1 : used;
}

/* ------------------------------------------------------------------------------------
 * End of a decode step (Sec. 4.3.4, the prune of Algorithm 1).  tok[r] is the token sampled for
 * live row r.  The step's input token has been appended, so the slot's depth grows by one (a full
 * slab stays full); the value is finished when its delimiter was sampled, and truncated when the
 * slab -- K_max tokens -- is full.  Returns the number of rows that stay alive; generation ends
 * when it is 0 ("every value is pruned") or, through the second rule, after K_max steps.
 * ---------------------------------------------------------------------------------- */
int hpdo_advance(int n_active, const int32_t* active_slot, const int32_t* tok, int32_t delimiter,
                 int32_t k_max, int32_t* slot_depth, uint8_t* slot_alive)
{
    int stay = 0;
    for (int r = 0; r < n_active; ++r) {
        int s = active_slot[r];
        if (slot_depth[s] < k_max) slot_depth[s] += 1;
        if (tok[r] == delimiter || slot_depth[s] >= k_max) slot_alive[s] = 0;
        else { slot_alive[s] = 1; ++stay; }
    }
    return stay;
}

/* ====================================================================================
 * Three sharing levels (Sec. 4.3.5: "the instruction and attribute definition is efficiently shared
 * among all documents"): a block of tokens common to several documents, then the document, then the
 * branch.  The sequence of a branch is [block ; document ; own tokens ; new token] at positions
 * 0, 1, 2, ...; its output is ordinary causal attention at the last index, exactly as if the block
 * had been stored in front of every document.
 * ==================================================================================== */
int hpdo_decode_step_shared3(int Hq, int Hkv, int D, double theta, double scale,
                             int n_active, const int32_t* doc_id, const int32_t* doc_block,
                             const int32_t* block_kv_start, const int32_t* block_len,
                             const int32_t* suffix_off, const int32_t* suffix_len,
                             const int32_t* doc_kv_start, const int32_t* doc_prefix_len,
                             const float* q, const float* k_new, const float* v_new,
                             const float* block_k, const float* block_v,
                             const float* prefix_k, const float* prefix_v,
                             const float* suffix_k, const float* suffix_v,
                             float* o, float* lse, float* q_rot, float* k_rot, int32_t* pos_out, int n_threads)
{
    int used = 1, fail = 0;
    size_t kvw = (size_t)Hkv * D, qw = (size_t)Hq * D;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel
    {
#ifdef _OPENMP
#pragma omp single
        used = omp_get_num_threads();
#endif
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n_active; ++r) {
            int d = doc_id[r], b = doc_block[d];
            int LB = block_len[b], L = doc_prefix_len[d], k = suffix_len[r];
            int n = LB + L + k + 1;
            int pos = LB + L + k;
            double* Kc = (double*)malloc(sizeof(double) * (size_t)n * kvw);
            double* Vc = (double*)malloc(sizeof(double) * (size_t)n * kvw);
            double* qr = (double*)malloc(sizeof(double) * qw);
            double* orow = (double*)malloc(sizeof(double) * qw);
            double* lrow = (double*)malloc(sizeof(double) * (size_t)Hq);
            double* sc = (double*)malloc(sizeof(double) * (size_t)n);
            if (!Kc || !Vc || !qr || !orow || !lrow || !sc) {
                fail = 1;
            } else {
                size_t at = 0;
                const float* bk = block_k + (size_t)block_kv_start[b] * kvw;
                const float* bv = block_v + (size_t)block_kv_start[b] * kvw;
                for (size_t i = 0; i < (size_t)LB * kvw; ++i) { Kc[at + i] = bk[i]; Vc[at + i] = bv[i]; }
                at += (size_t)LB * kvw;
                const float* pk = prefix_k + (size_t)doc_kv_start[d] * kvw;
                const float* pv = prefix_v + (size_t)doc_kv_start[d] * kvw;
                for (size_t i = 0; i < (size_t)L * kvw; ++i) { Kc[at + i] = pk[i]; Vc[at + i] = pv[i]; }
                at += (size_t)L * kvw;
                const float* sk = suffix_k + (size_t)suffix_off[r] * kvw;
                const float* sv = suffix_v + (size_t)suffix_off[r] * kvw;
                for (size_t i = 0; i < (size_t)k * kvw; ++i) { Kc[at + i] = sk[i]; Vc[at + i] = sv[i]; }
                at += (size_t)k * kvw;
                hpdo_rope(Hkv, D, theta, pos, k_new + (size_t)r * kvw, Kc + at);
                for (size_t i = 0; i < kvw; ++i) Vc[at + i] = v_new[(size_t)r * kvw + i];
                hpdo_rope(Hq, D, theta, pos, q + (size_t)r * qw, qr);
                hpdo_causal_attention_row(n - 1, Hq, Hkv, D, scale, qr, Kc, Vc, orow, lrow, sc);
                for (size_t i = 0; i < qw; ++i) o[(size_t)r * qw + i] = (float)orow[i];
                if (lse) for (int h = 0; h < Hq; ++h) lse[(size_t)r * Hq + h] = (float)lrow[h];
                if (q_rot) for (size_t i = 0; i < qw; ++i) q_rot[(size_t)r * qw + i] = (float)qr[i];
                if (k_rot) for (size_t i = 0; i < kvw; ++i) k_rot[(size_t)r * kvw + i] = (float)Kc[at + i];
                if (pos_out) pos_out[r] = pos;
            }
            free(Kc); free(Vc); free(qr); free(orow); free(lrow); free(sc);
        }
    }
    return fail ? -1 : used;
}

/* Two attention results over disjoint key sets, each a normalised output with the log-sum-exp of
 * its scores, combined into the result over the union: weights e^{lse_a} and e^{lse_b}. */
void hpdo_merge_lse(int n, int D, const double* o_a, const double* lse_a, const double* o_b, const double* lse_b,
                    double* o, double* lse)
{
    for (int i = 0; i < n; ++i) {
        double m = lse_a[i] > lse_b[i] ? lse_a[i] : lse_b[i];
        if (m == -INFINITY) {
            for (int d = 0; d < D; ++d) o[(size_t)i * D + d] = 0.0;
            lse[i] = -INFINITY;
            continue;
        }
        double wa = exp(lse_a[i] - m), wb = exp(lse_b[i] - m);
        for (int d = 0; d < D; ++d)
            o[(size_t)i * D + d] = (wa * o_a[(size_t)i * D + d] + wb * o_b[(size_t)i * D + d]) / (wa + wb);
        lse[i] = m + log(wa + wb);
    }
}

/* ====================================================================================
 * First inference step (Sec. 4.3.2 "First Inference Step"; the prefill of Algorithm 1): the model
 * input s = cat(p, a_1..a_N) of every group goes through ordinary causal attention -- in the
 * prefill the memory order IS the position order -- with the rotary embedding taken at
 * Algorithm 2's position IDs (a gap of K_max behind every attribute key).  The rotated keys and the
 * values are what the decode steps later find in the prefix cache; the rows at the attribute ends
 * are the ones whose outputs predict the first value tokens.
 *   q [T,Hq,D], k,v [T,Hkv,D] for the T = sum L_d prompt tokens, groups back to back;
 *   -> o [T,Hq,D], lse [T,Hq], k_rot [T,Hkv,D], q_rot [T,Hq,D], pos [T]   (fp32 outputs; may be NULL except o, pos)
 * ==================================================================================== */
int hpdo_prefill(int Hq, int Hkv, int D, double theta, double scale,
                 int n_docs, const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt, const int32_t* slot_vis,
                 int32_t k_max,
                 const float* q, const float* k, const float* v,
                 float* o, float* lse, float* q_rot, float* k_rot, int32_t* pos, int n_threads)
{
    int used = 1, fail = 0;
    size_t kvw = (size_t)Hkv * D, qw = (size_t)Hq * D;
    /* position IDs: Algorithm 2 per group, attribute j spanning (end of j-1, end of j] */
    {
        int t0 = 0, s0 = 0;
        for (int d = 0; d < n_docs; ++d) {
            int L = doc_prefix_len[d], c = doc_branch_cnt[d];
            int32_t* st = (int32_t*)malloc(sizeof(int32_t) * (size_t)(c > 0 ? c : 1));
            int32_t* en = (int32_t*)malloc(sizeof(int32_t) * (size_t)(c > 0 ? c : 1));
            if (!st || !en) { free(st); free(en); return -1; }
            for (int j = 0; j < c; ++j) {
                en[j] = slot_vis[s0 + j] - 1;
                st[j] = j ? en[j - 1] + 1 : 0;
            }
            hpdo_alg2_position_ids(L, c, st, en, k_max, pos + t0);
            free(st); free(en);
            t0 += L; s0 += c;
        }
    }
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
    int t0 = 0;
    for (int d = 0; d < n_docs; ++d) {
        int L = doc_prefix_len[d];
        double* Kc = (double*)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1) * kvw);
        double* Vc = (double*)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1) * kvw);
        if (!Kc || !Vc) { free(Kc); free(Vc); return -1; }
        for (int t = 0; t < L; ++t) {
            hpdo_rope(Hkv, D, theta, pos[t0 + t], k + (size_t)(t0 + t) * kvw, Kc + (size_t)t * kvw);
            for (size_t i = 0; i < kvw; ++i) Vc[(size_t)t * kvw + i] = v[(size_t)(t0 + t) * kvw + i];
            if (k_rot) for (size_t i = 0; i < kvw; ++i) k_rot[(size_t)(t0 + t) * kvw + i] = (float)Kc[(size_t)t * kvw + i];
        }
#pragma omp parallel
        {
#ifdef _OPENMP
#pragma omp single
            used = omp_get_num_threads();
#endif
            double* qr = (double*)malloc(sizeof(double) * qw);
            double* orow = (double*)malloc(sizeof(double) * qw);
            double* lrow = (double*)malloc(sizeof(double) * (size_t)Hq);
            double* sc = (double*)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
            if (!qr || !orow || !lrow || !sc) {
#pragma omp atomic write
                fail = 1;
            } else {
#pragma omp for schedule(dynamic, 4)
                for (int t = 0; t < L; ++t) {
                    hpdo_rope(Hq, D, theta, pos[t0 + t], q + (size_t)(t0 + t) * qw, qr);
                    hpdo_causal_attention_row(t, Hq, Hkv, D, scale, qr, Kc, Vc, orow, lrow, sc);
                    for (size_t i = 0; i < qw; ++i) o[(size_t)(t0 + t) * qw + i] = (float)orow[i];
                    if (lse) for (int h = 0; h < Hq; ++h) lse[(size_t)(t0 + t) * Hq + h] = (float)lrow[h];
                    if (q_rot) for (size_t i = 0; i < qw; ++i) q_rot[(size_t)(t0 + t) * qw + i] = (float)qr[i];
                }
            }
            free(qr); free(orow); free(lrow); free(sc);
        }
        free(Kc); free(Vc);
        t0 += L;
    }
    return fail ? -1 : used;
}
