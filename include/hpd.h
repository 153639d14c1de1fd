/*
 * libhpd -- decode-step attention of Hyper-Parallel Decoding (HPD) for NVIDIA B200 (sm_100a).
 *
 * HPD decodes many attribute values of many stacked documents in parallel: every live
 * "branch" (one value being generated) contributes ONE new token per decode step, and that
 * token may depend on its document and on the branch's own earlier tokens only (Eq. 4-6).
 * New tokens are appended to the KV cache out of logical order; position IDs, not memory
 * order, say where a token sits (Sec. 4.3.1-4.3.3).
 *
 * Conventions for every entry point
 *   - plain C ABI; returns 0 (HPD_OK) or a negative HPD_E_* code; nothing throws.
 *   - "dev" pointers are CUDA device memory owned by the caller; "host" pointers are ordinary
 *     host memory.  The library allocates no device memory.  Pointers to bf16 tensors must be
 *     16-byte aligned; the innermost dimension is contiguous; tensors are dense row-major
 *     with the shapes stated.
 *   - every call only ENQUEUES work on `stream` (a cudaStream_t passed as void*) and never
 *     synchronises.  Sizes that change per step (n_active) are read on the device.
 *   - problems detected on the device set bits (HPD_S_*) in the caller's `dev_status` word
 *     with the offending access suppressed; kernels never trap.
 *   - documents are numbered globally in prompt order; "slots" are all branches ever admitted,
 *     numbered globally and grouped by document; "rows" are the live slots of this step in
 *     ascending slot id.  G = Hq / Hkv.
 *   - call order of one step:  hpd_build_meta  (once per step; hpd_build_meta_skeleton in
 *                                               position-order mode)
 *                              per layer: hpd_rope_append  (or hpd_rope -> hpd_kv_append)
 *                                         -> hpd_attn_decode  (or _shared / _posorder)
 *                              hpd_advance  (once per step, after the last layer).
 *     The first inference step over the prompt tokens is hpd_prefill_meta -> hpd_prefill_attn.
 */
#ifndef HPD_H_
#define HPD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Attention geometry.  Supported: D in {64, 128}; Hq % Hkv == 0 with G in {1, 2, 4, 8};
 * 1 <= suffix_cap, and for hpd_attn_decode (128/G) * round_up(suffix_cap, 4) <= 65535 (i.e. suffix_cap
 * <= 508 / 1020 / 2044 / 4092 for G = 1 / 2 / 4 / 8; larger slabs return HPD_E_CAPACITY).  sm_scale multiplies q.k before the softmax (1/sqrt(D) in the paper's
 * "scaled dot-product attention", Sec. 4.3.2).  suffix_cap is the branch-cache slab size in
 * tokens: the K_max of Sec. 4.3.1 (values longer than K_max are truncated, Sec. 4.3.4). */
typedef struct hpd_geom {
    int32_t Hq, Hkv, D;
    float   rope_theta, sm_scale;
    int32_t suffix_cap;
} hpd_geom;

enum {
    HPD_OK          =  0,
    HPD_E_ARG       = -1,   /* null / misaligned pointer, negative size                        */
    HPD_E_GEOM      = -2,   /* geometry outside the supported set                              */
    HPD_E_WORKSPACE = -3,   /* workspace_bytes smaller than hpd_workspace_bytes() reports      */
    HPD_E_CAPACITY  = -4,   /* a size exceeds what the call can index (int32 tables, slab size) */
    HPD_E_CUDA      = -5    /* a CUDA runtime/driver call failed; see hpd_last_cuda_error()    */
};

/* bits of *dev_status */
enum {
    HPD_S_OVERFLOW  = 1,    /* hpd_kv_append: a branch slab was full, its write was suppressed */
    HPD_S_BAD_TABLE = 2,    /* a table entry pointed outside its tensor; the row was skipped   */
    HPD_S_TIMEOUT   = 4     /* an in-kernel wait on the kernel's own copies gave up            */
};

const char* hpd_strerror(int code);
/* cudaError_t (as int) of the last failing CUDA call made by this library on this thread. */
int hpd_last_cuda_error(void);

/* Bytes of workspace that hpd_build_meta + hpd_attn_decode need for problems up to the given
 * sizes.  The SAME workspace must be passed to hpd_build_meta and to the hpd_attn_decode calls
 * of that step: build_meta leaves its split-KV work list there. */
size_t hpd_workspace_bytes(const hpd_geom* geom /*host*/, int max_docs, int max_slots, int max_prefix_tokens);

/*
 * hpd_build_meta -- per-step bookkeeping as int32 device tables (Algorithm 2; Sec. 4.3.2-4.3.6).
 *
 * Inputs (dev):  doc_prefix_len[n_docs]  tokens of each document's shared prefix (L_d)
 *                doc_branch_cnt[n_docs]  slots of each document (sum = n_slots)
 *                slot_depth[n_slots]     branch tokens cached before this step
 *                slot_alive[n_slots]     non-zero while the branch is still decoding (pruning, Sec. 4.3.4)
 *                pos_gap                 0: positions continue the document, pos = L_d + depth;
 *                                        K_max: the j-th branch of a document is shifted by
 *                                        Algorithm 2's running offset j*K_max
 * Outputs (dev): doc_kv_start[n_docs+1]      exclusive scan of doc_prefix_len
 *                doc_slot_start[n_docs+1]    exclusive scan of doc_branch_cnt
 *                doc_active_start[n_docs+1]  CSR of rows per document
 *                per row r < n_active (arrays of n_slots entries, the rest set to -1):
 *                active_slot[r]  slot id (ascending)      doc_id[r]      its document
 *                branch_start[r] position ID of the branch's first token
 *                pos_id[r]       branch_start + depth (Sec. 4.3.3: previous ID + 1)
 *                suffix_off[r]   first row of the slot's slab in the branch cache (slot*suffix_cap)
 *                suffix_len[r]   depth
 *                n_active[1]     number of rows
 * Also writes the internal work list of hpd_attn_decode into `workspace`.
 * All tables are int32 and are reproducible bit for bit.  n_docs or n_slots may be 0.
 */
int hpd_build_meta(const hpd_geom* geom /*host*/, int n_docs, int n_slots,
                   const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt,
                   const int32_t* slot_depth, const uint8_t* slot_alive, int32_t pos_gap,
                   int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                   int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                   int32_t* suffix_off, int32_t* suffix_len, int32_t* n_active,
                   void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream);

/*
 * hpd_rope -- rotary embedding of the step's new q and k at each row's position ID, in place
 * (Sec. 4.3.1: the assigned position IDs define the positional embedding; Sec. 4.4).
 * Pairing is half-split: element i with i + D/2; angle = pos_id[r] * rope_theta^(-2i/D),
 * taken and reduced to [-pi, pi] in fp64; sine, cosine and the rotation in fp32; result rounded to bf16
 * (nearest even).
 *   q [max_rows, Hq, D] bf16 dev, k_new [max_rows, Hkv, D] bf16 dev; rows >= *n_active untouched.
 */
int hpd_rope(const hpd_geom* geom /*host*/, int max_rows, const int32_t* n_active /*dev*/,
             const int32_t* pos_id /*dev*/, void* q, void* k_new, void* stream);

/*
 * hpd_kv_append -- append each row's (rotated) key and its value to the branch cache
 * (Sec. 4.3.2: new tokens are appended to the cache; here every slot owns a slab of
 * suffix_cap rows, row suffix_off[r] + suffix_len[r] receives the token).
 *   k_new, v_new [max_rows, Hkv, D] bf16 dev;  suffix_k, suffix_v [n_slots*suffix_cap, Hkv, D] bf16 dev.
 * A full slab (suffix_len >= suffix_cap) gets no write and sets HPD_S_OVERFLOW.
 * The caller advances slot_depth for the next step.
 */
int hpd_kv_append(const hpd_geom* geom /*host*/, int max_rows, int n_slots, const int32_t* n_active,
                  const int32_t* suffix_off, const int32_t* suffix_len,
                  const void* k_new, const void* v_new, void* suffix_k, void* suffix_v,
                  int32_t* dev_status, void* stream);

/*
 * hpd_rope_append -- hpd_rope followed by hpd_kv_append in ONE launch (Sec. 4.3.1-4.3.2: the new token
 * is rotated at its assigned position ID and appended to the cache).  q and k_new are rotated in place
 * and the rotated key and the value go to row suffix_off[r] + suffix_len[r] of the branch cache; every
 * output bit equals that of the two separate calls, as do the status bits (a full slab still gets its q
 * and k rotated, no cache write, HPD_S_OVERFLOW).  Arguments as in the two calls.
 */
int hpd_rope_append(const hpd_geom* geom /*host*/, int max_rows, int n_slots, const int32_t* n_active,
                    const int32_t* pos_id, const int32_t* suffix_off, const int32_t* suffix_len,
                    void* q, void* k_new, const void* v_new, void* suffix_k, void* suffix_v,
                    int32_t* dev_status, void* stream);

/*
 * hpd_attn_decode -- the HPD decode attention (Eq. 5-6; Sec. 4.3.3).  For row r (document d,
 * slot s) and q head h:   o = softmax(sm_scale * q . [K_prefix(d) ; K_suffix(s)]^T) [V_prefix(d) ; V_suffix(s)]
 * over the document's L_d prefix tokens and the branch's own cached tokens.  The prefix of a
 * document is read from memory once per KV head for all of the document's rows.
 *   q [max_rows, Hq, D] bf16 (already rotated); prefix_k/v [total_prefix_tokens, Hkv, D] bf16
 *   (as cached, i.e. rotated); suffix_k/v [n_slots*suffix_cap, Hkv, D] bf16; tables from
 *   hpd_build_meta; suffix_includes_new = 1 when hpd_kv_append already ran this step (the branch
 *   then sees suffix_len+1 cached tokens, the new token among them), 0 to see suffix_len tokens.
 *   o [max_rows, Hq, D] bf16; lse [max_rows, Hq] fp32 natural-log sum-exp of the scaled scores,
 *   may be NULL.  Rows >= *n_active are not written.  A row with no visible token yields o = 0,
 *   lse = -inf.
 */
int hpd_attn_decode(const hpd_geom* geom /*host*/, int n_docs, int max_rows, int n_slots, int total_prefix_tokens,
                    const void* q, const void* prefix_k, const void* prefix_v,
                    const void* suffix_k, const void* suffix_v,
                    const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                    const int32_t* doc_id, const int32_t* suffix_off, const int32_t* suffix_len,
                    const int32_t* n_active, int suffix_includes_new,
                    void* o, float* lse,
                    void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream);

/*
 * hpd_advance -- the end of a decode step on the device (Sec. 4.3.4 "Early Stopping"; the prune of
 * Algorithm 1), so that the loop needs no host round trip per step.  token_id[r] is the token sampled
 * from row r's output.  For every row r < *n_active with slot s = active_slot[r]:
 *   slot_depth[s] = min(slot_depth[s] + 1, suffix_cap)      the step's input token is in the cache now
 *   slot_alive[s] = 0 if token_id[r] == delimiter_id        (the value is complete: its delimiter came)
 *                     or slot_depth[s] == suffix_cap        (K_max reached: the value is truncated)
 * and n_alive[0] (dev) = number of rows that stay alive: generation ends when it reaches 0.  The next
 * hpd_build_meta reads the updated slot tables.  token_id [max_rows] int32 dev.
 */
int hpd_advance(const hpd_geom* geom /*host*/, int max_rows, const int32_t* n_active, const int32_t* active_slot,
                const int32_t* token_id, int32_t delimiter_id, int32_t* slot_depth, uint8_t* slot_alive,
                int32_t* n_alive, void* stream);

/*
 * hpd_attn_decode_shared -- hpd_attn_decode with a third sharing level in the same launch (Sec. 4.3.5: the
 * instruction and the attribute definitions are shared among all documents): document d is preceded by block
 * doc_block[d], rows [block_kv_start[b], +block_len[b]) of block_k / block_v [total_block_tokens, Hkv, D] (dev),
 * stored once however many documents follow it.  Every (document, kv head) unit visits its block's tiles and its
 * document's tiles; the block's bytes come from HBM once and from L2 afterwards.  Results equal those of the
 * block stored in front of every document.  doc_block [n_docs], block_kv_start and block_len [n_blocks] int32 dev.
 * Position IDs must count the block: build the tables with hpd_build_meta_skeleton, slot_vis = block length + L_d,
 * pos_gap = 0.  Everything else as hpd_attn_decode (with total_block_tokens = 0 it is that call).
 */
int hpd_attn_decode_shared(const hpd_geom* geom /*host*/, int n_docs, int max_rows, int n_slots, int total_prefix_tokens,
                           const void* q, const void* prefix_k, const void* prefix_v,
                           const void* suffix_k, const void* suffix_v,
                           const void* block_k, const void* block_v, int total_block_tokens,
                           const int32_t* doc_block, const int32_t* block_kv_start, const int32_t* block_len,
                           const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                           const int32_t* doc_id, const int32_t* suffix_off, const int32_t* suffix_len,
                           const int32_t* n_active, int suffix_includes_new,
                           void* o, float* lse,
                           void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream);

/*
 * hpd_merge_lse -- three sharing levels as separate passes (the building block for caches that hpd_attn_decode_shared
 * does not cover, e.g. a block shared across calls).  A block of tokens common to several documents is attended ONCE per block
 * for all rows below it by a second hpd_attn_decode call whose "documents" are the blocks (tables from a
 * second hpd_build_meta over the blocks, its own workspace, an all-zero suffix_len table and
 * suffix_includes_new = 0, the block's K/V as prefix); this call combines the two results per (row, head):
 *     o = (e^{lse_a} o_a + e^{lse_b} o_b) / (e^{lse_a} + e^{lse_b}),   lse = log(e^{lse_a} + e^{lse_b}).
 * Both calls need their lse outputs.  o may alias o_a or o_b, lse may alias lse_a or lse_b or be NULL.
 * Position IDs then count the block too: build the document tables with hpd_build_meta_skeleton,
 * slot_vis = block length + L_d and pos_gap = 0.
 *   o_a, o_b, o [max_rows, Hq, D] bf16 dev; lse_a, lse_b, lse [max_rows, Hq] fp32 dev.
 */
int hpd_merge_lse(const hpd_geom* geom /*host*/, int max_rows, const int32_t* n_active,
                  const void* o_a, const float* lse_a, const void* o_b, const float* lse_b,
                  void* o, float* lse, void* stream);

/*
 * Position-order mode: the mask the paper's implementation runs (Sec. 4.3.2: "the triangular attention
 * mask is computed using the position ID ordering"; Fig. 3; Sec. 4.4; Algorithm 2).  A "document" of the
 * tables is then a whole stacked prompt: its prefix is the prompt followed by the skeleton, i.e. the
 * attribute-key tokens of its slots in slot order, and Algorithm 2 leaves a gap of pos_gap = K_max
 * position IDs behind every attribute key.  A new token sees every token of its group whose position ID
 * is not larger than its own: the prefix up to and including its own attribute key, and the cached
 * tokens of every slot of the group up to and including its own -- retired slots too, their tokens stay
 * in the cache (Sec. 4.3.4) -- which in the lock-step loop of Algorithm 1 is exactly the pattern of the
 * fine-tuning mask of Sec. 4.4.
 *
 * hpd_build_meta_skeleton -- hpd_build_meta with a per-slot anchor:
 *   slot_vis[n_slots] (dev)   prefix tokens of the slot's group up to and including its attribute key
 *                             (= end(a_j) + 1 in Algorithm 2's notation; 0 <= slot_vis <= L_d, ascending
 *                             inside a group).  The builder only uses it as the position anchor of the
 *                             slot's first token; hpd_merge_lse's three-level layout passes a larger one.
 *   branch_start[r] = slot_vis + j*pos_gap   (= pos_id[end(a_j)] + 1 of Algorithm 2)
 *   prefix_vis[r]   = slot_vis of the row's slot (n_slots entries, -1 past n_active)
 * Everything else as hpd_build_meta.
 *
 * hpd_attn_decode_posorder -- the attention under that mask.  Arguments as hpd_attn_decode, with the
 * slot tables (doc_slot_start, active_slot from the builder; the caller's slot_depth and slot_alive) in
 * place of suffix_off / suffix_len, and prefix_vis.  A slot's slab starts at row slot*suffix_cap; it
 * holds slot_depth tokens, one more for live slots when suffix_includes_new is set.  A group may have at
 * most 128 slots (larger groups set HPD_S_BAD_TABLE and their rows see the prefix only).
 */
int hpd_build_meta_skeleton(const hpd_geom* geom /*host*/, int n_docs, int n_slots,
                            const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt,
                            const int32_t* slot_depth, const uint8_t* slot_alive, const int32_t* slot_vis, int32_t pos_gap,
                            int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                            int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                            int32_t* suffix_off, int32_t* suffix_len, int32_t* prefix_vis, int32_t* n_active,
                            void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream);
int hpd_attn_decode_posorder(const hpd_geom* geom /*host*/, int n_docs, int max_rows, int n_slots, int total_prefix_tokens,
                             const void* q, const void* prefix_k, const void* prefix_v,
                             const void* suffix_k, const void* suffix_v,
                             const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                             const int32_t* doc_slot_start, const int32_t* doc_id, const int32_t* active_slot,
                             const int32_t* slot_depth, const uint8_t* slot_alive, const int32_t* prefix_vis,
                             const int32_t* n_active, int suffix_includes_new,
                             void* o, float* lse,
                             void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream);

/*
 * First inference step (Sec. 4.3.2 "First Inference Step"; the prefill of Algorithm 1): the whole model input
 * s = cat(prompt, skeleton) of every group through causal attention -- in the prefill the memory order is the
 * position order -- with the rotary embedding at Algorithm 2's position IDs.  Three calls:
 *   hpd_prefill_meta   per prompt token x (T = sum L_d of them, groups back to back): tok_doc[x] its group,
 *                      tok_pos[x] = t + pos_gap * #{slots of the group whose attribute key ends before t}
 *                      (Algorithm 2 with start(a_j) = end(a_{j-1}) + 1), tok_vis[x] = t + 1 (its causal bound),
 *                      t the token's index in its group; doc_kv_start, doc_slot_start; n_tokens[0] = T; and the
 *                      attention's work list in `workspace` (hpd_workspace_bytes(geom, n_docs, total_tokens, ..)).
 *                      At most 2048 groups per call (HPD_E_CAPACITY beyond).
 *   hpd_rope           with max_rows = total_tokens, n_active = n_tokens, pos_id = tok_pos, q = the prompt
 *                      tokens' queries and k_new = prefix_k itself: the keys are rotated in place in the prefix
 *                      cache, where the decode steps find them; the values are stored unrotated by the caller.
 *   hpd_prefill_attn   o[x] = causal attention of token x over its group's tokens 0..t; every 128/G tokens of a
 *                      group form one tensor-core tile and visit only the keys up to the tile's last token.
 * The rows that predict the first value tokens are those at the attribute ends, x = doc_kv_start[d] + slot_vis - 1
 * ("decoded from positions 12, 22 and 32" in the paper's figure); when only they are needed (last layer),
 * hpd_attn_decode_posorder on depth-0 slots with their queries does the same with 96 rows per prompt.
 *   q, o [total_tokens, Hq, D] bf16; prefix_k, prefix_v [total_tokens, Hkv, D] bf16; lse [total_tokens, Hq] or NULL.
 */
int hpd_prefill_meta(const hpd_geom* geom /*host*/, int n_docs, int n_slots, int total_tokens,
                     const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt, const int32_t* slot_vis, int32_t pos_gap,
                     int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* tok_doc, int32_t* tok_pos, int32_t* tok_vis,
                     int32_t* n_tokens, void* workspace, size_t workspace_bytes, void* stream);
int hpd_prefill_attn(const hpd_geom* geom /*host*/, int n_docs, int total_tokens,
                     const void* q, const void* prefix_k, const void* prefix_v,
                     const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* tok_doc, const int32_t* tok_vis,
                     const int32_t* n_tokens, void* o, float* lse,
                     void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream);

/*
 * std_attn_decode -- the in-repo comparison: standard batched decode in which every branch is a
 * sequence of its own with a private physical copy of [prefix ; branch tokens] (parallel streams
 * as batch elements, Sec. 2; standard batched inference, Sec. 4.3.6).  Same math as
 * hpd_attn_decode on the same tokens, GQA, split-KV.
 *   q [max_rows, Hq, D] bf16 (rotated); dup_k/v [total_tokens, Hkv, D] bf16, total_tokens <= 2^31-1
 *   (host value: the tensors' extent in token rows; tiles are fetched 16 tokens at a time, and
 *   whatever a tile holds beyond a sequence's last token -- other sequences' rows, or nothing at the
 *   end of the tensor -- is masked out and never read past total_tokens);
 *   seq_start [max_rows] int64 first token row of each sequence; seq_len [max_rows] int32;
 *   o [max_rows, Hq, D] bf16; lse nullable.
 * workspace: std_workspace_bytes(); may be NULL when that reports 0.
 */
size_t std_workspace_bytes(const hpd_geom* geom /*host*/, int max_rows, int max_seq_len);
int std_attn_decode(const hpd_geom* geom /*host*/, int max_rows, int max_seq_len, long long total_tokens,
                    const int32_t* n_active,
                    const void* q, const void* dup_k, const void* dup_v,
                    const int64_t* seq_start, const int32_t* seq_len,
                    void* o, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/*
 * std_attn_decode_static -- std_attn_decode without a workspace argument.  (The paper has no
 * counterpart: this is a convenience of the library.)
 *
 * For callers that cannot allocate device memory when they need the call: code that runs while a
 * framework's caching allocator is locked or exhausted, plug-ins of a host program that owns all
 * device memory, services that have committed the whole device heap to KV caches.  The split-KV
 * partials go to a fixed array of std_attn_decode_static_max_bytes() (16 MiB) that is part of the
 * library's device image: every GPU that loads the library holds it until the process exits.
 *   - Arguments, layouts and results are those of std_attn_decode.
 *   - A problem whose std_workspace_bytes() exceeds the array is rejected with HPD_E_WORKSPACE and
 *     nothing is launched; use std_attn_decode with your own workspace then.
 *   - The call allocates nothing (no cudaMalloc/cudaFree, no allocating library routine).
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress) and keeps
 *     it; make that first call outside any stream capture.  It is also the moment at which the CUDA
 *     runtime may place the library's device image, the array included, on that device, which can fail
 *     when the device heap is already exhausted: make one warm-up call at start-up, before memory gets
 *     tight.  From then on a call takes nothing from the device heap.
 *   - One process may use the library on several devices; every per-device cache of the library (this
 *     address, SM counts, kernel attributes) is keyed by the device that is current at the call.
 *   - All calls on one device share the array and it keeps the last call's contents.  Nothing needs
 *     clearing (each call writes every partial before its merge reads it), but two calls whose
 *     kernels can overlap on the GPU (different streams) race on it: keep them on one stream or
 *     order them with events.
 */
size_t std_attn_decode_static_max_bytes(void);
int std_attn_decode_static(const hpd_geom* geom /*host*/, int max_rows, int max_seq_len, long long total_tokens,
                           const int32_t* n_active,
                           const void* q, const void* dup_k, const void* dup_v,
                           const int64_t* seq_start, const int32_t* seq_len,
                           void* o, float* lse, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HPD_H_ */
