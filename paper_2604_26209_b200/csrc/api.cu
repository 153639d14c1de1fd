// extern "C" entry points of libhpd (see include/hpd.h): argument checks and kernel dispatch only.
#include <atomic>

#include "common.cuh"

namespace hpd {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int>(e); }

int geom_check(const hpd_geom* g)
{
    if (!g) return HPD_E_ARG;
    if (g->D != 64 && g->D != 128) return HPD_E_GEOM;
    if (g->Hq <= 0 || g->Hkv <= 0 || g->Hq % g->Hkv != 0) return HPD_E_GEOM;
    const int G = g->Hq / g->Hkv;
    if (G != 1 && G != 2 && G != 4 && G != 8) return HPD_E_GEOM;
    if (g->suffix_cap < 1) return HPD_E_GEOM;
    if (!(g->rope_theta > 0.f)) return HPD_E_GEOM;
    return HPD_OK;
}

int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return dev;
}

// SM count of the current device.  Looked up once per device; the table is only ever written with the value the
// driver reports for that device, so concurrent first calls store the same number.
int sm_count()
{
    static std::atomic<int> cached[kMaxDevices];
    const int dev = current_device();
    const bool slot = dev >= 0 && dev < kMaxDevices;
    if (slot) {
        const int c = cached[dev].load(std::memory_order_relaxed);
        if (c > 0) return c;
    }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) {
        if (slot) cached[dev].store(n, std::memory_order_relaxed);
        return n;
    }
    (void)cudaGetLastError();
    return 148;
}

}  // namespace hpd

using namespace hpd;

extern "C" {

const char* hpd_strerror(int code)
{
    switch (code) {
        case HPD_OK: return "ok";
        case HPD_E_ARG: return "invalid argument (null or misaligned pointer, negative size)";
        case HPD_E_GEOM: return "unsupported geometry (need D in {64,128}, Hq/Hkv in {1,2,4,8}, suffix_cap >= 1)";
        case HPD_E_WORKSPACE: return "workspace too small";
        case HPD_E_CAPACITY: return "size exceeds what the call can index (int32 tables; suffix_cap too large for the attention kernel)";
        case HPD_E_CUDA: return "CUDA call failed (see hpd_last_cuda_error)";
        default: return "unknown error code";
    }
}

int hpd_last_cuda_error(void) { return g_last_cuda_error; }

size_t hpd_workspace_bytes(const hpd_geom* geom, int max_docs, int max_slots, int /*max_prefix_tokens*/)
{
    if (geom_check(geom) != HPD_OK || max_docs < 0 || max_slots < 0) return 0;
    return ws_layout(*geom, max_docs, max_slots, sm_count()).total;
}

static int build_meta_common(const hpd_geom* geom, int n_docs, int n_slots,
                             const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt,
                             const int32_t* slot_depth, const uint8_t* slot_alive, const int32_t* slot_vis, int32_t pos_gap,
                             int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                             int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                             int32_t* suffix_off, int32_t* suffix_len, int32_t* prefix_vis, int32_t* n_active,
                             void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (n_docs < 0 || n_slots < 0 || pos_gap < 0) return HPD_E_ARG;
    if (n_docs == 0 && n_slots > 0) return HPD_E_ARG;
    if (!doc_kv_start || !doc_slot_start || !doc_active_start || !n_active || !workspace) return HPD_E_ARG;
    if (n_docs > 0 && (!doc_prefix_len || !doc_branch_cnt)) return HPD_E_ARG;
    if (n_slots > 0 && (!slot_depth || !slot_alive || !active_slot || !doc_id || !branch_start || !pos_id ||
                        !suffix_off || !suffix_len)) return HPD_E_ARG;
    if (static_cast<long long>(n_slots) * geom->suffix_cap > 0x7fffffffll) return HPD_E_CAPACITY;
    if (!aligned16(workspace)) return HPD_E_ARG;
    const int n_sm = sm_count();
    const WsLayout lay = ws_layout(*geom, n_docs, n_slots, n_sm);
    if (workspace_bytes < lay.total) return HPD_E_WORKSPACE;
    return launch_build_meta(*geom, n_docs, n_slots, doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive, pos_gap,
                             doc_kv_start, doc_slot_start, doc_active_start, active_slot, doc_id, branch_start, pos_id,
                             suffix_off, suffix_len, n_active, workspace, lay, n_sm, dev_status,
                             static_cast<cudaStream_t>(stream), slot_vis, prefix_vis);
}

int hpd_build_meta(const hpd_geom* geom, int n_docs, int n_slots,
                   const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt,
                   const int32_t* slot_depth, const uint8_t* slot_alive, int32_t pos_gap,
                   int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                   int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                   int32_t* suffix_off, int32_t* suffix_len, int32_t* n_active,
                   void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    return build_meta_common(geom, n_docs, n_slots, doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive, nullptr, pos_gap,
                             doc_kv_start, doc_slot_start, doc_active_start, active_slot, doc_id, branch_start, pos_id,
                             suffix_off, suffix_len, nullptr, n_active, workspace, workspace_bytes, dev_status, stream);
}

int hpd_build_meta_skeleton(const hpd_geom* geom, int n_docs, int n_slots,
                            const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt,
                            const int32_t* slot_depth, const uint8_t* slot_alive, const int32_t* slot_vis, int32_t pos_gap,
                            int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                            int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                            int32_t* suffix_off, int32_t* suffix_len, int32_t* prefix_vis, int32_t* n_active,
                            void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    if (n_slots > 0 && (!slot_vis || !prefix_vis)) return HPD_E_ARG;
    return build_meta_common(geom, n_docs, n_slots, doc_prefix_len, doc_branch_cnt, slot_depth, slot_alive, slot_vis, pos_gap,
                             doc_kv_start, doc_slot_start, doc_active_start, active_slot, doc_id, branch_start, pos_id,
                             suffix_off, suffix_len, prefix_vis, n_active, workspace, workspace_bytes, dev_status, stream);
}

int hpd_rope(const hpd_geom* geom, int max_rows, const int32_t* n_active, const int32_t* pos_id,
             void* q, void* k_new, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (max_rows < 0) return HPD_E_ARG;
    if (max_rows == 0) return HPD_OK;
    if (!n_active || !pos_id || !q || !k_new || !aligned16(q) || !aligned16(k_new)) return HPD_E_ARG;
    return launch_rope(*geom, max_rows, n_active, pos_id, static_cast<__nv_bfloat16*>(q),
                       static_cast<__nv_bfloat16*>(k_new), static_cast<cudaStream_t>(stream));
}

int hpd_kv_append(const hpd_geom* geom, int max_rows, int n_slots, const int32_t* n_active,
                  const int32_t* suffix_off, const int32_t* suffix_len,
                  const void* k_new, const void* v_new, void* suffix_k, void* suffix_v,
                  int32_t* dev_status, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (max_rows < 0 || n_slots < 0) return HPD_E_ARG;
    if (max_rows == 0) return HPD_OK;
    if (!n_active || !suffix_off || !suffix_len || !k_new || !v_new || !suffix_k || !suffix_v) return HPD_E_ARG;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(suffix_k) || !aligned16(suffix_v)) return HPD_E_ARG;
    return launch_kv_append(*geom, max_rows, n_slots, n_active, suffix_off, suffix_len,
                            static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
                            static_cast<__nv_bfloat16*>(suffix_k), static_cast<__nv_bfloat16*>(suffix_v), dev_status,
                            static_cast<cudaStream_t>(stream));
}

int hpd_rope_append(const hpd_geom* geom, int max_rows, int n_slots, const int32_t* n_active, const int32_t* pos_id,
                    const int32_t* suffix_off, const int32_t* suffix_len, void* q, void* k_new, const void* v_new,
                    void* suffix_k, void* suffix_v, int32_t* dev_status, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (max_rows < 0 || n_slots < 0) return HPD_E_ARG;
    if (max_rows == 0) return HPD_OK;
    if (!n_active || !pos_id || !suffix_off || !suffix_len || !q || !k_new || !v_new || !suffix_k || !suffix_v) return HPD_E_ARG;
    if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(suffix_k) || !aligned16(suffix_v)) return HPD_E_ARG;
    return launch_rope_append(*geom, max_rows, n_slots, n_active, pos_id, suffix_off, suffix_len,
                              static_cast<__nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(k_new),
                              static_cast<const __nv_bfloat16*>(v_new), static_cast<__nv_bfloat16*>(suffix_k),
                              static_cast<__nv_bfloat16*>(suffix_v), dev_status, static_cast<cudaStream_t>(stream));
}

int hpd_advance(const hpd_geom* geom, int max_rows, const int32_t* n_active, const int32_t* active_slot,
                const int32_t* token_id, int32_t delimiter_id, int32_t* slot_depth, uint8_t* slot_alive,
                int32_t* n_alive, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (max_rows < 0) return HPD_E_ARG;
    if (!n_alive) return HPD_E_ARG;
    if (max_rows > 0 && (!n_active || !active_slot || !token_id || !slot_depth || !slot_alive)) return HPD_E_ARG;
    return launch_advance(*geom, max_rows, n_active, active_slot, token_id, delimiter_id, slot_depth, slot_alive, n_alive,
                          static_cast<cudaStream_t>(stream));
}

int hpd_merge_lse(const hpd_geom* geom, int max_rows, const int32_t* n_active, const void* o_a, const float* lse_a,
                  const void* o_b, const float* lse_b, void* o, float* lse, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (max_rows < 0) return HPD_E_ARG;
    if (max_rows == 0) return HPD_OK;
    if (!n_active || !o_a || !lse_a || !o_b || !lse_b || !o) return HPD_E_ARG;
    if (!aligned16(o_a) || !aligned16(o_b) || !aligned16(o)) return HPD_E_ARG;
    return launch_merge_lse(*geom, max_rows, n_active, static_cast<const __nv_bfloat16*>(o_a), lse_a,
                            static_cast<const __nv_bfloat16*>(o_b), lse_b, static_cast<__nv_bfloat16*>(o), lse,
                            static_cast<cudaStream_t>(stream));
}

struct OrderTables {                 // extra tables of the position-order mode (all null in the branch-local mode)
    const int32_t *doc_slot_start, *active_slot, *slot_depth, *prefix_vis;
    const uint8_t* slot_alive;
    // third sharing level (branch-local mode only; all null otherwise)
    const void *block_k, *block_v;
    const int32_t *doc_block, *block_kv_start, *block_len;
    int total_block;
};

static int attn_common(const hpd_geom* geom, int n_docs, int max_rows, int n_slots, int total_prefix_tokens,
                       const void* q, const void* prefix_k, const void* prefix_v,
                       const void* suffix_k, const void* suffix_v,
                       const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                       const int32_t* doc_id, const int32_t* suffix_off, const int32_t* suffix_len,
                       const OrderTables& ord, const int32_t* n_active, int suffix_includes_new,
                       void* o, float* lse,
                       void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    // the attention kernel keeps each branch's packed column and cached-token count as 16-bit numbers
    if (attn_packed_columns(*geom) > kMaxPackedColumns) return HPD_E_CAPACITY;
    if (n_docs < 0 || max_rows < 0 || n_slots < 0 || total_prefix_tokens < 0) return HPD_E_ARG;
    if (max_rows == 0 || n_docs == 0) return HPD_OK;
    const bool order = ord.prefix_vis != nullptr;
    const bool slots = ord.active_slot != nullptr;       // position-order mode with branch caches (not the prefill)
    if (!q || !doc_kv_start || !doc_prefix_len || !doc_active_start || !doc_id || !n_active || !o || !workspace) return HPD_E_ARG;
    if ((!order || slots) && (!suffix_k || !suffix_v)) return HPD_E_ARG;
    if (!order && (!suffix_off || !suffix_len)) return HPD_E_ARG;
    if (slots && (!ord.doc_slot_start || !ord.slot_depth || !ord.slot_alive)) return HPD_E_ARG;
    if (total_prefix_tokens > 0 && (!prefix_k || !prefix_v)) return HPD_E_ARG;
    if (!aligned16(q) || !aligned16(prefix_k) || !aligned16(prefix_v) || !aligned16(suffix_k) ||
        !aligned16(suffix_v) || !aligned16(o) || !aligned16(workspace)) return HPD_E_ARG;
    const WsLayout lay = ws_layout(*geom, n_docs, n_slots, sm_count());
    if (workspace_bytes < lay.total) return HPD_E_WORKSPACE;

    AttnArgs a{};
    a.g = *geom;
    a.n_docs = n_docs; a.max_rows = max_rows; a.n_slots = n_slots; a.total_prefix = total_prefix_tokens;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.prefix_k = static_cast<const __nv_bfloat16*>(prefix_k);
    a.prefix_v = static_cast<const __nv_bfloat16*>(prefix_v);
    // without a branch cache (the prefill) the cache's tensor maps still need an address: the prefix tensors', never used
    a.suffix_k = static_cast<const __nv_bfloat16*>(suffix_k ? suffix_k : prefix_k);
    a.suffix_v = static_cast<const __nv_bfloat16*>(suffix_v ? suffix_v : prefix_v);
    a.doc_kv_start = doc_kv_start; a.doc_prefix_len = doc_prefix_len; a.doc_active_start = doc_active_start;
    a.doc_id = doc_id; a.suffix_off = suffix_off; a.suffix_len = suffix_len; a.n_active = n_active;
    a.suffix_extra = suffix_includes_new ? 1 : 0;
    a.doc_slot_start = ord.doc_slot_start; a.active_slot = ord.active_slot; a.slot_depth = ord.slot_depth;
    a.prefix_vis = ord.prefix_vis; a.slot_alive = ord.slot_alive;
    a.block_k = static_cast<const __nv_bfloat16*>(ord.block_k); a.block_v = static_cast<const __nv_bfloat16*>(ord.block_v);
    a.doc_block = ord.doc_block; a.block_kv_start = ord.block_kv_start; a.block_len = ord.block_len;
    a.total_block = ord.total_block;
    a.o = static_cast<__nv_bfloat16*>(o);
    a.lse = lse;
    a.workspace = workspace; a.lay = lay; a.dev_status = dev_status;
    a.stream = static_cast<cudaStream_t>(stream);
    return launch_attn_tc(a);
}

int hpd_attn_decode(const hpd_geom* geom, int n_docs, int max_rows, int n_slots, int total_prefix_tokens,
                    const void* q, const void* prefix_k, const void* prefix_v,
                    const void* suffix_k, const void* suffix_v,
                    const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                    const int32_t* doc_id, const int32_t* suffix_off, const int32_t* suffix_len,
                    const int32_t* n_active, int suffix_includes_new,
                    void* o, float* lse,
                    void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    return attn_common(geom, n_docs, max_rows, n_slots, total_prefix_tokens, q, prefix_k, prefix_v, suffix_k, suffix_v,
                       doc_kv_start, doc_prefix_len, doc_active_start, doc_id, suffix_off, suffix_len, OrderTables{},
                       n_active, suffix_includes_new, o, lse, workspace, workspace_bytes, dev_status, stream);
}

int hpd_attn_decode_shared(const hpd_geom* geom, int n_docs, int max_rows, int n_slots, int total_prefix_tokens,
                           const void* q, const void* prefix_k, const void* prefix_v,
                           const void* suffix_k, const void* suffix_v,
                           const void* block_k, const void* block_v, int total_block_tokens,
                           const int32_t* doc_block, const int32_t* block_kv_start, const int32_t* block_len,
                           const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                           const int32_t* doc_id, const int32_t* suffix_off, const int32_t* suffix_len,
                           const int32_t* n_active, int suffix_includes_new,
                           void* o, float* lse,
                           void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    if (total_block_tokens < 0) return HPD_E_ARG;
    if (total_block_tokens == 0)                         // no block at all: the plain call
        return hpd_attn_decode(geom, n_docs, max_rows, n_slots, total_prefix_tokens, q, prefix_k, prefix_v, suffix_k, suffix_v,
                               doc_kv_start, doc_prefix_len, doc_active_start, doc_id, suffix_off, suffix_len, n_active,
                               suffix_includes_new, o, lse, workspace, workspace_bytes, dev_status, stream);
    if (!block_k || !block_v || !doc_block || !block_kv_start || !block_len || !aligned16(block_k) || !aligned16(block_v))
        return HPD_E_ARG;
    OrderTables ord{};
    ord.block_k = block_k; ord.block_v = block_v; ord.doc_block = doc_block; ord.block_kv_start = block_kv_start;
    ord.block_len = block_len; ord.total_block = total_block_tokens;
    return attn_common(geom, n_docs, max_rows, n_slots, total_prefix_tokens, q, prefix_k, prefix_v, suffix_k, suffix_v,
                       doc_kv_start, doc_prefix_len, doc_active_start, doc_id, suffix_off, suffix_len, ord,
                       n_active, suffix_includes_new, o, lse, workspace, workspace_bytes, dev_status, stream);
}

int hpd_attn_decode_posorder(const hpd_geom* geom, int n_docs, int max_rows, int n_slots, int total_prefix_tokens,
                             const void* q, const void* prefix_k, const void* prefix_v,
                             const void* suffix_k, const void* suffix_v,
                             const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                             const int32_t* doc_slot_start, const int32_t* doc_id, const int32_t* active_slot,
                             const int32_t* slot_depth, const uint8_t* slot_alive, const int32_t* prefix_vis,
                             const int32_t* n_active, int suffix_includes_new,
                             void* o, float* lse,
                             void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    if (max_rows > 0 && n_docs > 0 && !active_slot) return HPD_E_ARG;
    const OrderTables ord{doc_slot_start, active_slot, slot_depth, prefix_vis, slot_alive};
    return attn_common(geom, n_docs, max_rows, n_slots, total_prefix_tokens, q, prefix_k, prefix_v, suffix_k, suffix_v,
                       doc_kv_start, doc_prefix_len, doc_active_start, doc_id, nullptr, nullptr, ord,
                       n_active, suffix_includes_new, o, lse, workspace, workspace_bytes, dev_status, stream);
}

int hpd_prefill_meta(const hpd_geom* geom, int n_docs, int n_slots, int total_tokens,
                     const int32_t* doc_prefix_len, const int32_t* doc_branch_cnt, const int32_t* slot_vis, int32_t pos_gap,
                     int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* tok_doc, int32_t* tok_pos, int32_t* tok_vis,
                     int32_t* n_tokens, void* workspace, size_t workspace_bytes, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (n_docs < 0 || n_slots < 0 || total_tokens < 0 || pos_gap < 0) return HPD_E_ARG;
    if (!doc_kv_start || !doc_slot_start || !n_tokens || !workspace || !aligned16(workspace)) return HPD_E_ARG;
    if (n_docs > 0 && (!doc_prefix_len || !doc_branch_cnt)) return HPD_E_ARG;
    if (n_slots > 0 && !slot_vis) return HPD_E_ARG;
    if (total_tokens > 0 && (!tok_doc || !tok_pos || !tok_vis)) return HPD_E_ARG;
    const int n_sm = sm_count();
    const WsLayout lay = ws_layout(*geom, n_docs, total_tokens, n_sm);
    if (workspace_bytes < lay.total) return HPD_E_WORKSPACE;
    return launch_prefill_meta(*geom, n_docs, total_tokens, pos_gap, doc_prefix_len, doc_branch_cnt, slot_vis, doc_kv_start,
                               doc_slot_start, tok_doc, tok_pos, tok_vis, n_tokens, workspace, lay, n_sm,
                               static_cast<cudaStream_t>(stream));
}

int hpd_prefill_attn(const hpd_geom* geom, int n_docs, int total_tokens,
                     const void* q, const void* prefix_k, const void* prefix_v,
                     const int32_t* doc_kv_start, const int32_t* doc_prefix_len, const int32_t* tok_doc, const int32_t* tok_vis,
                     const int32_t* n_tokens, void* o, float* lse,
                     void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream)
{
    if (total_tokens > 0 && n_docs > 0 && !tok_vis) return HPD_E_ARG;
    OrderTables ord{};
    ord.prefix_vis = tok_vis;
    // rows = tokens: a group's rows are its tokens (CSR of rows = doc_kv_start), no branch cache, max_slots = total_tokens
    return attn_common(geom, n_docs, total_tokens, total_tokens, total_tokens, q, prefix_k, prefix_v, nullptr, nullptr,
                       doc_kv_start, doc_prefix_len, doc_kv_start, tok_doc, nullptr, nullptr, ord, n_tokens, 0, o, lse,
                       workspace, workspace_bytes, dev_status, stream);
}

static int std_splits(const hpd_geom* g, int max_rows, int max_seq_len)
{
    // one persistent CTA per SM takes (sequence, block of 8 kv heads, split) items: split long sequences when the
    // batch alone gives fewer than two items per SM
    const long long items = static_cast<long long>(max_rows) * ((g->Hkv + 7) / 8);
    const long long target = 2ll * sm_count();
    if (items <= 0 || items >= target) return 1;
    long long s = (target + items - 1) / items;
    const long long by_len = max_seq_len / 256;       // at least 256 keys per split
    if (s > by_len) s = by_len;
    if (s > 32) s = 32;
    return s < 1 ? 1 : static_cast<int>(s);
}

size_t std_workspace_bytes(const hpd_geom* geom, int max_rows, int max_seq_len)
{
    if (geom_check(geom) != HPD_OK || max_rows <= 0) return 0;
    const int s = std_splits(geom, max_rows, max_seq_len);
    if (s <= 1) return 0;
    return sizeof(float) * static_cast<size_t>(max_rows) * geom->Hq * s * (geom->D + 2);
}

int std_attn_decode(const hpd_geom* geom, int max_rows, int max_seq_len, long long total_tokens, const int32_t* n_active,
                    const void* q, const void* dup_k, const void* dup_v,
                    const int64_t* seq_start, const int32_t* seq_len,
                    void* o, float* lse, void* workspace, size_t workspace_bytes, void* stream)
{
    int rc = geom_check(geom);
    if (rc != HPD_OK) return rc;
    if (max_rows < 0 || max_seq_len < 0 || total_tokens < 0) return HPD_E_ARG;
    if (total_tokens > 0x7fffffffll) return HPD_E_CAPACITY;
    if (max_rows == 0) return HPD_OK;
    if (!n_active || !q || !dup_k || !dup_v || !seq_start || !seq_len || !o) return HPD_E_ARG;
    if (!aligned16(q) || !aligned16(dup_k) || !aligned16(dup_v) || !aligned16(o)) return HPD_E_ARG;
    const int splits = std_splits(geom, max_rows, max_seq_len);
    const size_t need = std_workspace_bytes(geom, max_rows, max_seq_len);
    if (need > 0 && (!workspace || workspace_bytes < need)) return HPD_E_WORKSPACE;
    StdArgs s{};
    s.g = *geom;
    s.max_rows = max_rows; s.n_splits = splits; s.total_tokens = total_tokens; s.n_active = n_active;
    s.q = static_cast<const __nv_bfloat16*>(q);
    s.dup_k = static_cast<const __nv_bfloat16*>(dup_k); s.dup_v = static_cast<const __nv_bfloat16*>(dup_v);
    s.seq_start = seq_start; s.seq_len = seq_len;
    s.o = static_cast<__nv_bfloat16*>(o); s.lse = lse; s.part = static_cast<float*>(workspace);
    s.stream = static_cast<cudaStream_t>(stream);
    return launch_attn_std(s);
}

}  // extern "C"
