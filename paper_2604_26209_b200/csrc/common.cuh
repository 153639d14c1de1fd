// Shared declarations of the libhpd translation units (device side of the C ABI in include/hpd.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hpd.h"

namespace hpd {

// ---------------------------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------------------------
void set_last_cuda_error(cudaError_t e);

#define HPD_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) {                            \
            ::hpd::set_last_cuda_error(e__);                 \
            return HPD_E_CUDA;                               \
        }                                                    \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int kMaxDevices = 64;      // per-device caches (SM count, kernel attributes) are indexed by device ordinal

int geom_check(const hpd_geom* g);   // HPD_OK or HPD_E_GEOM / HPD_E_ARG
int current_device();                // ordinal of the calling thread's current device (0 if it cannot be queried)
int sm_count();                      // SMs of the current device (148 if it cannot be queried)

// hpd_attn_decode packs the cached tokens of the up to 128/G branches of a unit back to back and stores a branch's
// first column and length as 16-bit numbers (the limit is stated for slab sizes rounded up to a multiple of four).
constexpr long long kMaxPackedColumns = 65535;
inline long long attn_packed_columns(const hpd_geom& g)
{
    const long long G = g.Hq / g.Hkv;
    return (128 / G) * ((static_cast<long long>(g.suffix_cap) + 3) & ~3ll);
}

// ---------------------------------------------------------------------------------------------
// Workspace of one decode step.  hpd_build_meta writes the header and the work list;
// hpd_attn_decode consumes them and uses the partial area when a document's prefix is
// split over several work items.
//
//   [ WsHeader | WorkItem[work_cap] | DocSplit[max_docs] | part_ml | part_o ]
// ---------------------------------------------------------------------------------------------
constexpr int kTileM = 128;          // query rows of one tensor-core tile (rows = branches x G)
constexpr int kTileN = 128;          // keys of one tile

struct WsHeader {
    int32_t n_work;          // work items of this step
    int32_t chunk_tokens;    // prefix tokens per work item (0: documents are not split)
    int32_t n_part_rows;     // partial rows in use
    int32_t any_split;       // 1 if some document is split (the merge kernel has work)
    uint32_t ticket;         // dynamic scheduler: next work item
    uint32_t finished;       // CTAs that have drained the list (the last one resets both)
    int32_t work_cap, part_cap;
    int32_t longest_first;   // 1 if the list is in descending order of the units' estimated duration
    int32_t pad[23];
};
static_assert(sizeof(WsHeader) == 128, "header size");

// One unit of the attention kernel: rows [row_begin, row_begin+row_count) of document `doc`
// (indices relative to the document's first row) against prefix tokens
// [key_begin, key_begin+key_count) of that document, plus the rows' branch caches when
// with_suffix is set.  part_base < 0: the item produces the final output of its rows.
struct WorkItem {
    int32_t doc, key_begin, key_count, part_base;
    int32_t row_begin, row_count, with_suffix, pad;
};
static_assert(sizeof(WorkItem) == 32, "work item size");

struct DocSplit {                    // per document: where its partial results live
    int32_t part_base;               // first partial row of chunk 0 (chunk c: + c * n_rows(doc)), -1 if unsplit
    int32_t n_chunks;
};

struct WsLayout {
    size_t off_work, off_split, off_ml, off_o, total;
    int32_t work_cap, part_cap;
};
WsLayout ws_layout(const hpd_geom& g, int max_docs, int max_slots, int n_sm);

// ---------------------------------------------------------------------------------------------
// launches (one per translation unit)
// ---------------------------------------------------------------------------------------------
struct AttnArgs {
    hpd_geom g;
    int n_docs, max_rows, n_slots, total_prefix;
    const __nv_bfloat16 *q, *prefix_k, *prefix_v, *suffix_k, *suffix_v;
    const int32_t *doc_kv_start, *doc_prefix_len, *doc_active_start, *doc_id, *suffix_off, *suffix_len, *n_active;
    int suffix_extra;                // 1: suffix_len+1 cached tokens are visible
    // position-order mode only (all null otherwise): slot tables of the groups and the rows' visible prefix lengths
    const int32_t *doc_slot_start, *active_slot, *slot_depth, *prefix_vis;
    const uint8_t* slot_alive;
    // third sharing level only (all null otherwise): block K/V [total_block, Hkv, D], block of each document, blocks' rows
    const __nv_bfloat16 *block_k, *block_v;
    const int32_t *doc_block, *block_kv_start, *block_len;
    int total_block;
    __nv_bfloat16* o;
    float* lse;
    void* workspace;
    WsLayout lay;
    int32_t* dev_status;
    cudaStream_t stream;
};

// Standard batched decode over private per-sequence K/V copies (std_attn_decode).
struct StdArgs {
    hpd_geom g;
    int max_rows, n_splits;
    long long total_tokens;          // token rows of dup_k / dup_v
    const int32_t* n_active;
    const __nv_bfloat16 *q, *dup_k, *dup_v;
    const int64_t* seq_start;        // per row: first token row of the sequence
    const int32_t* seq_len;          // per row
    __nv_bfloat16* o;
    float* lse;
    float* part;                     // n_splits > 1: [max_rows, Hq, n_splits, D+2]
    cudaStream_t stream;
};

int launch_build_meta(const hpd_geom& g, int n_docs, int n_slots, const int32_t* doc_prefix_len,
                      const int32_t* doc_branch_cnt, const int32_t* slot_depth, const uint8_t* slot_alive,
                      int32_t pos_gap, int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                      int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                      int32_t* suffix_off, int32_t* suffix_len, int32_t* n_active, void* workspace,
                      const WsLayout& lay, int n_sm, int32_t* dev_status, cudaStream_t stream,
                      const int32_t* slot_vis = nullptr, int32_t* prefix_vis = nullptr);
int launch_prefill_meta(const hpd_geom& g, int n_docs, int total_tokens, int32_t pos_gap, const int32_t* doc_prefix_len,
                        const int32_t* doc_branch_cnt, const int32_t* slot_vis, int32_t* doc_kv_start, int32_t* doc_slot_start,
                        int32_t* tok_doc, int32_t* tok_pos, int32_t* tok_vis, int32_t* n_tokens, void* workspace,
                        const WsLayout& lay, int n_sm, cudaStream_t stream);
int launch_rope(const hpd_geom& g, int max_rows, const int32_t* n_active, const int32_t* pos_id,
                __nv_bfloat16* q, __nv_bfloat16* k_new, cudaStream_t stream);
int launch_kv_append(const hpd_geom& g, int max_rows, int n_slots, const int32_t* n_active, const int32_t* suffix_off,
                     const int32_t* suffix_len, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new,
                     __nv_bfloat16* suffix_k, __nv_bfloat16* suffix_v, int32_t* dev_status, cudaStream_t stream);
int launch_rope_append(const hpd_geom& g, int max_rows, int n_slots, const int32_t* n_active, const int32_t* pos_id,
                       const int32_t* suffix_off, const int32_t* suffix_len, __nv_bfloat16* q, __nv_bfloat16* k_new,
                       const __nv_bfloat16* v_new, __nv_bfloat16* suffix_k, __nv_bfloat16* suffix_v, int32_t* dev_status,
                       cudaStream_t stream);
int launch_advance(const hpd_geom& g, int max_rows, const int32_t* n_active, const int32_t* active_slot,
                   const int32_t* token_id, int32_t delimiter_id, int32_t* slot_depth, uint8_t* slot_alive,
                   int32_t* n_alive, cudaStream_t stream);
int launch_merge_lse(const hpd_geom& g, int max_rows, const int32_t* n_active, const __nv_bfloat16* o_a, const float* lse_a,
                     const __nv_bfloat16* o_b, const float* lse_b, __nv_bfloat16* o, float* lse, cudaStream_t stream);
int launch_attn_std(const StdArgs& a);         // TMA ring + warp-level tensor-core instructions
int launch_attn_tc(const AttnArgs& a);       // tcgen05 / TMA kernel

// ---------------------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace hpd
