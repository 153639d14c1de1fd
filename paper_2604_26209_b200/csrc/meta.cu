// hpd_build_meta: per-step int32 bookkeeping tables and the attention work list (device side).
//
// On the caller's stream, no host synchronisation.  Steps with up to 4096 documents take one launch
// (meta_fused_kernel); larger ones three:
//   doc_scan_kernel   exclusive scans over documents (prefix tokens, slots)
//   compact_kernel    stable compaction of live slots -> row tables, rows-per-document CSR
//   plan_kernel       split-KV policy + work list for the attention kernel; -1 fill of table tails
#include "common.cuh"

namespace hpd {

namespace {

constexpr int kScanThreads = 1024;
constexpr int kCompactThreads = 256;
constexpr int kPlanThreads = 1024;

__device__ __forceinline__ int warp_incl_scan(int v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Block-wide exclusive scan of one int per thread; returns the exclusive prefix and the block total.
template <int THREADS>
__device__ __forceinline__ int block_excl_scan(int v, int* smem /* THREADS/32 + 1 */, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = warp_incl_scan(v);
    if (lane == 31) smem[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = (lane < THREADS / 32) ? smem[lane] : 0;
        int wi = warp_incl_scan(w);
        if (lane < THREADS / 32) smem[lane] = wi - w;
        if (lane == 31) smem[THREADS / 32] = wi;
    }
    __syncthreads();
    int res = incl - v + smem[warp];
    total = smem[THREADS / 32];
    __syncthreads();
    return res;
}

// Two block-wide exclusive scans at the price of one: both values (and both totals) are below 2^31, so they share one
// 64-bit word without carrying into each other.
template <int THREADS>
__device__ __forceinline__ void block_excl_scan2(int a, int b, long long* smem /* THREADS/32 + 1 */, int& ea, int& eb, int& ta, int& tb) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long v = static_cast<long long>(static_cast<unsigned>(a)) | (static_cast<long long>(b) << 32);
    long long incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) smem[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const long long w = (lane < THREADS / 32) ? smem[lane] : 0;
        long long wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const long long t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        if (lane < THREADS / 32) smem[lane] = wi - w;
        if (lane == 31) smem[THREADS / 32] = wi;
    }
    __syncthreads();
    const long long res = incl - v + smem[warp], tot = smem[THREADS / 32];
    __syncthreads();
    ea = static_cast<int>(res & 0xffffffffll); eb = static_cast<int>(res >> 32);
    ta = static_cast<int>(tot & 0xffffffffll); tb = static_cast<int>(tot >> 32);
}

__global__ void __launch_bounds__(kScanThreads)
doc_scan_kernel(int n_docs, const int32_t* __restrict__ doc_prefix_len, const int32_t* __restrict__ doc_branch_cnt,
                int32_t* __restrict__ doc_kv_start, int32_t* __restrict__ doc_slot_start)
{
    __shared__ int sm[kScanThreads / 32 + 1];
    int run_kv = 0, run_sl = 0;
    for (int base = 0; base < n_docs; base += kScanThreads) {
        int d = base + threadIdx.x;
        int l = d < n_docs ? doc_prefix_len[d] : 0;
        int c = d < n_docs ? doc_branch_cnt[d] : 0;
        int tot;
        int el = block_excl_scan<kScanThreads>(l, sm, tot);
        int tl = tot;
        int ec = block_excl_scan<kScanThreads>(c, sm, tot);
        if (d < n_docs) {
            doc_kv_start[d] = run_kv + el;
            doc_slot_start[d] = run_sl + ec;
        }
        run_kv += tl;
        run_sl += tot;
    }
    if (threadIdx.x == 0) {
        doc_kv_start[n_docs] = run_kv;
        doc_slot_start[n_docs] = run_sl;
    }
}

// Each block owns kCompactThreads consecutive slots.  The number of live slots before the block is
// recounted by the block itself (reads at most n_slots bytes from L2), which keeps the kernel free of
// any inter-block dependency.
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(int n_docs, int n_slots, int32_t suffix_cap, int32_t pos_gap,
               const int32_t* __restrict__ doc_prefix_len, const int32_t* __restrict__ doc_branch_cnt,
               const int32_t* __restrict__ doc_slot_start,
               const int32_t* __restrict__ slot_depth, const uint8_t* __restrict__ slot_alive,
               const int32_t* __restrict__ slot_vis /* nullable: anchor = document length */,
               int32_t* __restrict__ doc_active_start, int32_t* __restrict__ active_slot,
               int32_t* __restrict__ doc_id, int32_t* __restrict__ branch_start, int32_t* __restrict__ pos_id,
               int32_t* __restrict__ suffix_off, int32_t* __restrict__ suffix_len,
               int32_t* __restrict__ prefix_vis /* nullable */, int32_t* __restrict__ n_active)
{
    __shared__ int sm[kCompactThreads / 32 + 1];
    const int first = blockIdx.x * kCompactThreads;

    // live slots in [0, first)
    int cnt = 0;
    {
        const uintptr_t addr = reinterpret_cast<uintptr_t>(slot_alive);
        int head = static_cast<int>((16 - (addr & 15)) & 15);
        if (head > first) head = first;
        for (int i = threadIdx.x; i < head; i += kCompactThreads) cnt += slot_alive[i] != 0;
        const int n_vec = (first - head) / 16;
        const uint4* v = reinterpret_cast<const uint4*>(slot_alive + head);
        for (int i = threadIdx.x; i < n_vec; i += kCompactThreads) {
            uint4 w = v[i];
            cnt += __popc(__vcmpne4(w.x, 0u) & 0x01010101u) + __popc(__vcmpne4(w.y, 0u) & 0x01010101u) +
                   __popc(__vcmpne4(w.z, 0u) & 0x01010101u) + __popc(__vcmpne4(w.w, 0u) & 0x01010101u);
        }
        for (int i = head + n_vec * 16 + threadIdx.x; i < first; i += kCompactThreads) cnt += slot_alive[i] != 0;
    }
    int before;
    {
        int tot;
        block_excl_scan<kCompactThreads>(cnt, sm, tot);
        before = tot;
    }

    const int s = first + threadIdx.x;
    const int alive = (s < n_slots) && slot_alive[s] != 0;
    int tot;
    const int excl = before + block_excl_scan<kCompactThreads>(alive, sm, tot);
    const int block_end = before + tot;

    if (s < n_slots) {
        // document of slot s: last d with doc_slot_start[d] <= s (documents without slots are skipped
        // automatically because their start equals the next document's start)
        int lo = 0, hi = n_docs;           // invariant: doc_slot_start[lo] <= s < doc_slot_start[hi]
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (doc_slot_start[mid] <= s) lo = mid; else hi = mid;
        }
        const int d = lo;
        const int j = s - doc_slot_start[d];
        if (j == 0) {
            // first slot of document d: rows before it; empty documents just before d share the value
            doc_active_start[d] = excl;
            for (int e = d - 1; e >= 0 && doc_branch_cnt[e] == 0; --e) doc_active_start[e] = excl;
        }
        if (alive) {
            const int depth = slot_depth[s];
            const int anchor = slot_vis ? slot_vis[s] : doc_prefix_len[d];
            const int bs = anchor + j * pos_gap;
            active_slot[excl] = s;
            doc_id[excl] = d;
            branch_start[excl] = bs;
            pos_id[excl] = bs + depth;
            suffix_off[excl] = s * suffix_cap;
            suffix_len[excl] = depth;
            if (prefix_vis) prefix_vis[excl] = anchor;
        }
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
        *n_active = block_end;
        doc_active_start[n_docs] = block_end;
        for (int e = n_docs - 1; e >= 0 && doc_branch_cnt[e] == 0; --e) doc_active_start[e] = block_end;
    }
}

// Split-KV policy.  A work item is (document, chunk of prefix tokens, block of <= 128/G branches).
// Documents are left whole unless the step has fewer items than SMs; then the largest chunk size
// 128 * 2^k that yields at least n_sm * Hkv^-1 items is taken, subject to the partial-result and
// work-list capacities of the workspace.  Chunks below 512 tokens are never taken: a chunk's fp32
// partial result and its merge then cost more than the chunk's keys (measured: batches of 2 to 4
// prompts with 512-token documents ran 10 % faster whole than in 128- or 256-token chunks).
constexpr int kCand = 9;             // chunk sizes 128 << 0..7, then "whole document"
constexpr int kMinCand = 2;          // smallest chunk size taken: 128 << 2 tokens

__device__ __forceinline__ int chunks_of(int L, int cand) {
    if (cand == kCand - 1 || L <= 0) return 1;
    const int S = kTileN << cand;
    return (L + S - 1) / S;
}

// Longest units first.  The attention kernel hands units out in list order, a few per pipeline, so a long unit drawn
// late leaves one pipeline running after the others have finished.  Lists of up to kSortItems items (from up to
// kSortDocs documents) whose items differ in length are therefore written in descending order of an estimate of
// their duration: one per prefix key, a constant per branch-cache column of the rows (the cached lengths are not
// looked at: one pass over every row would cost more than it saves) and a constant per unit.  Ties keep document
// order, so the list is reproducible.  Longer lists stay in document order: their units are short against the launch.
constexpr int kSortItems = 2048;
constexpr int kSortDocs = 2048;
constexpr int kPlanScratchInts = kSortItems;                  // the sort keys
constexpr uint32_t kCostMax = 0xFFFFFu;                       // 20 bits of cost above 12 bits of item index
constexpr int kUnitCost = 2 * kTileN;                         // a unit's fixed part, in key columns
constexpr int kBranchCost = 16;                               // per row and q head of the group: its cached tokens' columns

// estimate of a unit's duration, in key columns: keys of the prefix chunk, rows whose branch caches the unit visits
__device__ __forceinline__ int unit_cost(int keys, int branch_rows, int G) {
    return min(kUnitCost + keys + branch_rows * G * kBranchCost, static_cast<int>(kCostMax));
}

template <int THREADS>
__device__ __forceinline__ void sort_keys_ascending(uint32_t* key, int n2 /* power of two */)
{
    for (int k = 2; k <= n2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < n2 / 2; t += THREADS) {
                const int lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const int hi = lo + j;
                const uint32_t a = key[lo], b = key[hi];
                const bool up = (lo & k) == 0;
                if ((a > b) == up) { key[lo] = b; key[hi] = a; }
            }
            __syncthreads();
        }
    }
}

// The split-KV plan, run by ONE block of THREADS threads (doc_active_start must be complete and visible).  scratch: kPlanScratchInts ints of shared memory, rank: kSortItems entries.
template <int THREADS>
__device__ __forceinline__ void plan_block(int n_docs, int G, int Hkv, int n_sm,
                                           const int32_t* doc_prefix_len, const int32_t* doc_active_start,
                                           int* scratch, uint16_t* rank,
                                           WsHeader* __restrict__ hdr, WorkItem* __restrict__ work, DocSplit* __restrict__ split,
                                           int work_cap, int part_cap)
{
    constexpr int kPlanThreads = THREADS;
    __shared__ long long sm2[kPlanThreads / 32 + 1];
    __shared__ int sm1[kPlanThreads / 32 + 1];
    __shared__ long long red[kCand * 2];
    __shared__ int s_choice, s_cost_min, s_cost_max;
    const int rows_per_block = kTileM / G;

    // the usual case first: whole documents already give one unit per SM or more -> nothing to weigh
    // (the same pass weighs the whole documents' units: only lists whose units differ in length are put in order below)
    if (threadIdx.x < kCand * 2) red[threadIdx.x] = 0;
    if (threadIdx.x == 0) { s_cost_min = 0x7fffffff; s_cost_max = 0; }
    __syncthreads();
    {
        long long whole = 0;
        int cmin = 0x7fffffff, cmax = 0;
        for (int d = threadIdx.x; d < n_docs; d += kPlanThreads) {
            const int rows = __ldcg(doc_active_start + d + 1) - __ldcg(doc_active_start + d);
            if (rows > 0) {
                const int mb = (rows + rows_per_block - 1) / rows_per_block;
                whole += mb;
                const int L = min(max(doc_prefix_len[d], 0), static_cast<int>(kCostMax));
                cmin = min(cmin, unit_cost(L, rows - (mb - 1) * rows_per_block, G));
                cmax = max(cmax, unit_cost(L, min(rows, rows_per_block), G));
            }
        }
        for (int o = 16; o > 0; o >>= 1) {
            whole += __shfl_down_sync(0xffffffffu, whole, o);
            cmin = min(cmin, __shfl_xor_sync(0xffffffffu, cmin, o));
            cmax = max(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
        }
        if ((threadIdx.x & 31) == 0 && whole) {
            atomicAdd(reinterpret_cast<unsigned long long*>(&red[0]), static_cast<unsigned long long>(whole));
            atomicMin(&s_cost_min, cmin); atomicMax(&s_cost_max, cmax);
        }
    }
    __syncthreads();
    const bool enough = red[0] * Hkv >= n_sm;
    // worth the sort only when the units differ: more than a quarter between the shortest and the longest (a split
    // list always goes through the pass below: its chunks differ)
    const bool differ = !enough || (s_cost_max > s_cost_min && (s_cost_max - s_cost_min) * 4 > s_cost_max);
    __syncthreads();
    if (enough) {
        if (threadIdx.x == 0) s_choice = kCand - 1;
    } else {
    if (threadIdx.x < kCand * 2) red[threadIdx.x] = 0;
    __syncthreads();
    {
        long long items[kCand], prow[kCand];
#pragma unroll
        for (int c = 0; c < kCand; ++c) { items[c] = 0; prow[c] = 0; }
        for (int d = threadIdx.x; d < n_docs; d += kPlanThreads) {
            const int rows = __ldcg(doc_active_start + d + 1) - __ldcg(doc_active_start + d);
            if (rows <= 0) continue;
            const int mb = (rows + rows_per_block - 1) / rows_per_block;
            const int L = doc_prefix_len[d];
#pragma unroll
            for (int c = 0; c < kCand; ++c) {
                const int ch = chunks_of(L, c);
                items[c] += static_cast<long long>(ch) * mb;
                if (ch > 1) prow[c] += static_cast<long long>(ch) * rows;
            }
        }
#pragma unroll
        for (int c = 0; c < kCand; ++c) {
            long long a = items[c], b = prow[c];
            for (int o = 16; o > 0; o >>= 1) {
                a += __shfl_down_sync(0xffffffffu, a, o);
                b += __shfl_down_sync(0xffffffffu, b, o);
            }
            if ((threadIdx.x & 31) == 0) {
                atomicAdd(reinterpret_cast<unsigned long long*>(&red[c]), static_cast<unsigned long long>(a));
                atomicAdd(reinterpret_cast<unsigned long long*>(&red[kCand + c]), static_cast<unsigned long long>(b));
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int c = kCand - 1;                              // whole documents
        while (c > kMinCand && red[c] * Hkv < n_sm) {
            const int nc = c - 1;
            if (red[nc] > work_cap || red[kCand + nc] > part_cap) break;
            c = nc;
        }
        s_choice = c;
    }
    }
    __syncthreads();
    const int cand = s_choice;

    // ---- order of the list: rank[item in document order] = its place, longest first ----
    bool sorted = false;
    if (n_docs <= kSortDocs && differ) {
        uint32_t* s_key = reinterpret_cast<uint32_t*>(scratch);
        int n_items = 0;
        for (int base = 0; base < n_docs; base += kPlanThreads) {
            const int d = base + threadIdx.x;
            int rows = 0, L = 0, mb = 0, ch = 0;
            if (d < n_docs) {
                rows = __ldcg(doc_active_start + d + 1) - __ldcg(doc_active_start + d);
                L = doc_prefix_len[d];
                if (rows > 0) { mb = (rows + rows_per_block - 1) / rows_per_block; ch = chunks_of(L, cand); }
            }
            int tot;
            const int ei = n_items + block_excl_scan<kPlanThreads>(ch * mb, sm1, tot);
            if (d < n_docs) {
                const int S = (cand == kCand - 1) ? L : (kTileN << cand);
                for (int c = 0, w = ei; c < ch; ++c) {
                    const int kc = max(min(S, L - c * S), 0);
                    for (int m = 0; m < mb; ++m, ++w) {
                        const int nr = min(rows_per_block, rows - m * rows_per_block);
                        const int cost = unit_cost(min(kc, static_cast<int>(kCostMax)), c == ch - 1 ? nr : 0, G);
                        if (w < kSortItems) s_key[w] = ((kCostMax - static_cast<uint32_t>(cost)) << 12) | static_cast<uint32_t>(w);
                    }
                }
            }
            n_items += tot;
        }
        __syncthreads();
        if (n_items > 1 && n_items <= kSortItems) {
            sorted = true;
            int n2 = 2;
            while (n2 < n_items) n2 <<= 1;
            for (int w = n_items + threadIdx.x; w < n2; w += kPlanThreads) s_key[w] = 0xFFFFFFFFu;
            __syncthreads();
            sort_keys_ascending<kPlanThreads>(s_key, n2);
            for (int i = threadIdx.x; i < n_items; i += kPlanThreads) rank[s_key[i] & 0xFFFu] = static_cast<uint16_t>(i);
            __syncthreads();
        }
    }

    // emit the work list: exclusive scans of items and partial rows per document give an item's place in document
    // order, rank[] its place in the list
    int run_items = 0, run_part = 0, any_split = 0;
    for (int base = 0; base < n_docs; base += kPlanThreads) {
        const int d = base + threadIdx.x;
        int rows = 0, L = 0, mb = 0, ch = 0;
        if (d < n_docs) {
            rows = __ldcg(doc_active_start + d + 1) - __ldcg(doc_active_start + d);
            L = doc_prefix_len[d];
            if (rows > 0) {
                mb = (rows + rows_per_block - 1) / rows_per_block;
                ch = chunks_of(L, cand);
            }
        }
        const int my_items = ch * mb;
        const int my_part = ch > 1 ? ch * rows : 0;
        int tot_i, tot_p, ei, ep;
        block_excl_scan2<kPlanThreads>(my_items, my_part, sm2, ei, ep, tot_i, tot_p);
        ei += run_items; ep += run_part;
        if (d < n_docs) {
            split[d].part_base = ch > 1 ? ep : -1;
            split[d].n_chunks = ch;
            if (ch > 1) any_split = 1;
            const int S = (cand == kCand - 1) ? L : (kTileN << cand);
            int w = ei;
            for (int c = 0; c < ch; ++c) {
                const int kb = c * S;
                const int kc = min(S, L - kb);
                for (int m = 0; m < mb; ++m, ++w) {
                    WorkItem it;
                    it.doc = d;
                    it.key_begin = kb;
                    it.key_count = kc > 0 ? kc : 0;
                    it.row_begin = m * rows_per_block;
                    it.row_count = min(rows_per_block, rows - it.row_begin);
                    it.part_base = ch > 1 ? ep + c * rows : -1;
                    it.with_suffix = (c == ch - 1);
                    it.pad = 0;
                    work[sorted ? static_cast<int>(rank[w]) : w] = it;
                }
            }
        }
        run_items += tot_i;
        run_part += tot_p;
    }
    const int split_any = __syncthreads_or(any_split);
    if (threadIdx.x == 0) {
        hdr->n_work = run_items;
        hdr->chunk_tokens = (cand == kCand - 1) ? 0 : (kTileN << cand);
        hdr->n_part_rows = run_part;
        hdr->any_split = split_any;
        hdr->longest_first = sorted ? 1 : 0;
        hdr->ticket = 0;
        hdr->finished = 0;
        hdr->work_cap = work_cap;
        hdr->part_cap = part_cap;
    }
}

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(int n_docs, int n_slots, int G, int Hkv, int n_sm,
            const int32_t* __restrict__ doc_prefix_len, const int32_t* __restrict__ doc_active_start,
            const int32_t* __restrict__ n_active,
            int32_t* __restrict__ active_slot, int32_t* __restrict__ doc_id, int32_t* __restrict__ branch_start,
            int32_t* __restrict__ pos_id, int32_t* __restrict__ suffix_off, int32_t* __restrict__ suffix_len,
            int32_t* __restrict__ prefix_vis /* nullable */,
            WsHeader* __restrict__ hdr, WorkItem* __restrict__ work, DocSplit* __restrict__ split,
            int work_cap, int part_cap)
{
    if (blockIdx.x > 0) {
        // tail fill: entries past n_active read -1 in every per-row table
        const int na = *n_active;
        for (int i = na + (blockIdx.x - 1) * kPlanThreads + threadIdx.x; i < n_slots; i += (gridDim.x - 1) * kPlanThreads) {
            active_slot[i] = -1; doc_id[i] = -1; branch_start[i] = -1;
            pos_id[i] = -1; suffix_off[i] = -1; suffix_len[i] = -1;
            if (prefix_vis) prefix_vis[i] = -1;
        }
        return;
    }
    __shared__ int s_scratch[kPlanScratchInts];
    __shared__ uint16_t s_rank[kSortItems];
    plan_block<kPlanThreads>(n_docs, G, Hkv, n_sm, doc_prefix_len, doc_active_start, s_scratch, s_rank,
                             hdr, work, split, work_cap, part_cap);
}

// ---------------------------------------------------------------------------------------------------------------
// All of the above in ONE launch, for steps with at most kFusedDocs documents (the usual case).  Every block of 256
// slots repeats the two cheap global steps for itself -- the scans over documents (kept in shared memory) and the
// count of live slots before it and in total -- so that it can place its live slots' rows, its dead slots' -1 entries
// at the tail, and its documents' CSR entries without waiting for any other block.  The block that finishes last
// (counted in the workspace header) sees every block's CSR entries and writes the split-KV plan.
// ---------------------------------------------------------------------------------------------------------------
constexpr int kFusedDocs = 4096;
constexpr int kFusedThreads = 256;

__device__ __forceinline__ int count_alive(const uint8_t* __restrict__ slot_alive, int begin, int end)
{
    // live slots in [begin, end), 16 bytes at a time where the address allows
    int cnt = 0;
    const uintptr_t addr = reinterpret_cast<uintptr_t>(slot_alive + begin);
    int head = static_cast<int>((16 - (addr & 15)) & 15);
    if (head > end - begin) head = end - begin;
    for (int i = begin + threadIdx.x; i < begin + head; i += blockDim.x) cnt += slot_alive[i] != 0;
    const int n_vec = (end - begin - head) / 16;
    const uint4* v = reinterpret_cast<const uint4*>(slot_alive + begin + head);
    for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
        const uint4 w = v[i];
        cnt += __popc(__vcmpne4(w.x, 0u) & 0x01010101u) + __popc(__vcmpne4(w.y, 0u) & 0x01010101u) +
               __popc(__vcmpne4(w.z, 0u) & 0x01010101u) + __popc(__vcmpne4(w.w, 0u) & 0x01010101u);
    }
    for (int i = begin + head + n_vec * 16 + threadIdx.x; i < end; i += blockDim.x) cnt += slot_alive[i] != 0;
    return cnt;
}

__global__ void __launch_bounds__(kFusedThreads)
meta_fused_kernel(int n_docs, int n_slots, int32_t suffix_cap, int32_t pos_gap, int G, int Hkv, int n_sm,
                  const int32_t* __restrict__ doc_prefix_len, const int32_t* __restrict__ doc_branch_cnt,
                  const int32_t* __restrict__ slot_depth, const uint8_t* __restrict__ slot_alive,
                  const int32_t* __restrict__ slot_vis /* nullable */,
                  int32_t* __restrict__ doc_kv_start, int32_t* __restrict__ doc_slot_start, int32_t* doc_active_start,
                  int32_t* __restrict__ active_slot, int32_t* __restrict__ doc_id, int32_t* __restrict__ branch_start,
                  int32_t* __restrict__ pos_id, int32_t* __restrict__ suffix_off, int32_t* __restrict__ suffix_len,
                  int32_t* __restrict__ prefix_vis /* nullable */,
                  int32_t* __restrict__ n_active, WsHeader* hdr, WorkItem* __restrict__ work, DocSplit* __restrict__ split,
                  int work_cap, int part_cap)
{
    __shared__ int sm[kFusedThreads / 32 + 1];
    __shared__ long long sm2[kFusedThreads / 32 + 1];
    __shared__ int s_slot_start[kFusedDocs + 1];
    __shared__ int s_last;
    const int first = blockIdx.x * kFusedThreads;
    // this thread's slot: its flags are asked for now and used after the scans
    const int s = first + threadIdx.x;
    const int alive = (s < n_slots) && slot_alive[s] != 0;
    const int depth = s < n_slots ? slot_depth[s] : 0;
    const int my_vis = (slot_vis && s < n_slots) ? slot_vis[s] : 0;

    // ---- scans over documents: slot starts stay in shared memory, block 0 also publishes both scans ----
    {
        int run_kv = 0, run_sl = 0;
        for (int base = 0; base < n_docs; base += kFusedThreads) {
            const int d = base + threadIdx.x;
            const int l = d < n_docs ? doc_prefix_len[d] : 0;
            const int c = d < n_docs ? doc_branch_cnt[d] : 0;
            int tot_l, tot_c, el, ec;
            block_excl_scan2<kFusedThreads>(l, c, sm2, el, ec, tot_l, tot_c);
            if (d < n_docs) {
                s_slot_start[d] = run_sl + ec;
                if (blockIdx.x == 0) { doc_kv_start[d] = run_kv + el; doc_slot_start[d] = run_sl + ec; }
            }
            run_kv += tot_l;
            run_sl += tot_c;
        }
        if (threadIdx.x == 0) {
            s_slot_start[n_docs] = run_sl;
            if (blockIdx.x == 0) { doc_kv_start[n_docs] = run_kv; doc_slot_start[n_docs] = run_sl; }
        }
    }
    // ---- live slots before this block and in total ----
    int before, total;
    {
        int e0, e1, after;
        block_excl_scan2<kFusedThreads>(count_alive(slot_alive, 0, min(first, n_slots)),
                                        count_alive(slot_alive, min(first, n_slots), n_slots), sm2, e0, e1, before, after);
        total = before + after;
    }
    int tot;
    const int excl = before + block_excl_scan<kFusedThreads>(alive, sm, tot);

    if (s < n_slots) {
        int lo = 0, hi = n_docs;           // invariant: slot_start[lo] <= s < slot_start[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_slot_start[mid] <= s) lo = mid; else hi = mid;
        }
        const int d = lo;
        const int j = s - s_slot_start[d];
        if (j == 0) {
            // first slot of document d: rows before it; documents without slots just before d share the value
            doc_active_start[d] = excl;
            for (int e = d - 1; e >= 0 && s_slot_start[e + 1] == s_slot_start[e]; --e) doc_active_start[e] = excl;
        }
        if (alive) {
            const int anchor = slot_vis ? my_vis : doc_prefix_len[d];
            const int bs = anchor + j * pos_gap;
            active_slot[excl] = s;
            doc_id[excl] = d;
            branch_start[excl] = bs;
            pos_id[excl] = bs + depth;
            suffix_off[excl] = s * suffix_cap;
            suffix_len[excl] = depth;
            if (prefix_vis) prefix_vis[excl] = anchor;
        } else {
            const int t = total + (s - excl);            // the dead slots fill the tail of every row table with -1
            active_slot[t] = -1; doc_id[t] = -1; branch_start[t] = -1;
            pos_id[t] = -1; suffix_off[t] = -1; suffix_len[t] = -1;
            if (prefix_vis) prefix_vis[t] = -1;
        }
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
        *n_active = total;
        doc_active_start[n_docs] = total;
        for (int e = n_docs - 1; e >= 0 && s_slot_start[e + 1] == s_slot_start[e]; --e) doc_active_start[e] = total;
    }

    // ---- the block that finishes last writes the plan ----
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&hdr->finished, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    static_assert(kFusedDocs + 1 >= kPlanScratchInts, "the document scan's shared array doubles as the plan's scratch");
    __shared__ uint16_t s_rank[kSortItems];
    plan_block<kFusedThreads>(n_docs, G, Hkv, n_sm, doc_prefix_len, doc_active_start, s_slot_start, s_rank,
                              hdr, work, split, work_cap, part_cap);
}

// ---------------------------------------------------------------------------------------------------------------
// First inference step (Sec. 4.3.2): the rows are the prompt tokens themselves.  One launch writes, per token, its
// group, Algorithm 2's position ID (a gap of pos_gap behind every attribute key: t + pos_gap * #{slots whose key ends
// before t}) and its causal bound t + 1; and the attention's work list: (group, block of 128/G tokens) against the
// keys [0, end of the block) -- later keys are masked for every row of the block, so they are not visited at all.
// ---------------------------------------------------------------------------------------------------------------
constexpr int kPrefillDocs = 2048;
constexpr int kPrefillThreads = 256;

__global__ void __launch_bounds__(kPrefillThreads)
prefill_meta_kernel(int n_docs, int G, int32_t pos_gap,
                    const int32_t* __restrict__ doc_prefix_len, const int32_t* __restrict__ doc_branch_cnt,
                    const int32_t* __restrict__ slot_vis,
                    int32_t* __restrict__ doc_kv_start, int32_t* __restrict__ doc_slot_start,
                    int32_t* __restrict__ tok_doc, int32_t* __restrict__ tok_pos, int32_t* __restrict__ tok_vis,
                    int32_t* __restrict__ n_tokens, WsHeader* __restrict__ hdr, WorkItem* __restrict__ work,
                    DocSplit* __restrict__ split, int work_cap, int part_cap)
{
    __shared__ int sm[kPrefillThreads / 32 + 1];
    __shared__ int s_kv[kPrefillDocs + 1], s_slot[kPrefillDocs + 1], s_item[kPrefillDocs + 1];
    const int rpb = kTileM / G;                      // tokens per row block
    int run_kv = 0, run_sl = 0, run_it = 0;
    for (int base = 0; base < n_docs; base += kPrefillThreads) {
        const int d = base + threadIdx.x;
        const int l = d < n_docs ? doc_prefix_len[d] : 0;
        const int c = d < n_docs ? doc_branch_cnt[d] : 0;
        const int it = (l + rpb - 1) / rpb;
        int tl, tc, ti;
        const int el = block_excl_scan<kPrefillThreads>(l, sm, tl);
        const int ec = block_excl_scan<kPrefillThreads>(c, sm, tc);
        const int ei = block_excl_scan<kPrefillThreads>(it, sm, ti);
        if (d < n_docs) { s_kv[d] = run_kv + el; s_slot[d] = run_sl + ec; s_item[d] = run_it + ei; }
        run_kv += tl; run_sl += tc; run_it += ti;
    }
    if (threadIdx.x == 0) { s_kv[n_docs] = run_kv; s_slot[n_docs] = run_sl; s_item[n_docs] = run_it; }
    __syncthreads();
    const int n_tok = run_kv, n_items = min(run_it, work_cap);
    auto doc_of = [&](const int* start, int x) {      // last d with start[d] <= x (empty groups share a start and are skipped)
        int lo = 0, hi = n_docs;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (start[mid] <= x) lo = mid; else hi = mid;
        }
        return lo;
    };
    const int stride = gridDim.x * kPrefillThreads;
    for (int x = blockIdx.x * kPrefillThreads + threadIdx.x; x < n_tok; x += stride) {
        const int d = doc_of(s_kv, x);
        const int t = x - s_kv[d];
        int lo = s_slot[d], hi = s_slot[d + 1];       // slots of the group whose key ends before token t: slot_vis <= t
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (slot_vis[mid] <= t) lo = mid + 1; else hi = mid;
        }
        tok_doc[x] = d;
        tok_pos[x] = t + pos_gap * (lo - s_slot[d]);
        tok_vis[x] = t + 1;
    }
    for (int x = blockIdx.x * kPrefillThreads + threadIdx.x; x < n_items; x += stride) {
        const int d = doc_of(s_item, x);
        const int m = x - s_item[d];
        const int L = s_kv[d + 1] - s_kv[d];
        WorkItem it;
        it.doc = d; it.key_begin = 0; it.key_count = min(L, (m + 1) * rpb);
        it.part_base = -1; it.row_begin = m * rpb; it.row_count = min(rpb, L - m * rpb);
        it.with_suffix = 0; it.pad = 0;
        work[x] = it;
    }
    if (blockIdx.x == 0) {
        for (int d = threadIdx.x; d <= n_docs; d += kPrefillThreads) {
            doc_kv_start[d] = s_kv[d];
            doc_slot_start[d] = s_slot[d];
            if (d < n_docs) { split[d].part_base = -1; split[d].n_chunks = 1; }
        }
        if (threadIdx.x == 0) {
            *n_tokens = n_tok;
            hdr->n_work = n_items; hdr->chunk_tokens = 0; hdr->n_part_rows = 0; hdr->any_split = 0;
            hdr->ticket = 0; hdr->finished = 0; hdr->work_cap = work_cap; hdr->part_cap = part_cap; hdr->longest_first = 0;
        }
    }
}

}  // namespace

int launch_prefill_meta(const hpd_geom& g, int n_docs, int total_tokens, int32_t pos_gap, const int32_t* doc_prefix_len,
                        const int32_t* doc_branch_cnt, const int32_t* slot_vis, int32_t* doc_kv_start, int32_t* doc_slot_start,
                        int32_t* tok_doc, int32_t* tok_pos, int32_t* tok_vis, int32_t* n_tokens, void* workspace,
                        const WsLayout& lay, int n_sm, cudaStream_t stream)
{
    if (n_docs > kPrefillDocs) return HPD_E_CAPACITY;
    char* ws = static_cast<char*>(workspace);
    int blocks = (total_tokens + kPrefillThreads - 1) / kPrefillThreads;
    if (blocks < 1) blocks = 1;
    if (blocks > 4 * n_sm) blocks = 4 * n_sm;
    prefill_meta_kernel<<<blocks, kPrefillThreads, 0, stream>>>(
        n_docs, g.Hq / g.Hkv, pos_gap, doc_prefix_len, doc_branch_cnt, slot_vis, doc_kv_start, doc_slot_start, tok_doc, tok_pos,
        tok_vis, n_tokens, reinterpret_cast<WsHeader*>(ws), reinterpret_cast<WorkItem*>(ws + lay.off_work),
        reinterpret_cast<DocSplit*>(ws + lay.off_split), lay.work_cap, lay.part_cap);
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

WsLayout ws_layout(const hpd_geom& g, int max_docs, int max_slots, int n_sm)
{
    WsLayout l{};
    const int G = g.Hq / g.Hkv;
    const long long blocks = (static_cast<long long>(max_slots) * G + kTileM - 1) / kTileM;
    long long work_cap = 2ll * max_docs + 4 * (blocks + 1) + 2ll * n_sm + 64;
    long long part_cap = 2ll * max_slots + 1024;
    if (work_cap > 0x7fffffffll) work_cap = 0x7fffffffll;
    if (part_cap > 0x7fffffffll) part_cap = 0x7fffffffll;
    l.work_cap = static_cast<int32_t>(work_cap);
    l.part_cap = static_cast<int32_t>(part_cap);
    auto up = [](size_t x) { return (x + 255) & ~static_cast<size_t>(255); };
    size_t off = up(sizeof(WsHeader));
    l.off_work = off;  off = up(off + sizeof(WorkItem) * static_cast<size_t>(l.work_cap));
    l.off_split = off; off = up(off + sizeof(DocSplit) * static_cast<size_t>(max_docs > 0 ? max_docs : 1));
    l.off_ml = off;    off = up(off + sizeof(float) * 2 * static_cast<size_t>(l.part_cap) * g.Hq);
    l.off_o = off;     off = up(off + sizeof(float) * static_cast<size_t>(l.part_cap) * g.Hq * g.D);
    l.total = off;
    return l;
}

int launch_build_meta(const hpd_geom& g, int n_docs, int n_slots, const int32_t* doc_prefix_len,
                      const int32_t* doc_branch_cnt, const int32_t* slot_depth, const uint8_t* slot_alive,
                      int32_t pos_gap, int32_t* doc_kv_start, int32_t* doc_slot_start, int32_t* doc_active_start,
                      int32_t* active_slot, int32_t* doc_id, int32_t* branch_start, int32_t* pos_id,
                      int32_t* suffix_off, int32_t* suffix_len, int32_t* n_active, void* workspace,
                      const WsLayout& lay, int n_sm, int32_t* /*dev_status*/, cudaStream_t stream,
                      const int32_t* slot_vis, int32_t* prefix_vis)
{
    char* ws = static_cast<char*>(workspace);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws);
    WorkItem* work = reinterpret_cast<WorkItem*>(ws + lay.off_work);
    DocSplit* split = reinterpret_cast<DocSplit*>(ws + lay.off_split);

    if (n_docs <= kFusedDocs) {
        // the header's arrival counter must read 0 at launch: plan_block leaves it so (hdr->finished = 0) after every
        // step, and the very first step on a workspace finds whatever the caller's allocation holds -- clear it
        HPD_CUDA_TRY(cudaMemsetAsync(&hdr->finished, 0, sizeof(hdr->finished), stream));
        const int blocks = n_slots > 0 ? (n_slots + kFusedThreads - 1) / kFusedThreads : 1;
        meta_fused_kernel<<<blocks, kFusedThreads, 0, stream>>>(
            n_docs, n_slots, g.suffix_cap, pos_gap, g.Hq / g.Hkv, g.Hkv, n_sm, doc_prefix_len, doc_branch_cnt, slot_depth,
            slot_alive, slot_vis, doc_kv_start, doc_slot_start, doc_active_start, active_slot, doc_id, branch_start, pos_id,
            suffix_off, suffix_len, prefix_vis, n_active, hdr, work, split, lay.work_cap, lay.part_cap);
        HPD_CUDA_TRY(cudaGetLastError());
        return HPD_OK;
    }
    doc_scan_kernel<<<1, kScanThreads, 0, stream>>>(n_docs, doc_prefix_len, doc_branch_cnt, doc_kv_start, doc_slot_start);
    const int cblocks = n_slots > 0 ? (n_slots + kCompactThreads - 1) / kCompactThreads : 1;
    compact_kernel<<<cblocks, kCompactThreads, 0, stream>>>(
        n_docs, n_slots, g.suffix_cap, pos_gap, doc_prefix_len, doc_branch_cnt, doc_slot_start, slot_depth, slot_alive,
        slot_vis, doc_active_start, active_slot, doc_id, branch_start, pos_id, suffix_off, suffix_len, prefix_vis, n_active);
    int fill_blocks = (n_slots + kPlanThreads * 4 - 1) / (kPlanThreads * 4);
    if (fill_blocks < 1) fill_blocks = 1;
    if (fill_blocks > 64) fill_blocks = 64;
    plan_kernel<<<1 + fill_blocks, kPlanThreads, 0, stream>>>(
        n_docs, n_slots, g.Hq / g.Hkv, g.Hkv, n_sm, doc_prefix_len, doc_active_start, n_active, active_slot, doc_id,
        branch_start, pos_id, suffix_off, suffix_len, prefix_vis, hdr, work, split, lay.work_cap, lay.part_cap);
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

}  // namespace hpd
