// hpd_rope, hpd_kv_append and their fusion hpd_rope_append: the streaming kernels around the attention.
//
// All are pure HBM streaming (read + write of the step's new q/k/v rows); one CTA per four rows (rotation) or per
// row (append), 16-byte accesses, grid sized by max_rows with an early exit on the device-side row count.
// The fused kernel rotates q and k in place, and while a rotated key chunk is still in registers also
// stores it to the row's slot in the branch cache, then copies the value row there: one launch and one
// read of k instead of two, the same bits as the two separate calls.
#include "common.cuh"

namespace hpd {

namespace {

constexpr int kRopeThreads = 256;
constexpr int kRopeRows = 4;                         // rows per CTA: 4 x 64 angles give every thread one to evaluate

// One CTA per four rows.  Every thread first asks for its share of the rows' q / k / v chunks (up to ten 16-byte loads in
// flight per thread), then evaluates one of the rows' D/2 (cos, sin) pairs; they are kept in shared memory as fp32 and
// applied to all Hq + Hkv heads: a thread rotates 8 pairs at a time from one 16-byte chunk of the low half and one of the high half.
// Angles reach thousands of radians, where an fp32 product pos * inv_freq already loses ~1e-4 rad: the product and its
// reduction to [-pi, pi] are taken in fp64 (inverse frequencies computed in fp64 on the host, 2*pi split in two doubles),
// and only the reduced angle goes through the fp32 sine and cosine.
struct InvFreq { double f[64]; };                    // theta^(-2i/D), i < D/2 <= 64

struct AppendDst {                                   // fused kernel only: where the row's key and value go
    int32_t suffix_cap;
    int64_t cache_rows;
    const int32_t *suffix_off, *suffix_len;
    const __nv_bfloat16* v_new;
    __nv_bfloat16 *suffix_k, *suffix_v;
    int32_t* dev_status;
};

template <int D, bool FUSED>
__global__ void __launch_bounds__(kRopeThreads)
rope_kernel(int Hq, int Hkv, const InvFreq inv_freq, const int32_t* __restrict__ n_active,
            const int32_t* __restrict__ pos_id, __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k_new,
            const AppendDst ad)
{
    constexpr int HALF = D / 2;
    constexpr int CHUNKS = HALF / 8;                 // 16-byte chunks per half
    constexpr int R = kRopeRows;
    constexpr int B = 5;                             // items a thread has in flight (the usual 32 + 8 heads of 128: all of them)
    static_assert(R * HALF <= kRopeThreads, "one thread per angle of the CTA's rows");
    __shared__ float cs[R][HALF], sn[R][HALF];
    __shared__ long long s_dst[R];
    const int r0 = blockIdx.x * R;
    const int na = *n_active;
    if (r0 >= na) return;
    const int nr = min(R, na - r0);

    // ---- every load that needs no angle is issued first: positions, slot tables, the first items of q / k / v ----
    const int ar = threadIdx.x / HALF, ai = threadIdx.x % HALF;      // this thread's angle: row ar of the CTA, pair ai
    const int pos = ar < nr ? pos_id[r0 + ar] : 0;
    int t_len = 0;
    int64_t t_off = 0;
    if constexpr (FUSED) {
        if (threadIdx.x < nr) { t_len = ad.suffix_len[r0 + threadIdx.x]; t_off = ad.suffix_off[r0 + threadIdx.x]; }
    }
    const int items = (Hq + Hkv) * CHUNKS;           // 16-byte chunk pairs of one row
    const int total = nr * items;
    auto chunk_ptr = [&](int it, int& row, int& head, int& ch) -> uint4* {
        row = it / items;
        const int local = it - row * items;
        head = local / CHUNKS; ch = local - head * CHUNKS;
        __nv_bfloat16* base = head < Hq ? q + (static_cast<int64_t>(r0 + row) * Hq + head) * D
                                        : k_new + (static_cast<int64_t>(r0 + row) * Hkv + (head - Hq)) * D;
        return reinterpret_cast<uint4*>(base) + ch;
    };
    uint4 lo[B], hi[B];
#pragma unroll
    for (int k = 0; k < B; ++k) {
        const int it = threadIdx.x + k * kRopeThreads;
        if (it < total) {
            int row, head, ch;
            const uint4* pl = chunk_ptr(it, row, head, ch);
            lo[k] = pl[0]; hi[k] = pl[CHUNKS];
        }
    }
    // fused: the value rows' 16-byte pieces
    const int row_u4 = Hkv * D / 8;
    const int v_total = FUSED ? nr * row_u4 : 0;
    uint4 vv[2];
    if constexpr (FUSED) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int it = threadIdx.x + k * kRopeThreads;
            if (it < v_total) vv[k] = reinterpret_cast<const uint4*>(ad.v_new)[static_cast<int64_t>(r0) * row_u4 + it];
        }
    }

    // ---- angles, and where each row goes in the branch cache (-1: slab full or table entry out of range -> status bit, no write) ----
    if (ar < nr) {
        const double ang = static_cast<double>(pos) * inv_freq.f[ai];
        const double k = rint(ang * 0.15915494309189535);                       // turns
        double r = fma(-k, 6.283185307179586, ang);                             // minus k * 2*pi (high part, then the rest)
        r = fma(-k, 2.4492935982947064e-16, r);
        float s, c;
        sincosf(static_cast<float>(r), &s, &c);
        cs[ar][ai] = c;
        sn[ar][ai] = s;
    }
    if constexpr (FUSED) {
        if (threadIdx.x < nr) {
            long long dst = -1;
            if (t_len >= ad.suffix_cap || t_len < 0) {
                if (ad.dev_status) atomicOr(ad.dev_status, HPD_S_OVERFLOW);
            } else if (t_off < 0 || t_off + t_len >= ad.cache_rows) {
                if (ad.dev_status) atomicOr(ad.dev_status, HPD_S_BAD_TABLE);
            } else {
                dst = t_off + t_len;
            }
            s_dst[threadIdx.x] = dst;
        }
    }
    __syncthreads();

    // ---- rotate in place; the fused kernel also stores the rotated key chunks to the cache while they are in registers ----
    for (int base = 0; base < total; base += B * kRopeThreads) {
        if (base > 0) {
#pragma unroll
            for (int k = 0; k < B; ++k) {
                const int it = base + threadIdx.x + k * kRopeThreads;
                if (it < total) {
                    int row, head, ch;
                    const uint4* pl = chunk_ptr(it, row, head, ch);
                    lo[k] = pl[0]; hi[k] = pl[CHUNKS];
                }
            }
        }
#pragma unroll
        for (int k = 0; k < B; ++k) {
            const int it = base + threadIdx.x + k * kRopeThreads;
            if (it >= total) continue;
            int row, head, ch;
            uint4* pl = chunk_ptr(it, row, head, ch);
            uint32_t* l = reinterpret_cast<uint32_t*>(&lo[k]);
            uint32_t* h = reinterpret_cast<uint32_t*>(&hi[k]);
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const int i = ch * 8 + w * 2;
                const float a0 = bf16lo(l[w]), a1 = bf16hi(l[w]);
                const float b0 = bf16lo(h[w]), b1 = bf16hi(h[w]);
                const float c0 = cs[row][i], s0 = sn[row][i], c1 = cs[row][i + 1], s1 = sn[row][i + 1];
                l[w] = pack_bf16(fmaf(a0, c0, -b0 * s0), fmaf(a1, c1, -b1 * s1));
                h[w] = pack_bf16(fmaf(b0, c0, a0 * s0), fmaf(b1, c1, a1 * s1));
            }
            pl[0] = lo[k];
            pl[CHUNKS] = hi[k];
            if constexpr (FUSED) {
                const long long dst_row = s_dst[row];
                if (head >= Hq && dst_row >= 0) {
                    uint4* cd = reinterpret_cast<uint4*>(ad.suffix_k + (dst_row * Hkv + (head - Hq)) * D);
                    cd[ch] = lo[k];
                    cd[CHUNKS + ch] = hi[k];
                }
            }
        }
    }
    if constexpr (FUSED) {
        for (int base = 0; base < v_total; base += 2 * kRopeThreads) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int it = base + threadIdx.x + k * kRopeThreads;
                if (it >= v_total) continue;
                if (base > 0) vv[k] = reinterpret_cast<const uint4*>(ad.v_new)[static_cast<int64_t>(r0) * row_u4 + it];
                const int row = it / row_u4;
                const long long dst_row = s_dst[row];
                if (dst_row >= 0) reinterpret_cast<uint4*>(ad.suffix_v)[dst_row * row_u4 + (it - row * row_u4)] = vv[k];
            }
        }
    }
}

constexpr int kAppendThreads = 128;

__global__ void __launch_bounds__(kAppendThreads)
kv_append_kernel(int row_u4 /* Hkv*D*2/16 */, int32_t suffix_cap, int64_t cache_rows,
                 const int32_t* __restrict__ n_active, const int32_t* __restrict__ suffix_off,
                 const int32_t* __restrict__ suffix_len,
                 const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                 uint4* __restrict__ suffix_k, uint4* __restrict__ suffix_v, int32_t* __restrict__ dev_status)
{
    const int r = blockIdx.x;
    if (r >= *n_active) return;
    const int len = suffix_len[r];
    const int64_t off = suffix_off[r];
    if (len >= suffix_cap || len < 0) {
        if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, HPD_S_OVERFLOW);
        return;
    }
    const int64_t dst_row = off + len;
    if (off < 0 || dst_row >= cache_rows) {
        if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, HPD_S_BAD_TABLE);
        return;
    }
    const uint4* ks = k_new + static_cast<int64_t>(r) * row_u4;
    const uint4* vs = v_new + static_cast<int64_t>(r) * row_u4;
    uint4* kd = suffix_k + dst_row * row_u4;
    uint4* vd = suffix_v + dst_row * row_u4;
    for (int i = threadIdx.x; i < row_u4; i += kAppendThreads) {
        kd[i] = ks[i];
        vd[i] = vs[i];
    }
}

InvFreq inv_freq_table(const hpd_geom& g)
{
    InvFreq t{};
    for (int i = 0; i < g.D / 2; ++i) t.f[i] = pow(static_cast<double>(g.rope_theta), -2.0 * i / static_cast<double>(g.D));
    return t;
}

// End of a decode step (Sec. 4.3.4): one thread per row.
__global__ void __launch_bounds__(256)
advance_kernel(int max_rows, int32_t suffix_cap, int32_t delimiter_id, const int32_t* __restrict__ n_active,
               const int32_t* __restrict__ active_slot, const int32_t* __restrict__ token_id,
               int32_t* __restrict__ slot_depth, uint8_t* __restrict__ slot_alive, int32_t* __restrict__ n_alive)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    const int n = min(*n_active, max_rows);
    int stays = 0;
    if (r < n) {
        const int s = active_slot[r];
        const int d = min(slot_depth[s] + 1, suffix_cap);          // the step's token went into the slab (unless it was full)
        slot_depth[s] = d;
        stays = token_id[r] != delimiter_id && d < suffix_cap;
        slot_alive[s] = static_cast<uint8_t>(stays);
    }
    const int cnt = __syncthreads_count(stays);
    if (threadIdx.x == 0 && cnt) atomicAdd(n_alive, cnt);
}

// Merge of two attention results over disjoint key sets (three-level sharing): one warp per (row, q head).
template <int D>
__global__ void __launch_bounds__(256)
merge_lse_kernel(int Hq, int max_rows, const int32_t* __restrict__ n_active,
                 const __nv_bfloat16* o_a, const float* lse_a, const __nv_bfloat16* o_b, const float* lse_b,
                 __nv_bfloat16* o, float* lse)
{
    constexpr int E = D / 32;
    const int lane = threadIdx.x & 31;
    const int64_t w = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (w >= static_cast<int64_t>(min(*n_active, max_rows)) * Hq) return;
    const float la = lse_a[w], lb = lse_b[w];
    const float m = fmaxf(la, lb);
    float wa = 0.f, wb = 0.f, out_l = -INFINITY;
    if (m != -INFINITY) {
        const float ea = __expf(la - m), eb = __expf(lb - m);
        wa = ea / (ea + eb); wb = eb / (ea + eb);
        out_l = m + __logf(ea + eb);
    }
    const __nv_bfloat16* pa = o_a + w * D + lane * E;
    const __nv_bfloat16* pb = o_b + w * D + lane * E;
    __nv_bfloat16* po = o + w * D + lane * E;
    if constexpr (E == 4) {
        const uint2 a = *reinterpret_cast<const uint2*>(pa), b = *reinterpret_cast<const uint2*>(pb);
        uint2 r;
        r.x = pack_bf16(wa * bf16lo(a.x) + wb * bf16lo(b.x), wa * bf16hi(a.x) + wb * bf16hi(b.x));
        r.y = pack_bf16(wa * bf16lo(a.y) + wb * bf16lo(b.y), wa * bf16hi(a.y) + wb * bf16hi(b.y));
        *reinterpret_cast<uint2*>(po) = r;
    } else {
        const uint32_t a = *reinterpret_cast<const uint32_t*>(pa), b = *reinterpret_cast<const uint32_t*>(pb);
        *reinterpret_cast<uint32_t*>(po) = pack_bf16(wa * bf16lo(a) + wb * bf16lo(b), wa * bf16hi(a) + wb * bf16hi(b));
    }
    if (lse && lane == 0) lse[w] = out_l;
}

}  // namespace

int launch_merge_lse(const hpd_geom& g, int max_rows, const int32_t* n_active, const __nv_bfloat16* o_a, const float* lse_a,
                     const __nv_bfloat16* o_b, const float* lse_b, __nv_bfloat16* o, float* lse, cudaStream_t stream)
{
    if (max_rows <= 0) return HPD_OK;
    const int64_t warps = static_cast<int64_t>(max_rows) * g.Hq;
    const unsigned blocks = static_cast<unsigned>((warps + 7) / 8);
    if (g.D == 128) merge_lse_kernel<128><<<blocks, 256, 0, stream>>>(g.Hq, max_rows, n_active, o_a, lse_a, o_b, lse_b, o, lse);
    else merge_lse_kernel<64><<<blocks, 256, 0, stream>>>(g.Hq, max_rows, n_active, o_a, lse_a, o_b, lse_b, o, lse);
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

int launch_advance(const hpd_geom& g, int max_rows, const int32_t* n_active, const int32_t* active_slot,
                   const int32_t* token_id, int32_t delimiter_id, int32_t* slot_depth, uint8_t* slot_alive,
                   int32_t* n_alive, cudaStream_t stream)
{
    HPD_CUDA_TRY(cudaMemsetAsync(n_alive, 0, sizeof(int32_t), stream));
    if (max_rows <= 0) return HPD_OK;
    advance_kernel<<<(max_rows + 255) / 256, 256, 0, stream>>>(max_rows, g.suffix_cap, delimiter_id, n_active, active_slot,
                                                                token_id, slot_depth, slot_alive, n_alive);
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

int launch_rope(const hpd_geom& g, int max_rows, const int32_t* n_active, const int32_t* pos_id,
                __nv_bfloat16* q, __nv_bfloat16* k_new, cudaStream_t stream)
{
    if (max_rows <= 0) return HPD_OK;
    const InvFreq c = inv_freq_table(g);
    const AppendDst none{};
    if (g.D == 128)
        rope_kernel<128, false><<<(max_rows + kRopeRows - 1) / kRopeRows, kRopeThreads, 0, stream>>>(g.Hq, g.Hkv, c, n_active, pos_id, q, k_new, none);
    else
        rope_kernel<64, false><<<(max_rows + kRopeRows - 1) / kRopeRows, kRopeThreads, 0, stream>>>(g.Hq, g.Hkv, c, n_active, pos_id, q, k_new, none);
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

int launch_rope_append(const hpd_geom& g, int max_rows, int n_slots, const int32_t* n_active, const int32_t* pos_id,
                       const int32_t* suffix_off, const int32_t* suffix_len, __nv_bfloat16* q, __nv_bfloat16* k_new,
                       const __nv_bfloat16* v_new, __nv_bfloat16* suffix_k, __nv_bfloat16* suffix_v, int32_t* dev_status,
                       cudaStream_t stream)
{
    if (max_rows <= 0) return HPD_OK;
    const InvFreq c = inv_freq_table(g);
    const AppendDst ad{g.suffix_cap, static_cast<int64_t>(n_slots) * g.suffix_cap, suffix_off, suffix_len, v_new,
                       suffix_k, suffix_v, dev_status};
    if (g.D == 128)
        rope_kernel<128, true><<<(max_rows + kRopeRows - 1) / kRopeRows, kRopeThreads, 0, stream>>>(g.Hq, g.Hkv, c, n_active, pos_id, q, k_new, ad);
    else
        rope_kernel<64, true><<<(max_rows + kRopeRows - 1) / kRopeRows, kRopeThreads, 0, stream>>>(g.Hq, g.Hkv, c, n_active, pos_id, q, k_new, ad);
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

int launch_kv_append(const hpd_geom& g, int max_rows, int n_slots, const int32_t* n_active, const int32_t* suffix_off,
                     const int32_t* suffix_len, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new,
                     __nv_bfloat16* suffix_k, __nv_bfloat16* suffix_v, int32_t* dev_status, cudaStream_t stream)
{
    if (max_rows <= 0) return HPD_OK;
    const int row_u4 = g.Hkv * g.D * 2 / 16;
    kv_append_kernel<<<max_rows, kAppendThreads, 0, stream>>>(
        row_u4, g.suffix_cap, static_cast<int64_t>(n_slots) * g.suffix_cap, n_active, suffix_off, suffix_len,
        reinterpret_cast<const uint4*>(k_new), reinterpret_cast<const uint4*>(v_new),
        reinterpret_cast<uint4*>(suffix_k), reinterpret_cast<uint4*>(suffix_v), dev_status);
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

}  // namespace hpd
