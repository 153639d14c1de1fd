// Scalar (CUDA-core) flash-decode: one warp per (row, kv head, split) streams the row's keys once.
//
// This is the kernel behind std_attn_decode -- every branch owns a private copy of its whole
// sequence, so there is no sharing to exploit and the work is a pure stream over HBM with G query
// rows per key.  hpd_attn_decode uses it only for geometries the tensor-core kernel does not take.
//
// Mapping.  Scores: lane <-> key (32 keys per pass); the G query vectors sit in shared memory
// (pre-multiplied by sm_scale*log2(e)) and are read as broadcasts, so a score needs no cross-lane
// reduction.  Softmax: online, running max/sum per q head, two warp-shuffle reductions per pass.
// PV: lane <-> D/32 output columns; the probability of key j is broadcast with one shuffle per head.
#include "common.cuh"

namespace hpd {

namespace {

constexpr int kWarps = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int D, int G>
struct RowState {
    float o[G][D / 32];
    float m[G], l[G];
};

// Stream `cnt` consecutive token rows starting at token row `row0` of K/V [tokens, Hkv, D].
template <int D, int G>
__device__ __forceinline__ void stream_segment(RowState<D, G>& st, const float* __restrict__ qs,
                                               const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
                                               int64_t row0, int cnt, int Hkv, int hk, int lane)
{
    constexpr int E = D / 32;                       // output columns per lane
    const int64_t tok_stride = static_cast<int64_t>(Hkv) * D;
    for (int t = 0; t < cnt; t += 32) {
        const int key = t + lane;
        const bool valid = key < cnt;
        const uint4* kp = reinterpret_cast<const uint4*>(K + (row0 + (valid ? key : t)) * tok_stride + hk * D);
        float s[G];
#pragma unroll
        for (int g = 0; g < G; ++g) s[g] = 0.f;
#pragma unroll 4
        for (int c = 0; c < D / 8; ++c) {
            const uint4 kk = __ldg(kp + c);
            const float k0 = bf16lo(kk.x), k1 = bf16hi(kk.x), k2 = bf16lo(kk.y), k3 = bf16hi(kk.y);
            const float k4 = bf16lo(kk.z), k5 = bf16hi(kk.z), k6 = bf16lo(kk.w), k7 = bf16hi(kk.w);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float4 qa = *reinterpret_cast<const float4*>(qs + g * D + c * 8);
                const float4 qb = *reinterpret_cast<const float4*>(qs + g * D + c * 8 + 4);
                float a = s[g];
                a = fmaf(qa.x, k0, a); a = fmaf(qa.y, k1, a); a = fmaf(qa.z, k2, a); a = fmaf(qa.w, k3, a);
                a = fmaf(qb.x, k4, a); a = fmaf(qb.y, k5, a); a = fmaf(qb.z, k6, a); a = fmaf(qb.w, k7, a);
                s[g] = a;
            }
        }
        float p[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float sv = valid ? s[g] : -INFINITY;
            const float m_new = fmaxf(st.m[g], warp_max(sv));
            const float alpha = exp2f(st.m[g] - m_new);
            p[g] = exp2f(sv - m_new);
            st.l[g] = st.l[g] * alpha + warp_sum(p[g]);
            st.m[g] = m_new;
#pragma unroll
            for (int e = 0; e < E; ++e) st.o[g][e] *= alpha;
        }
        const int nk = min(32, cnt - t);
        const __nv_bfloat16* vp = V + (row0 + t) * tok_stride + hk * D + lane * E;
#pragma unroll 4
        for (int j = 0; j < nk; ++j) {
            float v[E];
            if constexpr (E == 4) {
                const uint2 w = __ldg(reinterpret_cast<const uint2*>(vp + j * tok_stride));
                v[0] = bf16lo(w.x); v[1] = bf16hi(w.x); v[2] = bf16lo(w.y); v[3] = bf16hi(w.y);
            } else {
                const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(vp + j * tok_stride));
                v[0] = bf16lo(w); v[1] = bf16hi(w);
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float pj = __shfl_sync(0xffffffffu, p[g], j);
#pragma unroll
                for (int e = 0; e < E; ++e) st.o[g][e] = fmaf(pj, v[e], st.o[g][e]);
            }
        }
    }
}

template <int D, int G>
__global__ void __launch_bounds__(kWarps * 32)
simt_attn_kernel(SimtArgs a)
{
    constexpr int E = D / 32;
    __shared__ __align__(16) float q_sm[kWarps][G * D];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int Hkv = a.g.Hkv, Hq = a.g.Hq;
    const int64_t wg = static_cast<int64_t>(blockIdx.x) * kWarps + warp;
    const int split = static_cast<int>(wg % a.n_splits);
    const int hk = static_cast<int>((wg / a.n_splits) % Hkv);
    const int64_t r = wg / (static_cast<int64_t>(a.n_splits) * Hkv);
    if (r >= *a.n_active) return;

    int n1, n2 = 0;
    int64_t base1, base2 = 0;
    if (a.doc_id) {
        const int d = a.doc_id[r];
        n1 = a.doc_prefix_len[d];
        base1 = a.doc_kv_start[d];
        n2 = a.suffix_len[r] + a.suffix_extra;
        if (n2 > a.g.suffix_cap) n2 = a.g.suffix_cap;
        if (n2 < 0) n2 = 0;
        base2 = a.suffix_off[r];
    } else {
        n1 = a.seq_len[r];
        base1 = a.seq_start[r];
    }
    const int total = n1 + n2;
    int lo = 0, hi = total;
    if (a.n_splits > 1) {
        int per = (total + a.n_splits - 1) / a.n_splits;
        per = (per + 31) & ~31;
        lo = min(total, split * per);
        hi = min(total, lo + per);
    }

    // q rows of this kv head, scaled so that exp2 can be used directly
    float* qs = q_sm[warp];
    const float qscale = a.g.sm_scale * kLog2e;
    const __nv_bfloat16* qrow = a.q + (r * Hq + static_cast<int64_t>(hk) * G) * D;
    for (int i = lane; i < G * D / 2; i += 32) {
        const uint32_t w = reinterpret_cast<const uint32_t*>(qrow)[i];
        qs[2 * i] = bf16lo(w) * qscale;
        qs[2 * i + 1] = bf16hi(w) * qscale;
    }
    __syncwarp();

    RowState<D, G> st;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        st.m[g] = -INFINITY;
        st.l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) st.o[g][e] = 0.f;
    }
    {
        const int b = min(lo, n1), e = min(hi, n1);
        if (e > b) stream_segment<D, G>(st, qs, a.k1, a.v1, base1 + b, e - b, Hkv, hk, lane);
    }
    if (n2 > 0) {
        const int b = max(lo, n1) - n1, e = max(hi, n1) - n1;
        if (e > b) stream_segment<D, G>(st, qs, a.k2, a.v2, base2 + b, e - b, Hkv, hk, lane);
    }

    if (a.n_splits == 1) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float inv = st.l[g] > 0.f ? 1.f / st.l[g] : 0.f;
            __nv_bfloat16* op = a.o + (r * Hq + static_cast<int64_t>(hk) * G + g) * D + lane * E;
            if constexpr (E == 4) {
                uint2 w;
                w.x = pack_bf16(st.o[g][0] * inv, st.o[g][1] * inv);
                w.y = pack_bf16(st.o[g][2] * inv, st.o[g][3] * inv);
                *reinterpret_cast<uint2*>(op) = w;
            } else {
                *reinterpret_cast<uint32_t*>(op) = pack_bf16(st.o[g][0] * inv, st.o[g][1] * inv);
            }
            if (a.lse && lane == 0)
                a.lse[r * Hq + hk * G + g] = st.l[g] > 0.f ? (st.m[g] + log2f(st.l[g])) * kLn2 : -INFINITY;
        }
    } else {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float* pp = a.part + ((r * Hq + static_cast<int64_t>(hk) * G + g) * a.n_splits + split) * (D + 2);
            if (lane == 0) { pp[0] = st.m[g]; pp[1] = st.l[g]; }
#pragma unroll
            for (int e = 0; e < E; ++e) pp[2 + lane * E + e] = st.o[g][e];
        }
    }
}

// Merge of split partials: one warp per (row, q head).
template <int D>
__global__ void __launch_bounds__(128)
simt_merge_kernel(int Hq, int n_splits, const int32_t* __restrict__ n_active, const float* __restrict__ part,
                  __nv_bfloat16* __restrict__ o, float* __restrict__ lse)
{
    constexpr int E = D / 32;
    const int lane = threadIdx.x & 31;
    const int64_t w = static_cast<int64_t>(blockIdx.x) * 4 + (threadIdx.x >> 5);
    const int64_t r = w / Hq;
    if (r >= *n_active) return;
    const float* pp = part + w * n_splits * (D + 2);
    float M = -INFINITY;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, pp[s * (D + 2)]);
    float L = 0.f, acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float m = pp[s * (D + 2)];
        const float sc = m == -INFINITY ? 0.f : exp2f(m - M);
        L += sc * pp[s * (D + 2) + 1];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = fmaf(sc, pp[s * (D + 2) + 2 + lane * E + e], acc[e]);
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    __nv_bfloat16* op = o + w * D + lane * E;
    if constexpr (E == 4) {
        uint2 v;
        v.x = pack_bf16(acc[0] * inv, acc[1] * inv);
        v.y = pack_bf16(acc[2] * inv, acc[3] * inv);
        *reinterpret_cast<uint2*>(op) = v;
    } else {
        *reinterpret_cast<uint32_t*>(op) = pack_bf16(acc[0] * inv, acc[1] * inv);
    }
    if (lse && lane == 0) lse[w] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
}

template <int D, int G>
int launch_t(const SimtArgs& a)
{
    const int64_t warps = static_cast<int64_t>(a.max_rows) * a.g.Hkv * a.n_splits;
    const int64_t blocks = (warps + kWarps - 1) / kWarps;
    if (blocks > 0x7fffffffll) return HPD_E_CAPACITY;
    simt_attn_kernel<D, G><<<static_cast<unsigned>(blocks), kWarps * 32, 0, a.stream>>>(a);
    if (a.n_splits > 1) {
        const int64_t mw = static_cast<int64_t>(a.max_rows) * a.g.Hq;
        simt_merge_kernel<D><<<static_cast<unsigned>((mw + 3) / 4), 128, 0, a.stream>>>(a.g.Hq, a.n_splits, a.n_active,
                                                                                         a.part, a.o, a.lse);
    }
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

}  // namespace

int launch_attn_simt(const SimtArgs& a)
{
    if (a.max_rows <= 0) return HPD_OK;
    const int G = a.g.Hq / a.g.Hkv;
#define HPD_CASE(DD, GG) if (a.g.D == DD && G == GG) return launch_t<DD, GG>(a);
    HPD_CASE(128, 1) HPD_CASE(128, 2) HPD_CASE(128, 4) HPD_CASE(128, 8)
    HPD_CASE(64, 1) HPD_CASE(64, 2) HPD_CASE(64, 4) HPD_CASE(64, 8)
#undef HPD_CASE
    return HPD_E_GEOM;
}

}  // namespace hpd
