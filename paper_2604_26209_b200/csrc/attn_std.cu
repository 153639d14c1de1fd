// std_attn_decode: standard batched decode over private per-sequence K/V copies (flash-decoding).
//
// Every branch is a sequence of its own, so there is nothing to share and the kernel is a pure stream
// over HBM: each K/V byte is read once and used by the G query heads of its kv head.  A persistent CTA
// walks work items (sequence, block of up to 8 kv heads, split); a producer warp streams the item's
// tokens through a shared-memory ring with TMA -- one box per stage and tensor, 16 tokens x all heads
// of the block, landing as one 128-byte-swizzled [16 tokens][64 elements] sub-tile per (head, half of
// D) -- and runs ahead into the next item while the consumers finish the current one.  Consumer warp w
// owns kv head w of the block and keeps keys on the M side of the warp-level tensor-core instruction,
// so no row of it is padding:
//     S^T[16 keys x 8] = K[16 x D] Q^T[D x 8]       (8 = the G <= 8 query heads, zero-padded)
//     O^T[D x 8]      += V^T[D x 16 keys] P^T[16 keys x 8]
// with an online softmax per query head in between (maximum over the 16 keys by warp shuffles, lazy
// rescaling of O^T, probabilities moved from accumulator to operand layout with movmatrix).  Split
// sequences (small batches) leave (m, l, O) partials that a second kernel merges.
#include <atomic>

#include "common.cuh"
#include "ptx.cuh"

namespace hpd {

namespace {

constexpr int kT = 16;                      // tokens per stage
constexpr int kStages = 3;
constexpr int kHB = 8;                      // kv heads per CTA = consumer warps
constexpr int kThreads = (kHB + 1) * 32;    // + the producer warp
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s

struct StdParams {
    hpd_geom g;
    int G, hb /* heads per block */, hchunks, n_splits, max_rows;
    const int32_t* n_active;
    const __nv_bfloat16* q;
    const int64_t* seq_start;
    const int32_t* seq_len;
    __nv_bfloat16* o;
    float* lse;
    float* part;                            // n_splits > 1: [max_rows, Hq, n_splits, D+2]
    int32_t* dev_status;                    // may be null
    float scale_log2;
    uint32_t tensor_bytes;                  // bytes of one stage's K (or V) box
};

struct Bars {
    unsigned long long full[kStages], empty[kStages];
    int abort_flag;
};

// Bounded wait: gives up after ~2 s or once another thread of the CTA has given up.
__device__ __forceinline__ bool wait_bar(unsigned long long* bar, uint32_t parity, Bars* b) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 1023) == 0) {
            if (*reinterpret_cast<volatile int*>(&b->abort_flag)) return false;
            if (clock64() - t0 > kWaitCycles) {
                *reinterpret_cast<volatile int*>(&b->abort_flag) = 1;
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t v) {
    uint32_t r;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}
// D[16x8] += A[16x16] B[16x8], bf16 operands, fp32 accumulate
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float group_max(float v) {       // over the 8 lanes that share lane % 4
    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
    return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
}
__device__ __forceinline__ float group_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    v += __shfl_xor_sync(0xffffffffu, v, 8);
    return v + __shfl_xor_sync(0xffffffffu, v, 16);
}

struct Item { int r, hc, split, lo, hi; int64_t start; };

// Work item `idx` -> (sequence, head block, split) and the token range of the split.
__device__ __forceinline__ Item decode_item(const StdParams& p, int64_t idx) {
    Item it;
    it.split = static_cast<int>(idx % p.n_splits);
    it.hc = static_cast<int>((idx / p.n_splits) % p.hchunks);
    it.r = static_cast<int>(idx / (static_cast<int64_t>(p.n_splits) * p.hchunks));
    const int len = max(p.seq_len[it.r], 0);
    it.start = p.seq_start[it.r];
    it.lo = 0; it.hi = len;
    if (p.n_splits > 1) {
        int per = (len + p.n_splits - 1) / p.n_splits;
        per = (per + kT - 1) / kT * kT;
        it.lo = min(len, it.split * per);
        it.hi = min(len, it.lo + per);
    }
    return it;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
std_attn_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const StdParams p)
{
    constexpr int HALVES = D / 64;
    constexpr int SUB = kT * 128;                       // one (head, half) sub-tile: 16 tokens x 128 B
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // the swizzle pattern is a function of the shared-memory address: stages start on 1024-byte boundaries
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const uint32_t stage_bytes = 2 * p.tensor_bytes;    // K then V
    Bars* bars = reinterpret_cast<Bars*>(smem + kStages * stage_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], kHB); }
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();

    const int64_t n_items = static_cast<int64_t>(max(min(*p.n_active, p.max_rows), 0)) * p.hchunks * p.n_splits;
    const int Hq = p.g.Hq, Hkv = p.g.Hkv, G = p.G;

    if (warp == kHB) {
        // ------------------------------------ producer ------------------------------------
        if (lane == 0) {
            uint32_t n = 0;
            bool ok = true;
            for (int64_t idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const Item it = decode_item(p, idx);
                for (int tok = it.lo; tok < it.hi; tok += kT, ++n) {
                    const int s = n % kStages;
                    ok = wait_bar(&bars->empty[s], ((n / kStages) & 1) ^ 1, bars);
                    if (!ok) break;
                    uint8_t* st = smem + s * stage_bytes;
                    mbar_expect_tx(&bars->full[s], stage_bytes);
                    const int c_tok = static_cast<int>(it.start + tok);
                    tma_load_4d(st, &map_k, &bars->full[s], 0, c_tok, 0, it.hc * p.hb);
                    tma_load_4d(st + p.tensor_bytes, &map_v, &bars->full[s], 0, c_tok, 0, it.hc * p.hb);
                }
            }
        }
    } else {
        // ------------------------------------ consumers -----------------------------------
        const int g8 = lane >> 2, t4 = lane & 3;         // fragment coordinates
        const int q0 = 2 * t4;                           // this thread's two query heads (columns of S^T, O^T)
        // per-lane ldmatrix row addresses inside a sub-tile (before the 16-byte chunk is chosen)
        const int k_tok = (lane & 7) + ((lane >> 3) & 1) * 8, k_sel = lane >> 4;
        const int v_key = (lane & 7) + (lane >> 4) * 8, v_sel = (lane >> 3) & 1;
        const uint32_t k_row = k_tok * 128, k_x = k_tok & 7;
        const uint32_t v_row = v_key * 128, v_x = v_key & 7;
        uint32_t n = 0;
        bool ok = true;
        for (int64_t idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
            const Item it = decode_item(p, idx);
            const int head = it.hc * p.hb + warp;
            const bool active = warp < p.hb && head < Hkv;
            // Q^T as the B operand: this thread needs q[head*G + g8][16 kk + 2 t4 + {0,1,8,9}]; rows >= G are zero
            uint32_t qf[D / 16][2];
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) { qf[kk][0] = 0u; qf[kk][1] = 0u; }
            if (active && g8 < G) {
                const uint32_t* qrow = reinterpret_cast<const uint32_t*>(p.q + (static_cast<int64_t>(it.r) * Hq + head * G + g8) * D);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    qf[kk][0] = qrow[kk * 8 + t4];
                    qf[kk][1] = qrow[kk * 8 + 4 + t4];
                }
            }
            float acc[D / 16][4];
#pragma unroll
            for (int mt = 0; mt < D / 16; ++mt) { acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f; }
            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

            for (int tok = it.lo; tok < it.hi; tok += kT, ++n) {
                const int s = n % kStages;
                ok = __all_sync(0xffffffffu, wait_bar(&bars->full[s], (n / kStages) & 1, bars));
                if (!ok) break;
                if (active) {
                    const uint32_t kb = smem_u32(smem + s * stage_bytes) + warp * HALVES * SUB;
                    const uint32_t vb = kb + p.tensor_bytes;
                    const int nv = min(kT, it.hi - tok);             // valid tokens of this tile
                    float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        uint32_t a[4];
                        ldsm_x4(kb + (kk >> 2) * SUB + k_row + ((((kk & 3) * 2 + k_sel) ^ k_x) << 4), a);
                        mma_16816(sc, a, qf[kk][0], qf[kk][1]);
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) sc[i] *= p.scale_log2;
                    if (nv < kT) {                                   // keys beyond the sequence: -inf by selection
                        if (g8 >= nv) { sc[0] = -INFINITY; sc[1] = -INFINITY; }
                        if (g8 + 8 >= nv) { sc[2] = -INFINITY; sc[3] = -INFINITY; }
                    }
                    const float mn0 = fmaxf(m0, group_max(fmaxf(sc[0], sc[2])));
                    const float mn1 = fmaxf(m1, group_max(fmaxf(sc[1], sc[3])));
                    if (__any_sync(0xffffffffu, mn0 > m0 || mn1 > m1)) {
                        const float a0 = ex2f(m0 - mn0), a1 = ex2f(m1 - mn1);      // m = -inf: 0, and acc is still 0
                        l0 *= a0; l1 *= a1;
#pragma unroll
                        for (int mt = 0; mt < D / 16; ++mt) { acc[mt][0] *= a0; acc[mt][1] *= a1; acc[mt][2] *= a0; acc[mt][3] *= a1; }
                        m0 = mn0; m1 = mn1;
                    }
                    const float p0 = ex2f(sc[0] - m0), p1 = ex2f(sc[1] - m1), p2 = ex2f(sc[2] - m0), p3 = ex2f(sc[3] - m1);
                    l0 += p0 + p2; l1 += p1 + p3;
                    // accumulator layout [key g8 (+8)][heads q0, q0+1] -> operand layout [keys 2 t4 + {0,1} (+8)][head g8]
                    const uint32_t b0 = movmatrix_trans(pack_bf16(p0, p1));
                    const uint32_t b1 = movmatrix_trans(pack_bf16(p2, p3));
                    uint32_t msk_lo = 0xffffffffu, msk_hi = 0xffffffffu;
                    if (nv < kT) {                                   // V rows beyond the sequence may hold anything: zero them
                        msk_lo = (2 * t4 < nv ? 0x0000ffffu : 0u) | (2 * t4 + 1 < nv ? 0xffff0000u : 0u);
                        msk_hi = (2 * t4 + 8 < nv ? 0x0000ffffu : 0u) | (2 * t4 + 9 < nv ? 0xffff0000u : 0u);
                    }
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt) {
                        uint32_t a[4];
                        ldsm_x4_trans(vb + (mt >> 2) * SUB + v_row + ((((mt & 3) * 2 + v_sel) ^ v_x) << 4), a);
                        if (nv < kT) { a[0] &= msk_lo; a[1] &= msk_lo; a[2] &= msk_hi; a[3] &= msk_hi; }
                        mma_16816(acc[mt], a, b0, b1);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->empty[s]);
            }
            if (!ok) break;

            // ---- item epilogue: O^T[d = 16 mt + g8 (+8)][head q0 (+1)] ----
            if (active) {
                l0 = group_sum(l0); l1 = group_sum(l1);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int qh = q0 + j;
                    if (qh >= G) continue;
                    const float m = j ? m1 : m0, l = j ? l1 : l0;
                    const int64_t row = static_cast<int64_t>(it.r) * Hq + head * G + qh;
                    if (p.n_splits == 1) {
                        const float inv = l > 0.f ? 1.f / l : 0.f;
                        __nv_bfloat16* op = p.o + row * D;
#pragma unroll
                        for (int mt = 0; mt < D / 16; ++mt) {
                            op[mt * 16 + g8] = __float2bfloat16_rn(acc[mt][j] * inv);
                            op[mt * 16 + 8 + g8] = __float2bfloat16_rn(acc[mt][2 + j] * inv);
                        }
                        if (p.lse && g8 == 0) p.lse[row] = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
                    } else {
                        float* pp = p.part + (row * p.n_splits + it.split) * (D + 2);
                        if (g8 == 0) { pp[0] = m; pp[1] = l; }
#pragma unroll
                        for (int mt = 0; mt < D / 16; ++mt) {
                            pp[2 + mt * 16 + g8] = acc[mt][j];
                            pp[2 + mt * 16 + 8 + g8] = acc[mt][2 + j];
                        }
                    }
                }
            }
        }
    }

    __syncthreads();
    if (bars->abort_flag) {
        if (threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, HPD_S_TIMEOUT);
        const long long t0 = clock64();                  // let copies that may still be in flight land
        while (clock64() - t0 < 20000000ll) { }
        __syncthreads();
    }
}

// Merge of split partials: one warp per (row, q head).
template <int D>
__global__ void __launch_bounds__(128)
std_merge_kernel(int Hq, int n_splits, const int32_t* __restrict__ n_active, const float* __restrict__ part,
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

// K or V [tokens, Hkv, D] bf16 seen as (64 elements, tokens, halves of D, heads): one box = 16 tokens x all halves x
// `hb` heads, which lands in shared memory as [head][half][token][128 B] with the 128-byte swizzle.
bool make_std_map(CUtensorMap* m, const void* base, int D, int Hkv, long long tokens, int hb)
{
    auto fn = tensor_map_encoder();
    if (!fn) return false;
    cuuint64_t dims[4] = {64, static_cast<cuuint64_t>(tokens > 0 ? tokens : 1), static_cast<cuuint64_t>(D / 64),
                          static_cast<cuuint64_t>(Hkv)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(Hkv) * D * 2, 128, static_cast<cuuint64_t>(D) * 2};
    cuuint32_t box[4] = {64, kT, static_cast<cuuint32_t>(D / 64), static_cast<cuuint32_t>(hb)};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
int launch_d(const StdArgs& a)
{
    const int hb = a.g.Hkv < kHB ? a.g.Hkv : kHB;
    StdParams p{};
    p.g = a.g;
    p.G = a.g.Hq / a.g.Hkv;
    p.hb = hb;
    p.hchunks = (a.g.Hkv + hb - 1) / hb;
    p.n_splits = a.n_splits;
    p.max_rows = a.max_rows;
    p.n_active = a.n_active; p.q = a.q; p.seq_start = a.seq_start; p.seq_len = a.seq_len;
    p.o = a.o; p.lse = a.lse; p.part = a.part; p.dev_status = nullptr;
    p.scale_log2 = a.g.sm_scale * kLog2e;
    p.tensor_bytes = static_cast<uint32_t>(kT) * hb * D * 2;
    const size_t smem = static_cast<size_t>(kStages) * 2 * p.tensor_bytes + sizeof(Bars) + 1024;

    static std::atomic<size_t> attr_bytes[kMaxDevices];          // largest dynamic shared memory enabled, per device
    const int dev = current_device();
    const bool slot = dev >= 0 && dev < kMaxDevices;
    if (!slot || attr_bytes[dev].load(std::memory_order_acquire) < smem) {
        HPD_CUDA_TRY(cudaFuncSetAttribute(std_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        if (slot) attr_bytes[dev].store(smem, std::memory_order_release);
    }
    CUtensorMap mk, mv;
    if (!make_std_map(&mk, a.dup_k, D, a.g.Hkv, a.total_tokens, hb) || !make_std_map(&mv, a.dup_v, D, a.g.Hkv, a.total_tokens, hb)) {
        set_last_cuda_error(cudaErrorInvalidValue);
        return HPD_E_CUDA;
    }
    const long long items = static_cast<long long>(a.max_rows) * p.hchunks * a.n_splits;
    const int n_sm = sm_count();
    const int grid = static_cast<int>(items < n_sm ? items : n_sm);
    std_attn_kernel<D><<<grid, kThreads, smem, a.stream>>>(mk, mv, p);
    if (a.n_splits > 1) {
        const int64_t mw = static_cast<int64_t>(a.max_rows) * a.g.Hq;
        std_merge_kernel<D><<<static_cast<unsigned>((mw + 3) / 4), 128, 0, a.stream>>>(a.g.Hq, a.n_splits, a.n_active,
                                                                                        a.part, a.o, a.lse);
    }
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

}  // namespace

int launch_attn_std(const StdArgs& a)
{
    if (a.max_rows <= 0) return HPD_OK;
    if (!(a.g.sm_scale > 0.f)) return HPD_E_GEOM;
    return a.g.D == 128 ? launch_d<128>(a) : launch_d<64>(a);
}

}  // namespace hpd
