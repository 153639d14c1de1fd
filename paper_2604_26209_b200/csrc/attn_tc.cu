// hpd_attn_decode on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
// One persistent CTA per SM walks the step's work units.  A unit = (work item, kv head): up to
// 128/G branches of one document (rows = branches x G query heads, the M dimension) against a chunk
// of that document's prefix, so each prefix K/V byte is read from HBM once for all of the document's
// branches.  The branches' own cached tokens ("suffix") are gathered into further K/V tiles of the
// same pipeline and masked block-diagonally (a row sees only its own branch's columns).
//
//   warp 0      TMA producer: Q tile, prefix K tiles, prefix V tiles (128B-swizzled boxes)
//   warp 1      MMA issuer:   S = Q K^T  (tcgen05.mma, accumulators in TMEM), O += P V
//   warps 2-5   softmax:      one thread per row; S from TMEM, online max/sum, P (bf16) to shared
//                             memory, rare rescale of O in TMEM, epilogue
//   warps 6-9   gather:       branch-cache rows -> swizzled K/V tiles with cp.async
//
// All waits are bounded: a wait that gives up raises HPD_S_TIMEOUT in the status word and the CTA
// drains and exits (TMEM is released on every path).
#include <cuda.h>
#include <cudaTypedefs.h>

#include <mutex>

#include "common.cuh"

namespace hpd {

namespace {

constexpr int kThreads = 320;
constexpr int kTile = 128;                 // rows and keys per tile
constexpr int kHalfBytes = kTile * 128;    // one 64-element half of a tile: 128 rows x 128 B
constexpr int kPBytes = 2 * kHalfBytes;    // P tile: 128 rows x 128 keys bf16
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleSlack = 8.0f;      // tolerated growth of the row maximum (log2 units) before O is rescaled
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s at 2 GHz

template <int D> struct Cfg {
    static constexpr int HALVES = D / 64;
    static constexpr int TILE_BYTES = HALVES * kHalfBytes;     // Q, K or V tile
    static constexpr int NK = D == 128 ? 3 : 4;                 // K stages
    static constexpr int NV = D == 128 ? 2 : 4;                 // V stages
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + TILE_BYTES;
    static constexpr int OFF_V = OFF_K + NK * TILE_BYTES;
    static constexpr int OFF_P = OFF_V + NV * TILE_BYTES;
    static constexpr int OFF_MISC = OFF_P + kPBytes;
    static constexpr int SMEM = OFF_MISC + 2048 + 1024;         // + misc + slack for 1024-B alignment
};

struct Misc {
    unsigned long long q_full, q_empty, p_full, p_empty;
    unsigned long long k_full[4], k_empty[4], v_full[4], v_empty[4];
    unsigned long long s_full[2], s_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int wt[2][4];
    int cs[2][kTile + 4];
};
static_assert(sizeof(Misc) <= 2048, "misc block");

struct TcParams {
    AttnArgs a;
    const WsHeader* hdr;
    const WorkItem* work;
    float* part_ml;
    float* part_o;
    float scale_log2;
    int G;
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false after ~2 s or once another thread of the CTA has given up.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, Misc* misc) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 1023) == 0) {
            if (*reinterpret_cast<volatile int*>(&misc->abort_flag)) return false;
            if (clock64() - t0 > kWaitCycles) {
                *reinterpret_cast<volatile int*>(&misc->abort_flag) = 1;
                return false;
            }
        }
    }
    return true;
}

// all lanes wait; the result is made warp-uniform so that warp-collective instructions stay converged
__device__ __forceinline__ bool mbar_wait_warp(unsigned long long* bar, uint32_t parity, Misc* misc) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, misc));
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, unsigned long long* bar, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, unsigned long long* bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

#define HPD_R8(a, o) "=r"(a[o + 0]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), "=r"(a[o + 6]), "=r"(a[o + 7])
#define HPD_W8(a, o) "r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), "r"(a[o + 6]), "r"(a[o + 7])
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : HPD_R8(v, 0), HPD_R8(v, 8), HPD_R8(v, 16), HPD_R8(v, 24) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), HPD_W8(v, 0), HPD_W8(v, 8), HPD_W8(v, 16), HPD_W8(v, 24) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void named_bar(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
// barrier over a 128-thread role group that also AND-reduces a flag, so that exits stay uniform
__device__ __forceinline__ bool named_bar_and(int id, bool v) {
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, %2, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r) : "r"(v ? 1u : 0u), "r"(id) : "memory");
    return r != 0;
}

// Shared-memory matrix descriptors (128-byte swizzle; version field = 1).
//   K-major  (Q, K, P): rows of 128 B; groups of 8 rows 1024 B apart (SBO); LBO unused.
//   MN-major (V):       rows (keys) of 128 B holding 64 head-dim elements; 8-key groups 1024 B apart
//                       (SBO); the next 64 head-dim elements 16 KiB further (LBO).
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
    return static_cast<uint64_t>((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr) {
    return static_cast<uint64_t>((saddr >> 4) & 0x3FFF) | (static_cast<uint64_t>(kHalfBytes >> 4) << 16) | (64ull << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N given; B either K-major (Q K^T) or MN-major (P V).
__device__ __forceinline__ uint32_t make_idesc(int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(b_mn_major) << 16) |
           (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(kTile >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// per-unit bookkeeping shared by all roles (every role recomputes it from the same global data)
// ------------------------------------------------------------------------------------------------
struct Unit {
    int doc, head, key_count, part_base, row_begin, nb /*branches*/, with_suffix;
    int row0;        // first global row
    int kv_row0;     // first global prefix token row
    int np;          // prefix tiles
};

__device__ __forceinline__ Unit load_unit(const TcParams& p, int w) {
    const int Hkv = p.a.g.Hkv;
    const WorkItem it = p.work[w / Hkv];
    Unit u;
    u.doc = it.doc; u.head = w % Hkv; u.key_count = it.key_count; u.part_base = it.part_base;
    u.row_begin = it.row_begin; u.nb = it.row_count; u.with_suffix = it.with_suffix;
    u.row0 = p.a.doc_active_start[it.doc] + it.row_begin;
    u.kv_row0 = p.a.doc_kv_start[it.doc] + it.key_begin;
    u.np = (it.key_count + kTile - 1) / kTile;
    return u;
}

__device__ __forceinline__ int branch_suffix_len(const TcParams& p, int row) {
    int n = p.a.suffix_len[row] + p.a.suffix_extra;
    n = n < 0 ? 0 : n;
    return n > p.a.g.suffix_cap ? p.a.g.suffix_cap : n;
}

// total cached tokens of the unit's branches (whole warp calls it)
__device__ __forceinline__ int suffix_total_warp(const TcParams& p, const Unit& u, int lane) {
    if (!u.with_suffix) return 0;
    int s = 0;
    for (int b = lane; b < u.nb; b += 32) s += branch_suffix_len(p, u.row0 + b);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

// exclusive scan of the branches' cached lengths over a 128-thread role group -> cs[0..128]; returns total
__device__ __forceinline__ int suffix_scan_group(const TcParams& p, const Unit& u, Misc* misc, int which, int t /*0..127*/, int bar_id) {
    int* cs = misc->cs[which];
    int* wt = misc->wt[which];
    int len = 0;
    if (u.with_suffix && t < u.nb) len = branch_suffix_len(p, u.row0 + t);
    int incl = len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, o);
        if ((t & 31) >= o) incl += v;
    }
    named_bar(bar_id);                       // previous unit's readers are done with cs/wt
    if ((t & 31) == 31) wt[t >> 5] = incl;
    named_bar(bar_id);
    int off = 0;
    for (int w = 0; w < (t >> 5); ++w) off += wt[w];
    const int total = wt[0] + wt[1] + wt[2] + wt[3];
    cs[t] = off + incl - len;
    if (t == kTile - 1) cs[kTile] = total;
    named_bar(bar_id);
    return total;
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
hpd_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const TcParams p)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    Misc* misc = reinterpret_cast<Misc*>(smem + C::OFF_MISC);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.G;
    const int n_units = p.hdr->n_work * p.a.g.Hkv;

    if (threadIdx.x == 0) {
        mbar_init(&misc->q_full, 1);  mbar_init(&misc->q_empty, 1);
        mbar_init(&misc->p_full, 4);  mbar_init(&misc->p_empty, 1);
        for (int i = 0; i < 4; ++i) {
            mbar_init(&misc->k_full[i], 1); mbar_init(&misc->k_empty[i], 1);
            mbar_init(&misc->v_full[i], 1); mbar_init(&misc->v_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(&misc->s_full[i], 1); mbar_init(&misc->s_empty[i], 4); }
        misc->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&misc->tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&misc->tmem_base);
    const uint32_t tmem_o = tmem + 2 * kTile;            // columns [256, 256 + D)

    if (warp == 0) {
        // ======================================= TMA producer =======================================
        uint32_t qi = 0, kc = 0, vc = 0;
        bool ok = true;
        for (int w = blockIdx.x; w < n_units && ok; w += gridDim.x) {
            const Unit u = load_unit(p, w);
            const int stot = suffix_total_warp(p, u, lane);
            const int ns = (stot + kTile - 1) / kTile;
            if (u.np + ns == 0) continue;
            if (lane == 0) {
                ok = mbar_wait(&misc->q_empty, (qi & 1) ^ 1, misc);
                if (ok) {
                    mbar_expect_tx(&misc->q_full, C::TILE_BYTES);
                    for (int h = 0; h < C::HALVES; ++h)
                        tma_load_4d(smem + C::OFF_Q + h * kHalfBytes, &map_q, &misc->q_full, h * 64, 0, u.head, u.row0);
                }
                // Every ring slot is waited for in order, also the suffix tiles' slots that the gather warps
                // fill: a waiter that skipped slots could otherwise test an mbarrier phase two behind.
                for (int t = 0; t < u.np + ns && ok; ++t) {
                    const int ks = kc % C::NK, vs = vc % C::NV;
                    ok = mbar_wait(&misc->k_empty[ks], ((kc / C::NK) & 1) ^ 1, misc);
                    if (!ok) break;
                    if (t < u.np) {
                        mbar_expect_tx(&misc->k_full[ks], C::TILE_BYTES);
                        for (int h = 0; h < C::HALVES; ++h)
                            tma_load_3d(smem + C::OFF_K + ks * C::TILE_BYTES + h * kHalfBytes, &map_k, &misc->k_full[ks],
                                        h * 64, u.head, u.kv_row0 + t * kTile);
                    }
                    ok = mbar_wait(&misc->v_empty[vs], ((vc / C::NV) & 1) ^ 1, misc);
                    if (!ok) break;
                    if (t < u.np) {
                        mbar_expect_tx(&misc->v_full[vs], C::TILE_BYTES);
                        for (int h = 0; h < C::HALVES; ++h)
                            tma_load_3d(smem + C::OFF_V + vs * C::TILE_BYTES + h * kHalfBytes, &map_v, &misc->v_full[vs],
                                        h * 64, u.head, u.kv_row0 + t * kTile);
                    }
                    ++kc; ++vc;
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            kc = __shfl_sync(0xffffffffu, kc, 0);
            vc = __shfl_sync(0xffffffffu, vc, 0);
            ++qi;
        }
    } else if (warp == 1) {
        // ======================================== MMA issuer ========================================
        uint32_t qi = 0, kc = 0, vc = 0, sc = 0, pc = 0;
        bool ok = true;
        const uint32_t q_addr = smem_u32(smem + C::OFF_Q), p_addr = smem_u32(smem + C::OFF_P);
        for (int w = blockIdx.x; w < n_units && ok; w += gridDim.x) {
            const Unit u = load_unit(p, w);
            const int stot = suffix_total_warp(p, u, lane);
            const int ns = (stot + kTile - 1) / kTile;
            const int nt = u.np + ns;
            if (nt == 0) continue;
            if (lane == 0) {
                ok = mbar_wait(&misc->q_full, qi & 1, misc);
                auto tile_cols = [&](int j) {
                    return j < u.np ? min(kTile, u.key_count - j * kTile) : min(kTile, stot - (j - u.np) * kTile);
                };
                auto issue_qk = [&](int j) {
                    const int ks = kc % C::NK, sb = sc & 1;
                    if (!mbar_wait(&misc->k_full[ks], (kc / C::NK) & 1, misc)) return false;
                    if (!mbar_wait(&misc->s_empty[sb], ((sc >> 1) & 1) ^ 1, misc)) return false;
                    tc_fence_after();
                    const int n_pad = (tile_cols(j) + 15) & ~15;
                    const uint32_t idesc = make_idesc(n_pad, 0);
                    const uint32_t k_addr = smem_u32(smem + C::OFF_K + ks * C::TILE_BYTES);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
                        tc_mma(tmem + sb * kTile, desc_kmajor(q_addr + off), desc_kmajor(k_addr + off), idesc, k > 0);
                    }
                    tc_commit(&misc->k_empty[ks]);
                    tc_commit(&misc->s_full[sb]);
                    if (j == nt - 1) tc_commit(&misc->q_empty);
                    ++kc; ++sc;
                    return true;
                };
                if (ok) ok = issue_qk(0);
                for (int j = 0; j < nt && ok; ++j) {
                    if (j + 1 < nt) { ok = issue_qk(j + 1); if (!ok) break; }
                    const int vs = vc % C::NV;
                    ok = mbar_wait(&misc->p_full, pc & 1, misc);
                    if (!ok) break;
                    ok = mbar_wait(&misc->v_full[vs], (vc / C::NV) & 1, misc);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t idesc = make_idesc(D, 1);
                    const uint32_t v_addr = smem_u32(smem + C::OFF_V + vs * C::TILE_BYTES);
                    const int nk = (tile_cols(j) + 15) >> 4;
                    for (int k = 0; k < nk; ++k) {
                        const uint32_t a_off = (k >> 2) * kHalfBytes + (k & 3) * 32;
                        tc_mma(tmem_o, desc_kmajor(p_addr + a_off), desc_mnmajor(v_addr + k * 2048), idesc, (j > 0 || k > 0));
                    }
                    tc_commit(&misc->v_empty[vs]);
                    tc_commit(&misc->p_empty);
                    ++vc; ++pc;
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            kc = __shfl_sync(0xffffffffu, kc, 0); vc = __shfl_sync(0xffffffffu, vc, 0);
            sc = __shfl_sync(0xffffffffu, sc, 0); pc = __shfl_sync(0xffffffffu, pc, 0);
            ++qi;
        }
    } else if (warp < 6) {
        // ========================================= softmax ==========================================
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;                // tile row = TMEM lane
        const int t128 = (warp - 2) * 32 + lane;         // index inside the role group (scan)
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        uint32_t sc = 0, pc_full = 0, pc_wait = 0;       // S tiles consumed, P tiles produced, PV completions waited
        uint8_t* p_tile = smem + C::OFF_P;
        bool ok = true;
        for (int w = blockIdx.x; w < n_units; w += gridDim.x) {
            if (!named_bar_and(1, ok)) break;            // uniform exit of the whole role group
            const Unit u = load_unit(p, w);
            const int stot = suffix_scan_group(p, u, misc, 0, t128, 1);
            const int ns = (stot + kTile - 1) / kTile;
            const int nt = u.np + ns;
            const int nrows = u.nb * G;
            const bool row_valid = row < nrows;
            const bool warp_active = quad * 32 < nrows;
            const int b = row / G, g = row - b * G;
            int my_cs = 0, my_len = 0;
            if (row_valid && u.with_suffix) { my_cs = misc->cs[0][b]; my_len = misc->cs[0][b + 1] - my_cs; }

            float m = -INFINITY, l = 0.f;
            for (int j = 0; j < nt && ok; ++j) {
                const int sb = sc & 1;
                ok = mbar_wait_warp(&misc->s_full[sb], (sc >> 1) & 1, misc);
                if (!ok) break;
                tc_fence_after();
                int lo = 0, hi = 0;
                if (row_valid) {
                    if (j < u.np) { hi = min(kTile, u.key_count - j * kTile); }
                    else {
                        const int base = (j - u.np) * kTile;
                        lo = max(0, my_cs - base);
                        hi = min(kTile, my_cs + my_len - base);
                        if (hi < lo) hi = lo;
                    }
                }
                uint32_t sv[kTile];
                if (warp_active) {
                    const uint32_t ta = tmem + lane_base + sb * kTile;
                    tmem_ld32(ta, sv); tmem_ld32(ta + 32, sv + 32); tmem_ld32(ta + 64, sv + 64); tmem_ld32(ta + 96, sv + 96);
                    tmem_ld_wait();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&misc->s_empty[sb]);
                ++sc;

                float lsum[4] = {0.f, 0.f, 0.f, 0.f};
                bool waited = false;
                if (warp_active) {
                    float tmax = -INFINITY;
                    const bool full = __all_sync(0xffffffffu, lo == 0 && hi == kTile);
                    if (full) {
#pragma unroll
                        for (int c = 0; c < kTile; ++c) tmax = fmaxf(tmax, __uint_as_float(sv[c]));
                    } else {
                        const unsigned span = static_cast<unsigned>(hi - lo);
#pragma unroll
                        for (int c = 0; c < kTile; ++c) {
                            const bool v = static_cast<unsigned>(c - lo) < span;
                            const float x = v ? __uint_as_float(sv[c]) : -INFINITY;
                            sv[c] = __float_as_uint(x);
                            tmax = fmaxf(tmax, x);
                        }
                    }
                    tmax *= p.scale_log2;
                    if (j == 0) {
                        m = tmax;
                    } else {
                        const bool grow = tmax > m + kRescaleSlack;
                        if (__any_sync(0xffffffffu, grow)) {
                            // O must be rescaled: wait until the previous P V product has landed in TMEM
                            ok = mbar_wait_warp(&misc->p_empty, pc_wait & 1, misc);
                            ++pc_wait; waited = true;
                            if (ok) {
                                tc_fence_after();
                                const float m_new = grow ? tmax : m;
                                const float f = grow ? ex2(m - m_new) : 1.f;
#pragma unroll
                                for (int c0 = 0; c0 < D; c0 += 32) {
                                    uint32_t ov[32];
                                    tmem_ld32(tmem_o + lane_base + c0, ov);
                                    tmem_ld_wait();
#pragma unroll
                                    for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * f);
                                    tmem_st32(tmem_o + lane_base + c0, ov);
                                }
                                tmem_st_wait();
                                l *= f;
                                m = m_new;
                            }
                        }
                    }
                }
                if (j > 0 && !waited) {
                    ok = ok && mbar_wait_warp(&misc->p_empty, pc_wait & 1, misc);   // previous P V has consumed the P tile
                    ++pc_wait;
                }
                if (!ok) break;
                if (warp_active) {
                    const float neg_m = (m == -INFINITY) ? 0.f : -m;
                    uint8_t* prow = p_tile + row * 128;
#pragma unroll
                    for (int kc8 = 0; kc8 < 16; ++kc8) {
                        float e[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            e[i] = ex2(fmaf(__uint_as_float(sv[kc8 * 8 + i]), p.scale_log2, neg_m));
                            lsum[i & 3] += e[i];
                        }
                        uint4 pk;
                        pk.x = pack_bf16(e[0], e[1]); pk.y = pack_bf16(e[2], e[3]);
                        pk.z = pack_bf16(e[4], e[5]); pk.w = pack_bf16(e[6], e[7]);
                        *reinterpret_cast<uint4*>(prow + (kc8 >> 3) * kHalfBytes + (((kc8 & 7) ^ (row & 7)) << 4)) = pk;
                    }
                    l += (lsum[0] + lsum[1]) + (lsum[2] + lsum[3]);
                    fence_async_smem();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&misc->p_full);
                ++pc_full;
            }
            if (!ok) continue;

            // -------- epilogue --------
            if (nt > 0) {
                ok = mbar_wait_warp(&misc->p_empty, pc_wait & 1, misc);
                ++pc_wait;
                if (!ok) continue;
                tc_fence_after();
            }
            const int grow_row = u.row0 + b;
            const bool store = row_valid && grow_row < p.a.max_rows;
            if (warp_active) {
                const int hq = u.head * G + g;
                if (u.part_base < 0) {
                    const float inv = l > 0.f ? 1.f / l : 0.f;
                    __nv_bfloat16* op = p.a.o + (static_cast<int64_t>(grow_row) * p.a.g.Hq + hq) * D;
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t ov[32];
                        if (nt > 0) { tmem_ld32(tmem_o + lane_base + c0, ov); tmem_ld_wait(); }
                        else {
#pragma unroll
                            for (int c = 0; c < 32; ++c) ov[c] = 0u;
                        }
                        if (store) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                uint4 pk;
                                pk.x = pack_bf16(__uint_as_float(ov[c + 0]) * inv, __uint_as_float(ov[c + 1]) * inv);
                                pk.y = pack_bf16(__uint_as_float(ov[c + 2]) * inv, __uint_as_float(ov[c + 3]) * inv);
                                pk.z = pack_bf16(__uint_as_float(ov[c + 4]) * inv, __uint_as_float(ov[c + 5]) * inv);
                                pk.w = pack_bf16(__uint_as_float(ov[c + 6]) * inv, __uint_as_float(ov[c + 7]) * inv);
                                *reinterpret_cast<uint4*>(op + c0 + c) = pk;
                            }
                        }
                    }
                    if (store && p.a.lse)
                        p.a.lse[static_cast<int64_t>(grow_row) * p.a.g.Hq + hq] = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
                } else {
                    const int64_t pr = (static_cast<int64_t>(u.part_base) + u.row_begin + b) * p.a.g.Hq + hq;
                    float* po = p.part_o + pr * D;
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t ov[32];
                        if (nt > 0) { tmem_ld32(tmem_o + lane_base + c0, ov); tmem_ld_wait(); }
                        else {
#pragma unroll
                            for (int c = 0; c < 32; ++c) ov[c] = 0u;
                        }
                        if (row_valid) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4)
                                *reinterpret_cast<uint4*>(po + c0 + c) = make_uint4(ov[c], ov[c + 1], ov[c + 2], ov[c + 3]);
                        }
                    }
                    if (row_valid) { p.part_ml[pr * 2] = m; p.part_ml[pr * 2 + 1] = l; }
                }
            }
            tc_fence_before();
        }
    } else {
        // ========================================== gather ==========================================
        const int t128 = (warp - 6) * 32 + lane;
        constexpr int CHUNKS = D / 8;                    // 16-byte chunks per row and head
        constexpr int COLS_PER_PASS = 128 / CHUNKS;
        const int chunk = t128 % CHUNKS, col_lane = t128 / CHUNKS;
        const int64_t cache_rows = static_cast<int64_t>(p.a.n_slots) * p.a.g.suffix_cap;
        const int64_t tok_stride = static_cast<int64_t>(p.a.g.Hkv) * D;
        uint32_t kc = 0, vc = 0;
        bool ok = true;
        for (int w = blockIdx.x; w < n_units; w += gridDim.x) {
            if (!named_bar_and(2, ok)) break;            // uniform exit of the whole role group
            const Unit u = load_unit(p, w);
            const int stot = suffix_scan_group(p, u, misc, 1, t128, 2);
            const int ns = (stot + kTile - 1) / kTile;
            const int* cs = misc->cs[1];
            // every ring slot is waited for in order (see the TMA producer); only suffix tiles are filled here
            for (int j = 0; j < u.np + ns; ++j) {
                const int ks = kc % C::NK, vs = vc % C::NV;
                bool w_ok = mbar_wait(&misc->k_empty[ks], ((kc / C::NK) & 1) ^ 1, misc);
                w_ok = mbar_wait(&misc->v_empty[vs], ((vc / C::NV) & 1) ^ 1, misc) && w_ok;
                ++kc; ++vc;
                if (j < u.np) { ok = ok && w_ok; continue; }
                ok = named_bar_and(2, ok && w_ok);
                if (!ok) break;
                const int s = j - u.np;
                const uint32_t k_dst = smem_u32(smem + C::OFF_K + ks * C::TILE_BYTES);
                uint8_t* v_gen = smem + C::OFF_V + vs * C::TILE_BYTES;
                const uint32_t v_dst = smem_u32(v_gen);
                const int valid = min(kTile, stot - s * kTile);
                const int padded = (valid + 15) & ~15;
                for (int cl = col_lane; cl < padded; cl += COLS_PER_PASS) {
                    const uint32_t off = (chunk >> 3) * kHalfBytes + cl * 128 + (((chunk & 7) ^ (cl & 7)) << 4);
                    if (cl < valid) {
                        const int c = s * kTile + cl;
                        int lo_b = 0, hi_b = u.nb;               // largest b with cs[b] <= c
                        while (hi_b - lo_b > 1) {
                            const int mid = (lo_b + hi_b) >> 1;
                            if (cs[mid] <= c) lo_b = mid; else hi_b = mid;
                        }
                        const int64_t srow = static_cast<int64_t>(p.a.suffix_off[u.row0 + lo_b]) + (c - cs[lo_b]);
                        if (srow >= 0 && srow < cache_rows) {
                            const int64_t e = srow * tok_stride + static_cast<int64_t>(u.head) * D + chunk * 8;
                            cp_async16(k_dst + off, p.a.suffix_k + e);
                            cp_async16(v_dst + off, p.a.suffix_v + e);
                        } else {
                            *reinterpret_cast<uint4*>(v_gen + off) = make_uint4(0, 0, 0, 0);
                            if (p.a.dev_status) atomicOr(p.a.dev_status, HPD_S_BAD_TABLE);
                        }
                    } else {
                        *reinterpret_cast<uint4*>(v_gen + off) = make_uint4(0, 0, 0, 0);   // padding keys: 0 * V must stay 0
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                fence_async_smem();
                named_bar(2);
                if (t128 == 0) { mbar_arrive(&misc->k_full[ks]); mbar_arrive(&misc->v_full[vs]); }
            }
        }
    }

    // ---------------------------------------- teardown ----------------------------------------
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (misc->abort_flag) {
        if (threadIdx.x == 0 && p.a.dev_status) atomicOr(p.a.dev_status, HPD_S_TIMEOUT);
        // give copies that may still be in flight time to land before the shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 20000000ll) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// Merge of the partial results of documents whose prefix was split over several work items.
template <int D>
__global__ void __launch_bounds__(256)
hpd_merge_kernel(TcParams p, const DocSplit* __restrict__ split)
{
    if (!p.hdr->any_split) return;
    const int lane = threadIdx.x & 31;
    const int Hq = p.a.g.Hq;
    const int64_t n_w = static_cast<int64_t>(*p.a.n_active) * Hq;
    constexpr int E = D / 32;
    for (int64_t w = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5); w < n_w; w += static_cast<int64_t>(gridDim.x) * 8) {
        const int r = static_cast<int>(w / Hq), h = static_cast<int>(w % Hq);
        const int d = p.a.doc_id[r];
        const DocSplit sp = split[d];
        if (sp.n_chunks <= 1) continue;
        const int rows_d = p.a.doc_active_start[d + 1] - p.a.doc_active_start[d];
        const int rl = r - p.a.doc_active_start[d];
        float M = -INFINITY;
        for (int c = 0; c < sp.n_chunks; ++c) {
            const int64_t pr = (static_cast<int64_t>(sp.part_base) + static_cast<int64_t>(c) * rows_d + rl) * Hq + h;
            M = fmaxf(M, p.part_ml[pr * 2]);
        }
        float L = 0.f, acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        for (int c = 0; c < sp.n_chunks; ++c) {
            const int64_t pr = (static_cast<int64_t>(sp.part_base) + static_cast<int64_t>(c) * rows_d + rl) * Hq + h;
            const float mc = p.part_ml[pr * 2];
            const float f = mc == -INFINITY ? 0.f : exp2f(mc - M);
            L += f * p.part_ml[pr * 2 + 1];
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] = fmaf(f, p.part_o[pr * D + lane * E + e], acc[e]);
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        __nv_bfloat16* op = p.a.o + w * D + lane * E;
        if constexpr (E == 4) {
            uint2 v;
            v.x = pack_bf16(acc[0] * inv, acc[1] * inv);
            v.y = pack_bf16(acc[2] * inv, acc[3] * inv);
            *reinterpret_cast<uint2*>(op) = v;
        } else {
            *reinterpret_cast<uint32_t*>(op) = pack_bf16(acc[0] * inv, acc[1] * inv);
        }
        if (p.a.lse && lane == 0) p.a.lse[w] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
    }
}

// ------------------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ------------------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 encode_fn()
{
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
    });
    return fn;
}

// K/V [tokens, Hkv, D] bf16: boxes of 128 tokens x 1 head x 64 elements, 128-byte swizzle
bool make_kv_map(CUtensorMap* m, const void* base, int D, int Hkv, long long tokens)
{
    auto fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(Hkv), static_cast<cuuint64_t>(tokens > 0 ? tokens : 1)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(Hkv) * D * 2};
    cuuint32_t box[3] = {64, 1, kTile};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q [rows, Hkv, G, D] bf16: boxes of 128/G rows x 1 kv head x G x 64 elements -> tile row = branch*G + g
bool make_q_map(CUtensorMap* m, const void* base, int D, int G, int Hkv, long long rows)
{
    auto fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(G), static_cast<cuuint64_t>(Hkv),
                          static_cast<cuuint64_t>(rows > 0 ? rows : 1)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(G) * D * 2,
                             static_cast<cuuint64_t>(Hkv) * G * D * 2};
    cuuint32_t box[4] = {64, static_cast<cuuint32_t>(G), 1, static_cast<cuuint32_t>(kTile / G)};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
int launch_d(const AttnArgs& a)
{
    using C = Cfg<D>;
    static bool attr_set = false;
    if (!attr_set) {
        HPD_CUDA_TRY(cudaFuncSetAttribute(hpd_attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
        attr_set = true;
    }
    const int G = a.g.Hq / a.g.Hkv;
    CUtensorMap mq, mk, mv;
    const void* kbase = a.total_prefix > 0 ? static_cast<const void*>(a.prefix_k) : static_cast<const void*>(a.suffix_k);
    const void* vbase = a.total_prefix > 0 ? static_cast<const void*>(a.prefix_v) : static_cast<const void*>(a.suffix_v);
    if (!make_q_map(&mq, a.q, D, G, a.g.Hkv, a.max_rows) || !make_kv_map(&mk, kbase, D, a.g.Hkv, a.total_prefix) ||
        !make_kv_map(&mv, vbase, D, a.g.Hkv, a.total_prefix)) {
        set_last_cuda_error(cudaErrorInvalidValue);
        return HPD_E_CUDA;
    }
    TcParams p{};
    p.a = a;
    char* ws = static_cast<char*>(a.workspace);
    p.hdr = reinterpret_cast<const WsHeader*>(ws);
    p.work = reinterpret_cast<const WorkItem*>(ws + a.lay.off_work);
    p.part_ml = reinterpret_cast<float*>(ws + a.lay.off_ml);
    p.part_o = reinterpret_cast<float*>(ws + a.lay.off_o);
    p.scale_log2 = a.g.sm_scale * kLog2e;
    p.G = G;
    const int n_sm = sm_count();
    hpd_attn_tc_kernel<D><<<n_sm, kThreads, C::SMEM, a.stream>>>(mq, mk, mv, p);
    hpd_merge_kernel<D><<<n_sm * 2, 256, 0, a.stream>>>(p, reinterpret_cast<const DocSplit*>(ws + a.lay.off_split));
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

}  // namespace

int launch_attn_tc(const AttnArgs& a)
{
    if (!(a.g.sm_scale > 0.f)) return HPD_E_GEOM;
    return a.g.D == 128 ? launch_d<128>(a) : launch_d<64>(a);
}

}  // namespace hpd
