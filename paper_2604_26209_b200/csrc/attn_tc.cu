// hpd_attn_decode on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
// One persistent CTA per SM runs two independent pipelines, each of which walks work units of its
// own.  A unit = (work item, kv head): up to 128/G branches of one document (rows = branches x G
// query heads, the M dimension) against a chunk of that document's prefix, so each prefix K/V byte
// is read from HBM once for all of the document's branches.  Keys are consumed in tiles of 64:
// first the tiles into which the branches' own cached tokens ("suffix") are packed back to back,
// one TMA box of the exact height (1..16 cache rows) per branch and half of D, masked
// block-diagonally (a row sees only its own branch's columns; in the position-order mode the
// columns of every slot up to its own); then the prefix tiles.  The
// suffix tiles come first because their many small copies are slow to issue and can be issued
// while the pipeline's previous unit is still being finished.
//
// Per unit a pipeline is latency-bound (one thread per row in the softmax, one thread issuing the
// MMAs, a serial epilogue); two of them on one SM overlap each other's waits and epilogues, which
// is what keeps HBM busy.  A pipeline owns a Q tile, a K and a V ring (shared memory), two score
// tiles and an output accumulator (tensor memory), and these warps:
//
//   warp 0 / 3    scheduler and TMA producer: draws the pipeline's units, publishes their
//                 descriptors, issues Q, K and V tiles (prefix: lane 0; suffix boxes: all lanes)
//   warp 1 / 2    MMA issuer: S = Q K^T (both operands in shared memory), two tiles ahead of the
//                 softmax, and O += P V (P in tensor memory, V in shared memory); tcgen05.mma
//   warps 4-7 /   softmax: one thread per row: S from TMEM, online max/sum, P as bf16 pairs written
//   warps 8-11    over the first half of the row's own scores, rare rescale of O in TMEM; epilogue:
//                 O / sum -> bf16 -> shared -> global
//
// TMEM columns of a pipeline (second pipeline + 256): S0 [0,64)  S1 [64,128)  O [128,256); the
// probabilities of a tile occupy the first 32 columns of the score tile they were computed from.
//
// All waits are bounded: a wait that gives up raises HPD_S_TIMEOUT in the status word and the CTA
// drains and exits (TMEM is released on every path).
#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "ptx.cuh"

namespace hpd {

namespace {

constexpr int kWarps = 12;
constexpr int kThreads = kWarps * 32;
constexpr int kM = 128;                    // rows of a tile
constexpr int kN = 64;                     // keys of a tile
constexpr int kQHalf = kM * 128;           // one 64-element half of the Q tile: 128 rows x 128 B
constexpr int kKHalf = kN * 128;           // one 64-element half of a K or V tile: 64 keys x 128 B
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleSlack = 8.0f;      // tolerated growth of the row maximum (log2 units) before O is rescaled
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s at 2 GHz
// TMEM columns of one pipeline (the second pipeline's start 256 columns further): two score tiles of 64 columns (the
// probabilities of a tile, bf16 pairs, overwrite the first 32 columns of its scores) and the output accumulator
constexpr uint32_t kColPipe = 256, kColS = 0, kColO = 128;
// registers per thread after the warpgroups have traded them (3 x 128 threads, 168 each at launch)
constexpr int kRegsIo = 104, kRegsSoftmax = 200;
// setmaxnreg only moves registers inside the CTA's own allocation (168 x 384 threads at launch): a request beyond
// that pool would block forever; using the pool exactly is fine
static_assert(kRegsIo + 2 * kRegsSoftmax <= 3 * 168, "registers traded between the warpgroups exceed the CTA's allocation");
constexpr int kRounds = 4;                 // a unit has at most 128 branches: 4 rounds of 32 lanes
constexpr int kDescReaders = 5;            // readers of a pipeline's unit descriptor: its MMA thread and its four softmax warps
constexpr int kMaxStages = 4;              // K or V stages of one pipeline (barrier storage)

template <int D> struct Cfg {
    static constexpr int HALVES = D / 64;
    static constexpr int Q_BYTES = HALVES * kQHalf;
    static constexpr int KV_BYTES = HALVES * kKHalf;            // one K or V tile
    static constexpr int NK = D == 128 ? 2 : 4;                  // K stages of each pipeline
    static constexpr int NV = D == 128 ? 2 : 4;                  // V stages of each pipeline
    static constexpr int OFF_Q = 0;                              // one Q tile per pipeline
    static constexpr int OFF_STAGE = OFF_Q + 2 * Q_BYTES;       // output transpose, 2 KB per softmax warp
    static constexpr int OFF_K = OFF_STAGE + 8 * 2048;
    static constexpr int OFF_V = OFF_K + 2 * NK * KV_BYTES;
    static constexpr int OFF_MISC = OFF_V + 2 * NV * KV_BYTES;
    static constexpr int SMEM = OFF_MISC + 4096;                 // + misc; the dynamic segment itself is 1024-B aligned
    static_assert(NK <= kMaxStages && NV <= kMaxStages, "barrier storage");
};
static_assert(Cfg<128>::SMEM <= 232448, "shared memory budget");

struct SufMaps {                            // tensor maps of the branch cache, one per box height: 1 .. 16 rows
    CUtensorMap k[16];
    CUtensorMap v[16];
};

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
// Unit descriptors.  A pipeline's producer warp draws work units from the step's ticket counter, gathers
// everything the other roles need to know about a unit -- tile counts, first rows, and per branch the
// number of cached tokens and the packed column of its first token -- and publishes it in the pipeline's
// shared-memory slot.  The MMA thread and the softmax warps copy what they need into registers at the start
// of the unit and release the slot at once, so no role ever waits for a dependent global load.
// ------------------------------------------------------------------------------------------------
struct UnitDesc {
    int nt;          // tiles of the unit (prefix + suffix); -1: no more units
    int np;          // prefix tiles
    int stot;        // cached tokens of all branches (= packed suffix columns)
    int head, key_count, part_base, row_begin, nb /*branches*/;
    int row0;        // first global row
    int kv_row0;     // first global prefix token row
    int blk_count;   // tokens of the block shared by several documents that precede this unit's prefix chunk (0: none)
    int blk_row0;    // first token row of that block in the block tensors
    uint16_t cs[kM];     // per branch: packed column of its first cached token
    uint16_t len[kM];    // per branch: cached tokens visible (0 for a bad table entry)
    // position-order mode: the branches above are ALL slots of the group up to the unit's last row (live or retired);
    uint16_t ridx[kM];   // per row-branch of the unit: its index among them
    int32_t pvis[kM];    // per row-branch: prefix tokens of this unit's chunk it may see
};
static_assert(sizeof(UnitDesc) == 48 + 10 * kM, "descriptor size");

struct Misc {
    unsigned long long q_full[2], q_empty[2];
    unsigned long long k_full[2][kMaxStages], k_empty[2][kMaxStages], v_full[2][kMaxStages], v_empty[2][kMaxStages];
    unsigned long long s_full[2][2], p_full[2][2], p_empty[2][2], o_full[2], o_free[2];
    unsigned long long desc_full[2], desc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int pad[2];
    UnitDesc desc[2];    // one per pipeline
};

static_assert(sizeof(Misc) <= 4096, "misc block");

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
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

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One tcgen05.mma; the two shared-memory descriptors are given as their low words (address and LBO fields, see
// below), the high word is the same for every operand of this kernel.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
                 "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(0x40004040u) : "memory");
}

// The same with the A operand in tensor memory (the probabilities, written there by the softmax threads).
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
                 "mov.b64 db, {%2, %5};\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(0x40004040u) : "memory");
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
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), HPD_W8(v, 0), HPD_W8(v, 8) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
template <int N> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

// Shared-memory matrix descriptors (128-byte swizzle; version field = 1).  High word, common to all operands:
// SBO = 1024 B (groups of 8 rows), version 1, swizzle mode 2 (128 B) = 0x40004040.  Low word: address / 16 in bits
// 0-13 and LBO / 16 in bits 16-29.  Shared-memory addresses are below 2^18, so moving a descriptor by a multiple
// of 16 bytes inside a tile is a plain addition to the low word.
//   K-major  (Q, K, P): rows of 128 B; LBO unused (1).
//   MN-major (V):       rows (keys) of 128 B holding 64 head-dim elements; the next 64 head-dim elements one tile
//                       half further (LBO).
__device__ __forceinline__ uint32_t desc_lo_kmajor(uint32_t saddr) { return (saddr >> 4) | (1u << 16); }
__device__ __forceinline__ uint32_t desc_lo_mnmajor(uint32_t saddr) { return (saddr >> 4) | (static_cast<uint32_t>(kKHalf >> 4) << 16); }
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N given; B either K-major (Q K^T) or MN-major (P V).
__device__ __forceinline__ uint32_t make_idesc(int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(b_mn_major) << 16) |
           (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(kM >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// per-unit bookkeeping
// ------------------------------------------------------------------------------------------------
struct Unit {        // the scalars of a descriptor, in registers
    int nt, np, stot, head, key_count, part_base, row_begin, nb, row0, kv_row0, blk_count, blk_row0;
};

__device__ __forceinline__ Unit read_unit(const UnitDesc& d) {
    Unit u;
    u.nt = d.nt; u.np = d.np; u.stot = d.stot; u.head = d.head; u.key_count = d.key_count; u.part_base = d.part_base;
    u.row_begin = d.row_begin; u.nb = d.nb; u.row0 = d.row0; u.kv_row0 = d.kv_row0;
    u.blk_count = d.blk_count; u.blk_row0 = d.blk_row0;
    return u;
}

// One K or V tile of a unit.  A prefix tile is two boxes issued by lane 0; a suffix tile is packed from one box per
// branch (and half), every lane placing the part of its branches that falls into the tile.  Boxes have the exact height
// of the piece (tensor maps for 1..16 rows), so nothing beyond a branch's length is ever read: whatever lies there in
// the cache -- possibly NaN -- must not meet a zero probability, and the packing needs no padding.
// Tile order of a unit: the suffix tiles, the tiles of the shared block (if any), the tiles of the document's prefix chunk.
__device__ __forceinline__ int block_tiles(const Unit& u) { return (u.blk_count + kN - 1) / kN; }

template <int D>
__device__ __forceinline__ void fill_tile(const Unit& u, int t, const int (&cs)[kRounds], const int (&len)[kRounds], const int (&off)[kRounds],
                                          int nrounds, int lane, uint8_t* tile, unsigned long long* full, const CUtensorMap* pre,
                                          const CUtensorMap* blk, const CUtensorMap* suf)
{
    using C = Cfg<D>;
    const int nbt = block_tiles(u);
    const int ns = u.nt - u.np - nbt;
    if (t >= ns) {
        if (lane == 0) {
            mbar_expect_tx(full, C::KV_BYTES);
            const bool in_block = t - ns < nbt;
            const CUtensorMap* m = in_block ? blk : pre;
            const int row = in_block ? u.blk_row0 + (t - ns) * kN : u.kv_row0 + (t - ns - nbt) * kN;
            for (int h = 0; h < C::HALVES; ++h)
                tma_load_3d(tile + h * kKHalf, m, full, h * 64, u.head, row);
        }
    } else {
        // the packing has no gaps: every column of [c_lo, c_hi) is some branch's cached token, so the tile receives
        // exactly c_hi - c_lo rows
        const int c_lo = t * kN, c_hi = min(u.stot, c_lo + kN);
        if (lane == 0) mbar_expect_tx(full, static_cast<uint32_t>(c_hi - c_lo) * D * 2);
#pragma unroll
        for (int r = 0; r < kRounds; ++r) {
            if (r >= nrounds) break;                     // rounds of 32 branches beyond the unit's last branch
            const int lo = max(cs[r], c_lo), hi = min(cs[r] + len[r], c_hi);
            int n = hi - lo;
            int row = off[r] + (lo - cs[r]);
            int col = lo - c_lo;
            while (n > 0) {
                const int hb = min(n, 16);
                const CUtensorMap* m = &suf[hb - 1];
                for (int h = 0; h < C::HALVES; ++h)
                    tma_load_3d(tile + h * kKHalf + col * 128, m, full, h * 64, u.head, row);
                row += hb; col += hb; n -= hb;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
// ORDER = false: branch-local mask (Eq. 5-6): a row sees its document's prefix and its own branch's cached tokens.
// ORDER = true:  position-order mask (Sec. 4.3.2, Fig. 3): a group is a whole stacked prompt; a row sees the first
//                prefix_vis[row] prefix tokens (prompt and the skeleton up to its own attribute key) and the cached
//                tokens of every slot of the group up to and including its own -- live or retired --, which is "position
//                ID not larger than mine" under Algorithm 2's K_max gaps.  Branch tokens are packed back to back in slot
//                order, so a row's visible packed columns are one range starting at 0.
// BLOCK = true:  a third sharing level (Sec. 4.3.5): the documents' prefixes are preceded by a block of tokens common to
//                several documents (instruction, attribute definitions), stored once in tensors of its own; a unit visits the
//                block's tiles between its suffix tiles and its document's tiles.
template <int D, bool ORDER, bool BLOCK>
__global__ void __launch_bounds__(kThreads, 1)
hpd_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_bk,
                   const __grid_constant__ CUtensorMap map_bv, const __grid_constant__ SufMaps smaps, const TcParams p)
{
    using C = Cfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    Misc* misc = reinterpret_cast<Misc*>(smem + C::OFF_MISC);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.G;
    if ((smem_u32(smem) & 1023u) != 0) {                 // swizzled tiles need 1024-byte alignment: refuse rather than misread
        if (threadIdx.x == 0 && p.a.dev_status) atomicOr(p.a.dev_status, HPD_S_BAD_TABLE);
        return;
    }

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&misc->q_full[i], 1);  mbar_init(&misc->q_empty[i], 1);
            for (int b = 0; b < 2; ++b) { mbar_init(&misc->s_full[i][b], 1); mbar_init(&misc->p_full[i][b], 4); mbar_init(&misc->p_empty[i][b], 1); }
            mbar_init(&misc->o_full[i], 1);  mbar_init(&misc->o_free[i], 4);
            mbar_init(&misc->desc_full[i], 1); mbar_init(&misc->desc_empty[i], kDescReaders);
            for (int k = 0; k < kMaxStages; ++k) {
                mbar_init(&misc->k_full[i][k], 1); mbar_init(&misc->k_empty[i][k], 1);
                mbar_init(&misc->v_full[i][k], 1); mbar_init(&misc->v_empty[i][k], 1);
            }
        }
        misc->abort_flag = 0;
        fence_mbar_init();
    }
    // stale tile contents are multiplied by zero probabilities: they must be finite from the start
    for (int i = threadIdx.x; i < (C::OFF_MISC - C::OFF_K) / 16; i += kThreads)
        reinterpret_cast<uint4*>(smem + C::OFF_K)[i] = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&misc->tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&misc->tmem_base);

    if (warp == 0 || warp == 3) {
        // ============================ scheduler and TMA producer of one pipeline =====================
        // Software pipeline over the pipeline's units, one stage per iteration, so that every global load is
        // consumed an iteration after it was issued: ticket (i+4) -> work item (i+3) -> document tables (i+2) ->
        // branch table (i+1) -> scan, publish and produce the tiles (i).  (An iteration lasts a whole unit, ten
        // microseconds or more, so one stage per iteration is ample for an L2 round trip.)
        reg_dealloc<kRegsIo>();
        const int x = warp == 0 ? 0 : 1;
        const int n_units = p.hdr->n_work * p.a.g.Hkv;
        const int Hkv = p.a.g.Hkv;
        const int64_t cache_rows = static_cast<int64_t>(p.a.n_slots) * p.a.g.suffix_cap;
        uint32_t* ticket = const_cast<uint32_t*>(&p.hdr->ticket);
        UnitDesc& d = misc->desc[x];
        uint8_t* k_ring = smem + C::OFF_K + x * C::NK * C::KV_BYTES;
        uint8_t* v_ring = smem + C::OFF_V + x * C::NV * C::KV_BYTES;
        uint8_t* q_tile = smem + C::OFF_Q + x * C::Q_BYTES;
        if (n_units == 0) {                              // nothing to do: publish the stop descriptor
            if (lane == 0) { d.nt = -1; mbar_arrive(&misc->desc_full[x]); }
        } else {
        // The first units of a pipeline are fixed (round i hands unit i * 2 * grid + j to the j-th pipeline; when the
        // list comes longest unit first, j counts upwards in even rounds and downwards in odd ones, which keeps the
        // pipelines' sums level), which fills the software pipeline without a chain of atomics and measured
        // slightly faster than drawing early; later units are drawn from the step's ticket counter, so faster SMs
        // (and the pipelines that got shorter units) take more.
        constexpr int kStatic = 6;
        const bool alternate = p.hdr->longest_first != 0;
        const uint32_t first_dynamic = static_cast<uint32_t>(kStatic) * 2u * gridDim.x;
        auto draw = [&]() {                              // next unit index (lane 0 draws, all lanes get it)
            uint32_t t = 0;
            if (lane == 0) t = atomicAdd(ticket, 1u);
            t = __shfl_sync(0xffffffffu, t, 0);
            return static_cast<int>(min(t + first_dynamic, static_cast<uint32_t>(n_units)));
        };
        auto fixed = [&](int i) {
            const uint32_t j = 2u * blockIdx.x + static_cast<uint32_t>(x);
            const uint32_t in_round = ((i & 1) && alternate) ? 2u * gridDim.x - 1u - j : j;
            return static_cast<int>(min(in_round + static_cast<uint32_t>(i) * 2u * gridDim.x, static_cast<uint32_t>(n_units)));
        };
        int w0 = fixed(0), w1 = fixed(1), w2 = fixed(2), w3 = fixed(3);
        auto item_of = [&](int w) { return p.work[min(w, max(n_units - 1, 0)) / Hkv]; };
        WorkItem it2 = item_of(w2), it1 = item_of(w1), it0 = item_of(w0);
        int das1 = p.a.doc_active_start[it1.doc], dks1 = p.a.doc_kv_start[it1.doc];
        int das0 = p.a.doc_active_start[it0.doc], dks0 = p.a.doc_kv_start[it0.doc];
        // shared block of the unit's document: its id one stage ahead of its first row and length
        int blk1 = 0, bks0 = 0, bln0 = 0;
        if constexpr (BLOCK) {
            blk1 = p.a.doc_block[it1.doc];
            const int blk0 = p.a.doc_block[it0.doc];
            bks0 = p.a.block_kv_start[blk0]; bln0 = p.a.block_len[blk0];
        }
        // position-order mode: first slot of the group and of the next one
        int dss1 = 0, dse1 = 0, dss0 = 0, dse0 = 0;
        const bool have_slots = ORDER && p.a.slot_depth != nullptr;      // false: no branch cache at all (the prefill)
        if (have_slots) {
            dss1 = p.a.doc_slot_start[it1.doc]; dse1 = p.a.doc_slot_start[it1.doc + 1];
            dss0 = p.a.doc_slot_start[it0.doc]; dse0 = p.a.doc_slot_start[it0.doc + 1];
        }
        // raw branch table of unit i.  Branch-local mode: per row, cached tokens (rl) and slab start (ro).  Position-order
        // mode: per slot of the group, cached tokens (rl) and the live flag (ro); per row, its slot (rs) and visible prefix (rp).
        int rl0[kRounds], ro0[kRounds], rs0[ORDER ? kRounds : 1], rp0[ORDER ? kRounds : 1];
        auto load_tab = [&](int w, const WorkItem& it, int das, int dss, int dse, int* rl, int* ro, int* rs, int* rp) {
#pragma unroll
            for (int r = 0; r < kRounds; ++r) {
                const int b = lane + 32 * r;
                rl[r] = 0; ro[r] = 0;
                if constexpr (ORDER) {
                    rs[r] = -1; rp[r] = 0;
                    if (w < n_units && b < it.row_count) {
                        const int row = das + it.row_begin + b;
                        rs[r] = have_slots ? p.a.active_slot[row] : 0;
                        rp[r] = p.a.prefix_vis[row];
                    }
                    if (have_slots && w < n_units && it.with_suffix && b < dse - dss) {
                        rl[r] = p.a.slot_depth[dss + b];
                        ro[r] = p.a.slot_alive[dss + b];
                    }
                } else {
                    if (w < n_units && it.with_suffix && b < it.row_count) {
                        const int row = das + it.row_begin + b;
                        rl[r] = p.a.suffix_len[row];
                        ro[r] = p.a.suffix_off[row];
                    }
                }
            }
        };
        load_tab(w0, it0, das0, dss0, dse0, rl0, ro0, rs0, rp0);
        uint32_t qc = 0, kc = 0, vc = 0;
        bool ok = true;
        for (uint32_t ui = 0; ok; ++ui) {
            // ---- issue the next stage of every unit in flight (results are used in the next iteration) ----
            const int w4 = static_cast<int>(ui) + 4 < kStatic ? fixed(static_cast<int>(ui) + 4) : draw();
            const WorkItem it3 = item_of(w3);
            const int das2 = p.a.doc_active_start[it2.doc], dks2 = p.a.doc_kv_start[it2.doc];
            int dss2 = 0, dse2 = 0;
            if (have_slots) { dss2 = p.a.doc_slot_start[it2.doc]; dse2 = p.a.doc_slot_start[it2.doc + 1]; }
            int rl1[kRounds], ro1[kRounds], rs1[ORDER ? kRounds : 1], rp1[ORDER ? kRounds : 1];
            load_tab(w1, it1, das1, dss1, dse1, rl1, ro1, rs1, rp1);
            int blk2 = 0, bks1 = 0, bln1 = 0;
            if constexpr (BLOCK) {
                blk2 = p.a.doc_block[it2.doc];
                bks1 = p.a.block_kv_start[blk1]; bln1 = p.a.block_len[blk1];
            }
            // ---- finish unit i: clamp, validate, scan, publish ----
            if (ui >= 1) {                               // the pipeline's consumers have copied the previous descriptor
                ok = mbar_wait_warp(&misc->desc_empty[x], (ui - 1) & 1, misc);
                if (!ok) break;
            }
            const bool live = w0 < n_units;
            int cs[kRounds], len[kRounds], off[kRounds];
            int carry = 0, bad = 0;
            int nbr = 0;                                 // position-order mode: slots of the group the unit's rows may see
            if constexpr (ORDER) {
                int last = -1;                           // index in the group of the unit's last row's slot
#pragma unroll
                for (int r = 0; r < kRounds; ++r) {
                    const int b = lane + 32 * r;
                    const int idx = (live && b < it0.row_count) ? rs0[r] - dss0 : -1;
                    if (b == it0.row_count - 1) last = idx;
                    if (have_slots && live && b < it0.row_count && (idx < 0 || idx >= kM || idx >= dse0 - dss0)) bad = 1;   // group too large or bad table
                    d.ridx[b] = static_cast<uint16_t>(idx < 0 || idx >= kM ? 0 : idx);
                    d.pvis[b] = (live && b < it0.row_count) ? rp0[r] - it0.key_begin : 0;
                }
                last = __reduce_max_sync(0xffffffffu, last);
                nbr = (have_slots && live && it0.with_suffix && last < kM) ? last + 1 : 0;
            }
#pragma unroll
            for (int r = 0; r < kRounds; ++r) {
                const int b = lane + 32 * r;
                int n = 0, o = 0;
                if constexpr (ORDER) {
                    if (b < nbr) {
                        n = rl0[r] + (ro0[r] ? p.a.suffix_extra : 0);
                        n = n < 0 ? 0 : (n > p.a.g.suffix_cap ? p.a.g.suffix_cap : n);
                        const int64_t o64 = static_cast<int64_t>(dss0 + b) * p.a.g.suffix_cap;
                        if (o64 + n > cache_rows) { bad = 1; n = 0; } else { o = static_cast<int>(o64); }
                    }
                } else if (live && it0.with_suffix && b < it0.row_count) {
                    n = rl0[r] + p.a.suffix_extra;
                    n = n < 0 ? 0 : (n > p.a.g.suffix_cap ? p.a.g.suffix_cap : n);
                    o = ro0[r];
                    if (o < 0 || static_cast<int64_t>(o) + n > cache_rows) { bad = 1; n = 0; o = 0; }
                }
                int incl = n;                                // columns the branch occupies
#pragma unroll
                for (int s = 1; s < 32; s <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, s);
                    if (lane >= s) incl += v;
                }
                cs[r] = carry + incl - n; len[r] = n; off[r] = o;
                d.cs[b] = static_cast<uint16_t>(cs[r]);
                d.len[b] = static_cast<uint16_t>(n);
                carry += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (__any_sync(0xffffffffu, bad) && lane == 0 && p.a.dev_status) atomicOr(p.a.dev_status, HPD_S_BAD_TABLE);
            const int nrounds = ((ORDER ? nbr : ((live && it0.with_suffix) ? it0.row_count : 0)) + 31) >> 5;
            Unit u;
            u.blk_count = (BLOCK && live && it0.key_begin == 0 && bln0 > 0) ? bln0 : 0;     // the block goes with the document's first chunk
            u.blk_row0 = bks0;
            u.np = live ? (it0.key_count + kN - 1) / kN : 0;
            u.nt = live ? u.np + block_tiles(u) + (carry + kN - 1) / kN : -1;
            u.stot = carry; u.head = w0 % Hkv; u.key_count = it0.key_count; u.part_base = it0.part_base;
            u.row_begin = it0.row_begin; u.nb = it0.row_count;
            u.row0 = das0 + it0.row_begin; u.kv_row0 = dks0 + it0.key_begin;
            if (lane == 0) {
                d.nt = u.nt; d.np = u.np; d.stot = u.stot; d.head = u.head; d.key_count = u.key_count; d.part_base = u.part_base;
                d.row_begin = u.row_begin; d.nb = u.nb; d.row0 = u.row0; d.kv_row0 = u.kv_row0;
                d.blk_count = u.blk_count; d.blk_row0 = u.blk_row0;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&misc->desc_full[x]);
            if (!live) break;
            // ---- the unit's tiles: K runs one tile ahead of V, the order in which the MMA warp consumes them ----
            const int nt = u.nt;
            for (int t = 0; t <= nt && ok; ++t) {
                if (t < nt) {
                    const int ks = kc % C::NK;
                    ok = mbar_wait_warp(&misc->k_empty[x][ks], ((kc / C::NK) & 1) ^ 1, misc);
                    if (!ok) break;
                    fill_tile<D>(u, t, cs, len, off, nrounds, lane, k_ring + ks * C::KV_BYTES, &misc->k_full[x][ks], &map_k, &map_bk, smaps.k);
                    ++kc;
                    if (t == 0) {
                        // The Q tile is asked for after the unit's first K tile: its buffer is released late in the
                        // previous unit, and waiting for it first would hold up the tile that can be fetched already.
                        ok = mbar_wait_warp(&misc->q_empty[x], (qc & 1) ^ 1, misc);
                        if (!ok) break;
                        if (lane == 0) {
                            mbar_expect_tx(&misc->q_full[x], C::Q_BYTES);
                            for (int h = 0; h < C::HALVES; ++h)
                                tma_load_4d(q_tile + h * kQHalf, &map_q, &misc->q_full[x], h * 64, 0, u.head, u.row0);
                        }
                        ++qc;
                    }
                }
                if (t >= 1) {
                    const int vs = vc % C::NV;
                    ok = mbar_wait_warp(&misc->v_empty[x][vs], ((vc / C::NV) & 1) ^ 1, misc);
                    if (!ok) break;
                    fill_tile<D>(u, t - 1, cs, len, off, nrounds, lane, v_ring + vs * C::KV_BYTES, &misc->v_full[x][vs], &map_v, &map_bv, smaps.v);
                    ++vc;
                }
                __syncwarp();
            }
            // ---- shift the pipeline ----
            w0 = w1; w1 = w2; w2 = w3; w3 = w4;
            it0 = it1; it1 = it2; it2 = it3;
            das0 = das1; dks0 = dks1; das1 = das2; dks1 = dks2;
            if constexpr (ORDER) { dss0 = dss1; dse0 = dse1; dss1 = dss2; dse1 = dse2; }
            if constexpr (BLOCK) { bks0 = bks1; bln0 = bln1; blk1 = blk2; }
#pragma unroll
            for (int r = 0; r < kRounds; ++r) {
                rl0[r] = rl1[r]; ro0[r] = ro1[r];
                if constexpr (ORDER) { rs0[r] = rs1[r]; rp0[r] = rp1[r]; }
            }
        }
        }
    } else if (warp < 3) {
        // ================================ MMA issuers (one per pipeline) =============================
        reg_dealloc<kRegsIo>();
        if (lane == 0) {
            const int x = warp - 1;
            uint32_t qc = 0, tiles = 0;                   // units with tiles so far; tiles of earlier units
            uint32_t sc = 0, pc = 0;                      // S tiles issued, P tiles consumed
            bool ok = true;
            const uint32_t q_lo = desc_lo_kmajor(smem_u32(smem + C::OFF_Q + x * C::Q_BYTES));
            const uint32_t k_lo0 = desc_lo_kmajor(smem_u32(smem + C::OFF_K + x * C::NK * C::KV_BYTES));
            const uint32_t v_lo0 = desc_lo_mnmajor(smem_u32(smem + C::OFF_V + x * C::NV * C::KV_BYTES));
            const uint32_t tmem_s = tmem + x * kColPipe + kColS, tmem_o = tmem + x * kColPipe + kColO;
            const uint32_t idesc_pv = make_idesc(D, 1);
            for (uint32_t ui = 0; ok; ++ui) {
                ok = mbar_wait(&misc->desc_full[x], ui & 1, misc);
                if (!ok) break;
                const Unit u = read_unit(misc->desc[x]);
                mbar_arrive(&misc->desc_empty[x]);
                if (u.nt < 0) break;
                const int nt = u.nt;
                if (nt == 0) continue;
                const int nbt = BLOCK ? block_tiles(u) : 0;
                const int ns = nt - u.np - nbt;
                // columns of tile j: only the last suffix tile, the last block tile and the last prefix tile can be partial
                const int last_s = u.stot - (ns - 1) * kN, last_p = u.key_count - (u.np - 1) * kN;
                const int last_b = u.blk_count - (nbt - 1) * kN;
                auto cols16 = [&](int j) {
                    int c = kN;
                    if (j == ns - 1) c = last_s;
                    else if (BLOCK && nbt > 0 && j == ns + nbt - 1) c = last_b;
                    else if (j == nt - 1 && u.np > 0) c = last_p;
                    return (c + 15) >> 4;
                };
                ok = mbar_wait(&misc->q_full[x], qc & 1, misc);
                ++qc;
                auto issue_qk = [&](int j) {
                    const uint32_t kt = tiles + j;
                    const int ks = kt % C::NK;
                    const uint32_t idesc = make_idesc(cols16(j) << 4, 0);
                    const uint32_t k_lo = k_lo0 + ks * (C::KV_BYTES >> 4);
                    if (!mbar_wait(&misc->k_full[x][ks], (kt / C::NK) & 1, misc)) return false;
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t qoff = ((k >> 2) * kQHalf + (k & 3) * 32) >> 4;
                        const uint32_t koff = ((k >> 2) * kKHalf + (k & 3) * 32) >> 4;
                        tc_mma(tmem_s + (sc & 1) * kN, q_lo + qoff, k_lo + koff, idesc, k > 0);
                    }
                    tc_commit(&misc->k_empty[x][ks]);
                    tc_commit(&misc->s_full[x][sc & 1]);
                    if (j + 1 >= nt) tc_commit(&misc->q_empty[x]);      // last use of the Q tile
                    ++sc;
                    return true;
                };
                // Scores run two tiles ahead: S(j+2) overwrites the tile in which S(j) was computed and P(j) was read,
                // and the tensor core executes this thread's MMAs in the order of issue, P(j) V(j) before it.
                if (ok) ok = issue_qk(0);
                if (ok && nt > 1) ok = issue_qk(1);
                for (int j = 0; j < nt && ok; ++j) {
                    const uint32_t vt = tiles + j;
                    const int vs = vt % C::NV;
                    const uint32_t v_lo = v_lo0 + vs * (C::KV_BYTES >> 4);
                    const int nk = cols16(j);
                    const uint32_t acc0 = j >= 1;
                    const int pb = pc & 1;
                    ok = mbar_wait(&misc->p_full[x][pb], (pc >> 1) & 1, misc);
                    if (!ok) break;
                    ok = mbar_wait(&misc->v_full[x][vs], (vt / C::NV) & 1, misc);
                    if (!ok) break;
                    if (j == 0 && ui > 0) {               // the previous unit's epilogue has read O
                        ok = mbar_wait(&misc->o_free[x], (ui - 1) & 1, misc);
                        if (!ok) break;
                    }
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < kN / 16; ++k)
                        if (k < nk) tc_mma_ts(tmem_o, tmem_s + pb * kN + k * 8, v_lo + k * 128, idesc_pv, k > 0 ? 1u : acc0);
                    tc_commit(&misc->v_empty[x][vs]);
                    tc_commit(&misc->p_empty[x][pb]);
                    if (j + 1 >= nt) tc_commit(&misc->o_full[x]);
                    ++pc;
                    if (j + 2 < nt) ok = issue_qk(j + 2);
                }
                tiles += nt;
            }
        }
    } else {
        // ======================================= softmax A / B =======================================
        reg_alloc<kRegsSoftmax>();
        const int x = warp >= 8 ? 1 : 0;                 // pipeline
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;                // tile row = TMEM lane
        const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tmem_s0 = tmem + lane_base + x * kColPipe + kColS;
        const uint32_t tmem_o = tmem + lane_base + x * kColPipe + kColO;
        uint8_t* stg = smem + C::OFF_STAGE + (x * 4 + quad) * 2048;      // this warp's output staging
        const int b_row = row / G;                       // branch of this row inside the unit
        const uint32_t g_magic = 0xFFFFFFFFu / static_cast<uint32_t>(G) + 1u;   // floor(r / G) = umulhi(r, g_magic) for r < 2^16, G > 1
        uint32_t pw = 0, of_cnt = 0;                     // tiles done (S read, P written), units with tiles
        bool ok = true;
        for (uint32_t unit_idx = 0; ok; ++unit_idx) {
            ok = mbar_wait_warp(&misc->desc_full[x], unit_idx & 1, misc);
            if (!ok) break;
            const Unit u = read_unit(misc->desc[x]);
            // branch-local mode: packed columns [my_cs, my_cs + my_len) hold this row's own cached tokens.  Position-order
            // mode: the row sees packed columns [0, my_cs + my_len) -- every slot up to its own -- and my_pv prefix tokens.
            int my_cs, my_len, my_pv = 0;
            if constexpr (ORDER) {
                const int ri = min(static_cast<int>(misc->desc[x].ridx[min(b_row, kM - 1)]), kM - 1);
                my_cs = 0;
                my_len = misc->desc[x].cs[ri] + misc->desc[x].len[ri];
                my_pv = misc->desc[x].pvis[min(b_row, kM - 1)];
            } else {
                my_cs = misc->desc[x].cs[b_row]; my_len = misc->desc[x].len[b_row];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&misc->desc_empty[x]);
            if (u.nt < 0) break;
            const int nt = u.nt;
            const int nrows = u.nb * G;
            const bool row_valid = row < nrows;
            const bool warp_active = quad * 32 < nrows;
            float m = -INFINITY, l = 0.f;
            for (int j = 0; j < nt && ok; ++j) {
                // Columns of this tile the row may see.  A suffix tile holds a few branches each; a warp whose rows see
                // none of them (known from the descriptor alone) skips the tile's scores and writes zero probabilities.
                int lo = 0, hi = 0;
                if (warp_active) {
                    const int nbt = BLOCK ? block_tiles(u) : 0;
                    const int ns = nt - u.np - nbt;
                    if (BLOCK && j >= ns && j < ns + nbt) {
                        hi = min(kN, u.blk_count - (j - ns) * kN);
                    } else if (j >= ns) {
                        hi = min(kN, (ORDER ? min(u.key_count, my_pv) : u.key_count) - (j - ns - nbt) * kN);
                        if (hi < 0) hi = 0;
                    } else {
                        const int base = j * kN;
                        lo = max(0, my_cs - base);
                        hi = min(kN, my_cs + my_len - base);
                        if (hi < lo) hi = lo;
                    }
                }
                const bool vis = __any_sync(0xffffffffu, hi > lo);
                const int pb = pw & 1;                   // the tile's S / P buffer
                const uint32_t tmem_s = tmem_s0 + pb * kN;
                ok = mbar_wait_warp(&misc->s_full[x][pb], (pw >> 1) & 1, misc);
                if (!ok) break;
                tc_fence_after();
                uint32_t sv[kN];
                if (vis) {
                    tmem_ld32(tmem_s, sv); tmem_ld32(tmem_s + 32, sv + 32);
                    tmem_ld_wait();
                }

                if (vis) {
                    if (!__all_sync(0xffffffffu, lo == 0 && hi == kN)) {
                        const unsigned span = static_cast<unsigned>(hi - lo);
#pragma unroll
                        for (int c = 0; c < kN; ++c)
                            if (static_cast<unsigned>(c - lo) >= span) sv[c] = 0xff800000u;   // -inf
                    }
                    float t8[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) t8[c] = fmaxf(__uint_as_float(sv[c]), __uint_as_float(sv[c + 8]));
#pragma unroll
                    for (int c = 16; c < kN; c += 16)
#pragma unroll
                        for (int k = 0; k < 8; ++k) t8[k] = fmax3(t8[k], __uint_as_float(sv[c + k]), __uint_as_float(sv[c + 8 + k]));
                    float tmax = fmax3(fmax3(t8[0], t8[1], t8[2]), fmax3(t8[3], t8[4], t8[5]), fmaxf(t8[6], t8[7]));
                    tmax *= p.scale_log2;
                    if (j == 0) {
                        m = tmax;
                    } else {
                        const bool fresh = m == -INFINITY;       // nothing visible so far: O row is still exactly zero
                        if (fresh) m = tmax;
                        const bool grow = !fresh && tmax > m + kRescaleSlack;
                        if (__any_sync(0xffffffffu, grow)) {
                            // O must be rescaled: wait until the previous P V product has landed in TMEM
                            ok = mbar_wait_warp(&misc->p_empty[x][(pw - 1) & 1], ((pw - 1) >> 1) & 1, misc);
                            if (ok) {
                                tc_fence_after();
                                const float m_new = grow ? tmax : m;
                                const float f = grow ? ex2(m - m_new) : 1.f;
#pragma unroll
                                for (int c0 = 0; c0 < D; c0 += 32) {
                                    uint32_t ov[32];
                                    tmem_ld32(tmem_o + c0, ov);
                                    tmem_ld_wait();
#pragma unroll
                                    for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * f);
                                    tmem_st32(tmem_o + c0, ov);
                                }
                                tmem_st_wait();
                                l *= f;
                                m = m_new;
                            }
                        }
                    }
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                // Probabilities go to tensor memory as bf16 pairs (column c holds keys 2c and 2c+1 of the row), over the
                // first half of the row's own scores, from where the tensor core reads them as the A operand of O += P V.
                if (warp_active) {
                    if (!vis) {                          // nothing visible for any row of the warp: zero probabilities
                        uint32_t pk[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c) pk[c] = 0u;
                        tmem_st16(tmem_s, pk);
                        tmem_st16(tmem_s + 16, pk);
                    } else {
                        const float neg_m = (m == -INFINITY) ? 0.f : -m;
                        float lsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int h = 0; h < 2; ++h) {    // 32 keys = 16 columns of bf16 pairs per store
                            uint32_t pk[16];
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const float e0 = ex2(fmaf(__uint_as_float(sv[h * 32 + 2 * c]), p.scale_log2, neg_m));
                                const float e1 = ex2(fmaf(__uint_as_float(sv[h * 32 + 2 * c + 1]), p.scale_log2, neg_m));
                                lsum[c & 1] += e0; lsum[2 + (c & 1)] += e1;
                                pk[c] = pack_bf16(e0, e1);
                            }
                            tmem_st16(tmem_s + h * 16, pk);
                        }
                        l += (lsum[0] + lsum[1]) + (lsum[2] + lsum[3]);
                    }
                    tmem_st_wait();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&misc->p_full[x][pb]);
                ++pw;
            }
            if (!ok) break;

            // ------------------------------------ epilogue ------------------------------------
            if (nt > 0) {                                // the unit's last P V product has landed (and the P tile is free)
                ok = mbar_wait_warp(&misc->o_full[x], of_cnt & 1, misc);
                ++of_cnt;
                if (!ok) break;
            }
            tc_fence_after();
            const int g_row = row - b_row * G;
            const int grow_row = u.row0 + b_row;
            const int hq = u.head * G + g_row;
            const bool store = row_valid && grow_row < p.a.max_rows;
            const bool final_out = u.part_base < 0;
            const float inv = final_out ? (l > 0.f ? 1.f / l : 0.f) : 1.f;
            const int64_t pr = (static_cast<int64_t>(final_out ? 0 : u.part_base) + u.row_begin + b_row) * p.a.g.Hq + hq;
            float* po = p.part_o + pr * D;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                float acc[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) acc[c] = 0.f;
                if (warp_active && nt > 0) {
                    uint32_t ov[32];
                    tmem_ld32(tmem_o + c0, ov);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) acc[c] = inv * __uint_as_float(ov[c]);
                }
                if (c0 + 32 >= D) {                      // all TMEM reads of this unit are done
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&misc->o_free[x]);
                }
                if (final_out) {
                    // transpose through this warp's 2 KB of shared memory: a row's 32 columns go out as one 64-byte
                    // piece, 8 rows per store instruction
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {
                        uint4 pk;
                        pk.x = pack_bf16(acc[c + 0], acc[c + 1]);
                        pk.y = pack_bf16(acc[c + 2], acc[c + 3]);
                        pk.z = pack_bf16(acc[c + 4], acc[c + 5]);
                        pk.w = pack_bf16(acc[c + 6], acc[c + 7]);
                        *reinterpret_cast<uint4*>(stg + lane * 64 + ((((c >> 3) ^ (lane >> 1)) & 3) << 4)) = pk;
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rl = 8 * i + (lane >> 2), ch = lane & 3;       // row inside the warp's 32, 16-byte piece
                        const uint4 pk = *reinterpret_cast<const uint4*>(stg + rl * 64 + (((ch ^ (rl >> 1)) & 3) << 4));
                        const int trow = quad * 32 + rl;
                        const int tb = G == 1 ? trow : static_cast<int>(__umulhi(static_cast<uint32_t>(trow), g_magic)), tg = trow - tb * G;
                        const int grow = u.row0 + tb;
                        if (trow < nrows && grow < p.a.max_rows)
                            *reinterpret_cast<uint4*>(p.a.o + (static_cast<int64_t>(grow) * p.a.g.Hq + u.head * G + tg) * D + c0 + ch * 8) = pk;
                    }
                    __syncwarp();
                } else if (store) {
#pragma unroll
                    for (int c = 0; c < 32; c += 4)
                        *reinterpret_cast<float4*>(po + c0 + c) = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
                }
            }
            if (store) {
                if (final_out) {
                    if (p.a.lse) p.a.lse[static_cast<int64_t>(grow_row) * p.a.g.Hq + hq] = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
                } else {
                    p.part_ml[pr * 2] = m; p.part_ml[pr * 2 + 1] = l;
                }
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

// Merge of the partial results of documents whose prefix was split over several work items.  One warp per (row, q
// head); the chunks' partials are fetched four at a time so that their loads are in flight together (the kernel is a
// chain of L2 round trips, not of bytes).
template <int D>
__global__ void __launch_bounds__(256)
hpd_merge_kernel(TcParams p, const DocSplit* __restrict__ split)
{
    // the attention kernel drew its units from the ticket counter: rewind it for the next launch on this workspace
    if (blockIdx.x == 0 && threadIdx.x == 0) const_cast<WsHeader*>(p.hdr)->ticket = 0;
    if (!p.hdr->any_split) return;
    const int lane = threadIdx.x & 31;
    const int Hq = p.a.g.Hq;
    const int64_t n_w = static_cast<int64_t>(*p.a.n_active) * Hq;
    constexpr int E = D / 32;
    constexpr int kBatch = 4;
    for (int64_t w = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5); w < n_w; w += static_cast<int64_t>(gridDim.x) * 8) {
        const int r = static_cast<int>(w / Hq), h = static_cast<int>(w % Hq);
        const int d = p.a.doc_id[r];
        const DocSplit sp = split[d];
        if (sp.n_chunks <= 1) continue;
        const int das = p.a.doc_active_start[d];
        const int rows_d = p.a.doc_active_start[d + 1] - das;
        const int64_t pr0 = (static_cast<int64_t>(sp.part_base) + (r - das)) * Hq + h;      // chunk c: pr0 + c * step
        const int64_t step = static_cast<int64_t>(rows_d) * Hq;
        float M = -INFINITY;
        for (int c0 = 0; c0 < sp.n_chunks; c0 += kBatch) {
            float m[kBatch];
#pragma unroll
            for (int i = 0; i < kBatch; ++i)
                m[i] = c0 + i < sp.n_chunks ? p.part_ml[(pr0 + (c0 + i) * step) * 2] : -INFINITY;
#pragma unroll
            for (int i = 0; i < kBatch; ++i) M = fmaxf(M, m[i]);
        }
        float L = 0.f, acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        for (int c0 = 0; c0 < sp.n_chunks; c0 += kBatch) {
            float2 ml[kBatch];
            float o[kBatch][E];
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const bool in = c0 + i < sp.n_chunks;
                const int64_t pr = pr0 + (in ? c0 + i : 0) * step;
                ml[i] = in ? *reinterpret_cast<const float2*>(p.part_ml + pr * 2) : make_float2(-INFINITY, 0.f);
                if constexpr (E == 4) {
                    const float4 v = *reinterpret_cast<const float4*>(p.part_o + pr * D + lane * E);
                    o[i][0] = v.x; o[i][1] = v.y; o[i][2] = v.z; o[i][3] = v.w;
                } else {
                    const float2 v = *reinterpret_cast<const float2*>(p.part_o + pr * D + lane * E);
                    o[i][0] = v.x; o[i][1] = v.y;
                }
            }
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                if (c0 + i >= sp.n_chunks) continue;
                const float f = ml[i].x == -INFINITY ? 0.f : exp2f(ml[i].x - M);
                L += f * ml[i].y;
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = fmaf(f, o[i][e], acc[e]);
            }
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
// K/V [tokens, Hkv, D] bf16: boxes of box_rows tokens x 1 head x 64 elements, 128-byte swizzle
bool make_kv_map(CUtensorMap* m, const void* base, int D, int Hkv, long long tokens, int box_rows)
{
    auto fn = tensor_map_encoder();
    if (!fn) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(Hkv), static_cast<cuuint64_t>(tokens > 0 ? tokens : 1)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(Hkv) * D * 2};
    cuuint32_t box[3] = {64, 1, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q [rows, Hkv, G, D] bf16: boxes of 128/G rows x 1 kv head x G x 64 elements -> tile row = branch*G + g
bool make_q_map(CUtensorMap* m, const void* base, int D, int G, int Hkv, long long rows)
{
    auto fn = tensor_map_encoder();
    if (!fn) return false;
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(G), static_cast<cuuint64_t>(Hkv),
                          static_cast<cuuint64_t>(rows > 0 ? rows : 1)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(G) * D * 2,
                             static_cast<cuuint64_t>(Hkv) * G * D * 2};
    cuuint32_t box[4] = {64, static_cast<cuuint32_t>(G), 1, static_cast<cuuint32_t>(kM / G)};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, bool ORDER, bool BLOCK>
int launch_d(const AttnArgs& a)
{
    using C = Cfg<D>;
    // the dynamic shared-memory limit is an attribute of the kernel on ONE device: set it once per device
    static std::atomic<bool> attr_set[kMaxDevices];
    const int dev = current_device();
    if (dev < 0 || dev >= kMaxDevices || !attr_set[dev].load(std::memory_order_acquire)) {
        HPD_CUDA_TRY(cudaFuncSetAttribute(hpd_attn_tc_kernel<D, ORDER, BLOCK>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM));
        if (dev >= 0 && dev < kMaxDevices) attr_set[dev].store(true, std::memory_order_release);
    }
    const int G = a.g.Hq / a.g.Hkv;
    // Tensor maps depend only on the tensors' addresses and extents: a decode loop calls with the same ones step
    // after step and layer after layer, so each thread keeps the maps of its last few distinct argument sets.
    struct MapKey {
        const void *q, *pk, *pv, *sk, *sv;
        long long max_rows, total_prefix, cache_rows;
        int Hkv, G;
        bool operator==(const MapKey& o) const {
            return q == o.q && pk == o.pk && pv == o.pv && sk == o.sk && sv == o.sv && max_rows == o.max_rows &&
                   total_prefix == o.total_prefix && cache_rows == o.cache_rows && Hkv == o.Hkv && G == o.G;
        }
    };
    struct MapSet { MapKey key; CUtensorMap mq, mk, mv; SufMaps sm; bool valid = false; };
    constexpr int kCached = 64;
    static thread_local MapSet cache[kCached];
    static thread_local unsigned next_victim = 0;
    const void* kbase = a.total_prefix > 0 ? static_cast<const void*>(a.prefix_k) : static_cast<const void*>(a.suffix_k);
    const void* vbase = a.total_prefix > 0 ? static_cast<const void*>(a.prefix_v) : static_cast<const void*>(a.suffix_v);
    const long long cache_rows = static_cast<long long>(a.n_slots) * a.g.suffix_cap;
    const MapKey key{a.q, kbase, vbase, a.suffix_k, a.suffix_v, a.max_rows, a.total_prefix, cache_rows, a.g.Hkv, G};
    MapSet* ms = nullptr;
    for (int i = 0; i < kCached && !ms; ++i)
        if (cache[i].valid && cache[i].key == key) ms = &cache[i];
    if (!ms) {
        ms = &cache[next_victim++ % kCached];
        ms->valid = false;
        bool maps_ok = make_q_map(&ms->mq, a.q, D, G, a.g.Hkv, a.max_rows) && make_kv_map(&ms->mk, kbase, D, a.g.Hkv, a.total_prefix, kN) &&
                       make_kv_map(&ms->mv, vbase, D, a.g.Hkv, a.total_prefix, kN);
        for (int i = 0; i < 16 && maps_ok; ++i) maps_ok = make_kv_map(&ms->sm.k[i], a.suffix_k, D, a.g.Hkv, cache_rows, i + 1);
        for (int i = 0; i < 16 && maps_ok; ++i) maps_ok = make_kv_map(&ms->sm.v[i], a.suffix_v, D, a.g.Hkv, cache_rows, i + 1);
        if (!maps_ok) {
            set_last_cuda_error(cudaErrorInvalidValue);
            return HPD_E_CUDA;
        }
        ms->key = key;
        ms->valid = true;
    }
    const CUtensorMap &mq = ms->mq, &mk = ms->mk, &mv = ms->mv;
    const SufMaps& sm = ms->sm;
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
    CUtensorMap mbk = mk, mbv = mv;                      // unused without a shared block
    if constexpr (BLOCK) {
        if (!make_kv_map(&mbk, a.block_k, D, a.g.Hkv, a.total_block, kN) || !make_kv_map(&mbv, a.block_v, D, a.g.Hkv, a.total_block, kN)) {
            set_last_cuda_error(cudaErrorInvalidValue);
            return HPD_E_CUDA;
        }
    }
    hpd_attn_tc_kernel<D, ORDER, BLOCK><<<n_sm, kThreads, C::SMEM, a.stream>>>(mq, mk, mv, mbk, mbv, sm, p);
    // one warp per (row, q head) where the rows allow it, at most one resident wave; with many documents nothing is
    // split as a rule (the kernel then only rewinds the ticket counter) and a small grid is launched sooner
    const long long merge_blocks = (static_cast<long long>(a.max_rows) * a.g.Hq + 7) / 8;
    const long long merge_cap = static_cast<long long>(a.n_docs) * a.g.Hkv < 4ll * n_sm ? 8ll * n_sm : 2ll * n_sm;
    const int merge_grid = static_cast<int>(std::min<long long>(std::max<long long>(merge_blocks, 1), merge_cap));
    hpd_merge_kernel<D><<<merge_grid, 256, 0, a.stream>>>(p, reinterpret_cast<const DocSplit*>(ws + a.lay.off_split));
    HPD_CUDA_TRY(cudaGetLastError());
    return HPD_OK;
}

}  // namespace

int launch_attn_tc(const AttnArgs& a)
{
    if (!(a.g.sm_scale > 0.f)) return HPD_E_GEOM;
    if (a.prefix_vis) return a.g.D == 128 ? launch_d<128, true, false>(a) : launch_d<64, true, false>(a);
    if (a.block_k) return a.g.D == 128 ? launch_d<128, false, true>(a) : launch_d<64, false, true>(a);
    return a.g.D == 128 ? launch_d<128, false, false>(a) : launch_d<64, false, false>(a);
}

}  // namespace hpd
