// Chunked causal linear attention for bf16 inputs on sm_100a: tcgen05 tensor-core tiles with TMEM
// accumulators, operands staged by TMA (Sec. 4.1 tiling of Eq. 2 with the causal mask).
//
// One CTA walks one (batch, head) sequence in tiles of 64 tokens: four compute warps plus one issuer
// warp whose lane 0 drives TMA and the tensor core (its own warp, so that its instruction stream is
// not interleaved with spinning lanes); roles meet only through mbarriers, every wait bounded.  The tensor core
// charges a tcgen05.mma by the instruction (about 46 cycles for any N <= 93 and any M <= 128), so the
// five 64 x 64 x 64 products of a tile are packed into M = 128 instructions:
//   TMA     : Q_i, K_i, V_i ([64 rows] x 128 B, 128-byte swizzle, adjacent in one stage of a 3-stage ring)
//   G1      : [Q_i ; K_i] Q_i^T                       -> TMEM tile PT; rows 64..127 are P^T = K_i Q_i^T
//   warps 2,3: P^T -> registers, causal mask (t >= s), bf16 -> shared tile (rows = s)
//   G2      : rows 0..63 of tile OS = Q_i S_hi + Q_i S_lo (A = [Q_i ; K_i], lanes 64..127 write-disabled)
//   G3      : OS += [P^T tile | K_i tile]^T V_i          rows 0..63 += P V_i (output), rows 64..127 += K_i^T V_i
//             (one MN-major A operand of two 64-wide atoms: the score tile and, through the descriptor's
//              leading-dimension offset, the K tile of the current stage)
//   warps 0,1: output rows -> scale, row normaliser -> swizzled staging -> TMA store
//   warps 2,3: state rows (fp32, never leave the SM) -> bf16 hi + lo -> shared (B operand of the next G2)
// The state is fed back to the tensor core as S_hi + S_lo (two bf16 terms, ~16 mantissa bits) so the
// inter-chunk term keeps fp32-like accuracy; P is rounded to bf16 once.
//
// Every wait is bounded: on a timeout the CTA records CHELA_ERR_TIMEOUT in the status word, drains its
// outstanding TMA loads (bounded), frees its TMEM and returns.
#include <cuda.h>

#include "common.cuh"

namespace chela {
namespace {

constexpr int kD = 64;            // head dimension handled by this kernel (d_k = d_v)
constexpr int kThreads = 160;            // 4 compute warps + 1 issuer warp
constexpr long long kWaitCycles = 2000000000LL;  // ~1 s at B200 clocks

// ------------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within kWaitCycles, or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > kWaitCycles || (abort_flag && *abort_flag)) return false;
    return true;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// The mbarrier receives one arrival once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread t of the warp receives lane (base lane + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&r)[32])
{
    uint32_t *u = reinterpret_cast<uint32_t *>(r);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]),
          "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]),
          "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]),
          "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
        : "r"(taddr)
        : "memory");
}
// Store counterpart: thread t of the warp writes 32 consecutive fp32 columns of lane (base lane + t).
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&r)[32])
{
    const uint32_t *u = reinterpret_cast<const uint32_t *>(r);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]),
          "r"(u[8]), "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]),
          "r"(u[16]), "r"(u[17]), "r"(u[18]), "r"(u[19]), "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]),
          "r"(u[24]), "r"(u[25]), "r"(u[26]), "r"(u[27]), "r"(u[28]), "r"(u[29]), "r"(u[30]), "r"(u[31]),
          "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ------------------------------------------------------------------------------- descriptors

// Shared-memory matrix descriptor for [rows] x 128-byte tiles with 128-byte swizzle (tile bases
// 1024-byte aligned).  Bits: [0,14) address >> 4, [16,30) leading byte offset >> 4, [32,46) stride byte
// offset >> 4 (distance between 8-row groups = 1024 B), [46,48) version = 1, [61,64) layout = 2
// (128-byte swizzle).  The same physical tile serves as a K-major operand (row = M/N index, 128 B along
// K) or as an MN-major operand (row = K index, 128 B along M/N); the instruction descriptor says which.
// For an MN-major operand wider than 64 elements the leading byte offset is the distance from one
// 64-element atom to the next; K-major operands here never use it.
// Only the low word depends on addresses, so the issuing thread keeps the high word constant and
// advances the low word: +2 per 32 bytes along a K-major row, +128 per 16 rows of an MN-major tile.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes = 16)
{
    return ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
}

// Instruction descriptor, kind::f16: fp32 accumulator (bits [4,6) = 1), bf16 A and B (bits [7,10),
// [10,13) = 1), A/B major (bit 15 / bit 16: 0 = K-major, 1 = MN-major), N >> 3 at [17,23), M >> 4 at [24,29).
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int a_mn_major, int b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem], bf16 operands, fp32 accumulate; issued by a single thread.
// upper_off != 0 write-disables TMEM lanes 64..127 (rows 64..127 of an M = 128 result).
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate,
                                          uint32_t upper_off = 0)
{
    const uint32_t m = upper_off ? 0xFFFFFFFFu : 0u;
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, {%6, %6, %7, %7}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi), "r"(0u), "r"(m)
        : "memory");
}

// TMA store of a shared-memory box to global memory (bulk async-group completion).
__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ------------------------------------------------------------------------------- kernel

constexpr int kC = 64;       // tokens per tile
constexpr int kStages = 3;
constexpr int kTile = kC * 128;   // one 64-row x 128-byte tile

template <typename TOut>
struct Smem {
    static constexpr int kOBoxes = (int)sizeof(TOut) * kD / 128;   // output staged as 128-byte wide boxes
    static constexpr int offPT = 0;                       // masked scores, transposed: rows = s, 64 t per row
    static constexpr int offShi = offPT + kTile;          // state, bf16 high part: rows = d_k
    static constexpr int offSlo = offShi + kTile;         // state, bf16 low part
    static constexpr int offO = offSlo + kTile;           // output staging
    static constexpr int offStage = offO + kOBoxes * kTile;   // per stage: Q, K, V tiles, adjacent
    static constexpr int offBar = offStage + kStages * 3 * kTile;   // full[kStages], p, o, pt, s
    static constexpr int offTmem = offBar + 8 * (kStages + 4);
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
};
constexpr int kTmemCols = 128;
constexpr int kColOS = 0;    // rows 0..63: output tile, rows 64..127: running state; 64 columns
constexpr int kColPT = 64;   // rows 64..127: transposed scores; 64 columns

// byte offset of element (row, 16-byte chunk) inside a 128-byte-swizzled [rows] x 128 B tile
__device__ __forceinline__ uint32_t sw128(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

#ifdef CHELA_TIMING
#define TMARK(n) do { long long tn = clock64(); tacc[n] += tn - tprev; tprev = tn; } while (0)
#define TDECL long long tacc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, tprev = clock64()
#define TDUMP(slot) do { for (int n_ = 0; n_ < 8; ++n_) reinterpret_cast<long long *>(status)[4 + 8 * (slot) + n_] = tacc[n_]; } while (0)
#else
#define TMARK(n)
#define TDECL
#define TDUMP(slot)
#endif

template <typename TOut>
__global__ void __launch_bounds__(kThreads)
linattn_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, int H, int L,
                     float scale, int norm, float eps, int *__restrict__ status, const float *__restrict__ s_part,
                     int G, int cpg)
{
    // Grid: one CTA per (batch*head, group).  Group g covers chunks [g*cpg, (g+1)*cpg) of its sequence and
    // starts from the state sum_{g' < g} s_part[bh][g'] (per-group K^T V sums written by the state kernel).
    using SM = Smem<TOut>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {  // swizzled tiles need a 1024-byte aligned base: report instead of corrupting
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x / G, g = blockIdx.x % G;
    const int b = bh / H, h = bh % H;
    const int c0 = g * cpg;                                        // first chunk of this group
    const int nchunks = min(cpg, (L + kC - 1) / kC - c0);          // chunks of this group
    const bool has_init = g > 0;

    const uint32_t bar_full0 = sbase + SM::offBar;
    const uint32_t bar_p = bar_full0 + 8 * kStages;   // G1 of a chunk has completed (tensor core -> warps 2,3)
    const uint32_t bar_o = bar_p + 8;                 // G2 + G3 of a chunk have completed (-> all roles)
    const uint32_t bar_pt = bar_o + 8;                // score tile of a chunk is in shared memory (warps 2,3 -> issuer)
    const uint32_t bar_s = bar_pt + 8;                // output/state rows read, state tiles written (4 warps -> issuer)
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM::offTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::offAbort);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(bar_full0 + 8 * s, 1);
        mbar_init(bar_p, 1);
        mbar_init(bar_o, 1);
        mbar_init(bar_pt, 2);
        mbar_init(bar_s, 4);
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_o);
    }
    if (warp == 0) {
        tmem_alloc(sbase + SM::offTmem, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        // =========================================== issuer: TMA loads and every tcgen05.mma ==========
        if (lane == 0) {
            TDECL;
            auto stage_base = [&](int chunk) { return sbase + SM::offStage + (chunk % kStages) * 3 * kTile; };
            auto issue_load = [&](int chunk) {
                const uint32_t bar = bar_full0 + 8 * (chunk % kStages), dst = stage_base(chunk);
                mbar_expect_tx(bar, 3 * kTile);
                tma_load_4d(dst, &tm_q, bar, 0, h, (c0 + chunk) * kC, b);
                tma_load_4d(dst + kTile, &tm_k, bar, 0, h, (c0 + chunk) * kC, b);
                tma_load_4d(dst + 2 * kTile, &tm_v, bar, 0, h, (c0 + chunk) * kC, b);
            };
            constexpr uint32_t idescG1 = make_idesc(128, kC, 0, 0);   // [Q;K] (K-major) x Q^T (K-major)
            constexpr uint32_t idescG2 = make_idesc(128, kD, 0, 1);   // [Q;K] (K-major) x S (MN-major)
            constexpr uint32_t idescG3 = make_idesc(128, kD, 1, 1);   // [P^T|K] (MN-major) x V (MN-major)
            // G1 of a chunk; false if the chunk's tiles never arrived
            auto issue_scores = [&](int chunk) -> bool {
                if (!mbar_wait(bar_full0 + 8 * (chunk % kStages), (chunk / kStages) & 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t qk_lo = desc_lo(stage_base(chunk));
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColPT, qk_lo + 2 * k, qk_lo + 2 * k, idescG1, k > 0);
                umma_commit(bar_p);
                return true;
            };
            const uint32_t shi_lo = desc_lo(sbase + SM::offShi), slo_lo = desc_lo(sbase + SM::offSlo);
            int loads_issued = 0, consumed = 0;
            for (; loads_issued < kStages && loads_issued < nchunks; ++loads_issued) issue_load(loads_issued);
            bool ok = issue_scores(0);
            uint32_t par_s = 0;
            for (int i = 0; ok && i < nchunks; ++i) {
                const uint32_t st = stage_base(i);
                if (i > 0 || has_init) {
                    // G2: rows 0..63 of OS = Q S_hi + Q S_lo; needs the state tiles of the previous chunk (or
                    // of the group's initial state) and the previous output rows out of TMEM
                    ok = mbar_wait(bar_s, par_s, abort_flag);
                    par_s ^= 1;
                    if (!ok) break;
                    tc_fence_after();
                    TMARK(0);
                    const uint32_t qk_lo = desc_lo(st);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColOS, qk_lo + 2 * k, shi_lo + 128 * k, idescG2, k > 0, 1);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColOS, qk_lo + 2 * k, slo_lo + 128 * k, idescG2, 1, 1);
                    TMARK(1);
                }
                // G3: OS += [P^T | K]^T V; atom 0 = score tile, atom 1 = K tile of this stage
                ok = mbar_wait(bar_pt, i & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                TMARK(2);
                const uint32_t a_lo = desc_lo(sbase + SM::offPT, st + kTile - (sbase + SM::offPT)), v_lo = desc_lo(st + 2 * kTile);
#pragma unroll
                for (int k = 0; k < kC / 16; ++k)
                    umma_bf16(tmem + kColOS, a_lo + 128 * k, v_lo + 128 * k, idescG3, (i > 0 || has_init || k > 0) ? 1u : 0u);
                umma_commit(bar_o);
                if (i + 1 < nchunks) {
                    ok = issue_scores(i + 1);
                    if (!ok) break;
                }
                TMARK(3);
                // the stage is free once G3 has completed: prefetch the chunk that will use it next
                ok = mbar_wait(bar_o, i & 1, abort_flag);
                if (!ok) break;
                consumed = i + 1;
                if (i + kStages < nchunks) {
                    issue_load(i + kStages);
                    ++loads_issued;
                }
                TMARK(4);
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(status, (int)CHELA_ERR_TIMEOUT);
                // drain loads that were issued but never consumed (bounded), so no copy lands after exit
                for (int c = consumed; c < loads_issued; ++c)
                    mbar_wait(bar_full0 + 8 * (c % kStages), (c / kStages) & 1, nullptr);
            }
#ifdef CHELA_TIMING
            if (blockIdx.x == 0) TDUMP(0);
#endif
        }
    } else {
        // =========================================== compute warps ====================================
        // TMEM lane = accumulator row = thread.  Warps 0,1 own output rows t = tid; warps 2,3 own row
        // r = tid - 64 of the transposed scores (s) and of the state (d_k).
        const bool upper = warp >= 2;
        const int r = tid & 63;
        const uint32_t tmem_warp = tmem + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
        TDECL;
        // state row r -> bf16 hi + lo -> shared (MN-major B operand of G2)
        auto write_state_tiles = [&](const float(&sv)[kD]) {
            uint8_t *sHi = smem + SM::offShi, *sLo = smem + SM::offSlo;
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
                uint32_t wh[4], wl[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float x0 = sv[c8 * 8 + e * 2], x1 = sv[c8 * 8 + e * 2 + 1];
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                    const float2 hf = __bfloat1622float2(hh);
                    wh[e] = *reinterpret_cast<const uint32_t *>(&hh);
                    wl[e] = pack_bf16(x0 - hf.x, x1 - hf.y);
                }
                const uint32_t off = sw128(r, c8);
                *reinterpret_cast<uint4 *>(sHi + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
                *reinterpret_cast<uint4 *>(sLo + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
            }
        };
        if (has_init) {
            // initial state of the group: sum of the preceding groups' K^T V, into TMEM rows 64..127 and
            // into the G2 operand tiles
            if (upper) {
                float sv[kD];
#pragma unroll
                for (int j = 0; j < kD; ++j) sv[j] = 0.f;
                for (int gp = 0; gp < g; ++gp) {
                    const float4 *src = reinterpret_cast<const float4 *>(s_part + (((size_t)bh * (G - 1) + gp) * kD + r) * kD);
#pragma unroll
                    for (int j = 0; j < kD / 4; ++j) {
                        const float4 x = src[j];
                        sv[4 * j] += x.x; sv[4 * j + 1] += x.y; sv[4 * j + 2] += x.z; sv[4 * j + 3] += x.w;
                    }
                }
                tmem_st32(tmem_warp + kColOS, *reinterpret_cast<const float(*)[32]>(&sv[0]));
                tmem_st32(tmem_warp + kColOS + 32, *reinterpret_cast<const float(*)[32]>(&sv[32]));
                tmem_st_wait();
                write_state_tiles(sv);
                fence_proxy_async();
                tc_fence_before();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_s);
        }
        for (int i = 0; i < nchunks; ++i) {
            if (upper) {
                // ---- P^T_i: TMEM -> causal mask -> bf16 -> shared (rows = s, 64 t per row) -------------
                ok = __all_sync(0xffffffffu, mbar_wait(bar_p, i & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                TMARK(0);
                // row s keeps t >= s; for warp 3 (s >= 32) the block t < 32 is all zeros: no TMEM read
                float p[2][32];
                if (warp == 2) tmem_ld32(tmem_warp + kColPT, p[0]);
                tmem_ld32(tmem_warp + kColPT + 32, p[1]);
                tmem_ld_wait();
                uint8_t *sP = smem + SM::offPT;
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    const bool live = cb == 1 || warp == 2;
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int t = cb * 32 + c8 * 8 + e * 2;
                            const float lo = (live && t >= r) ? p[cb][c8 * 8 + e * 2] : 0.f;
                            const float hi = (live && t + 1 >= r) ? p[cb][c8 * 8 + e * 2 + 1] : 0.f;
                            w[e] = pack_bf16(lo, hi);
                        }
                        *reinterpret_cast<uint4 *>(sP + sw128(r, cb * 4 + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pt);
                TMARK(1);
            }
            ok = __all_sync(0xffffffffu, mbar_wait(bar_o, i & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            TMARK(2);
            float acc[kD];
            if (!upper) {
                // ---- output row t: scale, normaliser -> swizzled staging -> TMA store (per warp: 32 rows) ----
                tmem_ld32(tmem_warp + kColOS, *reinterpret_cast<float(*)[32]>(&acc[0]));
                tmem_ld32(tmem_warp + kColOS + 32, *reinterpret_cast<float(*)[32]>(&acc[32]));
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar_s);     // the output rows are out of TMEM: G2 of the next chunk may overwrite them
                    bulk_wait_read0();      // this warp's previous output boxes have left shared memory
                }
                __syncwarp();
                float ss = 0.f;
#pragma unroll
                for (int j = 0; j < kD; ++j) {
                    acc[j] *= scale;
                    ss = fmaf(acc[j], acc[j], ss);
                }
                const float inv = norm ? rsqrtf(ss * (1.0f / kD) + eps) : 1.0f;
                uint8_t *sO = smem + SM::offO;
                if (sizeof(TOut) == 4) {
#pragma unroll
                    for (int j = 0; j < kD; j += 4)
                        *reinterpret_cast<float4 *>(sO + (j / 32) * kTile + sw128(r, (j % 32) / 4)) =
                            make_float4(acc[j] * inv, acc[j + 1] * inv, acc[j + 2] * inv, acc[j + 3] * inv);
                } else {
#pragma unroll
                    for (int j = 0; j < kD; j += 8)
                        *reinterpret_cast<uint4 *>(sO + sw128(r, j / 8)) =
                            make_uint4(pack_bf16(acc[j] * inv, acc[j + 1] * inv), pack_bf16(acc[j + 2] * inv, acc[j + 3] * inv),
                                       pack_bf16(acc[j + 4] * inv, acc[j + 5] * inv), pack_bf16(acc[j + 6] * inv, acc[j + 7] * inv));
                }
                fence_proxy_async();
                __syncwarp();
                // rows past L are clipped by the copy engine
                if (lane == 0) {
#pragma unroll
                    for (int bx = 0; bx < SM::kOBoxes; ++bx)
                        tma_store_4d(&tm_o, sbase + SM::offO + bx * kTile + warp * 32 * 128, bx * (128 / (int)sizeof(TOut)), h,
                                     (c0 + i) * kC + warp * 32, b);
                    bulk_commit();
                }
                TMARK(3);
            } else {
                // ---- state row d_k: bf16 hi + lo -> shared (MN-major B operand of the next chunk's G2) ------
                if (i + 1 < nchunks) {
                    tmem_ld32(tmem_warp + kColOS, *reinterpret_cast<float(*)[32]>(&acc[0]));
                    tmem_ld32(tmem_warp + kColOS + 32, *reinterpret_cast<float(*)[32]>(&acc[32]));
                    tmem_ld_wait();
                    write_state_tiles(acc);
                    fence_proxy_async();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_s);
                }
                TMARK(3);
            }
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicExch(status, (int)CHELA_ERR_TIMEOUT);
        }
        if (!upper && lane == 0) bulk_wait0();   // output boxes fully written before the CTA retires
#ifdef CHELA_TIMING
        if (blockIdx.x == 0 && (tid == 0 || tid == 64)) TDUMP(tid == 0 ? 1 : 2);
#endif
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------- state kernel

// Per-group state sums for sequences that are split along L: CTA (batch*head, g), g < G-1, writes
// s_part[bh][g] = sum over the group's chunks of K_i^T V_i (fp32, [d_k][d_v]).  Only K and V are read.
// One tcgen05.mma group per chunk: A = [K_i | V_i] (MN-major, two atoms), B = V_i; rows 0..63 of the
// accumulator are K^T V, rows 64..127 (V^T V) are ignored.
constexpr int kStStages = 4;
struct SmemState {
    static constexpr int offStage = 0;                              // per stage: K, V tiles, adjacent
    static constexpr int offBar = kStStages * 2 * kTile;            // full[kStStages], empty[kStStages], done
    static constexpr int offTmem = offBar + 8 * (2 * kStStages + 1);
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
};

__global__ void __launch_bounds__(kThreads)
linattn_state_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     float *__restrict__ s_part, int H, int G, int cpg, int *__restrict__ status)
{
    using SM = SmemState;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x / (G - 1), g = blockIdx.x % (G - 1);
    const int b = bh / H, h = bh % H;
    const int c0 = g * cpg, nchunks = cpg;    // every group but the last is full

    const uint32_t bar_full0 = sbase + SM::offBar, bar_empty0 = bar_full0 + 8 * kStStages,
                   bar_done = bar_empty0 + 8 * kStStages;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM::offTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::offAbort);
    if (tid == 0) {
        for (int s = 0; s < kStStages; ++s) {
            mbar_init(bar_full0 + 8 * s, 1);
            mbar_init(bar_empty0 + 8 * s, 1);
        }
        mbar_init(bar_done, 1);
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == 0) {
        tmem_alloc(sbase + SM::offTmem, 64);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        if (lane == 0) {
            auto issue_load = [&](int chunk) {
                const uint32_t bar = bar_full0 + 8 * (chunk % kStStages), dst = sbase + SM::offStage + (chunk % kStStages) * 2 * kTile;
                mbar_expect_tx(bar, 2 * kTile);
                tma_load_4d(dst, &tm_k, bar, 0, h, (c0 + chunk) * kC, b);
                tma_load_4d(dst + kTile, &tm_v, bar, 0, h, (c0 + chunk) * kC, b);
            };
            constexpr uint32_t idesc = make_idesc(128, kD, 1, 1);
            int loads_issued = 0, consumed = 0;
            for (; loads_issued < kStStages && loads_issued < nchunks; ++loads_issued) issue_load(loads_issued);
            bool ok = true;
            for (int i = 0; i < nchunks; ++i) {
                const int stage = i % kStStages;
                ok = mbar_wait(bar_full0 + 8 * stage, (i / kStStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t st = sbase + SM::offStage + stage * 2 * kTile;
                const uint32_t a_lo = desc_lo(st, kTile), v_lo = desc_lo(st + kTile);
#pragma unroll
                for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem, a_lo + 128 * k, v_lo + 128 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                umma_commit(bar_empty0 + 8 * stage);
                consumed = i + 1;
                if (i + kStStages < nchunks) {
                    ok = mbar_wait(bar_empty0 + 8 * stage, (i / kStStages) & 1, abort_flag);
                    if (!ok) break;
                    issue_load(i + kStStages);
                    ++loads_issued;
                }
            }
            if (ok) umma_commit(bar_done);
            else {
                *abort_flag = 1;
                atomicExch(status, (int)CHELA_ERR_TIMEOUT);
                for (int c = consumed; c < loads_issued; ++c)
                    mbar_wait(bar_full0 + 8 * (c % kStStages), (c / kStStages) & 1, nullptr);
            }
        }
    } else if (warp < 2) {
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_done, 0, abort_flag));
        if (ok) {
            tc_fence_after();
            float sv[kD];
            const uint32_t tmem_warp = tmem + ((uint32_t)(warp * 32) << 16);
            tmem_ld32(tmem_warp, *reinterpret_cast<float(*)[32]>(&sv[0]));
            tmem_ld32(tmem_warp + 32, *reinterpret_cast<float(*)[32]>(&sv[32]));
            tmem_ld_wait();
            float4 *dst = reinterpret_cast<float4 *>(s_part + (((size_t)bh * (G - 1) + g) * kD + tid) * kD);
#pragma unroll
            for (int j = 0; j < kD / 4; ++j) dst[j] = make_float4(sv[4 * j], sv[4 * j + 1], sv[4 * j + 2], sv[4 * j + 3]);
        } else if (lane == 0) {
            *abort_flag = 1;
            atomicExch(status, (int)CHELA_ERR_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 64);
}

// ------------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// [B, L, H, 64] viewed as a rank-4 tensor (d, H, L, B); box = (128 bytes of d) x 1 x C x 1, 128-byte
// swizzle.  Loads: rows past L are out of bounds for the copy engine and arrive as zeros.  Stores: rows
// past L are clipped.
bool make_map(CUtensorMap *map, const void *ptr, int B, int H, int L, int C, bool f32)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t es = f32 ? 4 : 2;
    const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)kD * es, (cuuint64_t)H * kD * es, (cuuint64_t)L * H * kD * es};
    const cuuint32_t box[4] = {(cuuint32_t)(128 / es), 1, (cuuint32_t)C, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr),
              dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// How a call is split along L.  The grid holds B*H*G CTAs, at most two per SM so that all of them are
// resident at once; a group never has fewer than 8 chunks.
struct SplitPlan {
    int G, cpg;
    size_t part_bytes;
};
SplitPlan split_plan(int B, int H, int L)
{
    int sms = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        sms <= 0)
        sms = 148;
    const long long bh = (long long)B * H;
    const int nchunks = (L + kC - 1) / kC;
    int G = 1;
    if (bh < 2LL * sms) {
        G = (int)((2LL * sms) / bh);
        if (G > nchunks / 8) G = nchunks / 8;
        if (G < 1) G = 1;
    }
    SplitPlan p;
    p.cpg = (nchunks + G - 1) / G;
    p.G = (nchunks + p.cpg - 1) / p.cpg;
    p.part_bytes = (size_t)bh * (p.G - 1) * kD * kD * sizeof(float);
    return p;
}
constexpr size_t kWsHeader = 512;   // word 0: asynchronous status; the rest: diagnostics

template <typename TOut>
chela_status_t launch_t(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int norm, float eps,
                        float scale, void *workspace, cudaStream_t stream)
{
    CUtensorMap mq, mk, mv, mo;
    if (!make_map(&mq, q, B, H, L, kC, false) || !make_map(&mk, k, B, H, L, kC, false) ||
        !make_map(&mv, v, B, H, L, kC, false) || !make_map(&mo, o, B, H, L, 32, sizeof(TOut) == 4))
        return CHELA_ERR_CUDA;
    const SplitPlan plan = split_plan(B, H, L);
    int *status = (int *)workspace;
    float *s_part = (float *)((char *)workspace + kWsHeader);
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return CHELA_ERR_CUDA;
    if (plan.G > 1) {
        if (cudaFuncSetAttribute(linattn_state_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemState::bytes) != cudaSuccess)
            return CHELA_ERR_CUDA;
        linattn_state_kernel<<<B * H * (plan.G - 1), kThreads, SmemState::bytes, stream>>>(mk, mv, s_part, H, plan.G, plan.cpg, status);
        if (cudaGetLastError() != cudaSuccess) return CHELA_ERR_CUDA;
    }
    auto kern = linattn_sm100_kernel<TOut>;
    const int smem = Smem<TOut>::bytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return CHELA_ERR_CUDA;
    kern<<<B * H * plan.G, kThreads, smem, stream>>>(mq, mk, mv, mo, H, L, scale, norm, eps, status, s_part, plan.G, plan.cpg);
    return last_launch_status();
}

}  // namespace

bool linattn_sm100_supported(int B, int H, int L, int d, int chunk, chela_dtype_t in_dtype, chela_dtype_t)
{
    (void)B; (void)H; (void)L;
    return in_dtype == CHELA_BF16 && d == kD && (chunk == 64 || chunk == 128);
}

// Header (word 0 = asynchronous status of the last launch that used this workspace) followed by the
// per-group state sums [B*H][G-1][64][64] fp32 of a call that is split along L.
size_t linattn_sm100_workspace_bytes(int B, int H, int L, int d, int)
{
    return d == kD ? kWsHeader + split_plan(B, H, L).part_bytes : 0;
}

chela_status_t launch_linattn_sm100(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int d,
                                    int chunk, chela_dtype_t, chela_dtype_t out_dtype, int norm, float eps,
                                    float scale, void *workspace, cudaStream_t stream)
{
    (void)d;
    // The result does not depend on the chunk size: both supported values run on 64-token tiles.
    (void)chunk;
    if (out_dtype == CHELA_F32) return launch_t<float>(q, k, v, o, B, H, L, norm, eps, scale, workspace, stream);
    return launch_t<__nv_bfloat16>(q, k, v, o, B, H, L, norm, eps, scale, workspace, stream);
}

}  // namespace chela
