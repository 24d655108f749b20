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
// Variants by template: operands given as bf16 pairs (kMask), the anti-causal mirror (kReverse) and the backward
// pass's gradient epilogue (kGrad); sequences of few (batch, head) pairs are split along L (linattn_state_kernel).
//
// Every wait is bounded: on a timeout the CTA records CHELA_ERR_TIMEOUT in the status word, drains its
// outstanding TMA loads (bounded), frees its TMEM and returns.
#include "sm100_ptx.cuh"

namespace chela {
namespace {

using namespace sm100;

constexpr int kD = 64;            // head dimension handled by this kernel (d_k = d_v)
constexpr int kThreads = 160;            // 4 compute warps + 1 issuer warp

// ------------------------------------------------------------------------------- kernel

constexpr int kC = 64;       // tokens per tile
constexpr int kTile = kC * 128;   // one 64-row x 128-byte tile

// kMask says which operands are bf16 pairs (hi + lo planes): bit 0 = Q, bit 1 = K, bit 2 = V, bit 3 = the score
// tile P (an internal operand: rounded once to bf16, or kept as hi + lo).  A product with a pair operand takes one
// more tensor-core term per pair side (hi*hi + hi*lo + lo*hi; lo*lo is dropped).  0 = the plain bf16 kernel, 15 = the
// mixer's attention; the backward pass uses 8 (recomputed forward), 9, 10 and 12 (one gradient operand is a pair).
__host__ __device__ constexpr int popc3(int m) { return (m & 1) + ((m >> 1) & 1) + ((m >> 2) & 1); }
// kGrad (backward pass, with kMask = 8): the epilogue does not store the output row but pulls the output gradient
// d_o back through the normaliser, G = scale (d_o - o <o, d_o> / d) / n, and stores G as a bf16 pair; the d_o tiles
// come through a two-slot ring of their own.
template <typename TOut, int kMask, bool kGrad = false>
struct Smem {
    static constexpr int kIn = kMask & 7;
    static constexpr bool kPPair = (kMask & 8) != 0;
    static constexpr int kTilesPerStage = 3 + popc3(kIn);   // Q, K, V (hi), then the low planes that exist, in that order
    static constexpr int iQlo = 3, iKlo = 3 + (kIn & 1), iVlo = 3 + popc3(kIn & 3);
    static constexpr int kStages = (kMask == 0) ? 3 : 2;
    static constexpr int kOBoxes = kGrad ? 2 : (int)sizeof(TOut) * kD / 128;   // output staged as 128-byte wide boxes (kGrad: hi, lo)
    static constexpr int offPT = 0;                       // masked scores, transposed: rows = s, 64 t per row (hi, lo)
    static constexpr int offShi = offPT + (kPPair ? 2 : 1) * kTile;   // state, bf16 high part: rows = d_k
    static constexpr int offSlo = offShi + kTile;         // state, bf16 low part
    static constexpr int offStage = offSlo + kTile;       // after the score tile: the G3 descriptor reaches K from P forwards
    // output staging; also what a 128-row operand that starts in the last tile of the last stage reads past it
    static constexpr int offO = offStage + kStages * kTilesPerStage * kTile;
    static constexpr int offD = offO + (kOBoxes > 1 ? kOBoxes : 1) * kTile;      // d_o tiles, two slots (kGrad)
    static constexpr int offBar = offD + (kGrad ? 2 : 0) * kTile;   // full[kStages], p, o, pt, s, dfull[2]
    static constexpr int offTmem = offBar + 8 * (kStages + 6);
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
};
constexpr int kTmemCols = 128;
// Diagnostics for a wait that gave up: words 8..11 of the workspace header keep, for the first such wait since the
// header was last zeroed by the caller, a site code (100 * kMask + site; 9000 + ... in the state kernel), the CTA,
// the chunk and the grid size.  The library never clears them.
#define DIAG(site, extra) do { if (atomicCAS(status + 8, 0, (site)) == 0) { status[9] = blockIdx.x; status[10] = (extra); status[11] = gridDim.x; } } while (0)
constexpr int kColOS = 0;    // rows 0..63: output tile, rows 64..127: running state; 64 columns
constexpr int kColPT = 64;   // rows 64..127: transposed scores; 64 columns

// kReverse: the anti-causal mirror (token t attends keys s >= t; the state accumulates from the end of the
// sequence).  Chunks are walked from the last to the first and the mask is the upper triangle; everything
// else, including the split into groups, works on the mirrored chunk index.  Used by the backward pass.
template <typename TOut, int kMask, bool kReverse, bool kGrad = false>
// Two CTAs per SM wherever shared memory allows (every mask but 15): 10 warps over the four register files put
// three on one of them, which caps a thread at 168 registers.
__global__ void __launch_bounds__(kThreads, kMask == 15 ? 1 : 2)
linattn_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                     const __grid_constant__ CUtensorMap tm_d, int H, int L,
                     float scale, int norm, float eps, int *__restrict__ status, const float *__restrict__ s_part,
                     int G, int cg0, int cg, const float *__restrict__ state_in, float *__restrict__ state_out, const WaitCtl wc)
{
    // Grid: one CTA per (group, batch*head), group-major.  Group 0 covers the first cg0 chunks of its sequence, group
    // g >= 1 the next cg chunks each (the last one what is left).  Group g starts from the state
    // sum_{g' < g} s_part[bh][g'] (per-group K^T V sums written by the state kernel), plus the caller's initial state
    // state_in[bh] if given; the last group writes the final state.  When G > 1 this kernel is launched as a
    // programmatic dependent of the state kernel: group 0 needs nothing from it and runs beside it (hence the longer
    // first group), the other groups wait for it before they read s_part.
    using SM = Smem<TOut, kMask, kGrad>;
    constexpr int kStages = SM::kStages;
    constexpr int kTPS = SM::kTilesPerStage;
    constexpr int kIn = SM::kIn;
    constexpr bool kPPair = SM::kPPair;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {  // swizzled tiles need a 1024-byte aligned base: report instead of corrupting
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nbh = gridDim.x / G;
    const int bh = blockIdx.x % nbh, g = blockIdx.x / nbh;
    const int b = bh / H, h = bh % H;
    const int c0 = g == 0 ? 0 : cg0 + (g - 1) * cg;                // first (mirrored) chunk of this group
    const int nch_total = (L + kC - 1) / kC;
    const int nchunks = min(g == 0 ? cg0 : cg, nch_total - c0);    // chunks of this group
    // token offset of the group's chunk number `chunk`
    auto tok = [&](int chunk) { return (kReverse ? nch_total - 1 - (c0 + chunk) : c0 + chunk) * kC; };
    const bool has_init = g > 0 || state_in != nullptr;

    const uint32_t bar_full0 = sbase + SM::offBar;
    const uint32_t bar_p = bar_full0 + 8 * kStages;   // G1 of a chunk has completed (tensor core -> warps 2,3)
    const uint32_t bar_o = bar_p + 8;                 // G2 + G3 of a chunk have completed (-> all roles)
    const uint32_t bar_pt = bar_o + 8;                // score tile of a chunk is in shared memory (warps 2,3 -> issuer)
    const uint32_t bar_s = bar_pt + 8;                // output/state rows read, state tiles written (4 warps -> issuer)
    const uint32_t bar_d0 = bar_s + 8;                // kGrad: the d_o tile of slot 0 / 1 has landed (copy engine -> epilogue warps)
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM::offTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::offAbort);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(bar_full0 + 8 * s, 1);
        mbar_init(bar_p, 1);
        mbar_init(bar_o, 1);
        mbar_init(bar_pt, 2);
        mbar_init(bar_s, 4);
        if (kGrad) {
            mbar_init(bar_d0, 1);
            mbar_init(bar_d0 + 8, 1);
            tma_prefetch_desc(&tm_d);
        }
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
            auto stage_base = [&](int chunk) { return sbase + SM::offStage + (chunk % kStages) * kTPS * kTile; };
            auto issue_load = [&](int chunk) {
                const uint32_t bar = bar_full0 + 8 * (chunk % kStages), dst = stage_base(chunk);
                mbar_expect_tx(bar, kTPS * kTile);
                tma_load_5d(dst, &tm_q, bar, 0, h, tok(chunk), b, 0);
                tma_load_5d(dst + kTile, &tm_k, bar, 0, h, tok(chunk), b, 0);
                tma_load_5d(dst + 2 * kTile, &tm_v, bar, 0, h, tok(chunk), b, 0);
                if (kIn & 1) tma_load_5d(dst + SM::iQlo * kTile, &tm_q, bar, 0, h, tok(chunk), b, 1);
                if (kIn & 2) tma_load_5d(dst + SM::iKlo * kTile, &tm_k, bar, 0, h, tok(chunk), b, 1);
                if (kIn & 4) tma_load_5d(dst + SM::iVlo * kTile, &tm_v, bar, 0, h, tok(chunk), b, 1);
            };
            constexpr uint32_t idescG1 = make_idesc(128, kC, 0, 0);   // [Q;K] (K-major) x Q^T (K-major)
            constexpr uint32_t idescG2 = make_idesc(128, kD, 0, 1);   // [Q;K] (K-major) x S (MN-major)
            constexpr uint32_t idescG3 = make_idesc(128, kD, 1, 1);   // [P^T|K] (MN-major) x V (MN-major)
            // G1 of a chunk; false if the chunk's tiles never arrived
            auto issue_scores = [&](int chunk) -> bool {
                if (!mbar_wait(bar_full0 + 8 * (chunk % kStages), (chunk / kStages) & 1, abort_flag, wc.limit)) { DIAG(1 + 100 * kMask, chunk); return false; }
                tc_fence_after();
                const uint32_t qk_lo = desc_lo(stage_base(chunk));
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColPT, qk_lo + 2 * k, qk_lo + 2 * k, idescG1, k > 0);
                if (kIn & 1) {   // + K_hi Q_lo^T
                    const uint32_t q2_lo = desc_lo(stage_base(chunk) + SM::iQlo * kTile);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColPT, qk_lo + 2 * k, q2_lo + 2 * k, idescG1, 1);
                }
                if (kIn & 2) {   // + K_lo Q_hi^T: the 128-row operand starts one tile before K_lo (rows 0..63 are not used)
                    const uint32_t xk2_lo = desc_lo(stage_base(chunk) + (SM::iKlo - 1) * kTile);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColPT, xk2_lo + 2 * k, qk_lo + 2 * k, idescG1, 1);
                }
                umma_commit(bar_p);
                return true;
            };
            const uint32_t shi_lo = desc_lo(sbase + SM::offShi), slo_lo = desc_lo(sbase + SM::offSlo);
            int loads_issued = 0, consumed = 0, d_issued = 0;
            // kGrad: d_o tile of a chunk into slot chunk % 2.  Slot and barrier are reused two chunks later, after the
            // epilogue warps have copied their rows: they say so with their arrival on bar_s, which the issuer has
            // waited for before it issues the reload, so the barrier never runs a phase ahead of its waiters.
            auto issue_d = [&](int chunk) {
                const uint32_t bar = bar_d0 + 8 * (chunk & 1);
                mbar_expect_tx(bar, kTile);
                tma_load_5d(sbase + SM::offD + (chunk & 1) * kTile, &tm_d, bar, 0, h, tok(chunk), b, 0);
            };
            for (; loads_issued < kStages && loads_issued < nchunks; ++loads_issued) issue_load(loads_issued);
            if (kGrad)
                for (; d_issued < 2 && d_issued < nchunks; ++d_issued) issue_d(d_issued);
            bool ok = issue_scores(0);
            uint32_t par_s = 0;
            for (int i = 0; ok && i < nchunks; ++i) {
                const uint32_t st = stage_base(i);
                if (i > 0 || has_init) {
                    // G2: rows 0..63 of OS = Q S_hi + Q S_lo; needs the state tiles of the previous chunk (or
                    // of the group's initial state) and the previous output rows out of TMEM
                    ok = mbar_wait(bar_s, par_s, abort_flag, wc.limit);
                    if (!ok) DIAG(2 + 100 * kMask, i);
                    par_s ^= 1;
                    if (!ok) break;
                    tc_fence_after();
                    if (kGrad && i >= 1 && i + 1 < nchunks) {   // the epilogue warps hold d_o of chunk i - 1: its slot takes chunk i + 1
                        issue_d(i + 1);
                        ++d_issued;
                    }
                    const uint32_t qk_lo = desc_lo(st);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColOS, qk_lo + 2 * k, shi_lo + 128 * k, idescG2, k > 0, 1);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColOS, qk_lo + 2 * k, slo_lo + 128 * k, idescG2, 1, 1);
                    if (kIn & 1) {   // + Q_lo S_hi (rows 64..127 of the operand: whatever follows Q_lo; their lanes are write-disabled)
                        const uint32_t qk2_lo = desc_lo(st + SM::iQlo * kTile);
#pragma unroll
                        for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColOS, qk2_lo + 2 * k, shi_lo + 128 * k, idescG2, 1, 1);
                    }
                }
                // G3: OS += [P^T | K]^T V; atom 0 = score tile, atom 1 = K tile of this stage
                ok = mbar_wait(bar_pt, i & 1, abort_flag, wc.limit);
                if (!ok) DIAG(3 + 100 * kMask, i);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_lo = desc_lo(sbase + SM::offPT, st + kTile - (sbase + SM::offPT)), v_lo = desc_lo(st + 2 * kTile);
#pragma unroll
                for (int k = 0; k < kC / 16; ++k)
                    umma_bf16(tmem + kColOS, a_lo + 128 * k, v_lo + 128 * k, idescG3, (i > 0 || has_init || k > 0) ? 1u : 0u);
                if (kIn & 4) {   // + [P_hi^T | K_hi]^T V_lo
                    const uint32_t v2_lo = desc_lo(st + SM::iVlo * kTile);
#pragma unroll
                    for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem + kColOS, a_lo + 128 * k, v2_lo + 128 * k, idescG3, 1);
                }
                if (kPPair || (kIn & 2)) {   // + [P_lo^T | K_lo]^T V_hi; a half that does not exist is write-disabled
                    const uint32_t atom0 = sbase + SM::offPT + (kPPair ? kTile : 0);
                    const uint32_t atom1 = st + ((kIn & 2) ? SM::iKlo : 1) * kTile;
                    const uint32_t a2_lo = desc_lo(atom0, atom1 - atom0);
                    const uint32_t lanes = (kPPair && (kIn & 2)) ? 0u : (kPPair ? 1u : 2u);
#pragma unroll
                    for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem + kColOS, a2_lo + 128 * k, v_lo + 128 * k, idescG3, 1, lanes);
                }
                umma_commit(bar_o);
                if (i + 1 < nchunks) {
                    ok = issue_scores(i + 1);
                    if (!ok) break;
                }
                // the stage is free once G3 has completed: prefetch the chunk that will use it next
                ok = mbar_wait(bar_o, i & 1, abort_flag, wc.limit);
                if (!ok) DIAG(4 + 100 * kMask, i);
                if (!ok) break;
                consumed = i + 1;
                if (i + kStages < nchunks) {
                    issue_load(i + kStages);
                    ++loads_issued;
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(status, (int)CHELA_ERR_TIMEOUT);
                // drain loads that were issued but never consumed (bounded), so no copy lands after exit
                for (int c = consumed; c < loads_issued; ++c)
                    mbar_wait(bar_full0 + 8 * (c % kStages), (c / kStages) & 1, nullptr, wc.limit);
                if (kGrad)
                    for (int c = d_issued > 2 ? d_issued - 2 : 0; c < d_issued; ++c) mbar_wait(bar_d0 + 8 * (c & 1), (c >> 1) & 1, nullptr, wc.limit);
            }
        }
    } else {
        // =========================================== compute warps ====================================
        // TMEM lane = accumulator row = thread.  Warps 0,1 own output rows t = tid; warps 2,3 own row
        // r = tid - 64 of the transposed scores (s) and of the state (d_k).
        const bool upper = warp >= 2;
        const int r = tid & 63;
        const uint32_t tmem_warp = tmem + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
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
                    float l0, l1;
                    sub2(l0, l1, x0, x1, hf.x, hf.y);
                    wh[e] = *reinterpret_cast<const uint32_t *>(&hh);
                    wl[e] = pack_bf16(l0, l1);
                }
                const uint32_t off = sw128(r, c8);
                *reinterpret_cast<uint4 *>(sHi + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
                *reinterpret_cast<uint4 *>(sLo + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
            }
        };
        // the same for one half of the row (32 columns: pieces 4 * hf .. 4 * hf + 3), for the per-chunk loop below
        auto write_state_half = [&](const float(&sv)[32], int hf) {
            uint8_t *sHi = smem + SM::offShi, *sLo = smem + SM::offSlo;
#pragma unroll
            for (int c8 = 0; c8 < 4; ++c8) {
                uint32_t wh[4], wl[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float x0 = sv[c8 * 8 + e * 2], x1 = sv[c8 * 8 + e * 2 + 1];
                    const __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                    const float2 hf2 = __bfloat1622float2(hh);
                    float l0, l1;
                    sub2(l0, l1, x0, x1, hf2.x, hf2.y);
                    wh[e] = *reinterpret_cast<const uint32_t *>(&hh);
                    wl[e] = pack_bf16(l0, l1);
                }
                const uint32_t off = sw128(r, 4 * hf + c8);
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
                if (state_in) {
                    const float4 *src = reinterpret_cast<const float4 *>(state_in + ((size_t)bh * kD + r) * kD);
#pragma unroll
                    for (int j = 0; j < kD / 4; ++j) {
                        const float4 x = src[j];
                        sv[4 * j] = x.x; sv[4 * j + 1] = x.y; sv[4 * j + 2] = x.z; sv[4 * j + 3] = x.w;
                    }
                }
                if (g > 0) griddep_wait();   // the state kernel has completed
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
                ok = __all_sync(0xffffffffu, mbar_wait(bar_p, i & 1, abort_flag, wc.limit));
                if (!ok && lane == 0) DIAG(6 + 100 * kMask, i);
                if (!ok) break;
                tc_fence_after();
                // row s keeps t >= s (mirrored: t <= s); all-zero blocks are not read from TMEM
                float p[2][32];
                // causal: rows s >= 32 (warp 3) have nothing at t < 32; mirrored: rows s < 32 (warp 2) nothing at t >= 32
                const bool live0 = kReverse || warp == 2, live1 = !kReverse || warp == 3;
                if (live0) tmem_ld32(tmem_warp + kColPT, p[0]);
                if (live1) tmem_ld32(tmem_warp + kColPT + 32, p[1]);
                tmem_ld_wait();
                uint8_t *sP = smem + SM::offPT;
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    const bool live = cb == 0 ? live0 : live1;
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        uint32_t w[4], w2[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int t = cb * 32 + c8 * 8 + e * 2;
                            const float x0 = (live && (kReverse ? t <= r : t >= r)) ? p[cb][c8 * 8 + e * 2] : 0.f;
                            const float x1 = (live && (kReverse ? t + 1 <= r : t + 1 >= r)) ? p[cb][c8 * 8 + e * 2 + 1] : 0.f;
                            const __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                            w[e] = *reinterpret_cast<const uint32_t *>(&hh);
                            if (kPPair) {
                                const float2 hf = __bfloat1622float2(hh);
                                w2[e] = pack_bf16(x0 - hf.x, x1 - hf.y);
                            }
                        }
                        *reinterpret_cast<uint4 *>(sP + sw128(r, cb * 4 + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
                        if (kPPair) *reinterpret_cast<uint4 *>(sP + kTile + sw128(r, cb * 4 + c8)) = make_uint4(w2[0], w2[1], w2[2], w2[3]);
                    }
                }
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && !(wc.skip_arrival && blockIdx.x == 0 && i == 0)) mbar_arrive(bar_pt);   // test hook: one arrival left out
            }
            ok = __all_sync(0xffffffffu, mbar_wait(bar_o, i & 1, abort_flag, wc.limit));
            if (!ok && lane == 0) DIAG(8 + 100 * kMask + 10 * warp, i);
            if (!ok) break;
            tc_fence_after();
            float acc[kD];
            if (!upper) {
                // ---- output row t: scale, normaliser -> swizzled staging -> TMA store (per warp: 32 rows) ----
                tmem_ld32(tmem_warp + kColOS, *reinterpret_cast<float(*)[32]>(&acc[0]));
                tmem_ld32(tmem_warp + kColOS + 32, *reinterpret_cast<float(*)[32]>(&acc[32]));
                tmem_ld_wait();
                uint4 dq4[kGrad ? 8 : 1];   // kGrad: row t of d_o (64 bf16), copied out of its slot before the arrival below
                if (kGrad) {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_d0 + 8 * (i & 1), (i >> 1) & 1, abort_flag, wc.limit));
                    if (!ok && lane == 0) DIAG(7 + 100 * kMask, i);
                    if (!ok) break;
                    const uint8_t *sD = smem + SM::offD + (i & 1) * kTile;
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) dq4[c8] = *reinterpret_cast<const uint4 *>(sD + sw128(r, c8));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar_s);     // the output rows are out of TMEM: G2 of the next chunk may overwrite them
                    bulk_wait_read0();      // this warp's previous output boxes have left shared memory
                }
                __syncwarp();
                float inv;
                if (kGrad) {   // the pull-back below needs the scaled row r itself
                    float ss = 0.f;
#pragma unroll
                    for (int j = 0; j < kD; ++j) {
                        acc[j] *= scale;
                        ss = fmaf(acc[j], acc[j], ss);
                    }
                    inv = norm ? rsqrtf(ss * (1.0f / kD) + eps) : 1.0f;
                } else {
                    // scaled and normalised in one multiplication, o = acc * scale / sqrt(scale^2 mean(acc^2) + eps),
                    // with two-wide fp32 instructions; the stores below then take the row as it is
                    float ss0 = 0.f, ss1 = 0.f;
#pragma unroll
                    for (int j = 0; j < kD; j += 2) sqacc2(ss0, ss1, acc[j], acc[j + 1]);
                    const float f = norm ? scale * rsqrtf((ss0 + ss1) * (scale * scale * (1.0f / kD)) + eps) : scale;
#pragma unroll
                    for (int j = 0; j < kD; j += 2) mul2(acc[j], acc[j + 1], acc[j], acc[j + 1], f);
                    inv = 1.0f;
                }
                uint8_t *sO = smem + SM::offO;
                if (kGrad) {
                    // acc = r (scaled); o = r inv; G = scale (d_o - o <o, d_o> / d) inv, stored as hi and lo planes
                    float od = 0.f;
                    const __nv_bfloat162 *dh = reinterpret_cast<const __nv_bfloat162 *>(dq4);
#pragma unroll
                    for (int j = 0; j < kD / 2; ++j) {
                        const float2 d2 = __bfloat1622float2(dh[j]);
                        od = fmaf(acc[2 * j] * inv, d2.x, od);
                        od = fmaf(acc[2 * j + 1] * inv, d2.y, od);
                    }
                    od *= 1.0f / kD;
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) {
                        uint32_t wh[4], wl[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int j = c8 * 4 + e;
                            const float2 d2 = __bfloat1622float2(dh[j]);
                            const float g0 = scale * (d2.x - acc[2 * j] * inv * od) * inv, g1 = scale * (d2.y - acc[2 * j + 1] * inv * od) * inv;
                            const __nv_bfloat162 hh = __floats2bfloat162_rn(g0, g1);
                            const float2 hf = __bfloat1622float2(hh);
                            wh[e] = *reinterpret_cast<const uint32_t *>(&hh);
                            wl[e] = pack_bf16(g0 - hf.x, g1 - hf.y);
                        }
                        *reinterpret_cast<uint4 *>(sO + sw128(r, c8)) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
                        *reinterpret_cast<uint4 *>(sO + kTile + sw128(r, c8)) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
                    }
                } else if (sizeof(TOut) == 4) {
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
                        if (kGrad)   // box = plane (hi, lo)
                            tma_store_5d(&tm_o, sbase + SM::offO + bx * kTile + warp * 32 * 128, 0, h, tok(i) + warp * 32, b, bx);
                        else
                            tma_store_5d(&tm_o, sbase + SM::offO + bx * kTile + warp * 32 * 128, bx * (128 / (int)sizeof(TOut)), h,
                                         tok(i) + warp * 32, b, 0);   // the map's rank is 5 (plane = 0)
                    bulk_commit();
                }
            } else {
                // ---- state row d_k: bf16 hi + lo -> shared (MN-major B operand of the next chunk's G2) ------
                if (i + 1 < nchunks) {
                    // (a loop over the two halves, not unrolled: the per-chunk code of these warps stays small)
#pragma unroll 1
                    for (int hf = 0; hf < 2; ++hf) {
                        float sv[32];
                        tmem_ld32(tmem_warp + kColOS + 32 * hf, sv);
                        tmem_ld_wait();
                        write_state_half(sv, hf);
                    }
                    fence_proxy_async();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_s);
                } else if (state_out && g == G - 1) {
                    // last chunk of the sequence: the fp32 state leaves the SM once, for the caller
                    tmem_ld32(tmem_warp + kColOS, *reinterpret_cast<float(*)[32]>(&acc[0]));
                    tmem_ld32(tmem_warp + kColOS + 32, *reinterpret_cast<float(*)[32]>(&acc[32]));
                    tmem_ld_wait();
                    float4 *dst = reinterpret_cast<float4 *>(state_out + ((size_t)bh * kD + r) * kD);
#pragma unroll
                    for (int j = 0; j < kD / 4; ++j) dst[j] = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
                }
            }
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicExch(status, (int)CHELA_ERR_TIMEOUT);
        }
        if (!upper && lane == 0) bulk_wait0();   // output boxes fully written before the CTA retires
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
template <int kMask>
struct SmemState {
    static constexpr int kKV = kMask & 6;                          // bit 1: K is a pair, bit 2: V is a pair
    static constexpr int kTilesPerStage = 2 + popc3(kKV);          // K, V (hi), then the low planes that exist
    static constexpr int iKlo = 2, iVlo = 2 + ((kKV >> 1) & 1);
    static constexpr int offStage = 0;
    // one spare tile after the ring: a two-atom operand that starts in the ring's last tile reads it
    static constexpr int offBar = (kStStages * kTilesPerStage + 1) * kTile;   // full[kStStages], empty[kStStages], done
    static constexpr int offTmem = offBar + 8 * (2 * kStStages + 1);
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
};

template <int kMask, bool kReverse>
__global__ void __launch_bounds__(kThreads)
linattn_state_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     float *__restrict__ s_part, int H, int L, int G, int cg0, int cg, int *__restrict__ status, const WaitCtl wc)
{
    using SM = SmemState<kMask>;
    constexpr int kKV = SM::kKV;
    constexpr int kTPS = SM::kTilesPerStage;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    griddep_launch_dependents();   // the main kernel's first groups may be scheduled beside this kernel
    // group-major like the main kernel, longest group (0) first
    const int nbh = gridDim.x / (G - 1);
    const int bh = blockIdx.x % nbh, g = blockIdx.x / nbh;
    const int b = bh / H, h = bh % H;
    const int c0 = g == 0 ? 0 : cg0 + (g - 1) * cg, nchunks = g == 0 ? cg0 : cg;    // every group but the last is full

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
                const uint32_t bar = bar_full0 + 8 * (chunk % kStStages), dst = sbase + SM::offStage + (chunk % kStStages) * kTPS * kTile;
                mbar_expect_tx(bar, kTPS * kTile);
                const int t0 = (kReverse ? (L + kC - 1) / kC - 1 - (c0 + chunk) : c0 + chunk) * kC;
                tma_load_5d(dst, &tm_k, bar, 0, h, t0, b, 0);
                tma_load_5d(dst + kTile, &tm_v, bar, 0, h, t0, b, 0);
                if (kKV & 2) tma_load_5d(dst + SM::iKlo * kTile, &tm_k, bar, 0, h, t0, b, 1);
                if (kKV & 4) tma_load_5d(dst + SM::iVlo * kTile, &tm_v, bar, 0, h, t0, b, 1);
            };
            constexpr uint32_t idesc = make_idesc(128, kD, 1, 1);
            int loads_issued = 0, consumed = 0;
            for (; loads_issued < kStStages && loads_issued < nchunks; ++loads_issued) issue_load(loads_issued);
            bool ok = true;
            for (int i = 0; i < nchunks; ++i) {
                const int stage = i % kStStages;
                ok = mbar_wait(bar_full0 + 8 * stage, (i / kStStages) & 1, abort_flag, wc.limit);
                if (!ok) DIAG(9001 + 100 * kMask, i);
                if (!ok) break;
                tc_fence_after();
                const uint32_t st = sbase + SM::offStage + stage * kTPS * kTile;
                const uint32_t a_lo = desc_lo(st, kTile), v_lo = desc_lo(st + kTile);
#pragma unroll
                for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem, a_lo + 128 * k, v_lo + 128 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                if (kKV & 4) {   // + K_hi^T V_lo
                    const uint32_t v2_lo = desc_lo(st + SM::iVlo * kTile);
#pragma unroll
                    for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem, a_lo + 128 * k, v2_lo + 128 * k, idesc, 1);
                }
                if (kKV & 2) {   // + K_lo^T V_hi (second atom: whatever tile follows; its rows are the ignored ones)
                    const uint32_t a2_lo = desc_lo(st + SM::iKlo * kTile, kTile);
#pragma unroll
                    for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem, a2_lo + 128 * k, v_lo + 128 * k, idesc, 1);
                }
                umma_commit(bar_empty0 + 8 * stage);
                consumed = i + 1;
                if (i + kStStages < nchunks) {
                    ok = mbar_wait(bar_empty0 + 8 * stage, (i / kStStages) & 1, abort_flag, wc.limit);
                    if (!ok) DIAG(9002 + 100 * kMask, i);
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
                    mbar_wait(bar_full0 + 8 * (c % kStStages), (c / kStStages) & 1, nullptr, wc.limit);
            }
        }
    } else if (warp < 2) {
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_done, 0, abort_flag, wc.limit));
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

// [B, L, H, 64] viewed as a rank-4 tensor (d, H, L, B); box = (128 bytes of d) x 1 x C x 1, 128-byte
// swizzle.  Loads: rows past L are out of bounds for the copy engine and arrive as zeros.  Stores: rows
// past L are clipped.
// `planes` = 2 for a bf16 pair (the low plane follows the high plane), else 1: always a rank-5 map.
bool make_map(CUtensorMap *map, const void *ptr, int B, int H, int L, int C, bool f32, int planes)
{
    const cuuint64_t es = f32 ? 4 : 2;
    const cuuint64_t dims[5] = {(cuuint64_t)kD, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B, (cuuint64_t)planes};
    const cuuint64_t strides[4] = {(cuuint64_t)kD * es, (cuuint64_t)H * kD * es, (cuuint64_t)L * H * kD * es,
                                   (cuuint64_t)B * L * H * kD * es};
    const cuuint32_t box[5] = {(cuuint32_t)(128 / es), 1, (cuuint32_t)C, 1, 1};
    return make_map_sw128(map, ptr, f32, 5, dims, strides, box);
}

// How a call is split along L.  The grid holds B*H*G CTAs, no more than are resident at once (two per SM,
// one per SM for the full-pair kernel); a group never has fewer than 16 chunks.  Group 0 is longer than the
// others when there are two: it runs beside the state kernel, the second starts when that has finished, and both
// should end together.
struct SplitPlan {
    int G, cg0, cg;
    size_t part_bytes;
};
SplitPlan split_plan(int B, int H, int L, bool pair, int sms = 0)   // pair: shared memory allows one CTA per SM only
{
    int dev = 0;
    if (sms <= 0 && (cudaGetDevice(&dev) != cudaSuccess ||
                     cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0))
        sms = 148;
    const long long bh = (long long)B * H;
    const int nchunks = (L + kC - 1) / kC;
    const long long slots = (pair ? 1LL : 2LL) * sms;   // resident CTAs: shared memory allows 2 per SM, 1 for pairs
    // Measured on B200: with fewer (batch, head) pairs than SMs, fill the resident slots (a lone CTA per SM is
    // bound by its own dependency chain, two per SM by HBM), but keep at least 16 chunks per group.
    int G = 1;
    if (bh < sms) {
        G = (int)(slots / bh);
        if (G > nchunks / 16) G = nchunks / 16;
        if (G < 1) G = 1;
    }
    SplitPlan p;
    if (G == 1) {
        p.G = 1;
        p.cg0 = p.cg = nchunks;
    } else {
        // cg / cg0, measured on B200 (L = 32K...128K, B*H = 32...128): with two groups everything is resident at once and
        // the first group should be twice the second; with more groups the later ones queue for CTA slots behind the
        // state kernel anyway and equal groups are best
        const double rho = G == 2 ? 0.5 : 1.0;
        p.cg0 = (int)((double)nchunks / (1.0 + (G - 1) * rho) + 0.999);
        if (p.cg0 > nchunks - (G - 1)) p.cg0 = nchunks - (G - 1);
        p.cg = (nchunks - p.cg0 + G - 2) / (G - 1);
        p.G = 1 + (nchunks - p.cg0 + p.cg - 1) / p.cg;
    }
    p.part_bytes = (size_t)bh * (p.G - 1) * kD * kD * sizeof(float);
    return p;
}

// The main kernel after the state kernel of the same call, allowed to start while that still runs.
template <typename Kern, typename... Args>
chela_status_t launch_dependent(Kern kern, int grid, int smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, args...) != cudaSuccess) {
        // without the attribute the launch is an ordinary stream-ordered one and griddepcontrol.wait returns at once
        (void)cudaGetLastError();
        kern<<<grid, kThreads, smem, stream>>>(args...);
    }
    return last_launch_status();
}
constexpr size_t kWsHeader = 512;   // word 0: asynchronous status; the rest: diagnostics

template <typename TOut, int kMask, bool kReverse>
chela_status_t launch_t(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int norm, float eps,
                        float scale, void *workspace, const float *state_in, float *state_out, cudaStream_t stream,
                        int planes_mask, bool keep_status = false)
{
    // planes_mask: which of q, k, v are given with two planes.  An operand that the kernel treats as a pair but
    // that has one plane gets a one-plane map: its "low plane" is then out of bounds for the copy engine and
    // arrives as zeros without touching memory (only the full-pair kernel, kMask = 15, is used that way).
    CUtensorMap mq, mk, mv, mo;
    const int pq = (planes_mask & 1) ? 2 : 1, pk = (planes_mask & 2) ? 2 : 1, pv = (planes_mask & 4) ? 2 : 1;
    if (!make_map(&mq, q, B, H, L, kC, false, pq) || !make_map(&mk, k, B, H, L, kC, false, pk) ||
        !make_map(&mv, v, B, H, L, kC, false, pv) || !make_map(&mo, o, B, H, L, 32, sizeof(TOut) == 4, 1))
        return CHELA_ERR_CUDA;
    const SplitPlan plan = split_plan(B, H, L, Smem<TOut, kMask>::bytes > 113 * 1024);
    const WaitCtl wc = current_wait_ctl();
    int *status = (int *)workspace;
    float *s_part = (float *)((char *)workspace + kWsHeader);
    // keep_status: a later launch of a multi-launch call must not erase what an earlier one reported
    if (!keep_status && cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return CHELA_ERR_CUDA;
    if (plan.G > 1) {
        auto skern = linattn_state_kernel<(kMask & 6), kReverse>;
        constexpr int ssmem = SmemState<(kMask & 6)>::bytes;
        if (cudaFuncSetAttribute(skern, cudaFuncAttributeMaxDynamicSharedMemorySize, ssmem) != cudaSuccess) return CHELA_ERR_CUDA;
        skern<<<B * H * (plan.G - 1), kThreads, ssmem, stream>>>(mk, mv, s_part, H, L, plan.G, plan.cg0, plan.cg, status, wc);
        if (cudaGetLastError() != cudaSuccess) return CHELA_ERR_CUDA;
    }
    auto kern = linattn_sm100_kernel<TOut, kMask, kReverse>;
    const int smem = Smem<TOut, kMask>::bytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return CHELA_ERR_CUDA;
    if (plan.G > 1)
        return launch_dependent(kern, B * H * plan.G, smem, stream, mq, mk, mv, mo, mo, H, L, scale, norm, eps, status,
                                (const float *)s_part, plan.G, plan.cg0, plan.cg, state_in, state_out, wc);
    kern<<<B * H, kThreads, smem, stream>>>(mq, mk, mv, mo, mo, H, L, scale, norm, eps, status, s_part, 1, plan.cg0, plan.cg,
                                            state_in, state_out, wc);
    return last_launch_status();
}

// Backward pass, first launch: recomputes the forward rows (scores and state kept as bf16 pairs) and writes
// G = d_o pulled back through the normaliser, as a bf16 pair (two planes at g).
chela_status_t launch_grad(const void *q, const void *k, const void *v, const void *d_o, void *g, int B, int H, int L, float eps,
                           float scale, void *workspace, cudaStream_t stream)
{
    CUtensorMap mq, mk, mv, mg, md;
    if (!make_map(&mq, q, B, H, L, kC, false, 1) || !make_map(&mk, k, B, H, L, kC, false, 1) || !make_map(&mv, v, B, H, L, kC, false, 1) ||
        !make_map(&md, d_o, B, H, L, kC, false, 1) || !make_map(&mg, g, B, H, L, 32, false, 2))
        return CHELA_ERR_CUDA;
    using SM = Smem<__nv_bfloat16, 8, true>;
    const SplitPlan plan = split_plan(B, H, L, SM::bytes > 113 * 1024);
    const WaitCtl wc = current_wait_ctl();
    int *status = (int *)workspace;
    float *s_part = (float *)((char *)workspace + kWsHeader);
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return CHELA_ERR_CUDA;
    if (plan.G > 1) {
        auto skern = linattn_state_kernel<0, false>;
        constexpr int ssmem = SmemState<0>::bytes;
        if (cudaFuncSetAttribute(skern, cudaFuncAttributeMaxDynamicSharedMemorySize, ssmem) != cudaSuccess) return CHELA_ERR_CUDA;
        skern<<<B * H * (plan.G - 1), kThreads, ssmem, stream>>>(mk, mv, s_part, H, L, plan.G, plan.cg0, plan.cg, status, wc);
        if (cudaGetLastError() != cudaSuccess) return CHELA_ERR_CUDA;
    }
    auto kern = linattn_sm100_kernel<__nv_bfloat16, 8, false, true>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::bytes) != cudaSuccess) return CHELA_ERR_CUDA;
    if (plan.G > 1)
        return launch_dependent(kern, B * H * plan.G, SM::bytes, stream, mq, mk, mv, mg, md, H, L, scale, 1, eps, status,
                                (const float *)s_part, plan.G, plan.cg0, plan.cg, (const float *)nullptr, (float *)nullptr, wc);
    kern<<<B * H, kThreads, SM::bytes, stream>>>(mq, mk, mv, mg, md, H, L, scale, 1, eps, status, s_part, 1, plan.cg0, plan.cg,
                                                 nullptr, nullptr, wc);
    return last_launch_status();
}

}  // namespace

chela_status_t launch_linattn_sm100_grad(const void *q, const void *k, const void *v, const void *d_o, void *g, int B, int H, int L,
                                         float eps, float scale, void *workspace, cudaStream_t stream)
{
    return launch_grad(q, k, v, d_o, g, B, H, L, eps, scale, workspace, stream);
}

void linattn_sm100_split(int B, int H, int L, int d, bool full_pair, int sms, int *G, int *cg0, int *cg)
{
    if (d == 128) {
        linattn_sm100_d128_split(B, H, L, sms, G, cg0, cg);
        return;
    }
    if (!full_pair) {
        // plain bf16: no groups of consecutive chunks; with fewer pairs than SMs a sequence is shared by stride
        const int stride = linattn_sm100_pipe_stride(B, H, L, sms);
        *G = stride > 1 ? stride : 1;
        *cg0 = *cg = stride > 1 ? 0 : (L + kC - 1) / kC;
        return;
    }
    const SplitPlan p = split_plan(B, H, L, full_pair, sms);
    *G = p.G;
    *cg0 = p.cg0;
    *cg = p.cg;
}

bool linattn_sm100_supported(int B, int H, int L, int d, int chunk, chela_dtype_t in_dtype, chela_dtype_t out_dtype)
{
    (void)B; (void)H; (void)L;
    return (in_dtype == CHELA_BF16 || in_dtype == CHELA_BF16_PAIR) && (out_dtype == CHELA_F32 || out_dtype == CHELA_BF16) &&
           (d == kD || d == 128) && (chunk == 64 || chunk == 128);
}

// Header (word 0 = asynchronous status of the last launch that used this workspace) followed by the
// per-group state sums [B*H][G-1][64][64] fp32 of a call that is split along L.
size_t linattn_sm100_workspace_bytes(int B, int H, int L, int d, int)
{
    if (d == 128) return linattn_sm100_d128_workspace_bytes(B, H, L);
    if (d != kD) return 0;
    const size_t a = split_plan(B, H, L, false).part_bytes, b = split_plan(B, H, L, true).part_bytes;
    return kWsHeader + (a > b ? a : b);   // the query does not know the input dtype: cover both plans
}

chela_status_t launch_linattn_sm100(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int d,
                                    int chunk, chela_dtype_t in_dtype, chela_dtype_t out_dtype, int norm, float eps,
                                    float scale, void *workspace, cudaStream_t stream, const float *state_in,
                                    float *state_out, bool reverse, int pair_mask, bool keep_status)
{
    if (d == 128)
        return launch_linattn_sm100_d128(q, k, v, o, B, H, L, in_dtype, out_dtype, norm, eps, scale, workspace, stream, state_in,
                                         state_out, reverse, pair_mask, keep_status);
    // The result does not depend on the chunk size: both supported values run on 64-token tiles.
    (void)chunk;
    const bool pair = in_dtype == CHELA_BF16_PAIR;
    const int pm = pair ? (pair_mask & 7) : 0;
    if (reverse) {   // anti-causal mirror: fp32 output, no state carry (the backward pass)
        if (out_dtype != CHELA_F32 || state_in || state_out) return CHELA_ERR_UNSUPPORTED;
        if (!pair) return launch_t<float, 0, true>(q, k, v, o, B, H, L, norm, eps, scale, workspace, nullptr, nullptr, stream, 0, keep_status);
        if (pm == 2) return launch_t<float, 10, true>(q, k, v, o, B, H, L, norm, eps, scale, workspace, nullptr, nullptr, stream, pm, keep_status);
        if (pm == 4) return launch_t<float, 12, true>(q, k, v, o, B, H, L, norm, eps, scale, workspace, nullptr, nullptr, stream, pm, keep_status);
        return CHELA_ERR_UNSUPPORTED;
    }
    if (pair) {
        // One gradient operand of the backward pass is a pair (or none: scores and state kept as pairs only):
        // kernels without the absent low planes; fp32 output, no state carry.
        if (pm != 7 && out_dtype == CHELA_F32 && !state_in && !state_out) {
            if (pm == 0) return launch_t<float, 8, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, nullptr, nullptr, stream, pm, keep_status);
            if (pm == 1) return launch_t<float, 9, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, nullptr, nullptr, stream, pm, keep_status);
        }
        if (out_dtype == CHELA_F32)
            return launch_t<float, 15, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, pm, keep_status);
        return launch_t<__nv_bfloat16, 15, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, pm, keep_status);
    }
    // plain bf16 with fewer (batch, head) pairs than SMs: the chain-free kernel, one CTA per SM, sequences shared by stride
    if (const int stride = linattn_sm100_pipe_stride(B, H, L, 0)) {
        if (!keep_status && cudaMemsetAsync(workspace, 0, sizeof(int), stream) != cudaSuccess) return CHELA_ERR_CUDA;
        return launch_linattn_sm100_pipe(q, k, v, o, B, H, L, stride, out_dtype, norm, eps, scale, (int *)workspace, state_in, state_out, stream);
    }
    if (out_dtype == CHELA_F32) return launch_t<float, 0, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, 0, keep_status);
    return launch_t<__nv_bfloat16, 0, false>(q, k, v, o, B, H, L, norm, eps, scale, workspace, state_in, state_out, stream, 0, keep_status);
}

}  // namespace chela
