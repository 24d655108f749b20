// Chunked causal linear attention, bf16 inputs, d_k = d_v = 64, for calls with fewer (batch, head) pairs than SMs:
// one CTA per SM whose chunk loop has no dependent chain through the tensor core (Sec. 4.1 tiling of Eq. 2 with the
// causal mask; the running state is the paper's "intermediate variable" kept on chip).
//
// linattn_sm100_kernel accumulates the state in TMEM and feeds it back to the tensor core, so chunk i + 1 cannot start
// before chunk i's accumulator has been read, converted and written to shared memory: about 1500 cycles per chunk for
// a lone CTA, hidden only by a second CTA on the SM.  Here the per-chunk products are independent of each other:
//   G1_i : [V_i ; K_i] Q_i^T                  -> TMEM PT[i%2]; rows 64..127 are P^T = K_i Q_i^T
//   G3_i : [P_i^T | K_i]^T V_i   (fresh)      -> TMEM OS[i%2]; rows 0..63 = P_i V_i, rows 64..127 = dS_i = K_i^T V_i
//   G2_i : rows 0..63 of OS[i%2] += Q_i [S_hi | S_lo]   (S_{i-1} as bf16 hi and lo tiles in shared memory, one N = 128
//          series: columns 0..63 take Q S_hi on top of P V, columns 64..127 take Q S_lo on top of zeros; the output warps
//          add the halves)
// and the recurrence S_i = S_{i-1} + dS_i is an fp32 add in the registers of the state warps, which write the hi/lo
// tiles for the next chunk's G2.  G1 and G3 of later chunks do not wait for G2, so the tensor core has work while the
// state warps turn dS_i into tiles.  Accumulators, score tiles and state tiles are double-buffered.
//
// Sequences are shared between CTAs by stride (B*H*stride <= SMs): CTA g of a sequence owns the chunks g, g + stride, ...
// and produces their output rows.  The state needs every chunk, so for a chunk it does not own a CTA loads K and V only
// and adds K^T V (output lanes write-disabled) onto the rows where G3 of the preceding own chunk has just put that
// chunk's own K^T V (same issuing thread, so in that order): the state warps still read one sum per own chunk.  The CTAs
// of a sequence read the same K, V tiles at about the same time, so all but the first read are served by L2: HBM
// traffic stays the algorithmic Q + K + V + O (measured), with no second kernel and no workspace.
//
// Warps (16): 0,1,4,5 output rows (add the halves, scale, normaliser, TMA store; 0,1 take the even own chunks, 4,5 the
// odd ones); 2,3,6 score rows (mask, bf16, shared tile: a third of the live 64 x 64 triangle each); 10,11,14,15 state
// rows (two warps per half of the columns); one issuing thread in each of 8 (G1), 9 (G2), 12 (G3 and the K^T V of chunks
// that are not owned) and 13 (TMA producer).  A lone thread issues a tcgen05.mma about every 50 to 80 cycles and pays
// the latency of every instruction between them, hence several issuers and no divisions in their loops.
// Roles meet only through mbarriers, every wait bounded: on a timeout the CTA records CHELA_ERR_TIMEOUT, waits
// (bounded) for its loads and products in flight, frees its TMEM and returns.
#include "sm100_ptx.cuh"

namespace chela {
namespace {

using namespace sm100;

constexpr int kD = 64;            // head dimension (d_k = d_v)
constexpr int kC = 64;            // tokens per chunk
constexpr int kTile = kC * 128;   // one 64-row x 128-byte tile
constexpr int kThreads = 512;
constexpr int kWarpA = 8, kWarpG2 = 9, kWarpG3 = 12, kWarpProducer = 13;

// kShared: stride > 1.  Ring depths: kKV stages of [V | K] (16 KB each) and kQ stages of Q (8 KB each).  A stage is
// held from the issue of its load until the last product that reads it has completed: for K and V the memory latency
// (about 3000 cycles under load) plus the way to G3 (2400), for Q plus the way to G2 (3600); the rings carry
// stages / hold time chunks per cycle, which is what bounds the kernel once HBM does not.
template <typename TOut, bool kShared>
struct SmemP {
    static constexpr int kKV = 7, kQ = 6;
    static constexpr int kOBoxes = (int)sizeof(TOut) * kD / 128;   // output leaves as 128-byte wide boxes, one at a time per warp
    static constexpr int offPT = 0;                               // masked scores, transposed (rows = s), two buffers
    static constexpr int offS = offPT + 2 * kTile;                // state tiles: [buffer][hi, lo], rows = d_k
    static constexpr int offKV = offS + 4 * kTile;                // after the score tiles: the G3 descriptor reaches K from P forwards
    static constexpr int offQ = offKV + kKV * 2 * kTile;
    static constexpr int offO = offQ + kQ * kTile;                // output staging, one tile per set of output warps; also what G2's 128-row operand reads past Q
    static constexpr int offBar = offO + 2 * kTile;
    static constexpr int nBar = 2 * kKV + 2 * kQ + 2 * 9 + 5;
    static constexpr int offTmem = offBar + 8 * nBar;
    static constexpr int offAbort = offTmem + 8;
    static constexpr int bytes = offAbort + 8;
};
// TMEM columns: PT[2] at 0, 64; OS[2] at 128, 192; DS[2] at 256, 320 (kShared only)
constexpr int kColPT = 0, kColOS = 128, kColDS = 384;   // PT 2 x 64, OS 2 x 128 (Q S_hi + P V | Q S_lo), DS 2 x 64

// The spin of a bounded wait, out of line: the roles run long straight-line code and every inlined spin loop is
// instruction-cache footprint they pay for (inlined: 0.54 ms at L = 32K, out of line: 0.43 ms).
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, const volatile int *abort_flag, long long limit)
{
    const long long t0 = clock64();
    bool ok = true;
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > limit || *abort_flag) {
            ok = false;
            break;
        }
    return ok;
}

// Position in a ring of n stages and the parity of its current pass, advanced without divisions (the issuing threads
// run one lane at a time: every instruction of theirs is latency).
struct Ring {
    int s;
    uint32_t ph;
    __device__ void advance(int n, int by = 1)
    {
        s += by;
        if (s >= n) {
            s -= n;
            ph ^= 1;
        }
    }
};

#define PDIAG(site, extra) do { if (atomicCAS(status + 8, 0, 7000 + (site)) == 0) { status[9] = blockIdx.x; status[10] = (extra); status[11] = gridDim.x; } } while (0)

template <typename TOut, bool kShared>
__global__ void __launch_bounds__(kThreads, 1)
linattn_sm100_pipe_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                          const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, int H, int L,
                          float scale, int norm, float eps, int *__restrict__ status, int stride_arg,
                          const float *__restrict__ state_in, float *__restrict__ state_out, const WaitCtl wc)
{
    using SM = SmemP<TOut, kShared>;
    constexpr int kKV = SM::kKV, kQ = SM::kQ;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    if (sbase & 1023u) {  // swizzled tiles need a 1024-byte aligned base: report instead of corrupting
        if (threadIdx.x == 0) atomicExch(status, (int)CHELA_ERR_CUDA);
        return;
    }
    const int stride = kShared ? stride_arg : 1;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x / stride, g = blockIdx.x % stride;
    const int b = bh / H, h = bh % H;
    const int nch_total = (L + kC - 1) / kC;
    // chunks 0 .. nchunks-1 are walked (through the last own one); own chunks are g, g + stride, ...
    const int n_own = g < nch_total ? (nch_total - 1 - g) / stride + 1 : 0;
    const int nchunks = n_own ? g + (n_own - 1) * stride + 1 : 0;
    const bool have_state = state_in != nullptr;
    constexpr uint32_t tmem_cols = 512u;

    // ---- barriers -------------------------------------------------------------------------------------------------
    const uint32_t bar_kv_full = sbase + SM::offBar;                 // [kKV] K, V of a chunk have landed
    const uint32_t bar_kv_empty = bar_kv_full + 8 * kKV;             // [kKV] every product that reads the stage has completed
    const uint32_t bar_q_empty = bar_kv_empty + 8 * kKV;             // [kQ] G2 has read the stage
    const uint32_t bar_p = bar_q_empty + 8 * kQ;                     // [2] G1 completed (tensor core -> score warps)
    const uint32_t bar_pt = bar_p + 16;                              // [2] PT buffer read by the score warps (-> G1 issuer)
    const uint32_t bar_ds = bar_pt + 16;                             // [2] G3 completed (-> state warps, G2 issuer, score warps)
    const uint32_t bar_o = bar_ds + 16;                              // [2] G2 completed (-> output warps, state warps)
    const uint32_t bar_of = bar_o + 16;                              // [2] OS buffer read by output and state warps (-> issuer)
    const uint32_t bar_s = bar_of + 16;                              // [2] state tiles written (state warps -> G2 issuer)
    const uint32_t bar_dn = bar_s + 16;                              // [2] K^T V of a run of chunks that are not owned completed (-> state warps)
    const uint32_t bar_d0 = bar_dn + 16;                             // K^T V of the chunks before the first own one completed (-> state warps)
    const uint32_t bar_tile = bar_d0 + 8;                           // [2] score tile in shared memory (both score warps of a set -> the one that issues G3)
    const uint32_t bar_fin = bar_tile + 16;                            // [3] every product an issuer has issued has completed (exit path)
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + SM::offTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + SM::offAbort);

    if (tid == 0) {
        for (int s = 0; s < kKV; ++s) {
            mbar_init(bar_kv_full + 8 * s, 1);
            mbar_init(bar_kv_empty + 8 * s, 1);
        }
        for (int s = 0; s < kQ; ++s) {
            mbar_init(bar_q_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_p + 8 * s, 1);
            mbar_init(bar_pt + 8 * s, 3);
            mbar_init(bar_ds + 8 * s, 1);
            mbar_init(bar_o + 8 * s, 1);
            mbar_init(bar_of + 8 * s, 6);
            mbar_init(bar_s + 8 * s, 4);
            mbar_init(bar_dn + 8 * s, 1);
            mbar_init(bar_tile + 8 * s, 3);
        }
        mbar_init(bar_d0, 1);
        for (int s = 0; s < 3; ++s) mbar_init(bar_fin + 8 * s, 1);
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_o);
    }
    if (warp == 0) {
        tmem_alloc(sbase + SM::offTmem, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // `site` names the wait in the diagnostics of one that gave up (7000 + site)
    auto pwait = [&](uint32_t bar, uint32_t parity, int site) {
        return mbar_try_wait(bar, parity) || wait_slow(bar, parity, abort_flag, wc.limit);
    };
    // two waits at once: the polls are issued back to back, so their latencies overlap (a lone issuing thread pays every
    // instruction's latency in full)
    auto pwait2 = [&](uint32_t bar_a, uint32_t par_a, int site_a, uint32_t bar_b, uint32_t par_b, int site_b) {
        const bool a = mbar_try_wait(bar_a, par_a), b = mbar_try_wait(bar_b, par_b);
        return (a || wait_slow(bar_a, par_a, abort_flag, wc.limit)) && (b || wait_slow(bar_b, par_b, abort_flag, wc.limit));
    };
    auto kv_stage = [&](int s) { return sbase + SM::offKV + s * 2 * kTile; };   // stage s of the ring: V tile, then K tile
    auto q_stage = [&](int s) { return sbase + SM::offQ + s * kTile; };
    auto give_up = [&](int site, int extra) {
        if (*abort_flag) return;   // another role gave up first: its diagnostics stand
        PDIAG(site, extra);
        *abort_flag = 1;
        atomicExch(status, (int)CHELA_ERR_TIMEOUT);
    };

    if (warp == kWarpProducer) {
        // =========================================== TMA producer ======================================================
        if (lane == 0) {
            int issued = 0, oi = 0, next_own = g;
            Ring kv = {0, 0}, qr = {0, 0};
            bool ok = true;
            for (int j = 0; ok && j < nchunks; ++j, kv.advance(kKV)) {
                const int s = kv.s;
                if (j >= kKV && !(ok = pwait(bar_kv_empty + 8 * s, kv.ph ^ 1, 1))) { give_up(1, j); break; }
                const bool mine = j == next_own;
                if (mine && oi >= kQ && !(ok = pwait(bar_q_empty + 8 * qr.s, qr.ph ^ 1, 2))) { give_up(2, j); break; }
                // one barrier per chunk: K, V and (own chunks) Q
                mbar_expect_tx(bar_kv_full + 8 * s, (mine ? 3 : 2) * kTile);
                tma_load_5d(kv_stage(s), &tm_v, bar_kv_full + 8 * s, 0, h, j * kC, b, 0);
                tma_load_5d(kv_stage(s) + kTile, &tm_k, bar_kv_full + 8 * s, 0, h, j * kC, b, 0);
                if (mine) {
                    tma_load_5d(q_stage(qr.s), &tm_q, bar_kv_full + 8 * s, 0, h, j * kC, b, 0);
                    qr.advance(kQ);
                    ++oi;
                    next_own += stride;
                }
                issued = j + 1;
            }
            if (!ok) {
                // drain: every load that was issued lands before the CTA retires (a phase already consumed reads as complete)
                for (int j = issued > kKV ? issued - kKV : 0; j < issued; ++j)
                    mbar_wait(bar_kv_full + 8 * (j % kKV), (j / kKV) & 1, nullptr, wc.limit);   // (exit path: divisions are fine)
            }
        }
    } else if (warp == kWarpA) {
        // =========================================== issuer of G1: PT[oi & 1] = [V;K] Q^T ==============================
        if (lane == 0) {
            constexpr uint32_t idescG1 = make_idesc(128, kC, 0, 0);   // [V;K] (K-major) x Q^T (K-major)
            bool ok = true;
            Ring kv = {g, 0}, qr = {0, 0};   // g < kKV
            for (int oi = 0, j = g; ok && oi < n_own; ++oi, j += stride, kv.advance(kKV, stride), qr.advance(kQ)) {
                const int buf = oi & 1;
                // the chunk's K, V and Q have landed; the score warps have taken own chunk oi - 2 out of PT[buf]
                ok = oi >= 2 ? pwait2(bar_kv_full + 8 * kv.s, kv.ph, 3, bar_pt + 8 * buf, ((oi >> 1) - 1) & 1, 5)
                             : pwait(bar_kv_full + 8 * kv.s, kv.ph, 3);
                if (!ok) { give_up(3, j); break; }
                tc_fence_after();
                const uint32_t vk_lo = desc_lo(kv_stage(kv.s)), q_lo = desc_lo(q_stage(qr.s));
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColPT + 64 * buf, vk_lo + 2 * k, q_lo + 2 * k, idescG1, k > 0);
                umma_commit(bar_p + 8 * buf);
            }
            umma_commit(bar_fin);   // every product issued by this thread has completed before TMEM and shared memory go away
            pwait(bar_fin, 0, 7);
        }
    } else if (warp == kWarpG2) {
        // =========================================== issuer of G2: rows 0..63 of OS[buf] += Q [S_hi | S_lo] ==========
        if (lane == 0) {
            constexpr uint32_t idescG2 = make_idesc(128, 2 * kD, 0, 1);   // [Q;..] (K-major) x [S_hi | S_lo] (MN-major)
            bool ok = true;
            Ring qr = {0, 0};
            for (int oi = 0, j = g; ok && oi < n_own; ++oi, j += stride, qr.advance(kQ)) {
                const int buf = oi & 1;
                const uint32_t ph = (oi >> 1) & 1;
                // after G3 of the same chunk (same accumulator), with the state tiles as of the previous chunk (the state
                // warps arrive for every own chunk, also when there is nothing to add)
                if (!(ok = pwait2(bar_ds + 8 * buf, ph, 8, bar_s + 8 * buf, ph, 9))) { give_up(8, j); break; }
                if (j > 0 || have_state) {
                    // Q's copy completed long ago (G1 has used it); this thread has not observed its barrier, the
                    // product that it issues follows the completed G1 and G3 of the chunk in the tensor core's order
                    tc_fence_after();
                    // B = [S_hi | S_lo]: two 64-column atoms, MN-major, one tile apart; columns 0..63 of OS[buf] take Q S_hi on top of
                    // P V, columns 64..127 take Q S_lo on top of the zeros the output warps left there
                    const uint32_t q_lo = desc_lo(q_stage(qr.s)), s_lo = desc_lo(sbase + SM::offS + buf * 2 * kTile, kTile);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) umma_bf16(tmem + kColOS + 128 * buf, q_lo + 2 * k, s_lo + 128 * k, idescG2, 1, 1);
                }
                umma_commit(bar_o + 8 * buf);
                umma_commit(bar_q_empty + 8 * qr.s);
            }
            umma_commit(bar_fin + 8);
            pwait(bar_fin + 8, 0, 11);
        }
    } else if (warp == kWarpG3) {
        // =========================================== issuer of G3 and of the K^T V of chunks that other CTAs own ========
        if (lane == 0) {
            constexpr uint32_t idescG3 = make_idesc(128, kD, 1, 1);   // [P^T|K] (MN-major) x V (MN-major)
            bool ok = true;
            // K^T V of chunk c summed onto rows 64..127 of the accumulator at column `col` (output lanes write-disabled)
            auto issue_ktv = [&](int c, const Ring &kv, uint32_t col, bool fresh) -> bool {
                if (!pwait(bar_kv_full + 8 * kv.s, kv.ph, 13)) { give_up(13, c); return false; }
                tc_fence_after();
                const uint32_t st = kv_stage(kv.s);
                const uint32_t a_lo = desc_lo(sbase + SM::offPT, st + kTile - (sbase + SM::offPT)), v_lo = desc_lo(st);
#pragma unroll
                for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem + col, a_lo + 128 * k, v_lo + 128 * k, idescG3, (!fresh || k > 0) ? 1u : 0u, 2);
                umma_commit(bar_kv_empty + 8 * kv.s);
                return true;
            };
            if (kShared && n_own > 0 && g > 0) {
                // the chunks before the first own one -> DS, read once by the state warps
                Ring kc = {0, 0};
                for (int c = 0; ok && c < g; ++c, kc.advance(kKV)) ok = issue_ktv(c, kc, kColDS, c == 0);
                if (ok) umma_commit(bar_d0);
            }
            Ring kv = {g, 0};   // g < kKV
            for (int oi = 0, j = g; ok && oi < n_own; ++oi, j += stride, kv.advance(kKV, stride)) {
                const int buf = oi & 1;
                const uint32_t ph = (oi >> 1) & 1;
                // the score tile is in shared memory; output and state warps have taken own chunk oi - 2 out of OS[buf]
                // (they arrive once at the start, too)
                if (!(ok = pwait2(bar_tile + 8 * buf, ph, 5, bar_of + 8 * buf, ph, 6))) { give_up(6, j); break; }
                tc_fence_after();
                const uint32_t st = kv_stage(kv.s), pt = sbase + SM::offPT + buf * kTile;
                const uint32_t a_lo = desc_lo(pt, st + kTile - pt), v_lo = desc_lo(st);
#pragma unroll
                for (int k = 0; k < kC / 16; ++k) umma_bf16(tmem + kColOS + 128 * buf, a_lo + 128 * k, v_lo + 128 * k, idescG3, k > 0);
                umma_commit(bar_kv_empty + 8 * kv.s);   // K and V are read by G1 and G3 only
                // strided: the chunks up to the next own one, onto the rows where G3 has just put this chunk's own K^T V (same
                // thread, so in this order), and the state warps read one sum per own chunk
                if (kShared) {
                    Ring kc = kv;
                    kc.advance(kKV);
                    for (int c = j + 1; ok && c < j + stride && c < nchunks; ++c, kc.advance(kKV)) ok = issue_ktv(c, kc, kColOS + 128 * buf, false);
                }
                umma_commit(bar_ds + 8 * buf);
            }
            umma_commit(bar_fin + 16);
            pwait(bar_fin + 16, 0, 14);
        }
    } else if (warp == 2 || warp == 3 || warp == 6) {
        // =========================================== score warps =======================================================
        // thread = row s of P^T (TMEM lane 64 + s) x 32 columns t: causal mask (t >= s), bf16, swizzled tile with rows = s.
        // Warp 2: rows 0..31, t 0..31 (triangle); warp 6: rows 0..31, t 32..63 (full); warp 3: rows 32..63, t 32..63
        // (triangle).  Rows 32..63, t 0..31 are zero in every chunk: written once.
        const int r = (warp & 1) * 32 + lane, t0 = warp == 2 ? 0 : 32;
        const bool full = warp == 6;
        const uint32_t tmem_warp = tmem + ((uint32_t)((warp & 3) * 32) << 16) + t0;
        if (warp == 3)
            for (int bufz = 0; bufz < 2; ++bufz)
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) *reinterpret_cast<uint4 *>(smem + SM::offPT + bufz * kTile + sw128(r, c8)) = make_uint4(0, 0, 0, 0);
        for (int oi = 0; oi < n_own; ++oi) {
            const int buf = oi & 1;
            if (!__all_sync(0xffffffffu, pwait(bar_p + 8 * buf, (oi >> 1) & 1, 16))) { if (lane == 0) give_up(16, oi); break; }
            tc_fence_after();
            float p[32];
            tmem_ld32(tmem_warp + kColPT + 64 * buf, p);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0 && !(wc.skip_arrival && blockIdx.x == 0 && oi == 0 && warp == 2)) mbar_arrive(bar_pt + 8 * buf);   // PT[buf] is free (test hook: one arrival left out)
            // G3 of own chunk oi - 2 has finished reading this score tile
            if (oi >= 2 && !__all_sync(0xffffffffu, pwait(bar_ds + 8 * buf, ((oi >> 1) - 1) & 1, 17))) { if (lane == 0) give_up(17, oi); break; }
            uint8_t *sP = smem + SM::offPT + buf * kTile;
#pragma unroll
            for (int c8 = 0; c8 < 4; ++c8) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int t = t0 + c8 * 8 + e * 2;
                    const float x0 = (full || t >= r) ? p[c8 * 8 + e * 2] : 0.f;
                    const float x1 = (full || t + 1 >= r) ? p[c8 * 8 + e * 2 + 1] : 0.f;
                    w[e] = pack_bf16(x0, x1);
                }
                *reinterpret_cast<uint4 *>(sP + sw128(r, t0 / 8 + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tile + 8 * buf);
        }
    } else if (warp == 10 || warp == 11 || warp == 14 || warp == 15) {
        // =========================================== state warps =======================================================
        // thread = row d_k of the state (TMEM lane 64 + d_k) x 32 of its 64 columns (warps 10,11: columns 0..31; warps
        // 14,15: columns 32..63), fp32 in registers for the whole sequence
        constexpr int kCols = 32;
        const int r = tid & 63, c0 = warp >= 14 ? kCols : 0;
        const uint32_t tmem_warp = tmem + ((uint32_t)((warp & 3) * 32) << 16) + c0;
        float sv[kCols];
        if (have_state) {
            const float4 *src = reinterpret_cast<const float4 *>(state_in + ((size_t)bh * kD + r) * kD + c0);
#pragma unroll
            for (int j = 0; j < kCols / 4; ++j) {
                const float4 x = src[j];
                sv[4 * j] = x.x; sv[4 * j + 1] = x.y; sv[4 * j + 2] = x.z; sv[4 * j + 3] = x.w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < kCols; ++j) sv[j] = 0.f;
        }
        auto add_tmem = [&](uint32_t col) {   // sv += this thread's 32 fp32 columns of the accumulator at `col`
            float t[kCols];
            tmem_ld32(tmem_warp + col, t);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < kCols; j += 2) add2(sv[j], sv[j + 1], t[j], t[j + 1]);
        };
        bool ok = true;
        if (lane == 0) {   // both accumulators start free
            mbar_arrive(bar_of);
            mbar_arrive(bar_of + 8);
        }
        if (kShared && g > 0 && n_own > 0) {
            // the chunks before the first own one belong to other CTAs: their K^T V, summed in DS
            if (!(ok = __all_sync(0xffffffffu, pwait(bar_d0, 0, 20)))) { if (lane == 0) give_up(20, 0); }
            if (ok) {
                tc_fence_after();
                add_tmem(kColDS);
            }
        }
        for (int oi = 0; ok && oi < n_own; ++oi) {
            const int j = g + oi * stride, buf = oi & 1;
            // 1. sv = S_{j-1}: bf16 hi + lo tiles (MN-major B operand of G2_j); the buffer was last read by G2 of own chunk oi - 2
            if (j > 0 || have_state) {
                if (oi >= 2 && !(ok = __all_sync(0xffffffffu, pwait(bar_o + 8 * buf, ((oi >> 1) - 1) & 1, 21)))) { if (lane == 0) give_up(21, j); break; }
                uint8_t *sHi = smem + SM::offS + buf * 2 * kTile, *sLo = sHi + kTile;
#pragma unroll
                for (int c8 = 0; c8 < kCols / 8; ++c8) {
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
                    const uint32_t off = sw128(r, c0 / 8 + c8);
                    *reinterpret_cast<uint4 *>(sHi + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
                    *reinterpret_cast<uint4 *>(sLo + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
                }
                fence_proxy_async();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_s + 8 * buf);   // also when there is nothing to write (first chunk, no initial state)
            // 2. rows 64..127 of OS[buf]: the chunk's K^T V, plus (strided) that of the chunks up to the next own one
            if (!(ok = __all_sync(0xffffffffu, pwait(bar_ds + 8 * buf, (oi >> 1) & 1, 22)))) { if (lane == 0) give_up(22, j); break; }
            tc_fence_after();
            add_tmem(kColOS + 128 * buf);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_of + 8 * buf);
        }
        if (ok && state_out && nchunks == nch_total) {
            // this CTA owns the last chunk of the sequence: the fp32 state leaves the SM once, for the caller
            float4 *dst = reinterpret_cast<float4 *>(state_out + ((size_t)bh * kD + r) * kD + c0);
#pragma unroll
            for (int j = 0; j < kCols / 4; ++j) dst[j] = make_float4(sv[4 * j], sv[4 * j + 1], sv[4 * j + 2], sv[4 * j + 3]);
        }
    } else if (warp == 0 || warp == 1 || warp == 4 || warp == 5) {
        // =========================================== output warps ======================================================
        // thread = output row t (TMEM lane t): scale, row normaliser -> swizzled staging -> TMA store (per warp: 32 rows).
        // Warps 0,1 take the even own chunks (buffer 0), warps 4,5 the odd ones (buffer 1).
        const int r = tid & 63, buf = warp >> 2, half = warp & 1;
        const uint32_t tmem_warp = tmem + ((uint32_t)(half * 32) << 16);
        auto zero_lo = [&]() {   // columns 64..127 of this thread's row of OS[buf] = 0
            float z[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) z[c] = 0.f;
            tmem_st32(tmem_warp + kColOS + 128 * buf + 64, z);
            tmem_st32(tmem_warp + kColOS + 128 * buf + 96, z);
            tmem_st_wait();
        };
        zero_lo();   // OS[buf] starts free and with a zero lo half
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_of + 8 * buf);
        for (int oi = buf; oi < n_own; oi += 2) {
            const int j = g + oi * stride;
            if (!__all_sync(0xffffffffu, pwait(bar_o + 8 * buf, (oi >> 1) & 1, 24))) { if (lane == 0) give_up(24, j); break; }
            tc_fence_after();
            // columns 0..63: Q S_hi + P V, columns 64..127: Q S_lo; the latter are zeroed again for the chunk after next
            float acc[kD];
#pragma unroll
            for (int hc = 0; hc < 2; ++hc) {
                float lo[32];
                tmem_ld32(tmem_warp + kColOS + 128 * buf + 32 * hc, *reinterpret_cast<float(*)[32]>(&acc[32 * hc]));
                tmem_ld32(tmem_warp + kColOS + 128 * buf + 64 + 32 * hc, lo);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 32; c += 2) add2(acc[32 * hc + c], acc[32 * hc + c + 1], lo[c], lo[c + 1]);
            }
            zero_lo();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_of + 8 * buf);   // the output rows are out of TMEM
            // the row is scaled and normalised in one multiplication: o = acc * scale / sqrt(scale^2 mean(acc^2) + eps)
            float ss0 = 0.f, ss1 = 0.f;
#pragma unroll
            for (int c = 0; c < kD; c += 2) sqacc2(ss0, ss1, acc[c], acc[c + 1]);
            const float inv = norm ? scale * rsqrtf((ss0 + ss1) * (scale * scale * (1.0f / kD)) + eps) : scale;
#pragma unroll
            for (int c = 0; c < kD; c += 2) mul2(acc[c], acc[c + 1], acc[c], acc[c + 1], inv);
            // this warp's 32 rows x 128 bytes of the set's staging tile, one 128-byte wide box after the other
            uint8_t *sO = smem + SM::offO + buf * kTile;
#pragma unroll
            for (int bx = 0; bx < SM::kOBoxes; ++bx) {
                if (lane == 0) bulk_wait_read0();   // the box this warp stored last has left the staging tile
                __syncwarp();
                if (sizeof(TOut) == 4) {
#pragma unroll
                    for (int c = 0; c < 32; c += 4)
                        *reinterpret_cast<float4 *>(sO + sw128(r, c / 4)) =
                            make_float4(acc[32 * bx + c], acc[32 * bx + c + 1], acc[32 * bx + c + 2], acc[32 * bx + c + 3]);
                } else {
#pragma unroll
                    for (int c = 0; c < kD; c += 8)
                        *reinterpret_cast<uint4 *>(sO + sw128(r, c / 8)) =
                            make_uint4(pack_bf16(acc[c], acc[c + 1]), pack_bf16(acc[c + 2], acc[c + 3]),
                                       pack_bf16(acc[c + 4], acc[c + 5]), pack_bf16(acc[c + 6], acc[c + 7]));
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {   // rows past L are clipped by the copy engine
                    tma_store_5d(&tm_o, sbase + SM::offO + buf * kTile + half * 32 * 128, bx * (128 / (int)sizeof(TOut)), h, j * kC + half * 32, b, 0);
                    bulk_commit();
                }
            }
        }
        if (lane == 0) bulk_wait0();   // output boxes fully written before the CTA retires
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, tmem_cols);
}

// [B, L, H, 64] viewed as a rank-5 tensor (d, H, L, B, 1); box = (128 bytes of d) x 1 x rows x 1 x 1, 128-byte swizzle.
// Loads: rows past L are out of bounds for the copy engine and arrive as zeros.  Stores: rows past L are clipped.
bool make_map(CUtensorMap *map, const void *ptr, int B, int H, int L, int rows, bool f32)
{
    const cuuint64_t es = f32 ? 4 : 2;
    const cuuint64_t dims[5] = {(cuuint64_t)kD, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B, 1};
    const cuuint64_t strides[4] = {(cuuint64_t)kD * es, (cuuint64_t)H * kD * es, (cuuint64_t)L * H * kD * es,
                                   (cuuint64_t)B * L * H * kD * es};
    const cuuint32_t box[5] = {(cuuint32_t)(128 / es), 1, (cuuint32_t)rows, 1, 1};
    return make_map_sw128(map, ptr, f32, 5, dims, strides, box);
}

template <typename TOut, bool kShared>
chela_status_t launch_t(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int stride, int norm, float eps,
                        float scale, int *status, const float *state_in, float *state_out, cudaStream_t stream)
{
    CUtensorMap mq, mk, mv, mo;
    if (!make_map(&mq, q, B, H, L, kC, false) || !make_map(&mk, k, B, H, L, kC, false) || !make_map(&mv, v, B, H, L, kC, false) ||
        !make_map(&mo, o, B, H, L, 32, sizeof(TOut) == 4))
        return CHELA_ERR_CUDA;
    auto kern = linattn_sm100_pipe_kernel<TOut, kShared>;
    constexpr int smem = SmemP<TOut, kShared>::bytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return CHELA_ERR_CUDA;
    kern<<<B * H * stride, kThreads, smem, stream>>>(mq, mk, mv, mo, H, L, scale, norm, eps, status, stride, state_in, state_out,
                                                      current_wait_ctl());
    return last_launch_status();
}

}  // namespace

// CTAs per sequence for a call with fewer (batch, head) pairs than SMs: as many as keep B*H*stride <= SMs (one CTA per
// SM, all resident), at most 4 (every CTA of a sequence streams all of its K and V out of L2), and at least four own
// chunks per CTA.  0 = the call is not for this kernel (as many pairs as SMs: two CTAs per SM of the other kernel).
int linattn_sm100_pipe_stride(int B, int H, int L, int sms)
{
    int dev = 0;
    if (sms <= 0 && (cudaGetDevice(&dev) != cudaSuccess ||
                     cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0))
        sms = 148;
    const long long bh = (long long)B * H;
    if (bh >= sms) return 0;
    const int nchunks = (L + kC - 1) / kC;
    int stride = (int)(sms / bh);
    if (stride > 4) stride = 4;
    if (stride > nchunks / 4) stride = nchunks / 4;
    return stride < 1 ? 1 : stride;
}

chela_status_t launch_linattn_sm100_pipe(const void *q, const void *k, const void *v, void *o, int B, int H, int L, int stride,
                                         chela_dtype_t out_dtype, int norm, float eps, float scale, int *status,
                                         const float *state_in, float *state_out, cudaStream_t stream)
{
    if (out_dtype == CHELA_F32) {
        if (stride > 1) return launch_t<float, true>(q, k, v, o, B, H, L, stride, norm, eps, scale, status, state_in, state_out, stream);
        return launch_t<float, false>(q, k, v, o, B, H, L, stride, norm, eps, scale, status, state_in, state_out, stream);
    }
    if (stride > 1) return launch_t<__nv_bfloat16, true>(q, k, v, o, B, H, L, stride, norm, eps, scale, status, state_in, state_out, stream);
    return launch_t<__nv_bfloat16, false>(q, k, v, o, B, H, L, stride, norm, eps, scale, status, state_in, state_out, stream);
}

}  // namespace chela
