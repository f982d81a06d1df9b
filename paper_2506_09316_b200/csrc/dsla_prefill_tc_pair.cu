// Tensor-core prefill of the dual-state linear attention layer for sm_100a, cluster variant (DSLA_IMPL_TENSOR_PAIR):
// bf16 inputs, d = 128, fp32 states.  Chunkwise form of the Sec. 4.1 recurrence (chunk C = 64 tokens; L^i_j = cumulative
// log2-gates of state i inside the chunk, inclusive):
//     P       = Q K^T                                                        tcgen05, fp32 in TMEM
//     P~      = P (.) [s<=j] (W1 2^(L1_j-L1_s) + W2 2^(L2_j-L2_s))           CUDA cores -> bf16 in smem
//     O_in^T  = V^T P~^T                                                     tcgen05
//     O^i^T   = S^i^T Q^T            (raw Q; state read from TMEM)           tcgen05
//     o_j     = O_in[j] + sum_i W_i 2^(L^i_j) O^i[j]                         fp32, registers
//     S^i^T  <- a^i S^i^T + (w^i (.) V)^T K                                  rescale on CUDA cores, MMA accumulates
// with W = (gamma, 1 - gamma) * scale, a^i = prod of the chunk's gates, w^i_s = 2^(L^i_last - L^i_s).
//
// The blended readout is a SUM over the two states, so the states are separable: a cluster of two
// CTAs works on one (sequence, head) pair and CTA i owns state i.  Each CTA keeps its fp32 state in
// TMEM for the whole sequence (d_v on the 128 lanes, everything is computed transposed so every MMA
// has M = 128), a bf16 copy of it as the A operand of the readout, and the scaled V^T of the chunk as
// the A operand of the update, written to TMEM by CUDA cores (no scaled copies in shared memory: Q, K,
// V tiles are read-only once TMA has landed them).  The chunk-local part (P, P~, O_in) is state
// independent; the two CTAs take it in turns (CTA i does the chunks with c mod 2 = i).  Each CTA
// finishes 32 of the chunk's 64 tokens: it sends the partial outputs of the other 32 to its peer
// through distributed shared memory and adds what the peer sends for its own.
//
// A sequence may be split into segments along T so that few (sequence, head) pairs still fill the
// GPU (dsla_prefill_summary.cu computes the segment summaries); this kernel folds the summaries of
// earlier segments into its initial state.  No TMA load uses cluster multicast: each CTA loads its
// own tiles and the L2 serves the second copy.
#include <cstdlib>

#include "dsla_prefill_tc.cuh"

namespace dsla {

namespace {

// Warp roles (20 warps).  A warp may touch only the 32 TMEM lanes of its quadrant (warp index mod 4), and the
// four warp schedulers of the SM take the warps of one quadrant each, so every role that works on TMEM has one
// warp per quadrant:
//   0, 1, 4, 5 : score tile warps (rows 0..31 / 32..63 of P x column halves): P~ = P (.) decay mask
//   2          : TMA producer; issues the state update
//   3          : issues the readout; allocates TMEM
//   7          : issues the chunk-local MMAs (scores, O_in)
//   6          : gate warp (cumulative log-gates and everything derived from them)
//   8..15      : state warps (two per quadrant, 64 d_k columns each): rescale + bf16 copy of the state
//   16..19     : V~ into TMEM, then the outputs (scale, exchange with the peer CTA, store)
constexpr int WARP_X = 2, WARP_Y = 3, WARP_GATE = 6, WARP_Z = 7, STATE_W0 = 8, VE_W0 = 16;
constexpr int NTHREADS = 24 * 32;
constexpr int NST = 3;                             // landing stages of {K, Q, V}
constexpr int STAGE_BYTES = 3 * 16384, ST_Q = 16384, ST_V = 32768;
constexpr int OFF_PT = NST * STAGE_BYTES;          // P~, 8 KB
constexpr int OFF_RECV = OFF_PT + 8192;            // partial outputs from the peer: 4 x [128 d_v][32 tokens] bf16
constexpr int RECV_BYTES = 8192, NRECV = 4;
constexpr int OFF_OUT = OFF_RECV + NRECV * RECV_BYTES;      // finished outputs, token-major: per finishing warp [32 tokens][32 d_v] bf16
constexpr int OUT_PITCH = 80, OUT_WARP_BYTES = 32 * OUT_PITCH;    // 64-byte rows padded to 80 (stmatrix rows hit distinct banks)
constexpr int SMEM_TILES = OFF_OUT + 4 * OUT_WARP_BYTES;
constexpr int SMEM_DYN = SMEM_TILES + 1024;        // + alignment slack
constexpr int NGA = 4, NGB = 2;                    // depth of the two rings of gate-derived factors
// TMEM columns
constexpr uint32_t COL_S = 0;       // fp32 state S^T, 128 columns (d_k)
constexpr uint32_t COL_SB = 128;    // bf16 copy, 64 columns
constexpr uint32_t COL_O = 192;     // readout O^T, 2 x 64 columns (tokens): chunks of even / odd index
constexpr uint32_t COL_OI = 320;    // chunk-local output O_in^T
constexpr uint32_t COL_P = 384;     // scores P (lanes 0..63 meaningful)
constexpr uint32_t COL_VT = 448;    // scaled V^T, bf16, 2 x 32 columns

// Factors every chunk needs (own state only).
struct alignas(16) GateA {
    float rowf[C];            // W_i 2^(L_j): weight of the state readout at token j
    __nv_bfloat16 w[C];       // 2^(L_last - L_s): weight of token s in the state update (0 past the end of the sequence)
    float a;                  // product of the chunk's gates
    float pad[3];
};
// Factors of a chunk whose local part this CTA computes (both states).
struct alignas(16) GateB {
    float L[2][C];            // cumulative log2-gates
};

struct alignas(16) Shared {
    uint64_t ld_full[NST], ld_empty[NST];
    uint64_t ga_full[NGA], ga_empty[NGA], gb_full[NGB], gb_empty[NGB];
    uint64_t vt_ready[2], vt_free[2];
    uint64_t s_ready, sb_ready, u_full, o_full[2], o_free[2];
    uint64_t p_full, pt_ready, pt_free, oi_full, oi_free;
    uint64_t x_full[NRECV][4], x_free[NRECV][4];
    uint32_t tmem_base;
    int abort_flag;
    GateA ga[NGA];
    GateB gb[NGB];
};

__global__ void __launch_bounds__(NTHREADS, 1)
prefill_tc_pair_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const TcParams tp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const PrefillParams& p = tp.p;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = (int)cluster_ctarank();          // = state index: 0 history, 1 recency
    const int peer = rank ^ 1;
    // Clusters are handed out in index order: the last segments first (they have the longest fold of summaries
    // ahead of them; when this grid starts as a programmatic dependent of the summary grid their prologue hides
    // behind its tail).
    const int units = p.N * p.H;
    const int u = (int)(blockIdx.x >> 1);
    const int g = tp.nseg - 1 - u / units;
    const int h = (u % units) % p.H;
    const int seq_rank = (u % units) / p.H;
    const int n = tp.order ? tp.order[seq_rank] : seq_rank;
    const SeqInfo sq = seq_info(p, n, g, tp.nseg, tp.cps, tp.skew8);
    // Every early exit below depends only on values both CTAs of the cluster share, and comes before any cluster
    // operation.
    if (sq.slot < 0 || sq.slot >= p.num_slots) return;
    // A sequence longer than the max_seqlen the host sized the segments for would lose its tail: say so.
    if (tid == 0 && g == 0 && sq.nchunks > seg_begin(tp.nseg, tp.nseg, tp.cps, tp.skew8)) atomicExch(p.status, (int)DSLA_ERR_INVALID_ARG);
    const size_t state_stride = (size_t)p.H * D * D;
    float* slot_i = p.state + (((size_t)sq.slot * 2 + rank) * p.H + h) * (size_t)(D * D);
    if (sq.len <= 0) {  // empty sequence: a fresh start leaves zero states, a resume leaves the slot alone
        if (g == 0 && !p.use_initial_state)
            for (int i = tid; i < D * D; i += NTHREADS) slot_i[i] = 0.f;
        return;
    }
    (void)state_stride;
    if (sq.c_begin >= sq.c_end) return;
    const int nc = sq.c_end - sq.c_begin;
    const int t0 = sq.t_begin + sq.c_begin * C;   // first token of this segment
    const int tok0 = sq.c_begin * C;              // its index inside the sequence
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent launch behind this grid (the decode step) may be scheduled early

    if (tid == 0) {
        for (int i = 0; i < NST; ++i) { mbar_init(&sh.ld_full[i], 1); mbar_init(&sh.ld_empty[i], 7); }   // three issuers + four V~ warps
        for (int i = 0; i < NGA; ++i) { mbar_init(&sh.ga_full[i], 1); mbar_init(&sh.ga_empty[i], 16); }  // eight state + eight output warps
        for (int i = 0; i < NGB; ++i) { mbar_init(&sh.gb_full[i], 1); mbar_init(&sh.gb_empty[i], 4); }
        for (int i = 0; i < 2; ++i) { mbar_init(&sh.vt_ready[i], 4); mbar_init(&sh.vt_free[i], 1); }
        mbar_init(&sh.s_ready, 8); mbar_init(&sh.sb_ready, 8); mbar_init(&sh.u_full, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&sh.o_full[i], 1); mbar_init(&sh.o_free[i], 8); }
        mbar_init(&sh.p_full, 1); mbar_init(&sh.pt_ready, 4); mbar_init(&sh.pt_free, 1);
        mbar_init(&sh.oi_full, 1); mbar_init(&sh.oi_free, 8);
        for (int b = 0; b < NRECV; ++b)
            for (int q = 0; q < 4; ++q) { mbar_init(&sh.x_full[b][q], 1); mbar_init(&sh.x_free[b][q], 1); }
        sh.abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == WARP_Y) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();        // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tb = sh.tmem_base;
    volatile int* abortp = &sh.abort_flag;
#define WAIT(bar, ph) mbar_wait(bar, (uint32_t)(ph), abortp, p.status)

    // Three threads issue the MMAs: a tcgen05 instruction costs its issuing thread some eighty cycles whatever its size, so
    // the small MMAs of this kernel are issue-bound per thread, and each thread drives one dependency chain.
    if (warp == WARP_X) {
        // ------------------------------------------------------------------ TMA producer; state update
        if (lane == 0) {
            prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_D = idesc_bf16(128, 128, 0, 1);    // S^T += V~^T K: A in TMEM, B = K as an MN-major N operand
            constexpr uint64_t ST_STEP = (uint64_t)(STAGE_BYTES >> 4);
            const uint64_t dk_n = smem_desc_sw128(sa, 8192, 1024);
            auto load = [&](int c) {
                const int s = c % NST;
                uint8_t* dst = tiles + s * STAGE_BYTES;
                const int t = t0 + c * C;
                mbar_arrive_expect_tx(&sh.ld_full[s], 6 * 8192);
                tma_load_4d(dst, &map_k, &sh.ld_full[s], 0, t, 0, h);
                tma_load_4d(dst + ST_V, &map_v, &sh.ld_full[s], 0, t, 0, h);
                tma_load_4d(dst + ST_Q, &map_q, &sh.ld_full[s], 0, t, 0, h);
                if (c + 3 < nc) {       // pull the tiles of a later chunk into L2 (one CTA of the pair each)
                    const int t3 = t + 3 * C;
                    if (rank == 0) { tma_prefetch_4d(&map_k, 0, t3, 0, h); tma_prefetch_4d(&map_q, 0, t3, 0, h); }
                    else tma_prefetch_4d(&map_v, 0, t3, 0, h);
                }
            };
            for (int c = 0; c < NST && c < nc; ++c) load(c);
#pragma unroll 1
            for (int c = 0; c < nc; ++c) {
                const int s = c % NST, b = c & 1;
                WAIT(&sh.ld_full[s], (c / NST) & 1);
                WAIT(&sh.vt_ready[b], (c >> 1) & 1);
                WAIT(&sh.s_ready, c & 1);
                tc_fence_after();
                const uint64_t bk = dk_n + (uint64_t)s * ST_STEP;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ts(tb + COL_S, tb + COL_VT + 32 * b + 8 * kk, bk + (uint64_t)(kk * 128), ID_D, 1);
                tc_commit(&sh.u_full);
                tc_commit(&sh.vt_free[b]);
                tc_commit(&sh.ld_empty[s]);
                // after the update is on its way: the stage of chunk c - 1 takes chunk c + 2
                if (c >= 1 && c + 2 < nc) {
                    WAIT(&sh.ld_empty[(c - 1) % NST], ((c - 1) / NST) & 1);
                    load(c + 2);
                }
            }
        }
    } else if (warp == WARP_Y) {
        // ------------------------------------------------------------------ readout
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_C = idesc_bf16(128, 64, 0, 0);     // O^T = S^T Q^T: A in TMEM, B = Q K-major
            constexpr uint64_t ST_STEP = (uint64_t)(STAGE_BYTES >> 4);
            const uint64_t dq_k = smem_desc_sw128(sa + ST_Q, 16, 1024);
#pragma unroll 1
            for (int c = 0; c < nc; ++c) {
                const int s = c % NST;
                WAIT(&sh.ld_full[s], (c / NST) & 1);
                if (c >= 2) WAIT(&sh.o_free[c & 1], ((c >> 1) - 1) & 1);     // the outputs of chunk c - 2 have left this accumulator
                WAIT(&sh.sb_ready, c & 1);
                tc_fence_after();
                const uint64_t bq = dq_k + (uint64_t)s * ST_STEP;
                const uint32_t od = tb + COL_O + 64 * (c & 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ts(od, tb + COL_SB + 8 * kk, bq + (uint64_t)(2 * kk), ID_C, kk ? 1u : 0u);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ts(od, tb + COL_SB + 32 + 8 * kk, bq + 512 + (uint64_t)(2 * kk), ID_C, 1u);
                tc_commit(&sh.o_full[c & 1]);
                tc_commit(&sh.ld_empty[s]);
            }
        }
    } else if (warp == WARP_Z) {
        // ------------------------------------------------------------------ chunk-local part: scores and O_in of the chunks this CTA owns
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_P = idesc_bf16(128, 64, 0, 0);     // P = Q K^T: both operands K-major
            constexpr uint32_t ID_B = idesc_bf16(128, 64, 1, 0);     // O_in^T = V^T P~^T: A = V as an MN-major operand
            constexpr uint64_t ST_STEP = (uint64_t)(STAGE_BYTES >> 4);
            const uint64_t dk_k = smem_desc_sw128(sa, 16, 1024), dq_k = smem_desc_sw128(sa + ST_Q, 16, 1024);
            const uint64_t dv_m = smem_desc_sw128(sa + ST_V, 8192, 1024);
            const uint64_t dpt = smem_desc_sw128(sa + OFF_PT, 16, 1024);
            // step n2 = -1 issues the scores of the first owned chunk; step n2 issues O_in of owned chunk n2 and the scores of the
            // next one, so the decay-mask work on chunk n2 + 1 runs while the outputs of chunk n2 are finished.  In between it
            // releases the stages of the chunks it does not touch (a commit with nothing pending arrives at once).
#pragma unroll 1
            for (int c = rank - 2; c < nc; c += 2) {
                const int n2 = c >> 1;       // index of owned chunk c (c >= 0)
                if (c >= 0) {
                    const int s = c % NST;
                    WAIT(&sh.pt_ready, n2 & 1);
                    if (n2 >= 1) WAIT(&sh.oi_free, (n2 - 1) & 1);
                    tc_fence_after();
                    const uint64_t av = dv_m + (uint64_t)s * ST_STEP;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_OI, av + (uint64_t)(kk * 128), dpt + (uint64_t)(2 * kk), ID_B, kk ? 1u : 0u);
                    tc_commit(&sh.oi_full);
                    tc_commit(&sh.pt_free);
                    tc_commit(&sh.ld_empty[s]);
                }
                if (c + 1 >= 0 && c + 1 < nc) {
                    // chunk c + 1 belongs to the peer CTA: release its stage, but only once the stage holds that chunk (an arrival
                    // before the refill would count for the stage's previous use)
                    WAIT(&sh.ld_full[(c + 1) % NST], ((c + 1) / NST) & 1);
                    tc_commit(&sh.ld_empty[(c + 1) % NST]);
                }
                if (c + 2 < nc) {
                    const int cn = c + 2, s = cn % NST;
                    WAIT(&sh.ld_full[s], (cn / NST) & 1);
                    // P is free: every tile warp arrived on pt_ready for the previous owned chunk after its last read of P
                    tc_fence_after();
                    const uint64_t sn = (uint64_t)s * ST_STEP;
#pragma unroll
                    for (int blk = 0; blk < 2; ++blk) {
                        const uint64_t a = dq_k + sn + (uint64_t)(512 * blk), b = dk_k + sn + (uint64_t)(512 * blk);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_P, a + (uint64_t)(2 * kk), b + (uint64_t)(2 * kk), ID_P, (blk | kk) ? 1u : 0u);
                    }
                    tc_commit(&sh.p_full);
                }
            }
        }
    } else if (warp == WARP_GATE) {
        // ------------------------------------------------------------------ gate warp
        // Everything a chunk needs from the gates comes from the cumulative log-gates
        //     L^i_j = sum_{t <= j} log2 g^i_t      (inclusive, from the chunk start; a zero gate counts as -200, so any
        //                                           product that contains one flushes to an exact zero)
        // through independent exponentials.  Lane l holds tokens l and l + 32.  The chunk decay a that carries the state
        // is the plain product of the gates.
        const float gam = p.gamma[h];
        const float W1 = gam * p.scale, W2 = (1.f - gam) * p.scale;
        const float Wown = rank == 0 ? W1 : W2;
        auto fetch = [&](int c, float2& lo, float2& hi2) {
            const int j = c * C + lane;
            const bool in = c < nc;
            // raw values: nothing may consume them here, or the warp would sit out the load latency in every chunk
            lo.x = load_gate(p.g_hist, t0 + j, p.H, h, in && tok0 + j < sq.len);
            lo.y = load_gate(p.g_rec, t0 + j, p.H, h, in && tok0 + j < sq.len);
            hi2.x = load_gate(p.g_hist, t0 + j + 32, p.H, h, in && tok0 + j + 32 < sq.len);
            hi2.y = load_gate(p.g_rec, t0 + j + 32, p.H, h, in && tok0 + j + 32 < sq.len);
        };
        float2 nlo, nhi;
        fetch(0, nlo, nhi);
        int nb = 0;
#pragma unroll 1
        for (int c = 0; c < nc; ++c) {
            const int k = c & (NGA - 1);
            const float2 glo = make_float2(fmaxf(nlo.x, 0.f), fmaxf(nlo.y, 0.f)), ghi = make_float2(fmaxf(nhi.x, 0.f), fmaxf(nhi.y, 0.f));
            fetch(c + 1, nlo, nhi);
            const float go_lo = rank == 0 ? glo.x : glo.y, go_hi = rank == 0 ? ghi.x : ghi.y;      // own state
            float la = warp_prefix_sum(lg2_gate(go_lo), lane), lb = warp_prefix_sum(lg2_gate(go_hi), lane);
            const float mid = __shfl_sync(0xffffffffu, la, 31);
            lb += mid;
            const float end = __shfl_sync(0xffffffffu, lb, 31);
            float pr = go_lo * go_hi;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) pr *= __shfl_xor_sync(0xffffffffu, pr, off);
            const int valid = min(C, sq.len - tok0 - c * C);
            if (c >= NGA) WAIT(&sh.ga_empty[k], ((c / NGA) - 1) & 1);
            GateA& ga = sh.ga[k];
            ga.rowf[lane] = Wown * ex2(la);
            ga.rowf[lane + 32] = Wown * ex2(lb);
            // tokens past the end of the sequence carry no weight in the state update
            ga.w[lane] = __float2bfloat16_rn(lane < valid ? ex2(end - la) : 0.f);
            ga.w[lane + 32] = __float2bfloat16_rn(lane + 32 < valid ? ex2(end - lb) : 0.f);
            if (lane == 0) ga.a = pr;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.ga_full[k]);
            if ((c & 1) == rank) {
                // this CTA computes the chunk-local part: it needs both states' logs
                const int kb = nb & (NGB - 1);
                const float gx_lo = rank == 0 ? glo.y : glo.x, gx_hi = rank == 0 ? ghi.y : ghi.x;  // the other state
                float ma = warp_prefix_sum(lg2_gate(gx_lo), lane), mb = warp_prefix_sum(lg2_gate(gx_hi), lane);
                const float midx = __shfl_sync(0xffffffffu, ma, 31);
                mb += midx;
                const float l1a = rank == 0 ? la : ma, l1b = rank == 0 ? lb : mb;
                const float l2a = rank == 0 ? ma : la, l2b = rank == 0 ? mb : lb;
                if (nb >= NGB) WAIT(&sh.gb_empty[kb], ((nb / NGB) - 1) & 1);
                GateB& gb = sh.gb[kb];
                gb.L[0][lane] = l1a; gb.L[0][lane + 32] = l1b;
                gb.L[1][lane] = l2a; gb.L[1][lane + 32] = l2b;
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.gb_full[kb]);
                ++nb;
            }
        }
    } else if (warp < STATE_W0) {
        {
            // ------------------------------------------------------------------ score tile warps 0, 1, 4, 5
            // P~ rows 32 q .. 32 q + 31, columns 32 half .. 32 half + 31 of the chunks whose local part this CTA computes
            const int q = warp & 3, half = warp >> 2;
            const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
            const int j = 32 * q + lane;
            const float gam = p.gamma[h];
            const float W1 = gam * p.scale, W2 = (1.f - gam) * p.scale;
            uint8_t* pt = tiles + OFF_PT;
#pragma unroll 1
            for (int c = rank, n2 = 0; c < nc; c += 2, ++n2) {
                const GateB& gb = sh.gb[n2 & (NGB - 1)];
                WAIT(&sh.gb_full[n2 & (NGB - 1)], (n2 / NGB) & 1);
                WAIT(&sh.p_full, n2 & 1);
                tc_fence_after();
                if (n2 >= 1) WAIT(&sh.pt_free, (n2 - 1) & 1);       // the previous P~ has been consumed
                // M[j][s] = W1 2^(L1_j - L1_s) + W2 2^(L2_j - L2_s) for s <= j (differences of logs, never positive), else 0;
                // eight columns per round, loop kept rolled (the code of all roles has to stay small)
                const float L1j = gb.L[0][j], L2j = gb.L[1][j];
#pragma unroll 1
                for (int m4 = 0; m4 < 4; ++m4) {
                    const int col0 = 32 * half + 8 * m4;
                    uint32_t pk[4] = {0u, 0u, 0u, 0u};
                    if (half <= q) {        // warp-uniform: the block above the diagonal is all zeros
                        uint32_t r[8];
                        tmem_ld8(lane_addr + COL_P + col0, r);
                        const float4 a0 = *reinterpret_cast<const float4*>(&gb.L[0][col0]), a1 = *reinterpret_cast<const float4*>(&gb.L[0][col0 + 4]);
                        const float4 b0 = *reinterpret_cast<const float4*>(&gb.L[1][col0]), b1 = *reinterpret_cast<const float4*>(&gb.L[1][col0 + 4]);
                        const float s1[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                        const float s2[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                        float m[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float mm = fmaf(W2, ex2(L2j - s2[e]), W1 * ex2(L1j - s1[e]));
                            m[e] = (col0 + e <= j) ? mm : 0.f;
                        }
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            pk[e] = pack_bf16(__uint_as_float(r[2 * e]) * m[2 * e], __uint_as_float(r[2 * e + 1]) * m[2 * e + 1]);
                    }
                    *reinterpret_cast<uint4*>(pt + sw128_offset(j, col0)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
                tc_fence_before();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.pt_ready); mbar_arrive(&sh.gb_empty[n2 & (NGB - 1)]); }
            }
        }
    } else if (warp < VE_W0) {
        // ------------------------------------------------------------------ state warps 8..15
        // One pass per chunk over this warp's 32 lanes x 64 columns of the fp32 state: the bf16 copy of S_c that the
        // readout of chunk c multiplies, and a_c S_c in place, onto which the update MMA of chunk c accumulates.
        const int q = warp & 3, ch = (warp - STATE_W0) >> 2;
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        const uint32_t s_addr = lane_addr + COL_S + 64 * ch, sb_addr = lane_addr + COL_SB + 32 * ch;
        const int v = 32 * q + lane;
#pragma unroll 1
        for (int c = 0; c < nc; ++c) {
            WAIT(&sh.ga_full[c & (NGA - 1)], (c / NGA) & 1);
            const float a = sh.ga[c & (NGA - 1)].a;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.ga_empty[c & (NGA - 1)]);
            if (c == 0) {
                // With programmatic dependent launch this grid may start while the summary grid is still running;
                // everything up to here (and all of chunk 0's operand work in the other warps) is independent of it.
                if (g > 0 && tp.ws) asm volatile("griddepcontrol.wait;" ::: "memory");
                const float* init = tp.init ? tp.init + ((size_t)(n * p.H + h) * 2 + rank) * (size_t)(D * D) : slot_i;
                init_state_pass(init, p.use_initial_state, tp.ws ? tp.ws + ((size_t)(n * p.H + h) * tp.nseg) * (SUMMARY_STRIDE / 4) : nullptr,
                                g, rank, v, a, lane_addr + COL_S, lane_addr + COL_SB, 2 * ch, 2 * ch + 2);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.s_ready); mbar_arrive(&sh.sb_ready); }
                continue;
            }
            WAIT(&sh.u_full, (c - 1) & 1);      // the update of chunk c - 1 is in the fp32 state
            WAIT(&sh.o_full[(c - 1) & 1], ((c - 1) >> 1) & 1);      // the readout of chunk c - 1 has read the previous bf16 copy
            tc_fence_after();
            const float2 a2 = make_float2(a, a);
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                uint32_t r0[32], pk[16];
                tmem_ld32(s_addr + 32 * i, r0);
                tc_wait_ld();
#pragma unroll
                for (int k = 0; k < 16; ++k) pk[k] = pack_bf16(__uint_as_float(r0[2 * k]), __uint_as_float(r0[2 * k + 1]));
                tmem_st16(sb_addr + 16 * i, pk);
#pragma unroll
                for (int k = 0; k < 32; k += 2) {
                    const float2 y = __fmul2_rn(make_float2(__uint_as_float(r0[k]), __uint_as_float(r0[k + 1])), a2);
                    r0[k] = __float_as_uint(y.x); r0[k + 1] = __float_as_uint(y.y);
                }
                tmem_st32(s_addr + 32 * i, r0);
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(&sh.s_ready); mbar_arrive(&sh.sb_ready); }
        }
        // ---- final state of this segment
        WAIT(&sh.u_full, (nc - 1) & 1);
        tc_fence_after();
        if (g == sq.last_seg) store_state(slot_i, v, lane_addr + COL_S, 2 * ch, 2 * ch + 2);
    } else {
        // ------------------------------------------------------------------ V~ and output warps 16..23
        // Two sets of four warps: warps 16..19 prepare V~ and send the peer CTA its half of every chunk's outputs, warps 20..23
        // finish this CTA's half; both read the same accumulators.
        const int q = warp & 3, set = (warp - VE_W0) >> 2;
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        const int v = 32 * q + lane;
        // V~^T[v][s] = w_s V[s][v] for the update, into TMEM as the A operand (d_v on the lanes, two tokens per 32-bit column).
        // ldmatrix with .trans hands a thread two consecutive tokens of one d_v column per register, which is the element
        // pair of the operand; a 16x128b TMEM store takes exactly that distribution (lane = t / 4, column = t % 4), so the
        // transpose costs no shuffles.  One round = 16 tokens x 16 d_v lanes: matrices (tokens 0..7 | 8..15) x (d_v 0..7 | 8..15).
        const int mk = lane >> 3, mr = lane & 7;                 // this thread addresses row mr of matrix mk
        auto make_vt = [&](int c) {
            const int s = c % NST, b = c & 1;
            WAIT(&sh.ld_full[s], (c / NST) & 1);
            WAIT(&sh.ga_full[c & (NGA - 1)], (c / NGA) & 1);
            if (c >= 2) WAIT(&sh.vt_free[b], ((c >> 1) - 1) & 1);  // the update of chunk c - 2 has read this buffer
            tc_fence_after();
            const uint32_t vtile = smem_u32(tiles + s * STAGE_BYTES + ST_V);
            const uint8_t* wp = reinterpret_cast<const uint8_t*>(sh.ga[c & (NGA - 1)].w) + 4 * (lane & 3);
#pragma unroll 1
            for (int hh = 0; hh < 2; ++hh) {       // the two 16-lane halves of this warp's TMEM quadrant
                const int d = 32 * q + 16 * hh + 8 * (mk & 1);            // first d_v column of the matrix this thread addresses
                // row of the V tile: token * 128 bytes, 16-byte piece (d / 8 mod 8) ^ (token mod 8); token mod 8 = mr in every round
                const uint32_t row0 = vtile + (uint32_t)(d >> 6) * 8192u + (uint32_t)((8 * (mk >> 1) + mr) * 128) +
                                      (((uint32_t)((d & 63) >> 3) ^ (uint32_t)mr) << 4);
                const uint32_t vt = tb + ((uint32_t)(32 * q + 16 * hh) << 16) + COL_VT + 32 * b;
                uint32_t r[16], w[8];
#pragma unroll
                for (int t16 = 0; t16 < 4; ++t16) {      // all loads of the half first: their latencies overlap
                    ldmatrix_x4_trans(row0 + (uint32_t)(t16 * 16 * 128), r[4 * t16], r[4 * t16 + 1], r[4 * t16 + 2], r[4 * t16 + 3]);
                    w[2 * t16] = *reinterpret_cast<const uint32_t*>(wp + 32 * t16);
                    w[2 * t16 + 1] = *reinterpret_cast<const uint32_t*>(wp + 32 * t16 + 16);
                }
#pragma unroll
                for (int t16 = 0; t16 < 4; ++t16) {
                    const __nv_bfloat162 ww0 = *reinterpret_cast<const __nv_bfloat162*>(&w[2 * t16]), ww1 = *reinterpret_cast<const __nv_bfloat162*>(&w[2 * t16 + 1]);
                    const __nv_bfloat162 y0 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16]), ww0);
                    const __nv_bfloat162 y1 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16 + 1]), ww0);
                    const __nv_bfloat162 y2 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16 + 2]), ww1);
                    const __nv_bfloat162 y3 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16 + 3]), ww1);
                    tmem_st_16x128b(vt + 8 * t16, *reinterpret_cast<const uint32_t*>(&y0), *reinterpret_cast<const uint32_t*>(&y1));
                    tmem_st_16x128b(vt + 8 * t16 + 4, *reinterpret_cast<const uint32_t*>(&y2), *reinterpret_cast<const uint32_t*>(&y3));
                }
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(&sh.vt_ready[b]); mbar_arrive(&sh.ld_empty[s]); }
        };
        __nv_bfloat16* og = reinterpret_cast<__nv_bfloat16*>(p.o);
        // The accumulators are read in the 16x256b distribution: per 16-lane half hh of this warp's quadrant, thread t holds the
        // d_v lanes 32 q + 16 hh + t / 4 (and + 8) and, per group i of 8 tokens, the token pair 8 i + 2 (t % 4), + 1.  A pair of
        // tokens of one d_v lane packs into one bf16x2 register, the unit of the exchange with the peer CTA (slot of 16 bytes
        // per thread, group pair and half) and of the transposing stmatrix that lays the finished outputs out token-major.
        // x[4 i + 0, 1]: lane t / 4, x[4 i + 2, 3]: lane t / 4 + 8 ; value = rowf_j O^i[j] [+ O_in[j]]
        const int tq = lane & 3;
        auto partial32 = [&](int c, int hh, int th, float2 (&x)[8]) {
            uint32_t ra[16], rc[16];
            const uint32_t ta = tb + ((uint32_t)(32 * q + 16 * hh) << 16) + 32 * th;
            const bool own = (c & 1) == rank;       // this CTA computed the chunk-local part
            tmem_ld_16x256b_x4(ta + COL_O + 64 * (c & 1), ra);
            if (own) tmem_ld_16x256b_x4(ta + COL_OI, rc);
            const float* rfp = sh.ga[c & (NGA - 1)].rowf + 32 * th + 2 * tq;
            float2 f[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) f[i] = *reinterpret_cast<const float2*>(rfp + 8 * i);
            tc_wait_ld();
            if (own) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    x[2 * i] = __ffma2_rn(make_float2(__uint_as_float(ra[4 * i]), __uint_as_float(ra[4 * i + 1])), f[i],
                                          make_float2(__uint_as_float(rc[4 * i]), __uint_as_float(rc[4 * i + 1])));
                    x[2 * i + 1] = __ffma2_rn(make_float2(__uint_as_float(ra[4 * i + 2]), __uint_as_float(ra[4 * i + 3])), f[i],
                                              make_float2(__uint_as_float(rc[4 * i + 2]), __uint_as_float(rc[4 * i + 3])));
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    x[2 * i] = __fmul2_rn(make_float2(__uint_as_float(ra[4 * i]), __uint_as_float(ra[4 * i + 1])), f[i]);
                    x[2 * i + 1] = __fmul2_rn(make_float2(__uint_as_float(ra[4 * i + 2]), __uint_as_float(ra[4 * i + 3])), f[i]);
                }
            }
        };
        auto release = [&](int c) {       // this warp has read its part of the accumulators and of the chunk's factors
            __syncwarp();
            if (lane == 0) {
                tc_fence_before();
                mbar_arrive(&sh.o_free[c & 1]);
                if ((c & 1) == rank) mbar_arrive(&sh.oi_free);
                mbar_arrive(&sh.ga_empty[c & (NGA - 1)]);
            }
        };
        // receive buffers: per warp q 2 KB = [half hh][piece k][lane] x 16 bytes (two bf16x2 group pairs per piece)
        const uint32_t slot = (uint32_t)(q * 2048 + lane * 16);
        if (set == 0) {
            // ---- sending warps: V~ one chunk ahead (it feeds the state chain), then the peer's 32 tokens of the chunk's outputs
            // as bf16 partial sums into the peer's receive buffer; the stores complete on the peer's barrier.
            const uint32_t recv_peer = map_to_cta(smem_u32(tiles + OFF_RECV), (uint32_t)peer) + slot;
            const uint32_t xfull_peer = map_to_cta(smem_u32(&sh.x_full[0][q]), (uint32_t)peer);     // + 32 bytes per buffer index
#pragma unroll 1
            for (int c = -1; c < nc; ++c) {
                if (c + 1 < nc) make_vt(c + 1);
                if (c < 0) continue;
                const int b = c & (NRECV - 1);
                WAIT(&sh.o_full[c & 1], (c >> 1) & 1);
                if ((c & 1) == rank) WAIT(&sh.oi_full, (c >> 1) & 1);
                if (c >= NRECV) WAIT(&sh.x_free[b][q], ((c / NRECV) - 1) & 1);     // the peer has read what chunk c - 4 left in buffer b
                tc_fence_after();
                const uint32_t dst = recv_peer + (uint32_t)b * RECV_BYTES, bar = xfull_peer + (uint32_t)b * 32u;
#pragma unroll 1
                for (int hh = 0; hh < 2; ++hh) {
                    float2 x[8];
                    partial32(c, hh, peer, x);
                    uint32_t pk[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) pk[k] = pack_bf16(x[k].x, x[k].y);
                    st_async_b32x4(dst + (uint32_t)(hh * 1024), pk[0], pk[1], pk[2], pk[3], bar);
                    st_async_b32x4(dst + (uint32_t)(hh * 1024 + 512), pk[4], pk[5], pk[6], pk[7], bar);
                }
                release(c);
            }
        } else {
            // ---- finishing warps: this CTA's 32 tokens: own partial sums + what the peer sent -> bf16 -> token-major staging tile
            // (stmatrix, transposed) -> 16-byte stores to global memory
            const uint32_t xfree_peer = map_to_cta(smem_u32(&sh.x_free[0][q]), (uint32_t)peer);     // + 32 bytes per buffer index
            uint8_t* stage = tiles + OFF_OUT + q * OUT_WARP_BYTES;                 // [32 tokens][32 d_v] bf16, rows OUT_PITCH bytes apart
            const uint32_t st_row = smem_u32(stage) + (uint32_t)((lane & 7) * OUT_PITCH + (lane >> 3) * 16);   // stmatrix: row lane % 8 of matrix lane / 8
#pragma unroll 1
            for (int c = 0; c < nc; ++c) {
                const int b = c & (NRECV - 1);
                if (lane == 0) mbar_arrive_expect_tx(&sh.x_full[b][q], 32 * 64);      // the peer's warp q sends 64 bytes per lane
                WAIT(&sh.o_full[c & 1], (c >> 1) & 1);
                if ((c & 1) == rank) WAIT(&sh.oi_full, (c >> 1) & 1);
                tc_fence_after();
                uint32_t out[2][8];          // [hh][2 i + (lane t/4 | lane t/4 + 8)] : bf16x2 of the token pair
                float2 x[8];
                partial32(c, 0, rank, x);
                mbar_wait_cluster(&sh.x_full[b][q], (uint32_t)((c / NRECV) & 1), abortp, p.status);
                const uint8_t* src = tiles + OFF_RECV + b * RECV_BYTES + slot;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    if (hh == 1) partial32(c, 1, rank, x);
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const uint4 y = *reinterpret_cast<const uint4*>(src + hh * 1024 + k * 512);
                        const uint32_t yy[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 s2 = __fadd2_rn(x[4 * k + e], make_float2(__uint_as_float(yy[e] << 16), __uint_as_float(yy[e] & 0xffff0000u)));
                            out[hh][4 * k + e] = pack_bf16(s2.x, s2.y);
                        }
                    }
                }
                release(c);
                if (lane == 0) mbar_arrive_cluster_relaxed(xfree_peer + (uint32_t)b * 32u);     // after release(): the reads have returned
                // matrices of group i: d_v blocks (hh 0: t/4, t/4 + 8; hh 1: t/4, t/4 + 8) x tokens 8 i .. 8 i + 7
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    stmatrix_x4_trans(st_row + (uint32_t)(8 * i * OUT_PITCH), out[0][2 * i], out[0][2 * i + 1], out[1][2 * i], out[1][2 * i + 1]);
                __syncwarp();
                const int valid = min(C, sq.len - tok0 - c * C) - 32 * rank;     // tokens of this CTA's half that exist
                // a warp store covers 8 tokens x 64 contiguous bytes
                __nv_bfloat16* dst = og + ((size_t)(t0 + c * C + 32 * rank) * p.H + h) * D + 32 * q + 8 * (lane & 3);
                const size_t row = (size_t)p.H * D;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const int tok = (lane >> 2) + 8 * m;
                    const uint4 y = *reinterpret_cast<const uint4*>(stage + tok * OUT_PITCH + (lane & 3) * 16);
                    if (tok < valid) *reinterpret_cast<uint4*>(dst + tok * row) = y;
                }
                __syncwarp();
            }
        }
    }
#undef WAIT
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();        // the peer may still be sending to this CTA's shared memory until it gets here too
    if (warp == WARP_Y) tmem_dealloc(tb, 512);
}

// ---- host side -------------------------------------------------------------------------------
// Number of 2-CTA clusters of the main kernel that can be resident at once on the current device
// (falls back to half the SM count of a B200 when there is no device to ask).
}  // namespace

int pair_resident_clusters() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 74; }
    if (cached[dev] > 0) return cached[dev];
    int sms = 0, n = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) { (void)cudaGetLastError(); return 74; }
    n = sms / 2;
    if (cudaFuncSetAttribute(prefill_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN) == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * sms));
        cfg.blockDim = dim3(NTHREADS);
        cfg.dynamicSmemBytes = SMEM_DYN;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int m = 0;
        if (cudaOccupancyMaxActiveClusters(&m, prefill_tc_pair_kernel, &cfg) == cudaSuccess && m > 0 && m < n) n = m;
    }
    (void)cudaGetLastError();
    cached[dev] = n;
    return n;
}

dsla_status launch_main_pair(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& tp, bool dependent,
                             cudaStream_t s) {
    if (cudaFuncSetAttribute(prefill_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN) != cudaSuccess) return DSLA_ERR_CUDA;
    // Clusters of two CTAs (one per state).  With segments, a programmatic dependent launch after the summary grid: the
    // prologue and the first chunk's operand work overlap the summary grid's tail; the state warps wait for it before they
    // read the summaries.
    const long long units = (long long)tp.p.N * tp.p.H;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * units * tp.nseg));
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = SMEM_DYN;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, prefill_tc_pair_kernel, mq, mk, mv, tp) != cudaSuccess) return DSLA_ERR_CUDA;
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // namespace dsla
