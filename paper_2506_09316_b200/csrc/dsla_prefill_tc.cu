// Tensor-core prefill of the dual-state linear attention layer for sm_100a (DSLA_IMPL_TENSOR): bf16 inputs,
// d = 128, fp32 states, both states of a (sequence, head) pair in one CTA.  Chunkwise form of the Sec. 4.1
// recurrence (chunk C = 64 tokens, cumulative log-gates b^i_j inside the chunk, a^i = e^{b^i_last},
// w^i_s = e^{b^i_last - b^i_s}, r^i_j = weight_i e^{b^i_j}, weight = (gamma, 1 - gamma) * scale):
//     P      = Q K^T                                        tcgen05, fp32 in TMEM
//     P~     = P (.) [s<=j] (w1 e^{b1_j-b1_s} + w2 e^{b2_j-b2_s})     CUDA cores -> bf16 in smem
//     O^T    = V^T P~^T + S1^T (r1 (.) Q)^T + S2^T (r2 (.) Q)^T       tcgen05, states read from TMEM
//     S^i^T <- a^i S^i^T + V^T (w^i (.) K)                            rescale on CUDA cores, MMA accumulates
// Everything is computed transposed (d_v on the 128 TMEM lanes, tokens or d_k on the columns) so
// every MMA has M = 128.  The two fp32 states live in TMEM for the whole sequence; a bf16 copy in
// TMEM is the A operand of the readout.  TMA lands K and Q in one of three buffers and V in one of
// two (128-byte swizzle); the gate terms come from cumulative log2-gates of the chunk.
//
// A sequence may be split into segments along T so that few (sequence, head) pairs still fill the
// GPU (dsla_prefill_summary.cu computes the segment summaries); the main kernel, launched as the
// summary grid's programmatic dependent, folds the summaries of earlier segments into its initial
// state.  Packed batches are visited longest sequence first.  This file also holds the host side
// of both tensor-core variants (segment plan, workspace layout, launches).
#include "dsla_prefill_tc.cuh"

namespace dsla {

namespace {

// Warp roles of the main kernel: 0 = TMA producer that also issues the score and state-update MMAs, 1 = issuer of
// the MMAs that build the output tile, 2..9 = tile warps (masked scores, operand scaling), 10..17 = state warps
// (state rescale + bf16 copy, outputs, initial/final state), 18..19 = gate warps.
// A warp may touch only the 32 TMEM lanes of its quadrant (warp index mod 4).
constexpr int WARP_TMA = 0, WARP_MMA = 1, TILE_W0 = 2, STATE_W0 = 10;
constexpr int GATE_W0 = 18;               // warps 18,19: gates, decay mask M, per-token factors
constexpr int NTHREADS = 20 * 32;
// Shared-memory tiles (16 KB each, 128-byte swizzle).  K and Q land in one of three buffers and are scaled in
// place for state 1; the state-2 copies and V live in one of two buffers.  The third landing buffer takes the TMA
// latency and the score MMAs off the chain "operands of chunk c -> MMAs of chunk c -> buffers free again".
constexpr int KQ_BYTES = 2 * 16384;      // [K / K~1][Q / Q~1]
constexpr int KQ_Q = 16384;
constexpr int X_BYTES = 3 * 16384;       // [K~2][Q~2][V]
constexpr int X_Q = 16384, X_V = 32768;
constexpr int OFF_X = 3 * KQ_BYTES;
constexpr int OFF_PT = OFF_X + 2 * X_BYTES;  // P~, 8 KB (freed as soon as the V part of the output has read it)
constexpr int OFF_MASK = OFF_PT + 8192;      // decay mask M, bf16 [2][64][MASK_PITCH] (one buffer per chunk parity)
constexpr int MASK_PITCH = 72;               // bf16 elements; 144-byte rows keep 16-byte row accesses conflict-free
constexpr int MASK_BYTES = 64 * MASK_PITCH * 2;
constexpr int SMEM_TILES = OFF_MASK + 2 * MASK_BYTES;
constexpr int SMEM_DYN = SMEM_TILES + 1024;  // + alignment slack
// TMEM columns
constexpr uint32_t COL_S = 0;      // fp32 S1^T [0,128), S2^T [128,256)
constexpr uint32_t COL_SB = 256;   // bf16 copies: S1^T [256,320), S2^T [320,384)
constexpr uint32_t COL_O = 384;    // O^T, 64 columns (tokens)
constexpr uint32_t COL_P = 448;    // P, 64 columns (lanes 0..63 meaningful)


// Per-token factors of one chunk, per state.
struct alignas(16) GateSmem {
    uint32_t rowf[2][C]; // weight_i * (decay from the chunk start through token j), bf16 in both halves
    uint32_t w[2][C];    // decay from token s to the end of the chunk (or segment), bf16 in both halves
};

struct alignas(16) Shared {
    uint64_t kq_full[3], kq_empty[3], v_full[2], x_empty[2], p_full[2], p_free, pt_free, prep_ready[2], sb_ready[2], s_ready[2], o_full[2], o_free,
        u_full[2], m_ready[2], m_free[2], init_done;
    uint32_t tmem_base;
    int abort_flag;
    GateSmem gs[2];
};

// ============================================================================================
// Main kernel
// ============================================================================================
__global__ void __launch_bounds__(NTHREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const TcParams tp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const PrefillParams& p = tp.p;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Blocks are handed out in index order: the last segments first.  When this grid starts as a programmatic dependent
    // of the summary grid, the blocks that fit next to it are then the ones with the longest fold of summaries ahead of
    // them, and their prologue (TMEM, first tiles, first scores) is hidden behind the summary grid's tail.
    const int units = p.N * p.H;
    const int g = tp.nseg - 1 - (int)(blockIdx.x / units);
    const int h = (blockIdx.x % units) % p.H;
    const int rank = (blockIdx.x % units) / p.H;
    const int n = tp.order ? tp.order[rank] : rank;
    const SeqInfo sq = seq_info(p, n, g, tp.nseg, tp.cps, tp.skew8);
    if (sq.slot < 0 || sq.slot >= p.num_slots) return;
    if (tid == 0 && g == 0 && sq.nchunks > seg_begin(tp.nseg, tp.nseg, tp.cps, tp.skew8)) atomicExch(p.status, (int)DSLA_ERR_INVALID_ARG);
    float* slot1 = p.state + (((size_t)sq.slot * p.n_total + p.state_first) * p.H + h) * (size_t)(D * D);
    const size_t state_stride = (size_t)p.H * D * D;
    // where the initial state is read: the slot, or the snapshot taken before this grid (split sequences)
    const float* init1 = tp.init ? tp.init + (size_t)(n * p.H + h) * 2 * (size_t)(D * D) : slot1;
    const size_t init_stride = tp.init ? (size_t)(D * D) : state_stride;
    if (sq.len <= 0) {  // empty sequence: a fresh start leaves zero states, a resume leaves the slot alone
        if (g == 0 && !p.use_initial_state)
            for (int i = tid; i < (p.single ? 1 : 2) * D * D; i += NTHREADS) slot1[(size_t)(i / (D * D)) * state_stride + i % (D * D)] = 0.f;
        return;
    }
    if (sq.c_begin >= sq.c_end) return;
    const int nc = sq.c_end - sq.c_begin;
    const int t0 = sq.t_begin + sq.c_begin * C;   // first token of this segment
    const int tok0 = sq.c_begin * C;              // its index inside the sequence
    const bool init_shared = (g > 0 && tp.ws) || p.use_initial_state;   // the initial state is loaded, not just zero
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent launch behind this grid (the decode step) may be scheduled early

    if (tid == 0) {
        for (int i = 0; i < 3; ++i) { mbar_init(&sh.kq_full[i], 1); mbar_init(&sh.kq_empty[i], 2); }   // both issuers release a buffer
        for (int i = 0; i < 2; ++i) { mbar_init(&sh.v_full[i], 1); mbar_init(&sh.x_empty[i], 2); }
        mbar_init(&sh.pt_free, 1);
        mbar_init(&sh.init_done, 8);     // the tile warps' share of the initial state
        mbar_init(&sh.p_full[0], 1); mbar_init(&sh.p_free, 8);   // every tile warp passes p_full before P is overwritten
        mbar_init(&sh.prep_ready[0], 8);
        mbar_init(&sh.sb_ready[0], 4); mbar_init(&sh.sb_ready[1], 4); mbar_init(&sh.s_ready[0], 4); mbar_init(&sh.s_ready[1], 4);
        mbar_init(&sh.o_full[0], 1); mbar_init(&sh.o_free, 8); mbar_init(&sh.u_full[0], 1); mbar_init(&sh.u_full[1], 1);
        mbar_init(&sh.m_ready[0], 2); mbar_init(&sh.m_ready[1], 2);
        mbar_init(&sh.m_free[0], 8); mbar_init(&sh.m_free[1], 8);
        sh.abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == WARP_MMA) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = sh.tmem_base;
    volatile int* abortp = &sh.abort_flag;
#define WAIT(bar, ph) mbar_wait(bar, (uint32_t)(ph), abortp, p.status)

    if (warp == WARP_TMA) {
        // ------------------------------------------------------------------ TMA producer + issuer of P and the state updates
        // Two threads issue the MMAs of a chunk.  This one loads the tiles, issues the state updates
        // S^i^T += V^T K~i (which wait only for the state warps' rescale) and the scores P = Q K^T two chunks ahead;
        // the other issues everything that accumulates into the output tile.
        if (lane == 0) {
            prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_P = idesc_bf16(128, 64, 0, 0);
            constexpr uint32_t ID_U = idesc_bf16(128, 128, 1, 1);
            constexpr uint64_t KQ_STEP = (uint64_t)(KQ_BYTES >> 4), X_STEP = (uint64_t)(X_BYTES >> 4);
            const uint64_t dq0 = smem_desc_sw128(sa + KQ_Q, 16, 1024), dk0 = smem_desc_sw128(sa, 16, 1024);         // K-major (scores)
            const uint64_t dkn1 = smem_desc_sw128(sa, 8192, 1024), dkn2 = smem_desc_sw128(sa + OFF_X, 8192, 1024);   // K~1, K~2 as N operands
            const uint64_t dv0 = smem_desc_sw128(sa + OFF_X + X_V, 8192, 1024);
            // Iteration c: state updates of chunk c, refills of the buffers chunk c used, scores of chunk c + 2.
            // Iterations -3..-1 only start the first loads and the first two score tiles (one copy of each code path).
            int k3 = 0, ph3 = 0;        // c mod 3 and the parity of c / 3 (valid for c >= 0)
            int k3p = 0;                // (c + 2) mod 3 for c >= -2
#pragma unroll 1
            for (int c = -3; c < nc; ++c) {
                const int s = c & 1;
                if (c >= 0) {
                    WAIT(&sh.prep_ready[0], c & 1);            // K~1, K~2 are in place
                    WAIT(&sh.v_full[s], (c >> 1) & 1);
                    const uint64_t a = dv0 + (uint64_t)s * X_STEP;
#pragma unroll 1
                    for (int i = 0; i < 2; ++i) {
                        WAIT(&sh.s_ready[i], c & 1);           // fp32 state i has been rescaled
                        tc_fence_after();
                        const uint64_t b = i == 0 ? dkn1 + (uint64_t)k3 * KQ_STEP : dkn2 + (uint64_t)s * X_STEP;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_S + 128 * i, a + (uint64_t)(kk * 128), b + (uint64_t)(kk * 128), ID_U, 1);
                        tc_commit(&sh.u_full[i]);
                    }
                    tc_commit(&sh.kq_empty[k3]);
                    tc_commit(&sh.x_empty[s]);
                }
                if (c + 3 < nc) {
                    if (c >= 0) WAIT(&sh.kq_empty[k3], ph3);   // both issuers' MMAs on this buffer are done
                    const int i3 = c >= 0 ? k3 : c + 3;
                    uint8_t* dst = tiles + i3 * KQ_BYTES;
                    const int t = t0 + (c + 3) * C;
                    mbar_arrive_expect_tx(&sh.kq_full[i3], 4 * 8192);
                    tma_load_4d(dst, &map_k, &sh.kq_full[i3], 0, t, 0, h);
                    tma_load_4d(dst + KQ_Q, &map_q, &sh.kq_full[i3], 0, t, 0, h);
                }
                if (c >= -2 && c + 2 < nc) {
                    if (c >= 0) WAIT(&sh.x_empty[s], (c >> 1) & 1);
                    mbar_arrive_expect_tx(&sh.v_full[s], 2 * 8192);
                    tma_load_4d(tiles + OFF_X + s * X_BYTES + X_V, &map_v, &sh.v_full[s], 0, t0 + (c + 2) * C, 0, h);
                    // scores of chunk c + 2: K-major operands, four 32-byte k-steps inside a 64-element block, the next block 8 KB further
                    const int cp = c + 2;
                    WAIT(&sh.kq_full[k3p], (cp / 3) & 1);
                    if (cp >= 1) WAIT(&sh.p_free, (cp - 1) & 1);          // every tile warp has seen the previous P
                    tc_fence_after();
                    const uint64_t sn = (uint64_t)k3p * KQ_STEP;
#pragma unroll 1
                    for (int blk = 0; blk < 2; ++blk) {
                        const uint64_t a = dq0 + sn + (uint64_t)(512 * blk), b = dk0 + sn + (uint64_t)(512 * blk);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_P, a + (uint64_t)(2 * kk), b + (uint64_t)(2 * kk), ID_P, (blk | kk) ? 1u : 0u);
                    }
                    tc_commit(&sh.p_full[0]);
                }
                if (c >= 0 && ++k3 == 3) { k3 = 0; ph3 ^= 1; }
                if (c >= -2 && ++k3p == 3) k3p = 0;
            }
        }
    } else if (warp == WARP_MMA) {
        // ------------------------------------------------------------------ MMA issuer of the output tile
        // O^T = V^T P~^T + S1^T Q~1^T + S2^T Q~2^T : the first part does not need the states; each state has its own
        // hand-off, so the bf16 copy of one runs under the MMAs of the other.  Groups of four MMAs with compile-time
        // operand steps cost about half the issue time of a rolled loop.
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_OS = idesc_bf16(128, 64, 0, 0);
            constexpr uint32_t ID_OV = idesc_bf16(128, 64, 1, 0);
            constexpr uint64_t KQ_STEP = (uint64_t)(KQ_BYTES >> 4), X_STEP = (uint64_t)(X_BYTES >> 4);
            const uint64_t dq1 = smem_desc_sw128(sa + KQ_Q, 16, 1024), dq2 = smem_desc_sw128(sa + OFF_X + X_Q, 16, 1024);
            const uint64_t dv0 = smem_desc_sw128(sa + OFF_X + X_V, 8192, 1024);
            const uint64_t dp0 = smem_desc_sw128(sa + OFF_PT, 16, 1024);
            int k3 = 0;
#pragma unroll 1
            for (int c = 0; c < nc; ++c) {
                const int s = c & 1;
                WAIT(&sh.prep_ready[0], c & 1);
                WAIT(&sh.v_full[s], (c >> 1) & 1);
                if (c > 0) WAIT(&sh.o_free, (c - 1) & 1);
                tc_fence_after();
                {
                    const uint64_t a = dv0 + (uint64_t)s * X_STEP;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_O, a + (uint64_t)(kk * 128), dp0 + (uint64_t)(2 * kk), ID_OV, kk ? 1u : 0u);
                    tc_commit(&sh.pt_free);       // P~ may be overwritten
                }
#pragma unroll 1
                for (int i = 0; i < 2; ++i) {
                    WAIT(&sh.sb_ready[i], c & 1);
                    tc_fence_after();
                    const uint64_t dq = i == 0 ? dq1 + (uint64_t)k3 * KQ_STEP : dq2 + (uint64_t)s * X_STEP;
                    const uint32_t at = tb + COL_SB + 64 * i;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ts(tb + COL_O, at + 8 * kk, dq + (uint64_t)(2 * kk), ID_OS, 1);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ts(tb + COL_O, at + 32 + 8 * kk, dq + 512 + (uint64_t)(2 * kk), ID_OS, 1);
                }
                tc_commit(&sh.o_full[0]);
                tc_commit(&sh.kq_empty[k3]);
                tc_commit(&sh.x_empty[s]);
                if (++k3 == 3) k3 = 0;
            }
        }
    } else if (warp < STATE_W0) {
        // ------------------------------------------------------------------ tile warps 2..9
        // All eight warps work on every chunk: P~ = P (.) M (the four warps of quadrants 0 and 1) and the scaled
        // copies of Q and K (everyone).
        const int tt = tid - TILE_W0 * 32;                // 0..255
        const int q = warp & 3;                           // TMEM lane quadrant
        const int half = (warp - TILE_W0) >> 2;           // column half: 32 score columns / 32 output tokens
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);

        int k3 = 0, ph3 = 0;      // c mod 3, parity of c / 3
        if (init_shared) {
            // rows 64..127 of the initial state of state `half` for this lane quadrant, while the first tiles are in flight
            const float* gsrc = half == 0 ? p.g_hist : p.g_rec;
            float a0 = fmaxf(load_gate(gsrc, t0 + 2 * lane, p.H, h, tok0 + 2 * lane < sq.len), 0.f) *
                       fmaxf(load_gate(gsrc, t0 + 2 * lane + 1, p.H, h, tok0 + 2 * lane + 1 < sq.len), 0.f);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) a0 *= __shfl_xor_sync(0xffffffffu, a0, off);      // decay of chunk 0
            if (g > 0 && tp.ws) asm volatile("griddepcontrol.wait;" ::: "memory");
            init_state_pass(init1 + (size_t)half * init_stride, p.use_initial_state && !(p.single && half == 1),
                            tp.ws ? tp.ws + ((size_t)(n * p.H + h) * tp.nseg) * (SUMMARY_STRIDE / 4) : nullptr, g, half, 32 * q + lane, a0,
                            lane_addr + COL_S + 128 * half, lane_addr + COL_SB + 64 * half, 2, 4);
            tc_wait_st();
            tc_fence_before();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.init_done);
        for (int c = 0; c < nc; ++c, k3 = k3 == 2 ? 0 : k3 + 1, ph3 ^= (k3 == 0)) {
            const int s = c & 1;
            GateSmem& gs = sh.gs[s];
            uint8_t* kq = tiles + k3 * KQ_BYTES;            // K (-> K~1) and Q (-> Q~1) of this chunk
            uint8_t* xb = tiles + OFF_X + s * X_BYTES;      // K~2, Q~2 (and V) of this chunk
            const uint8_t* Mm = tiles + OFF_MASK + s * MASK_BYTES;
            {
                WAIT(&sh.m_ready[s], (c >> 1) & 1);
                WAIT(&sh.kq_full[k3], ph3);   // TMA writes of K, Q visible to this thread
                // P ready: the MMA is done reading raw Q, K.  The second issuer put P_c behind its wait for the MMAs of
                // chunk c - 2, so the K~2 / Q~2 buffer of this parity is free as well.
                WAIT(&sh.p_full[0], c & 1);
                tc_fence_after();
                if (q >= 2 && lane == 0) mbar_arrive(&sh.p_free);   // these warps do not read P; they only had to see this phase
                if (q < 2) {
                    // ---- P~ rows 32q..32q+31, columns 32 half .. +31
                    const int j = 32 * q + lane;
                    uint8_t* pt = tiles + OFF_PT;
                    const bool any = half <= q;               // block not entirely above the diagonal
                    uint32_t r[32];
                    if (any) { tmem_ld32(lane_addr + COL_P + 32 * half, r); tc_wait_ld(); }
                    __syncwarp();
                    if (lane == 0) { tc_fence_before(); mbar_arrive(&sh.p_free); }
                    if (c >= 1) WAIT(&sh.pt_free, (c - 1) & 1);     // the V part of chunk c - 1 has read P~
                    const uint4* mrow = reinterpret_cast<const uint4*>(Mm + j * (MASK_PITCH * 2) + 64 * half);
#pragma unroll
                    for (int m4 = 0; m4 < 4; ++m4) {
                        uint32_t pk[4] = {0u, 0u, 0u, 0u};
                        // columns 32 half + 8 m4 .. +7 ; everything right of the row's 16-block is zero
                        if (any && 32 * half + 8 * m4 <= (j | 15)) {
                            const uint4 mm = mrow[m4];
                            const uint32_t mw[4] = {mm.x, mm.y, mm.z, mm.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(&mw[e]);
                                pk[e] = pack_bf16(__uint_as_float(r[8 * m4 + 2 * e]) * __low2float(m2),
                                                  __uint_as_float(r[8 * m4 + 2 * e + 1]) * __high2float(m2));
                            }
                        }
                        *reinterpret_cast<uint4*>(pt + sw128_offset(j, 32 * half + 8 * m4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
                {
                    // ---- scaled copies: every thread handles four 16-byte pieces of Q and of K
#pragma unroll 1
                    for (int m = 0; m < 4; ++m) {
                        const int idx = tt + 256 * m;             // 16-byte piece inside a 16 KB tile
                        const int row = (idx >> 3) & 63;
                        const uint4 xq = reinterpret_cast<const uint4*>(kq + KQ_Q)[idx], xk = reinterpret_cast<const uint4*>(kq)[idx];
                        const uint32_t f0 = gs.rowf[0][row], f1 = gs.rowf[1][row], w0 = gs.w[0][row], w1 = gs.w[1][row];
                        reinterpret_cast<uint4*>(kq + KQ_Q)[idx] = scale8(xq, f0);
                        reinterpret_cast<uint4*>(xb + X_Q)[idx] = scale8(xq, f1);
                        reinterpret_cast<uint4*>(kq)[idx] = scale8(xk, w0);
                        reinterpret_cast<uint4*>(xb)[idx] = scale8(xk, w1);
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.prep_ready[0]); mbar_arrive(&sh.m_free[s]); }
            }
        }
    } else if (warp >= GATE_W0) {
        // ------------------------------------------------------------------ gate warps 18,19
        // Everything the chunk needs from the gates comes from the cumulative log-gates
        //     L^i_j = sum_{t <= j} log2 g^i_t        (inclusive, from the chunk start; a zero gate counts as -200,
        //                                             so any product that contains one flushes to an exact zero)
        // through independent exponentials (no serial chains):
        //   M[j][s]  = W1 2^(L1_j - L1_s) + W2 2^(L2_j - L2_s)  for s <= j, else 0      (decay mask)
        //   rowf^i_j = W_i 2^(L^i_j)                  (decay from the chunk start through token j)
        //   w^i_s    = 2^(L^i_last - L^i_s)           (decay from token s to the end of the chunk)
        // Lane l holds tokens l and l + 32.  Warp 18 writes the triangle of rows/columns 0..31, warp 19 the
        // triangle of 32..63; the full block (rows 32..63, columns 0..31) factors through token 31,
        // 2^(L_j - L_31) 2^(L_31 - L_s) with both factors <= 1, and is split between the two warps.
        const int gw = warp - GATE_W0;
        const float W1 = (p.weights ? p.weights[(size_t)h * p.n_total + p.state_first] : p.gamma[h]) * p.scale;
        const float W2 = p.single ? 0.f : (p.weights ? p.weights[(size_t)h * p.n_total + p.state_first + 1] : 1.f - p.gamma[h]) * p.scale;
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
        for (int c = 0; c < nc; ++c) {
            const int s = c & 1;
            GateSmem& gs = sh.gs[s];
            __nv_bfloat16* Mm = reinterpret_cast<__nv_bfloat16*>(tiles + OFF_MASK + s * MASK_BYTES);
            const float2 glo = make_float2(fmaxf(nlo.x, 0.f), fmaxf(nlo.y, 0.f)), ghi = make_float2(fmaxf(nhi.x, 0.f), fmaxf(nhi.y, 0.f));
            fetch(c + 1, nlo, nhi);
            float l1a = warp_prefix_sum(lg2_gate(glo.x), lane), l2a = warp_prefix_sum(lg2_gate(glo.y), lane);
            float l1b = warp_prefix_sum(lg2_gate(ghi.x), lane), l2b = warp_prefix_sum(lg2_gate(ghi.y), lane);
            const float mid1 = __shfl_sync(0xffffffffu, l1a, 31), mid2 = __shfl_sync(0xffffffffu, l2a, 31);   // L at token 31
            l1b += mid1; l2b += mid2;
            const float end1 = __shfl_sync(0xffffffffu, l1b, 31), end2 = __shfl_sync(0xffffffffu, l2b, 31);   // L at token 63
            if (c >= 2) WAIT(&sh.m_free[s], ((c >> 1) - 1) & 1);
            {
                // per-token factors of this warp's state
                const float la = gw == 0 ? l1a : l2a, lb = gw == 0 ? l1b : l2b, le = gw == 0 ? end1 : end2;
                const float Wi = gw == 0 ? W1 : W2;
                const int valid = min(C, sq.len - tok0 - c * C);
                gs.rowf[gw][lane] = dup_bf16(Wi * ex2(la));
                gs.rowf[gw][lane + 32] = dup_bf16(Wi * ex2(lb));
                // rows past the end of the sequence carry no weight in the state update
                gs.w[gw][lane] = dup_bf16(lane < valid ? ex2(le - la) : 0.f);
                gs.w[gw][lane + 32] = dup_bf16(lane + 32 < valid ? ex2(le - lb) : 0.f);
            }
            {
                // triangle block of this warp: rows and columns 32 gw .. 32 gw + 31, this lane = column
                const float x1 = gw == 0 ? l1a : l1b, x2 = gw == 0 ? l2a : l2b;
                __nv_bfloat16* mcol = Mm + (32 * gw) * MASK_PITCH + 32 * gw + lane;
#pragma unroll 8
                for (int jj = 0; jj < 32; ++jj) {
                    const float r1 = __shfl_sync(0xffffffffu, x1, jj), r2 = __shfl_sync(0xffffffffu, x2, jj);
                    const float m = fmaf(W2, ex2(r2 - x2), W1 * ex2(r1 - x1));
                    mcol[jj * MASK_PITCH] = __float2bfloat16_rn(jj >= lane ? m : 0.f);
                }
                // full block: rows 32 + 16 gw .. + 15, columns 0..31
                const float f1 = ex2(mid1 - l1a), f2 = ex2(mid2 - l2a);                 // column factors (token s -> 31)
                const float e1 = W1 * ex2(l1b - mid1), e2 = W2 * ex2(l2b - mid2);       // row factors (31 -> token 32 + lane)
                __nv_bfloat16* mrow = Mm + (32 + 16 * gw) * MASK_PITCH + lane;
#pragma unroll 8
                for (int jj = 0; jj < 16; ++jj) {
                    const float a1 = __shfl_sync(0xffffffffu, e1, 16 * gw + jj), a2 = __shfl_sync(0xffffffffu, e2, 16 * gw + jj);
                    mrow[jj * MASK_PITCH] = __float2bfloat16_rn(fmaf(a2, f2, a1 * f1));
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.m_ready[s]);
        }
    } else {
        // ------------------------------------------------------------------ state warps 10..17
        const int q = warp & 3, hi = (warp - STATE_W0) >> 2;   // TMEM lane quadrant, state index
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        const uint32_t s_addr = lane_addr + COL_S + 128 * hi;
        const uint32_t sb_addr = lane_addr + COL_SB + 64 * hi;
        const int v = 32 * q + lane;
        const float* gsrc = hi == 0 ? p.g_hist : p.g_rec;
        // Outputs of chunk c, tokens 32 hi .. 32 hi + 31 of this warp's lane quadrant: each thread owns one d_v lane of
        // O^T; a warp's store of one token is 64 contiguous bytes (two full sectors), so the values go straight from
        // registers to global memory.  The state warps do this after their pass over the state, in the time they would
        // otherwise wait for the next update MMA.
        __nv_bfloat16* og = reinterpret_cast<__nv_bfloat16*>(p.o);
        auto outputs = [&](int c) {
            uint32_t r[32];
            tmem_ld32(lane_addr + COL_O + 32 * hi, r);
            tc_wait_ld();
            __syncwarp();
            if (lane == 0) { tc_fence_before(); mbar_arrive(&sh.o_free); }
            const int valid = min(C, sq.len - tok0 - c * C) - 32 * hi;     // tokens of this warp's half that exist
            __nv_bfloat16* dst = og + ((size_t)(t0 + c * C + 32 * hi) * p.H + h) * D + v;
            const size_t row = (size_t)p.H * D;
            if (valid >= 32) {
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) dst[jj * row] = __float2bfloat16_rn(__uint_as_float(r[jj]));
            } else {
#pragma unroll 1
                for (int jj = 0; jj < valid; ++jj) {   // ragged tail (cold): pick the register with a shuffle-free select chain
                    float x = 0.f;
#pragma unroll
                    for (int e = 0; e < 32; ++e) x = e == jj ? __uint_as_float(r[e]) : x;
                    dst[jj * row] = __float2bfloat16_rn(x);
                }
            }
        };
        // chunk decay a = prod of this state's gates over the chunk (two tokens per lane).  The gates of chunk c + 1
        // are requested at the top of iteration c and multiplied together at its end, so the load latency hides
        // behind the waits and the two passes.
        auto gate_pair = [&](int c) -> float2 {
            const int j = c * C + 2 * lane;
            const bool in = c < nc;
            return make_float2(load_gate(gsrc, t0 + j, p.H, h, in && tok0 + j < sq.len),
                               load_gate(gsrc, t0 + j + 1, p.H, h, in && tok0 + j + 1 < sq.len));
        };
        auto warp_prod = [&](float2 gp) -> float {
            float pr = fmaxf(gp.x, 0.f) * fmaxf(gp.y, 0.f);
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) pr *= __shfl_xor_sync(0xffffffffu, pr, off);
            return pr;
        };
        float a_next = warp_prod(gate_pair(0));
        for (int c = 0; c < nc; ++c) {
            const float a = a_next;
            const float2 gp_next = gate_pair(c + 1);
            if (c == 0) {
                // With programmatic dependent launch this grid may start while the summary grid is still running;
                // everything up to here (and all of chunk 0's operand work in the other warps) is independent of it.
                if (g > 0 && tp.ws) asm volatile("griddepcontrol.wait;" ::: "memory");
                init_state_pass(init1 + (size_t)hi * init_stride, p.use_initial_state && !(p.single && hi == 1),
                                tp.ws ? tp.ws + ((size_t)(n * p.H + h) * tp.nseg) * (SUMMARY_STRIDE / 4) : nullptr, g, hi, v, a, s_addr, sb_addr,
                                0, init_shared ? 2 : 4);
                tc_wait_st();
                mbar_wait(&sh.init_done, 0, abortp, p.status);     // the other half (or nothing) from the tile warps
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.sb_ready[hi]); mbar_arrive(&sh.s_ready[hi]); }
                a_next = warp_prod(gp_next);
                continue;
            }
            WAIT(&sh.u_full[hi], (c - 1) & 1);
            WAIT(&sh.o_full[0], (c - 1) & 1);   // the readout of chunk c-1 (other issuer) has read the bf16 copy
            tc_fence_after();
            // ---- one pass over the state (TMEM -> registers once): the bf16 copy of S_{c-1} that the readout of chunk c
            // multiplies, and a_c S_{c-1} in place, onto which the update MMA of chunk c accumulates
            {
                const float2 a2 = make_float2(a, a);
                uint32_t r0[32], r1[32];
                tmem_ld32(s_addr, r0);
                tmem_ld32(s_addr + 32, r1);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    tc_wait_ld();
                    uint32_t pk[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) pk[k] = pack_bf16(__uint_as_float(r0[2 * k]), __uint_as_float(r0[2 * k + 1]));
                    tmem_st16(sb_addr + 32 * half, pk);
#pragma unroll
                    for (int k = 0; k < 16; ++k) pk[k] = pack_bf16(__uint_as_float(r1[2 * k]), __uint_as_float(r1[2 * k + 1]));
                    tmem_st16(sb_addr + 32 * half + 16, pk);
#pragma unroll
                    for (int k = 0; k < 32; k += 2) {
                        const float2 y0 = __fmul2_rn(make_float2(__uint_as_float(r0[k]), __uint_as_float(r0[k + 1])), a2);
                        const float2 y1 = __fmul2_rn(make_float2(__uint_as_float(r1[k]), __uint_as_float(r1[k + 1])), a2);
                        r0[k] = __float_as_uint(y0.x); r0[k + 1] = __float_as_uint(y0.y);
                        r1[k] = __float_as_uint(y1.x); r1[k + 1] = __float_as_uint(y1.y);
                    }
                    tmem_st32(s_addr + 64 * half, r0);
                    tmem_st32(s_addr + 64 * half + 32, r1);
                    if (half == 0) { tmem_ld32(s_addr + 64, r0); tmem_ld32(s_addr + 96, r1); }
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.sb_ready[hi]); mbar_arrive(&sh.s_ready[hi]); }
            }
            outputs(c - 1);       // o_full of chunk c - 1 was awaited at the top of this iteration
            a_next = warp_prod(gp_next);
        }
        // ---- outputs of the last chunk, final states of this segment
        mbar_wait(&sh.o_full[0], (nc - 1) & 1, abortp, p.status);
        tc_fence_after();
        outputs(nc - 1);
        mbar_wait(&sh.u_full[hi], (nc - 1) & 1, abortp, p.status);
        tc_fence_after();
        if (g == sq.last_seg && !(p.single && hi == 1)) store_state(slot1 + (size_t)hi * state_stride, v, s_addr, 0, 4);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == WARP_MMA) tmem_dealloc(tb, 512);
}

}  // namespace

namespace {

bool wants_order(const dsla_prefill_args* a) { return a->cu_seqlens != nullptr && a->N > 1 && a->N <= ORDER_MAX_N; }

int sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
        (void)cudaGetLastError();
        return 148;      // a B200, when there is no device to ask (sizing a workspace on a build machine)
    }
    return sms;
}

// Segments per sequence: enough work items (CTAs, or clusters of the pair variant) to cover the SMs when there
// are few (sequence, head) pairs, never shorter than 4 chunks per segment.
void plan(const dsla_prefill_args* a, bool pair, int* nseg, int* cps, int* skew8) {
    const int max_chunks = (a->max_seqlen + C - 1) / C;
    const long long units = (long long)a->N * a->H;
    const int room = pair ? pair_resident_clusters() : sm_count();     // work items resident at once
    int ns = 1;
    if (units > 0 && units < room) ns = (int)(room / units);
    if (ns > 16) ns = 16;
    while (ns > 1 && (max_chunks + ns - 1) / ns < 4) --ns;
    if (max_chunks <= 0) ns = 1;
    *nseg = ns;
    *cps = max_chunks > 0 ? (max_chunks + ns - 1) / ns : 1;
    // later segments fold more summaries into their initial state before they start (about 0.8 chunk times each):
    // make consecutive segments 3/4 chunk shorter, as far as the shortest keeps at least three chunks
    int sk = ns > 1 ? (8 * (*cps - 3)) / (ns - 1) : 0;
    *skew8 = sk < 0 ? 0 : (sk > 3 ? 3 : sk);
}

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
size_t summaries_bytes(const dsla_prefill_args* a, int nseg) { return nseg > 1 ? (size_t)a->N * a->H * nseg * SUMMARY_STRIDE : 0; }
size_t order_bytes(const dsla_prefill_args* a) { return wants_order(a) ? up256((size_t)a->N * sizeof(int)) : 0; }
// room for the snapshot of the initial states of split sequences (used when use_initial_state is set)
size_t snapshot_bytes(const dsla_prefill_args* a, int nseg) { return nseg > 1 ? (size_t)a->N * a->H * 2 * D * D * sizeof(float) : 0; }

dsla_status launch_main(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& tp, bool dependent,
                        cudaStream_t s) {
    if (cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN) != cudaSuccess) return DSLA_ERR_CUDA;
    const long long units = (long long)tp.p.N * tp.p.H;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * tp.nseg));
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = SMEM_DYN;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, prefill_tc_kernel, mq, mk, mv, tp) != cudaSuccess) return DSLA_ERR_CUDA;
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // namespace

bool prefill_tc_available() { return true; }

size_t prefill_tc_workspace_bytes(const dsla_prefill_args* a, bool pair) {
    int nseg, cps, skew8;
    plan(a, pair, &nseg, &cps, &skew8);
    return summaries_bytes(a, nseg) + order_bytes(a) + snapshot_bytes(a, nseg);     // each a multiple of 256
}

dsla_status launch_prefill_tc(const PrefillParams& p, const dsla_prefill_args* a, bool pair, cudaStream_t s) {
    if (p.N == 0 || a->T_total == 0) {
        // only empty sequences: the CUDA-core kernel handles the slot bookkeeping
        return launch_prefill_simt(p, D, C, DSLA_BF16, s);
    }
    TcParams tp;
    tp.p = p;
    plan(a, pair, &tp.nseg, &tp.cps, &tp.skew8);
    char* wsp = static_cast<char*>(a->workspace);
    tp.ws = tp.nseg > 1 ? reinterpret_cast<float*>(wsp) : nullptr;
    tp.order = nullptr;
    tp.init = nullptr;
    if (wants_order(a)) {
        int* order = reinterpret_cast<int*>(wsp + summaries_bytes(a, tp.nseg));
        launch_seq_order(p.cu_seqlens, p.N, order, s);
        tp.order = order;
    }
    if (tp.nseg > 1 && p.use_initial_state) {
        // The CTA of a sequence's last segment overwrites the slot with the final state; CTAs of earlier segments read the
        // slot as their initial state and nothing orders the two inside the grid: they read a copy taken beforehand.
        float* snap = reinterpret_cast<float*>(wsp + summaries_bytes(a, tp.nseg) + order_bytes(a));
        launch_state_snapshot(p, snap, s);
        tp.init = snap;
    }
    CUtensorMap mq, mk, mv;
    if (!make_tile_map(&mq, p.q, a->T_total, p.H) || !make_tile_map(&mk, p.k, a->T_total, p.H) || !make_tile_map(&mv, p.v, a->T_total, p.H))
        return DSLA_ERR_CUDA;
    const long long units = (long long)p.N * p.H;
    if (2 * units * tp.nseg > 0x7fffffffLL) return DSLA_ERR_UNSUPPORTED;
    if (tp.nseg > 1) {
        const dsla_status rc = launch_summary(mk, mv, tp, s);
        if (rc != DSLA_OK) return rc;
    }
    return pair ? launch_main_pair(mq, mk, mv, tp, tp.nseg > 1, s) : launch_main(mq, mk, mv, tp, tp.nseg > 1, s);
}

}  // namespace dsla
