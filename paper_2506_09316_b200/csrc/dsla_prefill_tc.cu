// Tensor-core prefill of the dual-state linear attention layer for sm_100a: bf16 inputs, d = 128,
// fp32 states.  Chunkwise form of the Sec. 4.1 recurrence (chunk C = 64 tokens, cumulative
// log-gates b^i_j inside the chunk, a^i = e^{b^i_last}, w^i_s = e^{b^i_last - b^i_s},
// r^i_j = weight_i e^{b^i_j}, weight = (gamma, 1 - gamma) * scale):
//     P      = Q K^T                                        tcgen05, fp32 in TMEM
//     P~     = P (.) [s<=j] (w1 e^{b1_j-b1_s} + w2 e^{b2_j-b2_s})     CUDA cores -> bf16 in smem
//     O^T    = V^T P~^T + S1^T (r1 (.) Q)^T + S2^T (r2 (.) Q)^T       tcgen05, states read from TMEM
//     S^i^T <- a^i S^i^T + V^T (w^i (.) K)                            rescale on CUDA cores, MMA accumulates
// Everything is computed transposed (d_v on the 128 TMEM lanes, tokens or d_k on the columns) so
// every MMA has M = 128.  The two fp32 states live in TMEM for the whole sequence; a bf16 copy in
// TMEM is the A operand of the readout.  TMA lands K and Q in one of three buffers and V in one of
// two (128-byte swizzle); the gate terms come from cumulative log2-gates of the chunk.
//
// A sequence may be split into `nseg` segments along T so that few (sequence, head) pairs still
// fill the GPU: a first kernel computes each segment's state summary from zero
// (U_g = sum_s (prod of later gates in the segment) k_s^T v_s and A_g = prod of the segment's
// gates) into the workspace; the main kernel, launched as its programmatic dependent, combines the
// summaries of earlier segments into its initial state and then runs its segment.  Packed batches
// are visited longest sequence first.
#include "dsla_internal.cuh"
#include "tc_utils.cuh"

namespace dsla {

using namespace tc;

namespace {

constexpr int C = 64;                 // tokens per chunk
constexpr int D = 128;                // head size
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
// summary kernel: 4 stages of [K/K~1][K~2][V]
constexpr int SUM_STAGES = 4, SUM_STAGE_BYTES = 3 * 16384, SUM_OFF_V = 32768;
constexpr int SUM_NTHREADS = 384, SUM_NCOMPUTE = 256;
constexpr int SUM_GATE_AHEAD = 6;        // chunks between the L2 prefetch and the load of a chunk's gates
constexpr int SUM_PREFETCH = 8;          // chunks between the L2 prefetch and the load of a tile
constexpr int SUM_SMEM_DYN = SUM_STAGES * SUM_STAGE_BYTES + 1024;
// TMEM columns
constexpr uint32_t COL_S = 0;      // fp32 S1^T [0,128), S2^T [128,256)
constexpr uint32_t COL_SB = 256;   // bf16 copies: S1^T [256,320), S2^T [320,384)
constexpr uint32_t COL_O = 384;    // O^T, 64 columns (tokens)
constexpr uint32_t COL_P = 448;    // P, 64 columns (lanes 0..63 meaningful)
constexpr size_t SUMMARY_STRIDE = 2 * D * D * sizeof(float) + 256;  // U (both states) + A[2], padded

#ifdef DSLA_TIMELINE
__device__ long long* g_timeline = nullptr;   // [role 6][chunk 64][event 8], then per-CTA start/end times, then counters
__device__ int g_timeline_block = 0;
#define TL(role, c, ev) do { if (tlp && (unsigned)(c) < 64u) tlp[((role) * 64 + (c)) * 8 + (ev)] = clock64(); } while (0)
__device__ __forceinline__ long long gtime() { long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#ifdef DSLA_TLW   // per-thread wait / section counters on top of the event timeline (costs ~20 registers)
#define TL_INIT long long* const tlp = (int)blockIdx.x == g_timeline_block ? g_timeline : nullptr; \
    long long tl_w[10] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0}; const long long tl_t0 = clock64()
#define WAITP(tag, bar, ph) do { const long long _a = clock64(); mbar_wait(bar, ph, abortp, p.status); tl_w[tag] += clock64() - _a; } while (0)
#define TLT(var) const long long var = clock64()
#define TLACC(tag, expr) tl_w[tag] += (expr)
#define TLW_BEGIN const long long _tlb = clock64()
#define TLW_END(tag) tl_w[tag] += clock64() - _tlb
#define TL_DUMP(role) do { if (tlp) { for (int _k = 0; _k < 10; ++_k) tlp[3800 + 12 * (role) + _k] = tl_w[_k]; tlp[3800 + 12 * (role) + 10] = clock64() - tl_t0; } } while (0)
#else
#ifdef DSLA_TIMELINE_SUMMARY   // events of the summary kernel only
#define TL_INIT long long* const tlp = nullptr
#else
#define TL_INIT long long* const tlp = (int)blockIdx.x == g_timeline_block ? g_timeline : nullptr
#endif
#define WAITP(tag, bar, ph) mbar_wait(bar, ph, abortp, p.status)
#define TLT(var) do { } while (0)
#define TLACC(tag, expr) do { } while (0)
#define TLW_BEGIN do { } while (0)
#define TLW_END(tag) do { } while (0)
#define TL_DUMP(role) do { } while (0)
#endif
#else
#define WAITP(tag, bar, ph) mbar_wait(bar, ph, abortp, p.status)
#define TLT(var) do { } while (0)
#define TLACC(tag, expr) do { } while (0)
#define TLW_BEGIN do { } while (0)
#define TLW_END(tag) do { } while (0)
#define TL_DUMP(role) do { } while (0)
#define TL(role, c, ev) do { } while (0)
#define TL_INIT do { } while (0)
#endif

struct TcParams {
    PrefillParams p;
    float* ws;          // summaries: [(n*H + h)*nseg + g] -> {U[2][D][D], A[2]}
    int nseg;           // segments per sequence (grid dimension)
    int cps;            // chunks per segment (mean)
    int skew8;          // eighths of a chunk by which consecutive segments get shorter (later segments start later: they
                        // first fold the summaries of all earlier segments into their initial state)
    const int* order;   // sequences by descending length (longest first), or nullptr for index order
};

// Per-token factors of one chunk, per state.
struct alignas(16) GateSmem {
    uint32_t rowf[2][C]; // weight_i * (decay from the chunk start through token j), bf16 in both halves
    uint32_t w[2][C];    // decay from token s to the end of the chunk (or segment), bf16 in both halves
};

struct alignas(16) Shared {
    uint64_t kq_full[3], kq_empty[3], v_full[2], x_empty[2], p_full[2], p_free, pt_free, prep_ready[2], sb_ready[2], s_ready[2], o_full[2], o_free,
        u_full[2], m_ready[2], m_free[2], init_done;
    uint64_t full[4], empty[4];   // summary kernel
    uint32_t tmem_base;
    int abort_flag;
    GateSmem gs[2];
};

// f rounded to bf16, duplicated into both halves of a 32-bit word
__device__ __forceinline__ uint32_t dup_bf16(float f) {
    const uint32_t h = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(f));
    return h | (h << 16);
}

__device__ __forceinline__ float load_gate(const float* g, int t, int H, int h, bool ok) {
    return ok ? __ldg(g + (size_t)t * H + h) : 1.f;
}

// Multiplies the eight bf16 of a 16-byte piece by the bf16 factor held in both halves of f.
__device__ __forceinline__ uint4 scale8(const uint4 x, const uint32_t f) {
    uint4 y;
    const uint32_t* xi = reinterpret_cast<const uint32_t*>(&x);
    uint32_t* yi = reinterpret_cast<uint32_t*>(&y);
    const __nv_bfloat162 ff = *reinterpret_cast<const __nv_bfloat162*>(&f);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 r = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&xi[e]), ff);
        yi[e] = *reinterpret_cast<const uint32_t*>(&r);
    }
    return y;
}

struct SeqInfo {
    int t_begin, len, slot, nchunks, c_begin, c_end, last_seg;
};

// First chunk of segment g: equal parts of cps chunks, shifted so that segment g is about skew8 (nseg - 2g - 1) / 8
// chunks longer than the mean.  seg_begin(0) = 0 and seg_begin(nseg) = nseg cps.
__host__ __device__ __forceinline__ int seg_begin(int g, int nseg, int cps, int skew8) { return g * cps + (skew8 * g * (nseg - g)) / 8; }

__device__ __forceinline__ SeqInfo seq_info(const PrefillParams& p, int n, int g, int nseg, int cps, int skew8) {
    SeqInfo s;
    s.t_begin = p.cu_seqlens ? p.cu_seqlens[n] : n * p.T;
    const int t_end = p.cu_seqlens ? p.cu_seqlens[n + 1] : (n + 1) * p.T;
    s.len = t_end - s.t_begin;
    s.slot = p.slots ? p.slots[n] : n;
    s.nchunks = (s.len + C - 1) / C;
    s.c_begin = seg_begin(g, nseg, cps, skew8);
    s.c_end = min(s.nchunks, seg_begin(g + 1, nseg, cps, skew8));
    s.last_seg = 0;     // the last segment that holds a chunk of this sequence
    for (int j = 1; j < nseg; ++j)
        if (seg_begin(j, nseg, cps, skew8) < s.nchunks) s.last_seg = j;
    return s;
}

// Initial state of a segment (cold path, kept out of line so the chunk loop stays small): the slot
// contents (or zero) pushed through the summaries of the earlier segments, S <- A_j S + U_j; writes the bf16
// copy for the readout and a_0 S for the first update.  One thread = one d_v lane of one state and the d_k rows
// 32 bt_begin .. 32 bt_end - 1.  The fold is a chain of dependent rounds of loads (about a microsecond per earlier
// segment for one warp per lane quadrant), so when there is something to load the tile warp of the same quadrant,
// which would otherwise wait for the first tiles, takes half of the rows.
__device__ __noinline__ void init_state_pass(const float* base, int use_initial_state, const float* wsu, int g, int hi, int v,
                                             float a, uint32_t s_addr, uint32_t sb_addr, int bt_begin, int bt_end) {
#pragma unroll 1
    for (int bt = bt_begin; bt < bt_end; ++bt) {
        float acc[32];
#pragma unroll
        for (int k = 0; k < 32; ++k) acc[k] = use_initial_state ? base[(size_t)(32 * bt + k) * D + v] : 0.f;
#pragma unroll 1
        for (int jg = 0; jg < g; ++jg) {
            const float* u = wsu + (size_t)jg * (SUMMARY_STRIDE / 4);
            const float A = __ldg(u + 2 * D * D + hi);
            const float* uu = u + (size_t)hi * D * D;
            float x[32];
#pragma unroll
            for (int k = 0; k < 32; ++k) x[k] = __ldg(uu + (size_t)(32 * bt + k) * D + v);
#pragma unroll
            for (int k = 0; k < 32; ++k) acc[k] = fmaf(A, acc[k], x[k]);
        }
        uint32_t pk[16], sc[32];
#pragma unroll
        for (int k = 0; k < 16; ++k) pk[k] = pack_bf16(acc[2 * k], acc[2 * k + 1]);
#pragma unroll
        for (int k = 0; k < 32; ++k) sc[k] = __float_as_uint(acc[k] * a);
        tmem_st16(sb_addr + 16 * bt, pk);
        tmem_st32(s_addr + 32 * bt, sc);
    }
}

// Final fp32 state of one (state, d_v lane) from TMEM to global memory [d_k][d_v] (cold path, out of line).
__device__ __noinline__ void store_state(float* dst, int v, uint32_t s_addr) {
#pragma unroll 1
    for (int bt = 0; bt < 4; ++bt) {
        uint32_t r[32];
        tmem_ld32(s_addr + 32 * bt, r);
        tc_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) dst[(size_t)(32 * bt + k) * D + v] = __uint_as_float(r[k]);
    }
}

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
    float* slot1 = p.state + (((size_t)sq.slot * 2) * p.H + h) * (size_t)(D * D);
    const size_t state_stride = (size_t)p.H * D * D;
    if (sq.len <= 0) {  // empty sequence: a fresh start leaves zero states, a resume leaves the slot alone
        if (g == 0 && !p.use_initial_state)
            for (int i = tid; i < 2 * D * D; i += NTHREADS) slot1[(size_t)(i / (D * D)) * state_stride + i % (D * D)] = 0.f;
        return;
    }
    if (sq.c_begin >= sq.c_end) return;
    const int nc = sq.c_end - sq.c_begin;
    const int t0 = sq.t_begin + sq.c_begin * C;   // first token of this segment
    const int tok0 = sq.c_begin * C;              // its index inside the sequence
    const bool init_shared = (g > 0 && tp.ws) || p.use_initial_state;   // the initial state is loaded, not just zero
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent launch behind this grid (the decode step) may be scheduled early
    TL_INIT;
    if (tid == 0) TL(0, 63, 6);
#ifdef DSLA_TIMELINE
    if (tid == 0 && g_timeline) g_timeline[3072 + 4 * blockIdx.x] = gtime();
#endif

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
                    WAITP(0, &sh.prep_ready[0], c & 1);            // K~1, K~2 are in place
                    WAITP(3, &sh.v_full[s], (c >> 1) & 1);
                    TL(4, c, 3);
                    const uint64_t a = dv0 + (uint64_t)s * X_STEP;
#pragma unroll 1
                    for (int i = 0; i < 2; ++i) {
                        WAITP(1, &sh.s_ready[i], c & 1);           // fp32 state i has been rescaled
                        TL(4, c, 4 + i);
                        tc_fence_after();
                        const uint64_t b = i == 0 ? dkn1 + (uint64_t)k3 * KQ_STEP : dkn2 + (uint64_t)s * X_STEP;
                        TLW_BEGIN;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_S + 128 * i, a + (uint64_t)(kk * 128), b + (uint64_t)(kk * 128), ID_U, 1);
                        tc_commit(&sh.u_full[i]);
                        TLW_END(6);
                    }
                    tc_commit(&sh.kq_empty[k3]);
                    tc_commit(&sh.x_empty[s]);
                    TL(4, c, 6);
                }
                if (c + 3 < nc) {
                    if (c >= 0) WAITP(2, &sh.kq_empty[k3], ph3);   // both issuers' MMAs on this buffer are done
                    if (c >= 0) TL(4, c, 7);
                    const int i3 = c >= 0 ? k3 : c + 3;
                    uint8_t* dst = tiles + i3 * KQ_BYTES;
                    const int t = t0 + (c + 3) * C;
                    mbar_arrive_expect_tx(&sh.kq_full[i3], 4 * 8192);
                    tma_load_4d(dst, &map_k, &sh.kq_full[i3], 0, t, 0, h);
                    tma_load_4d(dst + KQ_Q, &map_q, &sh.kq_full[i3], 0, t, 0, h);
                    TL(4, c + 3, 0);
                }
                if (c >= -2 && c + 2 < nc) {
                    if (c >= 0) WAITP(2, &sh.x_empty[s], (c >> 1) & 1);
                    mbar_arrive_expect_tx(&sh.v_full[s], 2 * 8192);
                    tma_load_4d(tiles + OFF_X + s * X_BYTES + X_V, &map_v, &sh.v_full[s], 0, t0 + (c + 2) * C, 0, h);
                    // scores of chunk c + 2: K-major operands, four 32-byte k-steps inside a 64-element block, the next block 8 KB further
                    const int cp = c + 2;
                    WAITP(4, &sh.kq_full[k3p], (cp / 3) & 1);
                    if (cp >= 1) WAITP(4, &sh.p_free, (cp - 1) & 1);          // every tile warp has seen the previous P
                    TL(4, cp, 1);
                    tc_fence_after();
                    const uint64_t sn = (uint64_t)k3p * KQ_STEP;
                    TLW_BEGIN;
#pragma unroll 1
                    for (int blk = 0; blk < 2; ++blk) {
                        const uint64_t a = dq0 + sn + (uint64_t)(512 * blk), b = dk0 + sn + (uint64_t)(512 * blk);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_P, a + (uint64_t)(2 * kk), b + (uint64_t)(2 * kk), ID_P, (blk | kk) ? 1u : 0u);
                    }
                    tc_commit(&sh.p_full[0]);
                    TLW_END(5);
                    TL(4, cp, 2);
                }
                if (c >= 0 && ++k3 == 3) { k3 = 0; ph3 ^= 1; }
                if (c >= -2 && ++k3p == 3) k3p = 0;
            }
            TL_DUMP(0);
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
                TL(1, c, 0);
                WAITP(0, &sh.prep_ready[0], c & 1);
                WAITP(3, &sh.v_full[s], (c >> 1) & 1);
                if (c > 0) WAITP(1, &sh.o_free, (c - 1) & 1);
                TL(1, c, 1);
                tc_fence_after();
                {
                    TLW_BEGIN;
                    const uint64_t a = dv0 + (uint64_t)s * X_STEP;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_O, a + (uint64_t)(kk * 128), dp0 + (uint64_t)(2 * kk), ID_OV, kk ? 1u : 0u);
                    tc_commit(&sh.pt_free);       // P~ may be overwritten
                    TLW_END(4);
                    TL(1, c, 2);
                }
#pragma unroll 1
                for (int i = 0; i < 2; ++i) {
                    WAITP(2, &sh.sb_ready[i], c & 1);
                    TL(1, c, 3 + i);
                    tc_fence_after();
                    TLW_BEGIN;
                    const uint64_t dq = i == 0 ? dq1 + (uint64_t)k3 * KQ_STEP : dq2 + (uint64_t)s * X_STEP;
                    const uint32_t at = tb + COL_SB + 64 * i;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ts(tb + COL_O, at + 8 * kk, dq + (uint64_t)(2 * kk), ID_OS, 1);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ts(tb + COL_O, at + 32 + 8 * kk, dq + 512 + (uint64_t)(2 * kk), ID_OS, 1);
                    TLW_END(5);
                }
                tc_commit(&sh.o_full[0]);
                tc_commit(&sh.kq_empty[k3]);
                tc_commit(&sh.x_empty[s]);
                TL(1, c, 6);
                if (++k3 == 3) k3 = 0;
            }
            TL_DUMP(1);
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
            init_state_pass(slot1 + (size_t)half * state_stride, p.use_initial_state,
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
            if ((warp == 4 || warp == 6) && lane == 0) TL(warp == 4 ? 2 : 5, c, 0);
            {
                WAITP(2, &sh.m_ready[s], (c >> 1) & 1);
                WAITP(3, &sh.kq_full[k3], ph3);   // TMA writes of K, Q visible to this thread
                // P ready: the MMA is done reading raw Q, K.  The second issuer put P_c behind its wait for the MMAs of
                // chunk c - 2, so the K~2 / Q~2 buffer of this parity is free as well.
                WAITP(4, &sh.p_full[0], c & 1);
                tc_fence_after();
                if ((warp == 4 || warp == 6) && lane == 0) TL(warp == 4 ? 2 : 5, c, 1);
                TLT(tlm0);
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
                    if (c >= 1) WAITP(1, &sh.pt_free, (c - 1) & 1);     // the V part of chunk c - 1 has read P~
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
                TLT(tlm1); TLACC(8, tlm1 - tlm0);
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
                TLACC(9, clock64() - tlm1);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.prep_ready[0]); mbar_arrive(&sh.m_free[s]); }
                if ((warp == 4 || warp == 6) && lane == 0) TL(warp == 4 ? 2 : 5, c, 2);
            }
        }
        if (warp == 4 && lane == 0) TL_DUMP(2);
        if (warp == 6 && lane == 0) TL_DUMP(3);
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
        const float gam = p.gamma[h];
        const float W1 = gam * p.scale, W2 = (1.f - gam) * p.scale;
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
            TLT(tlg0);
            float l1a = warp_prefix_sum(lg2_gate(glo.x), lane), l2a = warp_prefix_sum(lg2_gate(glo.y), lane);
            float l1b = warp_prefix_sum(lg2_gate(ghi.x), lane), l2b = warp_prefix_sum(lg2_gate(ghi.y), lane);
            const float mid1 = __shfl_sync(0xffffffffu, l1a, 31), mid2 = __shfl_sync(0xffffffffu, l2a, 31);   // L at token 31
            l1b += mid1; l2b += mid2;
            const float end1 = __shfl_sync(0xffffffffu, l1b, 31), end2 = __shfl_sync(0xffffffffu, l2b, 31);   // L at token 63
            if (c >= 2) WAITP(0, &sh.m_free[s], ((c >> 1) - 1) & 1);
            if (warp == GATE_W0 && lane == 0) TL(0, c, 1);
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
            TLT(tlg1); TLACC(1, tlg1 - tlg0);
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
            TLACC(2, clock64() - tlg1);
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.m_ready[s]);
            if (warp == GATE_W0 && lane == 0) TL(0, c, 2);
        }
        if (warp == GATE_W0 && lane == 0) TL_DUMP(6);
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
            if (warp == 12 && lane == 0) TL(3, c, 0);
            if (c == 0) {
                // With programmatic dependent launch this grid may start while the summary grid is still running;
                // everything up to here (and all of chunk 0's operand work in the other warps) is independent of it.
                if (g > 0 && tp.ws) asm volatile("griddepcontrol.wait;" ::: "memory");
                init_state_pass(slot1 + (size_t)hi * state_stride, p.use_initial_state,
                                tp.ws ? tp.ws + ((size_t)(n * p.H + h) * tp.nseg) * (SUMMARY_STRIDE / 4) : nullptr, g, hi, v, a, s_addr, sb_addr,
                                0, init_shared ? 2 : 4);
                tc_wait_st();
                mbar_wait(&sh.init_done, 0, abortp, p.status);     // the other half (or nothing) from the tile warps
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.sb_ready[hi]); mbar_arrive(&sh.s_ready[hi]); }
#ifdef DSLA_TIMELINE
                if (warp == 12 && lane == 0 && g_timeline) g_timeline[3072 + 4 * blockIdx.x + 2] = gtime();
#endif
                a_next = warp_prod(gp_next);
                continue;
            }
            WAITP(0, &sh.u_full[hi], (c - 1) & 1);
            WAITP(1, &sh.o_full[0], (c - 1) & 1);   // the readout of chunk c-1 (other issuer) has read the bf16 copy
            tc_fence_after();
            if (warp == 12 && lane == 0) TL(3, c, 1);
            if (warp == 16 && lane == 0) TL(3, c, 4);
            TLT(tls0);
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
            if (warp == 12 && lane == 0) TL(3, c, 2);
            if (warp == 16 && lane == 0) TL(3, c, 5);
            TLT(tls1); TLACC(2, tls1 - tls0);
            outputs(c - 1);       // o_full of chunk c - 1 was awaited at the top of this iteration
            TLACC(3, clock64() - tls1);
            a_next = warp_prod(gp_next);
            if (warp == 12 && lane == 0) TL(3, c, 3);
            if (warp == 16 && lane == 0) TL(3, c, 6);
        }
        if (warp == 12 && lane == 0) TL_DUMP(4);
        if (warp == 16 && lane == 0) TL_DUMP(5);
        // ---- outputs of the last chunk, final states of this segment
        mbar_wait(&sh.o_full[0], (nc - 1) & 1, abortp, p.status);
        tc_fence_after();
        outputs(nc - 1);
        mbar_wait(&sh.u_full[hi], (nc - 1) & 1, abortp, p.status);
#ifdef DSLA_TIMELINE
        if (warp == 12 && lane == 0 && g_timeline) g_timeline[3072 + 4 * blockIdx.x + 3] = gtime();
#endif
        tc_fence_after();
        if (g == sq.last_seg) store_state(slot1 + (size_t)hi * state_stride, v, s_addr);
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 0) TL(0, 63, 7);
#ifdef DSLA_TIMELINE
    if (tid == 0 && g_timeline) g_timeline[3072 + 4 * blockIdx.x + 1] = gtime();
#endif
    if (warp == WARP_MMA) tmem_dealloc(tb, 512);
}

// ============================================================================================
// Segment summaries: U_g (both states, from zero) and A_g for every segment but a sequence's last.
// The chunks are walked from the END of the segment backwards while a running product R^i of all
// later gates is carried, so every token's weight prod_{t > s} g^i_t (to the end of the segment) is a
// plain product: no logarithms, no rescaling of the accumulator, and a zero gate is exact.
// A pure streaming pipeline, four chunks deep: warps 10, 11 derive the weights (one state each),
// warps 0..7 scale K into the two weighted copies, warp 8 drives TMA, warp 9 issues the MMAs.
// ============================================================================================
__global__ void __launch_bounds__(SUM_NTHREADS, 1)
prefill_tc_summary_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const TcParams tp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    __shared__ alignas(16) uint32_t wts[SUM_STAGES][2][C];     // per-token weights, bf16 in both halves
    __shared__ uint64_t w_ready[SUM_STAGES], w_free[SUM_STAGES], k_ready[SUM_STAGES];
    const PrefillParams& p = tp.p;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef DSLA_TIMELINE
    if (threadIdx.x == 0 && g_timeline) g_timeline[4096 + 4 * blockIdx.x] = gtime();
#endif
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the main grid may be scheduled as SMs become free
#ifdef DSLA_TIMELINE_SUMMARY
    long long* const tlp = (int)blockIdx.x == g_timeline_block ? g_timeline : nullptr;
#else
    long long* const tlp = nullptr; (void)tlp;
#endif
    const int nsum = tp.nseg - 1;
    const int g = blockIdx.x % nsum;
    const int h = (blockIdx.x / nsum) % p.H;
    const int rank = blockIdx.x / (nsum * p.H);
    const int n = tp.order ? tp.order[rank] : rank;
    const SeqInfo sq = seq_info(p, n, g, tp.nseg, tp.cps, tp.skew8);
    if (sq.slot < 0 || sq.slot >= p.num_slots) return;
    if (sq.len <= 0 || g >= sq.last_seg) return;      // only segments that have a successor
    const int nc = sq.c_end - sq.c_begin;             // full chunks only (not the sequence's last segment)
    const int t0 = sq.t_begin + sq.c_begin * C;
    float* out = tp.ws + ((size_t)(n * p.H + h) * tp.nseg + g) * (SUMMARY_STRIDE / 4);

    if (tid == 0) {
        for (int s = 0; s < SUM_STAGES; ++s) {
            mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1);
            mbar_init(&w_ready[s], 2); mbar_init(&w_free[s], 8); mbar_init(&k_ready[s], 8);
        }
        mbar_init(&sh.u_full[0], 1);
        sh.abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 9) { tmem_alloc(&sh.tmem_base, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = sh.tmem_base;
    volatile int* abortp = &sh.abort_flag;

    // iteration it = 0 .. nc-1 handles chunk nc-1-it; stage s = it % 4, use u = it / 4 of that stage
    if (warp == 8) {
        if (lane == 0) {
            prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
            for (int it = 0; it < nc; ++it) {
                const int s = it % SUM_STAGES, u = it / SUM_STAGES;
                TL(0, it, 0);
                if (u >= 1) mbar_wait(&sh.empty[s], (u - 1) & 1, abortp, p.status);
                TL(0, it, 1);
                uint8_t* st = tiles + s * SUM_STAGE_BYTES;
                const int t = t0 + (nc - 1 - it) * C;
                mbar_arrive_expect_tx(&sh.full[s], 4 * 8192);
                tma_load_4d(st, &map_k, &sh.full[s], 0, t, 0, h);
                tma_load_4d(st + SUM_OFF_V, &map_v, &sh.full[s], 0, t, 0, h);
                if (it + SUM_PREFETCH < nc) {   // pull a tile well ahead into L2: the four stages alone do not cover the HBM latency
                    const int tp2 = t - SUM_PREFETCH * C;
                    tma_prefetch_4d(&map_k, 0, tp2, 0, h);
                    tma_prefetch_4d(&map_v, 0, tp2, 0, h);
                }
            }
        }
    } else if (warp == 9) {
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_U = idesc_bf16(128, 256, 1, 1);
            for (int it = 0; it < nc; ++it) {
                const int s = it % SUM_STAGES, u = it / SUM_STAGES;
                TL(1, it, 0);
                mbar_wait(&k_ready[s], u & 1, abortp, p.status);
                TL(1, it, 1);
                tc_fence_after();
                const uint32_t st = sa + s * SUM_STAGE_BYTES;
                const uint64_t dv = smem_desc_sw128(st + SUM_OFF_V, 8192, 1024), dkk = smem_desc_sw128(st, 8192, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ss(tb, dv + (uint64_t)(kk * 128), dkk + (uint64_t)(kk * 128), ID_U, (it | kk) > 0);
                tc_commit(&sh.empty[s]);
                TL(1, it, 2);
                if (it == nc - 1) tc_commit(&sh.u_full[0]);
            }
        }
    } else if (warp >= 10) {
        // ---- weights: warp 10 the history state, warp 11 the recency state; lane l holds the adjacent tokens 2l and 2l + 1,
        // so one suffix scan over the 32 pair products gives every token's weight
        const int i = warp - 10;
        const float* gsrc = i == 0 ? p.g_hist : p.g_rec;
        float R = 1.f;                                 // product of the gates of all later chunks
        float n0 = load_gate(gsrc, t0 + (nc - 1) * C + 2 * lane, p.H, h, true);     // raw; clamped where it is used
        float n1 = load_gate(gsrc, t0 + (nc - 1) * C + 2 * lane + 1, p.H, h, true);
        for (int it = 0; it < nc; ++it) {
            const int s = it % SUM_STAGES, u = it / SUM_STAGES;
            const float g0 = fmaxf(n0, 0.f), g1 = fmaxf(n1, 0.f);
            if (it + 1 < nc) {
                const int t = t0 + (nc - 2 - it) * C + 2 * lane;
                n0 = load_gate(gsrc, t, p.H, h, true);      // consumed in the next iteration
                n1 = load_gate(gsrc, t + 1, p.H, h, true);
            }
            if (it + 1 + SUM_GATE_AHEAD < nc) {
                // One chunk of look-ahead does not cover the DRAM latency (this warp's iteration is shorter): pull the gates
                // of a chunk further ahead into L2 so that the load above becomes an L2 hit.
                const float* gp = gsrc + (size_t)(t0 + (nc - 2 - it - SUM_GATE_AHEAD) * C + 2 * lane) * p.H + h;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(gp));
                asm volatile("prefetch.global.L2 [%0];" ::"l"(gp + p.H));
            }
            const float sfx = warp_suffix_prod(g0 * g1, lane);        // product of the gates of tokens >= 2l
            const float tot = __shfl_sync(0xffffffffu, sfx, 0);
            float ex = __shfl_down_sync(0xffffffffu, sfx, 1);         // ... of tokens > 2l + 1
            if (lane == 31) ex = 1.f;
            ex *= R;
            if (warp == 10 && lane == 0) TL(3, it, 0);
            if (u >= 1) mbar_wait(&w_free[s], (u - 1) & 1, abortp, p.status);
            if (warp == 10 && lane == 0) TL(3, it, 1);
            *reinterpret_cast<uint2*>(&wts[s][i][2 * lane]) = make_uint2(dup_bf16(g1 * ex), dup_bf16(ex));
            R *= tot;
            __syncwarp();
            if (lane == 0) mbar_arrive(&w_ready[s]);
            if (warp == 10 && lane == 0) TL(3, it, 2);
        }
        if (lane == 0) out[2 * D * D + i] = R;         // A_g: product of every gate of the segment
    } else {
        // ---- K~1 (in place) and K~2: four 16-byte pieces per thread and chunk
        const int q = warp & 3, hi = warp >> 2;
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        for (int it = 0; it < nc; ++it) {
            const int s = it % SUM_STAGES, u = it / SUM_STAGES;
            uint8_t* st = tiles + s * SUM_STAGE_BYTES;
            if (tid == 0) TL(2, it, 0);
            mbar_wait(&w_ready[s], u & 1, abortp, p.status);
            if (tid == 0) TL(2, it, 1);
            mbar_wait(&sh.full[s], u & 1, abortp, p.status);
            if (tid == 0) TL(2, it, 2);
#ifdef DSLA_TIMELINE
            if (tid == 0 && it == 0 && g_timeline) g_timeline[4096 + 4 * blockIdx.x + 2] = gtime();
#endif
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const int idx = tid + SUM_NCOMPUTE * m;
                const int row = (idx >> 3) & 63;
                uint4* kp = reinterpret_cast<uint4*>(st) + idx;
                const uint4 xk = *kp;
                const uint32_t w0 = wts[s][0][row], w1 = wts[s][1][row];
                *kp = scale8(xk, w0);
                *(kp + 1024) = scale8(xk, w1);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) { mbar_arrive(&k_ready[s]); mbar_arrive(&w_free[s]); }
            if (tid == 0) TL(2, it, 3);
        }
        mbar_wait(&sh.u_full[0], 0, abortp, p.status);
#ifdef DSLA_TIMELINE
        if (tid == 0 && g_timeline) g_timeline[4096 + 4 * blockIdx.x + 3] = gtime();
#endif
        tc_fence_after();
        store_state(out + (size_t)hi * D * D, 32 * q + lane, lane_addr + 128 * hi);
    }
    tc_fence_before();
    __syncthreads();
#ifdef DSLA_TIMELINE
    if (tid == 0 && g_timeline) g_timeline[4096 + 4 * blockIdx.x + 1] = gtime();
#endif
    if (warp == 9) tmem_dealloc(tb, 256);
}

// ---- host side -------------------------------------------------------------------------------
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
    static EncodeFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        cudaDriverEntryPointQueryResult qr;
        void* ptr = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(ptr);
        (void)cudaGetLastError();
    }
    return fn;
}

// Tensor [T_total][H][128] bf16 viewed as (d, H, T); a box is 64 d-elements (128 B) x 1 head x 64 tokens.
// [T_total, H, 128] bf16 seen as (x: 64 elements, t, half: the two 64-element halves of a row, h) so that one
// copy of box {64, 64 tokens, 2, 1} lands as two consecutive 8 KB tiles [half][token][64], each in the 128-byte
// swizzle the MMA descriptors expect.
bool make_map(CUtensorMap* m, const void* base, int T_total, int H) {
    EncodeFn fn = get_encode();
    if (!fn) return false;
    cuuint64_t dims[4] = {64, (cuuint64_t)T_total, 2, (cuuint64_t)H};
    cuuint64_t strides[3] = {(cuuint64_t)H * D * 2, 128, (cuuint64_t)D * 2};
    cuuint32_t box[4] = {64, 64, 2, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Segments per sequence: enough CTAs to cover the SMs when there are few (sequence, head) pairs,
// never shorter than 4 chunks per segment.
// Ragged batches: blocks are handed to the SMs in index order, so sequences are visited longest first (a long
// sequence that starts late would otherwise run on alone at the end).  order[r] = index of the r-th longest
// sequence, ties by index; one thread per sequence counts how many sequences come before its own.
constexpr int ORDER_MAX_N = 8192;
__global__ void seq_order_kernel(const int32_t* __restrict__ cu, int N, int* __restrict__ order) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int len_i = cu[i + 1] - cu[i];
    int before = 0;
    int prev = __ldg(cu);
    for (int j = 0; j < N; ++j) {
        const int next = __ldg(cu + j + 1);
        const int len_j = next - prev;
        prev = next;
        before += (len_j > len_i || (len_j == len_i && j < i)) ? 1 : 0;
    }
    order[before] = i;
}

bool wants_order(const dsla_prefill_args* a) { return a->cu_seqlens != nullptr && a->N > 1 && a->N <= ORDER_MAX_N; }

void plan(const dsla_prefill_args* a, int* nseg, int* cps, int* skew8) {
    const int max_chunks = (a->max_seqlen + C - 1) / C;
    const long long units = (long long)a->N * a->H;
    int ns = 1;
    if (units > 0 && units < 148) ns = (int)(148 / units);
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

}  // namespace

#ifdef DSLA_TIMELINE
extern "C" int dsla_debug_set_timeline(long long* dev_ptr, int block) {
    cudaMemcpyToSymbol(g_timeline_block, &block, sizeof(block));
    return (int)cudaMemcpyToSymbol(g_timeline, &dev_ptr, sizeof(dev_ptr));
}
#endif

bool prefill_tc_available() { return true; }

size_t prefill_tc_workspace_bytes(const dsla_prefill_args* a) {
    int nseg, cps, skew8;
    plan(a, &nseg, &cps, &skew8);
    const size_t summaries = nseg > 1 ? (size_t)a->N * a->H * nseg * SUMMARY_STRIDE : 0;     // a multiple of 256
    const size_t order = wants_order(a) ? (((size_t)a->N * sizeof(int) + 255) & ~(size_t)255) : 0;
    return summaries + order;
}

dsla_status launch_prefill_tc(const PrefillParams& p, const dsla_prefill_args* a, cudaStream_t s) {
    if (p.N == 0 || a->T_total == 0) {
        // only empty sequences: the CUDA-core kernel handles the slot bookkeeping
        return launch_prefill_simt(p, D, C, DSLA_BF16, s);
    }
    TcParams tp;
    tp.p = p;
    plan(a, &tp.nseg, &tp.cps, &tp.skew8);
    tp.ws = tp.nseg > 1 ? static_cast<float*>(a->workspace) : nullptr;
    tp.order = nullptr;
    if (wants_order(a)) {
        const size_t summaries = tp.nseg > 1 ? (size_t)a->N * a->H * tp.nseg * SUMMARY_STRIDE : 0;
        int* order = reinterpret_cast<int*>(static_cast<char*>(a->workspace) + summaries);
        seq_order_kernel<<<dim3((unsigned)((p.N + 255) / 256)), dim3(256), 0, s>>>(p.cu_seqlens, p.N, order);
        count_launch();
        tp.order = order;
    }
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, p.q, a->T_total, p.H) || !make_map(&mk, p.k, a->T_total, p.H) || !make_map(&mv, p.v, a->T_total, p.H))
        return DSLA_ERR_CUDA;
    if (cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN) != cudaSuccess ||
        cudaFuncSetAttribute(prefill_tc_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SUM_SMEM_DYN) != cudaSuccess)
        return DSLA_ERR_CUDA;
    const long long units = (long long)p.N * p.H;
    if (units * tp.nseg > 0x7fffffffLL) return DSLA_ERR_UNSUPPORTED;
    if (tp.nseg > 1) {
        prefill_tc_summary_kernel<<<dim3((unsigned)(units * (tp.nseg - 1))), dim3(SUM_NTHREADS), SUM_SMEM_DYN, s>>>(mk, mv, tp);
        count_launch();
    }
    {
        // Programmatic dependent launch after the summary grid: the main grid's prologue and the first chunk's
        // operand work overlap the summary grid's tail; the state warps wait for it before they read the summaries.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(units * tp.nseg));
        cfg.blockDim = dim3(NTHREADS);
        cfg.dynamicSmemBytes = SMEM_DYN;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = tp.nseg > 1 ? 1 : 0;
        if (cudaLaunchKernelEx(&cfg, prefill_tc_kernel, mq, mk, mv, tp) != cudaSuccess) return DSLA_ERR_CUDA;
    }
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // namespace dsla
