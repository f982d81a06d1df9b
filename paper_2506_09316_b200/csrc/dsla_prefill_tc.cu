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
// TMEM is the A operand of the readout.  TMA stages Q/K/V tiles (128-byte swizzle, 2 stages).
//
// A sequence may be split into `nseg` segments along T so that few (sequence, head) pairs still
// fill the GPU: a first kernel computes each segment's state summary from zero
// (U_g = sum_s (prod of later gates in the segment) k_s^T v_s and A_g = prod of the segment's
// gates) into the workspace; the main kernel combines the summaries of earlier segments into its
// initial state and then runs its segment.
#include "dsla_internal.cuh"
#include "tc_utils.cuh"

namespace dsla {

using namespace tc;

namespace {

constexpr int C = 64;                 // tokens per chunk
constexpr int D = 128;                // head size
constexpr int NCOMPUTE = 256;         // warps 0-7
constexpr int WARP_TMA = 8, WARP_MMA = 9;
constexpr int NTHREADS = 320;
constexpr int STAGE_BYTES = 5 * 16384;   // [K/K~1][K~2][Q/Q~1][Q~2][V]
constexpr int OFF_K = 0, OFF_Q = 32768, OFF_V = 65536;
constexpr int OFF_PT = 2 * STAGE_BYTES;  // P~ double buffer, 8 KB each
constexpr int SMEM_TILES = 2 * STAGE_BYTES + 2 * 8192;
constexpr int SMEM_DYN = SMEM_TILES + 1024;  // + alignment slack
// TMEM columns
constexpr uint32_t COL_S = 0;      // fp32 S1^T [0,128), S2^T [128,256)
constexpr uint32_t COL_SB = 256;   // bf16 copies: S1^T [256,320), S2^T [320,384)
constexpr uint32_t COL_O = 384;    // O^T, 64 columns (tokens)
constexpr uint32_t COL_P = 448;    // P, 64 columns (lanes 0..63 meaningful)
constexpr size_t SUMMARY_STRIDE = 2 * D * D * sizeof(float) + 256;  // U (both states) + A[2], padded

struct TcParams {
    PrefillParams p;
    float* ws;          // summaries: [(n*H + h)*nseg + g] -> {U[2][D][D], A[2]}
    int nseg;           // segments per sequence (grid dimension)
    int cps;            // chunks per segment
};

struct GateSmem {
    float b[2][C];      // cumulative log-gate inside the chunk (zero gates skipped)
    int zc[2][C];       // zero-gate count, inclusive
    float rowf[2][C];   // weight_i * e^{b_j}, 0 behind a zero gate
    float w[2][C];      // e^{b_last - b_s} (main) or decay to the end of the segment (summary)
    float a[2];         // chunk decay
    float pad[2];
};

struct Shared {
    uint64_t full[2], empty[2], p_full, p_free, ready, o_full, o_free, u_full;
    uint32_t tmem_base;
    int abort_flag;
    GateSmem gs[2];
    double red_b[2][8];
    int red_z[2][8];
};

// Inclusive scan of log-gates over one chunk by warps 0 (history) and 1 (recency); each lane owns two
// consecutive tokens whose gate values (`g0`, `g1`) were fetched earlier.
__device__ __forceinline__ void gate_scan(GateSmem& gs, int i, int lane, float g0, float g1) {
    const bool z0 = !(g0 > 0.f), z1 = !(g1 > 0.f);
    const double l0 = z0 ? 0.0 : (double)__logf(g0), l1 = z1 ? 0.0 : (double)__logf(g1);
    double run = l0 + l1;
    int zrun = (int)z0 + (int)z1;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, run, off);
        const int zup = __shfl_up_sync(0xffffffffu, zrun, off);
        if (lane >= off) { run += up; zrun += zup; }
    }
    const double excl = run - (l0 + l1);
    const int zexcl = zrun - ((int)z0 + (int)z1);
    gs.b[i][2 * lane] = (float)(excl + l0);
    gs.b[i][2 * lane + 1] = (float)run;
    gs.zc[i][2 * lane] = zexcl + (int)z0;
    gs.zc[i][2 * lane + 1] = zrun;
}

__device__ __forceinline__ float load_gate(const float* g, int t, int H, int h, bool ok) {
    return ok ? __ldg(g + (size_t)t * H + h) : 1.f;
}

// Multiplies the eight bf16 of a 16-byte chunk by f.
__device__ __forceinline__ uint4 scale8(const uint4 x, float f) {
    uint4 y;
    const uint32_t* xi = reinterpret_cast<const uint32_t*>(&x);
    uint32_t* yi = reinterpret_cast<uint32_t*>(&y);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162*>(&xi[e]);
        yi[e] = pack_bf16(__low2float(v) * f, __high2float(v) * f);
    }
    return y;
}

struct SeqInfo {
    int t_begin, len, slot, nchunks, c_begin, c_end, last_seg;
};

__device__ __forceinline__ SeqInfo seq_info(const PrefillParams& p, int n, int g, int cps) {
    SeqInfo s;
    s.t_begin = p.cu_seqlens ? p.cu_seqlens[n] : n * p.T;
    const int t_end = p.cu_seqlens ? p.cu_seqlens[n + 1] : (n + 1) * p.T;
    s.len = t_end - s.t_begin;
    s.slot = p.slots ? p.slots[n] : n;
    s.nchunks = (s.len + C - 1) / C;
    s.c_begin = g * cps;
    s.c_end = min(s.nchunks, (g + 1) * cps);
    s.last_seg = s.nchunks > 0 ? (s.nchunks - 1) / cps : 0;
    return s;
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
    const int g = blockIdx.x % tp.nseg;
    const int h = (blockIdx.x / tp.nseg) % p.H;
    const int n = blockIdx.x / (tp.nseg * p.H);
    const SeqInfo sq = seq_info(p, n, g, tp.cps);
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

    if (tid == 0) {
        mbar_init(&sh.full[0], 1); mbar_init(&sh.full[1], 1);
        mbar_init(&sh.empty[0], 1); mbar_init(&sh.empty[1], 1);
        mbar_init(&sh.p_full, 1); mbar_init(&sh.p_free, 4);
        mbar_init(&sh.ready, 8); mbar_init(&sh.o_full, 1); mbar_init(&sh.o_free, 8); mbar_init(&sh.u_full, 1);
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
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
            for (int c = 0; c < nc; ++c) {
                const int s = c & 1;
                if (c >= 2) mbar_wait(&sh.empty[s], ((c >> 1) & 1) ^ 1, abortp, p.status);
                uint8_t* st = tiles + s * STAGE_BYTES;
                const int t = t0 + c * C;
                mbar_arrive_expect_tx(&sh.full[s], 6 * 8192);
                tma_load_3d(st + OFF_Q, &map_q, &sh.full[s], 0, h, t);
                tma_load_3d(st + OFF_Q + 8192, &map_q, &sh.full[s], 64, h, t);
                tma_load_3d(st + OFF_K, &map_k, &sh.full[s], 0, h, t);
                tma_load_3d(st + OFF_K + 8192, &map_k, &sh.full[s], 64, h, t);
                tma_load_3d(st + OFF_V, &map_v, &sh.full[s], 0, h, t);
                tma_load_3d(st + OFF_V + 8192, &map_v, &sh.full[s], 64, h, t);
            }
        }
    } else if (warp == WARP_MMA) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_P = idesc_bf16(128, 64, 0, 0);
            constexpr uint32_t ID_OS = idesc_bf16(128, 64, 0, 0);
            constexpr uint32_t ID_OV = idesc_bf16(128, 64, 1, 0);
            constexpr uint32_t ID_U = idesc_bf16(128, 256, 1, 1);
            auto issue_p = [&](int c) {
                const uint32_t st = sa + (c & 1) * STAGE_BYTES;
                const uint64_t dq = smem_desc_sw128(st + OFF_Q, 16, 1024), dk = smem_desc_sw128(st + OFF_K, 16, 1024);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * 8192 + (kk & 3) * 32) >> 4);
                    mma_ss(tb + COL_P, dq + off, dk + off, ID_P, kk > 0);
                }
                tc_commit(&sh.p_full);
            };
            mbar_wait(&sh.full[0], 0, abortp, p.status);
            tc_fence_after();
            issue_p(0);
            for (int c = 0; c < nc; ++c) {
                const int s = c & 1;
                if (c + 1 < nc) {
                    mbar_wait(&sh.full[(c + 1) & 1], ((c + 1) >> 1) & 1, abortp, p.status);
                    mbar_wait(&sh.p_free, c & 1, abortp, p.status);
                    tc_fence_after();
                    issue_p(c + 1);
                }
                mbar_wait(&sh.ready, c & 1, abortp, p.status);
                if (c > 0) mbar_wait(&sh.o_free, (c - 1) & 1, abortp, p.status);
                tc_fence_after();
                const uint32_t st = sa + s * STAGE_BYTES;
                // O^T = S1^T Q~1^T + S2^T Q~2^T + V^T P~^T
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const uint64_t dq = smem_desc_sw128(st + OFF_Q + i * 16384, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint64_t off = (uint64_t)(((kk >> 2) * 8192 + (kk & 3) * 32) >> 4);
                        mma_ts(tb + COL_O, tb + COL_SB + 64 * i + 8 * kk, dq + off, ID_OS, (i | kk) > 0);
                    }
                }
                const uint64_t dv = smem_desc_sw128(st + OFF_V, 8192, 1024);
                const uint64_t dp = smem_desc_sw128(sa + OFF_PT + s * 8192, 16, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_O, dv + (uint64_t)(kk * 128), dp + (uint64_t)(kk * 2), ID_OV, 1);
                tc_commit(&sh.o_full);
                // S^T += V^T [K~1 | K~2]
                const uint64_t dkk = smem_desc_sw128(st + OFF_K, 8192, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ss(tb + COL_S, dv + (uint64_t)(kk * 128), dkk + (uint64_t)(kk * 128), ID_U, 1);
                tc_commit(&sh.u_full);
                tc_commit(&sh.empty[s]);
            }
        }
    } else {
        // ------------------------------------------------------------------ compute warps 0..7
        const int q = warp & 3, hi = warp >> 2;          // TMEM lane quadrant, column half / state index
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        const float gam = p.gamma[h];
        const float W1 = gam * p.scale, W2 = (1.f - gam) * p.scale;
        __nv_bfloat16* og = reinterpret_cast<__nv_bfloat16*>(p.o);
        // gate prefetch registers (warps 0, 1 only): two tokens per lane
        const float* gsrc = warp == 0 ? p.g_hist : p.g_rec;
        float g0 = 1.f, g1 = 1.f;
        if (warp < 2) {
            const int j = 2 * lane;
            g0 = load_gate(gsrc, t0 + j, p.H, h, sq.c_begin * C + j < sq.len);
            g1 = load_gate(gsrc, t0 + j + 1, p.H, h, sq.c_begin * C + j + 1 < sq.len);
        }
        for (int c = 0; c <= nc; ++c) {
            const int s = c & 1;
            GateSmem& gs = sh.gs[s];
            uint8_t* st = tiles + s * STAGE_BYTES;
            if (c < nc) {
                // ---- a. gates of this chunk; prefetch the next chunk's
                if (warp < 2) {
                    gate_scan(gs, warp, lane, g0, g1);
                    const int j = (c + 1) * C + 2 * lane;
                    const bool more = c + 1 < nc;
                    g0 = load_gate(gsrc, t0 + j, p.H, h, more && sq.c_begin * C + j < sq.len);
                    g1 = load_gate(gsrc, t0 + j + 1, p.H, h, more && sq.c_begin * C + j + 1 < sq.len);
                }
                named_bar_sync(1, NCOMPUTE);
                if (tid < 2 * C) {
                    const int i = tid / C, j = tid % C;
                    const float bl = gs.b[i][C - 1], b = gs.b[i][j];
                    const int zl = gs.zc[i][C - 1], z = gs.zc[i][j];
                    const int valid = min(C, sq.len - (sq.c_begin + c) * C);
                    gs.rowf[i][j] = z == 0 ? (i == 0 ? W1 : W2) * __expf(b) : 0.f;
                    gs.w[i][j] = (j < valid && z == zl) ? __expf(bl - b) : 0.f;   // rows past the sequence end carry no weight
                    if (j == 0) gs.a[i] = zl == 0 ? __expf(bl) : 0.f;
                }
                named_bar_sync(1, NCOMPUTE);
                // ---- b. mask (warps 0,1,4,5) and operand scaling (warps 2,3,6,7)
                mbar_wait(&sh.full[s], (c >> 1) & 1, abortp, p.status);
                mbar_wait(&sh.p_full, c & 1, abortp, p.status);
                tc_fence_after();
                if (q < 2) {
                    const int j = 32 * q + lane;
                    uint8_t* pt = tiles + OFF_PT + s * 8192;
                    uint32_t r[32];
                    const bool any = 32 * hi <= 32 * q + 31;     // column block not entirely above the diagonal
                    if (any) { tmem_ld32(lane_addr + COL_P + 32 * hi, r); tc_wait_ld(); }
                    __syncwarp();
                    if (lane == 0) { tc_fence_before(); mbar_arrive(&sh.p_free); }
                    const float b1 = gs.b[0][j], b2 = gs.b[1][j];
                    const int z1 = gs.zc[0][j], z2 = gs.zc[1][j];
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        uint32_t pk[4];
#pragma unroll
                        for (int e = 0; e < 8; e += 2) {
                            float val[2];
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const int sc = 32 * hi + 8 * m + e + u;
                                float mk = 0.f;
                                if (any && sc <= j) {
                                    const float d1 = gs.zc[0][sc] == z1 ? __expf(b1 - gs.b[0][sc]) : 0.f;
                                    const float d2 = gs.zc[1][sc] == z2 ? __expf(b2 - gs.b[1][sc]) : 0.f;
                                    mk = W1 * d1 + W2 * d2;
                                }
                                val[u] = (any && sc <= j) ? __uint_as_float(r[8 * m + e + u]) * mk : 0.f;
                            }
                            pk[e >> 1] = pack_bf16(val[0], val[1]);
                        }
                        *reinterpret_cast<uint4*>(pt + sw128_offset(j, 32 * hi + 8 * m)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                } else {
                    const int pt_id = (q - 2) * 32 + lane + 64 * hi;   // 0..127
#pragma unroll 4
                    for (int m = 0; m < 8; ++m) {
                        const int idx = pt_id + 128 * m;               // 16-byte chunk inside a 16 KB tile
                        const int row = (idx >> 3) & 63;
                        uint4* qp = reinterpret_cast<uint4*>(st + OFF_Q) + idx;
                        uint4* kp = reinterpret_cast<uint4*>(st + OFF_K) + idx;
                        const uint4 xq = *qp, xk = *kp;
                        *qp = scale8(xq, gs.rowf[0][row]);
                        *(qp + 1024) = scale8(xq, gs.rowf[1][row]);
                        *kp = scale8(xk, gs.w[0][row]);
                        *(kp + 1024) = scale8(xk, gs.w[1][row]);
                    }
                }
                fence_proxy_async_smem();
            }
            // ---- c. outputs of the previous chunk
            if (c > 0) {
                const int cp = c - 1;
                mbar_wait(&sh.o_full, cp & 1, abortp, p.status);
                tc_fence_after();
                uint32_t r[32];
                tmem_ld32(lane_addr + COL_O + 32 * hi, r);
                tc_wait_ld();
                __syncwarp();
                if (lane == 0) { tc_fence_before(); mbar_arrive(&sh.o_free); }
                const int valid = min(C, sq.len - (sq.c_begin + cp) * C);
                __nv_bfloat16* orow = og + ((size_t)(t0 + cp * C + 32 * hi) * p.H + h) * D + 32 * q + lane;
#pragma unroll
                for (int jj = 0; jj < 32; ++jj)
                    if (32 * hi + jj < valid) orow[(size_t)jj * p.H * D] = __float2bfloat16_rn(__uint_as_float(r[jj]));
            }
            if (c == nc) break;
            // ---- d. state pass: bf16 copy of S_c for the readout, then S <- a_c S for the update
            {
                const float a = gs.a[hi];
                const uint32_t s_addr = lane_addr + COL_S + 128 * hi;
                const uint32_t sb_addr = lane_addr + COL_SB + 64 * hi;
                const int v = 32 * q + lane;
                if (c == 0) {
                    // initial state of this segment: slot contents (or zero) pushed through the summaries of
                    // the earlier segments, S <- A_j S + U_j
                    const float* base = slot1 + (size_t)hi * state_stride;
                    const float* wsu = tp.ws ? tp.ws + ((size_t)(n * p.H + h) * tp.nseg) * (SUMMARY_STRIDE / 4) : nullptr;
#pragma unroll 1
                    for (int bt = 0; bt < 4; ++bt) {
                        float acc[32];
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            acc[k] = p.use_initial_state ? base[(size_t)(32 * bt + k) * D + v] : 0.f;
                        for (int jg = 0; jg < g; ++jg) {
                            const float* u = wsu + (size_t)jg * (SUMMARY_STRIDE / 4);
                            const float A = u[2 * D * D + hi];
                            const float* uu = u + (size_t)hi * D * D;
#pragma unroll
                            for (int k = 0; k < 32; ++k) acc[k] = fmaf(A, acc[k], uu[(size_t)(32 * bt + k) * D + v]);
                        }
                        uint32_t pk[16], sc[32];
#pragma unroll
                        for (int k = 0; k < 16; ++k) pk[k] = pack_bf16(acc[2 * k], acc[2 * k + 1]);
#pragma unroll
                        for (int k = 0; k < 32; ++k) sc[k] = __float_as_uint(acc[k] * a);
                        tmem_st16(sb_addr + 16 * bt, pk);
                        tmem_st32(s_addr + 32 * bt, sc);
                    }
                } else {
                    mbar_wait(&sh.u_full, (c - 1) & 1, abortp, p.status);
                    tc_fence_after();
                    uint32_t r[2][32];
                    tmem_ld32(s_addr, r[0]);
#pragma unroll
                    for (int bt = 0; bt < 4; ++bt) {
                        tc_wait_ld();
                        if (bt + 1 < 4) tmem_ld32(s_addr + 32 * (bt + 1), r[(bt + 1) & 1]);
                        uint32_t (&x)[32] = r[bt & 1];
                        uint32_t pk[16];
#pragma unroll
                        for (int k = 0; k < 16; ++k) pk[k] = pack_bf16(__uint_as_float(x[2 * k]), __uint_as_float(x[2 * k + 1]));
                        tmem_st16(sb_addr + 16 * bt, pk);
#pragma unroll
                        for (int k = 0; k < 32; ++k) x[k] = __float_as_uint(__uint_as_float(x[k]) * a);
                        tmem_st32(s_addr + 32 * bt, x);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.ready);
            }
        }
        // ---- final states of this segment's last chunk
        mbar_wait(&sh.u_full, (nc - 1) & 1, abortp, p.status);
        tc_fence_after();
        if (g == sq.last_seg) {
            float* dst = slot1 + (size_t)hi * state_stride;
            const int v = 32 * q + lane;
#pragma unroll 1
            for (int bt = 0; bt < 4; ++bt) {
                uint32_t r[32];
                tmem_ld32(lane_addr + COL_S + 128 * hi + 32 * bt, r);
                tc_wait_ld();
#pragma unroll
                for (int k = 0; k < 32; ++k) dst[(size_t)(32 * bt + k) * D + v] = __uint_as_float(r[k]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == WARP_MMA) tmem_dealloc(tb, 512);
}

// ============================================================================================
// Segment summaries: U_g (both states, from zero) and A_g for every segment but a sequence's last.
// Weights are taken relative to the END of the segment, so the MMAs accumulate over the whole
// segment without any rescaling pass.
// ============================================================================================
__global__ void __launch_bounds__(NTHREADS, 1)
prefill_tc_summary_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const TcParams tp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ Shared sh;
    const PrefillParams& p = tp.p;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nsum = tp.nseg - 1;
    const int g = blockIdx.x % nsum;
    const int h = (blockIdx.x / nsum) % p.H;
    const int n = blockIdx.x / (nsum * p.H);
    const SeqInfo sq = seq_info(p, n, g, tp.cps);
    if (sq.slot < 0 || sq.slot >= p.num_slots) return;
    if (sq.len <= 0 || g >= sq.last_seg) return;      // only segments that have a successor
    const int nc = sq.c_end - sq.c_begin;             // full chunks only (not the sequence's last segment)
    const int t0 = sq.t_begin + sq.c_begin * C;
    float* out = tp.ws + ((size_t)(n * p.H + h) * tp.nseg + g) * (SUMMARY_STRIDE / 4);

    if (tid == 0) {
        mbar_init(&sh.full[0], 1); mbar_init(&sh.full[1], 1);
        mbar_init(&sh.empty[0], 1); mbar_init(&sh.empty[1], 1);
        mbar_init(&sh.ready, 8); mbar_init(&sh.u_full, 1);
        sh.abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == WARP_MMA) { tmem_alloc(&sh.tmem_base, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = sh.tmem_base;
    volatile int* abortp = &sh.abort_flag;

    if (warp == WARP_TMA) {
        if (lane == 0) {
            prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
            for (int c = 0; c < nc; ++c) {
                const int s = c & 1;
                if (c >= 2) mbar_wait(&sh.empty[s], ((c >> 1) & 1) ^ 1, abortp, p.status);
                uint8_t* st = tiles + s * STAGE_BYTES;
                const int t = t0 + c * C;
                mbar_arrive_expect_tx(&sh.full[s], 4 * 8192);
                tma_load_3d(st + OFF_K, &map_k, &sh.full[s], 0, h, t);
                tma_load_3d(st + OFF_K + 8192, &map_k, &sh.full[s], 64, h, t);
                tma_load_3d(st + OFF_V, &map_v, &sh.full[s], 0, h, t);
                tma_load_3d(st + OFF_V + 8192, &map_v, &sh.full[s], 64, h, t);
            }
        }
    } else if (warp == WARP_MMA) {
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_U = idesc_bf16(128, 256, 1, 1);
            for (int c = 0; c < nc; ++c) {
                const int s = c & 1;
                mbar_wait(&sh.ready, c & 1, abortp, p.status);
                tc_fence_after();
                const uint32_t st = sa + s * STAGE_BYTES;
                const uint64_t dv = smem_desc_sw128(st + OFF_V, 8192, 1024), dkk = smem_desc_sw128(st + OFF_K, 8192, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ss(tb, dv + (uint64_t)(kk * 128), dkk + (uint64_t)(kk * 128), ID_U, (c | kk) > 0);
                tc_commit(&sh.empty[s]);
                if (c == nc - 1) tc_commit(&sh.u_full);
            }
        }
    } else {
        const int q = warp & 3, hi = warp >> 2;
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        // ---- total log-decay and zero-gate count of the whole segment (fp64 sums)
        double tot[2] = {0.0, 0.0};
        int ztot[2] = {0, 0};
        {
            const int ntok = nc * C;
            for (int j = tid; j < ntok; j += NCOMPUTE) {
                const float a = __ldg(p.g_hist + (size_t)(t0 + j) * p.H + h), b = __ldg(p.g_rec + (size_t)(t0 + j) * p.H + h);
                if (a > 0.f) tot[0] += (double)__logf(a); else ztot[0]++;
                if (b > 0.f) tot[1] += (double)__logf(b); else ztot[1]++;
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    tot[i] += __shfl_xor_sync(0xffffffffu, tot[i], off);
                    ztot[i] += __shfl_xor_sync(0xffffffffu, ztot[i], off);
                }
                if (lane == 0) { sh.red_b[i][warp] = tot[i]; sh.red_z[i][warp] = ztot[i]; }
            }
            named_bar_sync(1, NCOMPUTE);
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                tot[i] = 0.0; ztot[i] = 0;
                for (int w8 = 0; w8 < 8; ++w8) { tot[i] += sh.red_b[i][w8]; ztot[i] += sh.red_z[i][w8]; }
            }
        }
        double pre[2] = {0.0, 0.0};   // log-decay of the chunks already processed
        int zpre[2] = {0, 0};
        const float* gsrc = warp == 0 ? p.g_hist : p.g_rec;
        float g0 = 1.f, g1 = 1.f;
        if (warp < 2) {
            g0 = load_gate(gsrc, t0 + 2 * lane, p.H, h, true);
            g1 = load_gate(gsrc, t0 + 2 * lane + 1, p.H, h, true);
        }
        for (int c = 0; c < nc; ++c) {
            const int s = c & 1;
            GateSmem& gs = sh.gs[s];
            uint8_t* st = tiles + s * STAGE_BYTES;
            if (warp < 2) {
                gate_scan(gs, warp, lane, g0, g1);
                const bool more = c + 1 < nc;
                const int j = (c + 1) * C + 2 * lane;
                g0 = load_gate(gsrc, t0 + j, p.H, h, more);
                g1 = load_gate(gsrc, t0 + j + 1, p.H, h, more);
            }
            named_bar_sync(1, NCOMPUTE);
            if (tid < 2 * C) {
                const int i = tid / C, j = tid % C;
                const bool open = (ztot[i] - zpre[i] - gs.zc[i][j]) == 0;   // no zero gate after token j
                gs.w[i][j] = open ? __expf((float)(tot[i] - pre[i] - (double)gs.b[i][j])) : 0.f;
            }
            named_bar_sync(1, NCOMPUTE);
#pragma unroll
            for (int i = 0; i < 2; ++i) { pre[i] += (double)gs.b[i][C - 1]; zpre[i] += gs.zc[i][C - 1]; }
            mbar_wait(&sh.full[s], (c >> 1) & 1, abortp, p.status);
#pragma unroll 4
            for (int m = 0; m < 4; ++m) {
                const int idx = tid + NCOMPUTE * m;
                const int row = (idx >> 3) & 63;
                uint4* kp = reinterpret_cast<uint4*>(st + OFF_K) + idx;
                const uint4 xk = *kp;
                *kp = scale8(xk, gs.w[0][row]);
                *(kp + 1024) = scale8(xk, gs.w[1][row]);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.ready);
        }
        mbar_wait(&sh.u_full, 0, abortp, p.status);
        tc_fence_after();
        {
            float* dst = out + (size_t)hi * D * D;
            const int v = 32 * q + lane;
#pragma unroll 1
            for (int bt = 0; bt < 4; ++bt) {
                uint32_t r[32];
                tmem_ld32(lane_addr + 128 * hi + 32 * bt, r);
                tc_wait_ld();
#pragma unroll
                for (int k = 0; k < 32; ++k) dst[(size_t)(32 * bt + k) * D + v] = __uint_as_float(r[k]);
            }
            if (tid < 2) out[2 * D * D + tid] = ztot[tid] == 0 ? __expf((float)tot[tid]) : 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == WARP_MMA) tmem_dealloc(tb, 256);
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
bool make_map(CUtensorMap* m, const void* base, int T_total, int H) {
    EncodeFn fn = get_encode();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)T_total};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2};
    cuuint32_t box[3] = {64, 1, 64};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Segments per sequence: enough CTAs to cover the SMs when there are few (sequence, head) pairs,
// never shorter than 4 chunks per segment.
void plan(const dsla_prefill_args* a, int* nseg, int* cps) {
    const int max_chunks = (a->max_seqlen + C - 1) / C;
    const long long units = (long long)a->N * a->H;
    int ns = 1;
    if (units > 0 && units < 148) ns = (int)(148 / units);
    if (ns > 16) ns = 16;
    while (ns > 1 && (max_chunks + ns - 1) / ns < 4) --ns;
    if (max_chunks <= 0) ns = 1;
    *nseg = ns;
    *cps = max_chunks > 0 ? (max_chunks + ns - 1) / ns : 1;
}

}  // namespace

bool prefill_tc_available() { return true; }

size_t prefill_tc_workspace_bytes(const dsla_prefill_args* a) {
    int nseg, cps;
    plan(a, &nseg, &cps);
    if (nseg <= 1) return 0;
    return (size_t)a->N * a->H * nseg * SUMMARY_STRIDE;
}

dsla_status launch_prefill_tc(const PrefillParams& p, const dsla_prefill_args* a, cudaStream_t s) {
    if (p.N == 0 || a->T_total == 0) {
        // only empty sequences: the CUDA-core kernel handles the slot bookkeeping
        return launch_prefill_simt(p, D, C, DSLA_BF16, s);
    }
    TcParams tp;
    tp.p = p;
    plan(a, &tp.nseg, &tp.cps);
    tp.ws = tp.nseg > 1 ? static_cast<float*>(a->workspace) : nullptr;
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, p.q, a->T_total, p.H) || !make_map(&mk, p.k, a->T_total, p.H) || !make_map(&mv, p.v, a->T_total, p.H))
        return DSLA_ERR_CUDA;
    if (cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN) != cudaSuccess ||
        cudaFuncSetAttribute(prefill_tc_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_DYN) != cudaSuccess)
        return DSLA_ERR_CUDA;
    const long long units = (long long)p.N * p.H;
    if (units * tp.nseg > 0x7fffffffLL) return DSLA_ERR_UNSUPPORTED;
    if (tp.nseg > 1) {
        prefill_tc_summary_kernel<<<dim3((unsigned)(units * (tp.nseg - 1))), dim3(NTHREADS), SMEM_DYN, s>>>(mk, mv, tp);
        count_launch();
    }
    prefill_tc_kernel<<<dim3((unsigned)(units * tp.nseg)), dim3(NTHREADS), SMEM_DYN, s>>>(mq, mk, mv, tp);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // namespace dsla
