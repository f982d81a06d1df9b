// Helper kernels of the tensor-core prefill: the state summaries of the segments a sequence is split
// into, the longest-first visiting order of a packed batch, and the snapshot of the initial states.
//
// Segment summaries: U_g (both states, accumulated from zero) and A_g (product of the segment's gates)
// for every segment but a sequence's last, so that a later segment can start from
// S_in = fold over earlier segments of (S <- A_j S + U_j) -- the inter-segment level of the state scan
// of the Sec. 4.1 recurrence.  The chunks are walked from the END of the segment backwards while a
// running product R^i of all later gates is carried, so every token's weight prod_{t > s} g^i_t (to the
// end of the segment) is a plain product: no logarithms, no rescaling of the accumulator, and a zero
// gate is exact.  A pure streaming pipeline: warps 10, 11 derive the weights (one state each), warps
// 0..3 build the weighted, transposed V~i^T of both states in TMEM straight from the V tile (ldmatrix
// with .trans hands a thread two consecutive tokens of one d_v column, which is the element pair a
// 16x128b TMEM store takes: no shuffles and no scaled copy in shared memory), warp 8 drives TMA,
// warp 9 issues the MMAs  S^i^T += V~i^T K  (M = 128, N = 128, K = 64 tokens; A in TMEM, B = the raw
// K tile), warps 4..7 only help with the final store.
#include "dsla_prefill_tc.cuh"

namespace dsla {

namespace {

constexpr int SUM_STAGES = 6, SUM_STAGE_BYTES = 2 * 16384, SUM_OFF_V = 16384;   // stage = [K][V]
constexpr int SUM_WSTAGES = 4;           // ring of per-chunk weights
constexpr int SUM_NTHREADS = 384;
constexpr int SUM_GATE_AHEAD = 6;        // chunks between the L2 prefetch and the load of a chunk's gates
constexpr int SUM_PREFETCH = 8;          // chunks between the L2 prefetch and the load of a tile
constexpr int SUM_SMEM_DYN = SUM_STAGES * SUM_STAGE_BYTES + 1024;
constexpr uint32_t SUM_COL_VT = 256;     // V~^T, bf16: [chunk parity][state] x 32 columns

struct alignas(16) SumShared {
    uint64_t full[SUM_STAGES], empty[SUM_STAGES], w_ready[SUM_WSTAGES], w_free[SUM_WSTAGES], vt_ready[2], vt_free[2], u_full;
    uint32_t tmem_base;
    int abort_flag;
    __nv_bfloat16 wts[SUM_WSTAGES][2][C];     // per-token weights
};

__global__ void __launch_bounds__(SUM_NTHREADS, 1)
prefill_tc_summary_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const TcParams tp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ SumShared sh;
    const PrefillParams& p = tp.p;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the main grid may be scheduled as SMs become free
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
        for (int s = 0; s < SUM_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 5); }   // four V~ warps + the MMAs on K
        for (int s = 0; s < SUM_WSTAGES; ++s) { mbar_init(&sh.w_ready[s], 2); mbar_init(&sh.w_free[s], 4); }
        for (int b = 0; b < 2; ++b) { mbar_init(&sh.vt_ready[b], 4); mbar_init(&sh.vt_free[b], 1); }
        mbar_init(&sh.u_full, 1);
        sh.abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 9) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = sh.tmem_base;
    volatile int* abortp = &sh.abort_flag;

    // iteration it = 0 .. nc-1 handles chunk nc-1-it; tile stage it % 6, weight stage it % 4, V~ buffer it % 2
    if (warp == 8) {
        if (lane == 0) {
            prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
            for (int it = 0; it < nc; ++it) {
                const int s = it % SUM_STAGES, u = it / SUM_STAGES;
                if (u >= 1) mbar_wait(&sh.empty[s], (u - 1) & 1, abortp, p.status);
                uint8_t* st = tiles + s * SUM_STAGE_BYTES;
                const int t = t0 + (nc - 1 - it) * C;
                mbar_arrive_expect_tx(&sh.full[s], 4 * 8192);
                tma_load_4d(st + SUM_OFF_V, &map_v, &sh.full[s], 0, t, 0, h);
                tma_load_4d(st, &map_k, &sh.full[s], 0, t, 0, h);
                if (it + SUM_PREFETCH < nc) {   // pull a tile well ahead into L2: the stages alone do not cover the HBM latency
                    const int tp2 = t - SUM_PREFETCH * C;
                    tma_prefetch_4d(&map_k, 0, tp2, 0, h);
                    tma_prefetch_4d(&map_v, 0, tp2, 0, h);
                }
            }
        }
    } else if (warp == 9) {
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            constexpr uint32_t ID_U = idesc_bf16(128, 128, 0, 1);       // A in TMEM, B = K as an MN-major N operand
            for (int it = 0; it < nc; ++it) {
                const int s = it % SUM_STAGES, u = it / SUM_STAGES, b = it & 1;
                mbar_wait(&sh.full[s], u & 1, abortp, p.status);
                mbar_wait(&sh.vt_ready[b], (it >> 1) & 1, abortp, p.status);
                tc_fence_after();
                const uint64_t dkk = smem_desc_sw128(sa + s * SUM_STAGE_BYTES, 8192, 1024);
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ts(tb + 128 * i, tb + SUM_COL_VT + 64 * b + 32 * i + 8 * kk, dkk + (uint64_t)(kk * 128), ID_U, (it | kk) > 0);
                tc_commit(&sh.empty[s]);
                tc_commit(&sh.vt_free[b]);
                if (it == nc - 1) tc_commit(&sh.u_full);
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
            const int s = it % SUM_WSTAGES, u = it / SUM_WSTAGES;
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
            if (u >= 1) mbar_wait(&sh.w_free[s], (u - 1) & 1, abortp, p.status);
            *reinterpret_cast<__nv_bfloat162*>(&sh.wts[s][i][2 * lane]) = __floats2bfloat162_rn(g1 * ex, ex);
            R *= tot;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.w_ready[s]);
        }
        if (lane == 0) out[2 * D * D + i] = R;         // A_g: product of every gate of the segment
    } else {
        const int q = warp & 3, hi = warp >> 2;
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        if (warp < 4) {
            // ---- V~i^T[v][s] = w^i_s V[s][v] for both states into TMEM (d_v on the lanes, two tokens per 32-bit column).
            // One round = 16 tokens x 16 d_v lanes: matrices (tokens 0..7 | 8..15) x (d_v 0..7 | 8..15); a 16x128b TMEM store
            // takes the ldmatrix.trans distribution as it is (lane = t / 4, column = t % 4).
            const int mk = lane >> 3, mr = lane & 7;                 // this thread addresses row mr of matrix mk
            for (int it = 0; it < nc; ++it) {
                const int s = it % SUM_STAGES, u = it / SUM_STAGES, ws = it % SUM_WSTAGES, b = it & 1;
                mbar_wait(&sh.w_ready[ws], (it / SUM_WSTAGES) & 1, abortp, p.status);
                mbar_wait(&sh.full[s], u & 1, abortp, p.status);
                if (it >= 2) mbar_wait(&sh.vt_free[b], ((it >> 1) - 1) & 1, abortp, p.status);     // the MMAs of chunk it - 2 have read this buffer
                tc_fence_after();
                const uint32_t vtile = smem_u32(tiles + s * SUM_STAGE_BYTES + SUM_OFF_V);
                const uint8_t* wp0 = reinterpret_cast<const uint8_t*>(sh.wts[ws][0]) + 4 * (lane & 3);
                const uint8_t* wp1 = reinterpret_cast<const uint8_t*>(sh.wts[ws][1]) + 4 * (lane & 3);
#pragma unroll 1
                for (int hh = 0; hh < 2; ++hh) {       // the two 16-lane halves of this warp's TMEM quadrant
                    const int d = 32 * q + 16 * hh + 8 * (mk & 1);            // first d_v column of the matrix this thread addresses
                    // row of the V tile: token * 128 bytes, 16-byte piece (d / 8 mod 8) ^ (token mod 8); token mod 8 = mr in every round
                    const uint32_t row0 = vtile + (uint32_t)(d >> 6) * 8192u + (uint32_t)((8 * (mk >> 1) + mr) * 128) +
                                          (((uint32_t)((d & 63) >> 3) ^ (uint32_t)mr) << 4);
                    const uint32_t vt = tb + ((uint32_t)(32 * q + 16 * hh) << 16) + SUM_COL_VT + 64 * b;
                    uint32_t r[16];
#pragma unroll
                    for (int t16 = 0; t16 < 4; ++t16)      // all loads of the half first: their latencies overlap
                        ldmatrix_x4_trans(row0 + (uint32_t)(t16 * 16 * 128), r[4 * t16], r[4 * t16 + 1], r[4 * t16 + 2], r[4 * t16 + 3]);
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const uint8_t* wp = i == 0 ? wp0 : wp1;
#pragma unroll
                        for (int t16 = 0; t16 < 4; ++t16) {
                            const __nv_bfloat162 ww0 = *reinterpret_cast<const __nv_bfloat162*>(wp + 32 * t16);
                            const __nv_bfloat162 ww1 = *reinterpret_cast<const __nv_bfloat162*>(wp + 32 * t16 + 16);
                            const __nv_bfloat162 y0 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16]), ww0);
                            const __nv_bfloat162 y1 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16 + 1]), ww0);
                            const __nv_bfloat162 y2 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16 + 2]), ww1);
                            const __nv_bfloat162 y3 = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&r[4 * t16 + 3]), ww1);
                            tmem_st_16x128b(vt + 32 * i + 8 * t16, *reinterpret_cast<const uint32_t*>(&y0), *reinterpret_cast<const uint32_t*>(&y1));
                            tmem_st_16x128b(vt + 32 * i + 8 * t16 + 4, *reinterpret_cast<const uint32_t*>(&y2), *reinterpret_cast<const uint32_t*>(&y3));
                        }
                    }
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&sh.vt_ready[b]); mbar_arrive(&sh.empty[s]); mbar_arrive(&sh.w_free[ws]); }
            }
        }
        mbar_wait(&sh.u_full, 0, abortp, p.status);
        tc_fence_after();
        store_state(out + (size_t)hi * D * D, 32 * q + lane, lane_addr + 128 * hi, 0, 4);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tb, 512);
}

// Ragged batches: blocks are handed to the SMs in index order, so sequences are visited longest first (a long
// sequence that starts late would otherwise run on alone at the end).  order[r] = index of the r-th longest
// sequence, ties by index; one thread per sequence counts how many sequences come before its own.
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

// Copies the two states of every (sequence, head) out of the sequence's slot: snap[(n*H + h)][2][D][D].
__global__ void __launch_bounds__(256) state_snapshot_kernel(const PrefillParams p, float* __restrict__ snap) {
    const int unit = blockIdx.x >> 1, i = blockIdx.x & 1;
    const int n = unit / p.H, h = unit % p.H;
    const int slot = p.slots ? p.slots[n] : n;
    if (slot < 0 || slot >= p.num_slots || (p.single && i == 1)) return;
    const float4* src = reinterpret_cast<const float4*>(p.state + (((size_t)slot * p.n_total + p.state_first + i) * p.H + h) * (size_t)(D * D));
    float4* dst = reinterpret_cast<float4*>(snap + ((size_t)unit * 2 + i) * (size_t)(D * D));
    for (int k = threadIdx.x; k < D * D / 4; k += 256) dst[k] = src[k];
}

// The give-up path of the bounded waits, on its own: one warp, one barrier that nobody ever arrives at, nothing
// asynchronous in flight.  The wait runs out after max_polls polls, raises the status word and the kernel returns.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(int* status, unsigned max_polls) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncwarp();
    volatile int* abortp = &abort_flag;
    if (threadIdx.x == 0) mbar_wait(&bar, 0, abortp, status, max_polls);
    __syncwarp();
    // a wait that starts after the abort flag is up returns on its first poll
    mbar_wait(&bar, 0, abortp, status, MBAR_WAIT_LIMIT);
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
    static EncodeFn fn = [] {
        cudaDriverEntryPointQueryResult qr;
        void* ptr = nullptr;
        EncodeFn f = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            f = reinterpret_cast<EncodeFn>(ptr);
        (void)cudaGetLastError();
        return f;
    }();
    return fn;
}

}  // namespace

// [T_total, H, 128] bf16 seen as (x: 64 elements, t, half: the two 64-element halves of a row, h) so that one
// copy of box {64, 64 tokens, 2, 1} lands as two consecutive 8 KB tiles [half][token][64], each in the 128-byte
// swizzle the MMA descriptors expect.
bool make_tile_map(CUtensorMap* m, const void* base, int T_total, int H) {
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

void launch_bounded_wait_selftest(int* status, unsigned max_polls, cudaStream_t s) {
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(status, max_polls);
    count_launch();
}

void launch_seq_order(const int32_t* cu, int N, int* order, cudaStream_t s) {
    seq_order_kernel<<<dim3((unsigned)((N + 255) / 256)), dim3(256), 0, s>>>(cu, N, order);
    count_launch();
}

void launch_state_snapshot(const PrefillParams& p, float* snap, cudaStream_t s) {
    state_snapshot_kernel<<<dim3((unsigned)(2 * p.N * p.H)), dim3(256), 0, s>>>(p, snap);
    count_launch();
}

dsla_status launch_summary(const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& tp, cudaStream_t s) {
    if (cudaFuncSetAttribute(prefill_tc_summary_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SUM_SMEM_DYN) != cudaSuccess)
        return DSLA_ERR_CUDA;
    const long long units = (long long)tp.p.N * tp.p.H;
    prefill_tc_summary_kernel<<<dim3((unsigned)(units * (tp.nseg - 1))), dim3(SUM_NTHREADS), SUM_SMEM_DYN, s>>>(mk, mv, tp);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // namespace dsla
