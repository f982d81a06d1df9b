// Gate producer of the dual-state layer: the activated gates come from single linear layers on the layer input
// (Sec. 5.3; zero bias at initialisation, App. B),
//     [g_hist | g_rec][t, :] = logistic(x[t, :] W^T + b),        x: [T, D_model] bf16,  W: [2 H, D_model] bf16,
// written straight in the [T, H] fp32 layout the prefill and decode kernels read, so no pre-activation tensor
// crosses HBM.  A tcgen05 GEMM: CTA = 128 tokens, M = 128 (tokens on the TMEM lanes), N = 2 H, K = D_model in
// steps of 64; TMA lands the x and W tiles (128-byte swizzle) in a four-stage ring; the epilogue reads the fp32
// accumulator from TMEM (one token per thread), adds the bias, applies the logistic and stores 16 bytes at a time (the
// H outputs of a token and gate tensor are contiguous).  Bound by reading x once from HBM (T * D_model * 2 bytes).
//
// Few tokens mean few CTAs (32 at T = 4096), and one CTA streams its rows at a fraction of what the SM could
// take: then K is split over the 2 or 4 CTAs of a thread-block cluster.  Each CTA accumulates its share of the
// K steps; ranks 1.. send their fp32 partial tile to rank 0's shared memory (st.async with a transaction-count
// barrier that rank 0 arms), rank 0 adds them to its own accumulator and runs the epilogue.
#include "dsla_internal.cuh"
#include "tc_utils.cuh"

namespace dsla {

using namespace tc;

namespace {

constexpr int GP_STAGES = 4, GP_KB = 64, GP_M = 128, GP_MAXN = 256;
constexpr int GP_NTHREADS = 6 * 32;      // warp 0: TMA, warp 1: MMA issue + TMEM, warps 2..5: epilogue (one per lane quadrant)
__device__ int g_gate_status = 0;        // raised when a bounded wait gives up

struct GateProjectParams {
    const float* bias;       // [n_out] or nullptr
    float* g_hist;           // [T, H]
    float* g_rec;            // [T, H]
    int T, H, D_model, n_out;
    int split;               // CTAs per cluster that share one 128-token tile (1, 2 or 4); divides D_model / 64
};

__global__ void __launch_bounds__(GP_NTHREADS, 1)
gate_project_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const GateProjectParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full[GP_STAGES], empty[GP_STAGES], acc_full, red_full;
    __shared__ uint32_t tmem_base;
    __shared__ int abort_flag;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = p.split;
    const int rank = split > 1 ? (int)cluster_ctarank() : 0;
    const int t0 = (int)(blockIdx.x / split) * GP_M;
    const int nk = p.D_model / GP_KB / split;          // K steps of this CTA
    const int kb0 = rank * nk;
    const int a_bytes = GP_M * GP_KB * 2, b_bytes = p.n_out * GP_KB * 2;
    const int stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);
    uint32_t ncols = 32;
    while ((int)ncols < p.n_out) ncols <<= 1;       // TMEM allocations are powers of two >= 32 columns

    if (tid == 0) {
        for (int s = 0; s < GP_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(&acc_full, 1);
        mbar_init(&red_full, 1);
        abort_flag = 0;
        fence_barrier_init();
        // rank 0 expects one fp32 tile (128 tokens x n_out) from every other rank of the cluster
        if (split > 1 && rank == 0) mbar_arrive_expect_tx(&red_full, (uint32_t)((split - 1) * GP_M * p.n_out * 4));
    }
    if (warp == 1) { tmem_alloc(&tmem_base, ncols); tmem_relinquish(); }
    tc_fence_before();
    if (split > 1) cluster_sync_all();      // every barrier of the cluster is initialised before anything is sent
    else __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base;
    // partial tiles land behind the stages: [rank - 1][token][n_out] fp32, the 16-byte pieces of a row rotated by the
    // token index so that a warp (one token per lane) reads and writes without bank conflicts
    uint8_t* red = tiles + GP_STAGES * stage_bytes;
    const int npieces = p.n_out / 4;
    volatile int* abortp = &abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&map_x); prefetch_tensormap(&map_w);
            for (int kb = 0; kb < nk; ++kb) {
                const int s = kb % GP_STAGES, u = kb / GP_STAGES;
                if (u >= 1) mbar_wait(&empty[s], (u - 1) & 1, abortp, &g_gate_status);
                uint8_t* st = tiles + s * stage_bytes;
                const int kcol = (kb0 + kb) * GP_KB;
                mbar_arrive_expect_tx(&full[s], (uint32_t)(a_bytes + b_bytes));
                tma_load_2d(st, &map_x, &full[s], kcol, t0);                       // rows past T are filled with zeros
                tma_load_2d(st + a_bytes, &map_w, &full[s], kcol, 0);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t sa = smem_u32(tiles);
            const uint32_t idesc = idesc_bf16(GP_M, p.n_out, 0, 0);               // both operands K-major
            for (int kb = 0; kb < nk; ++kb) {
                const int s = kb % GP_STAGES, u = kb / GP_STAGES;
                mbar_wait(&full[s], u & 1, abortp, &g_gate_status);
                tc_fence_after();
                const uint64_t da = smem_desc_sw128(sa + s * stage_bytes, 16, 1024), db = smem_desc_sw128(sa + s * stage_bytes + a_bytes, 16, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) mma_ss(tb, da + (uint64_t)(2 * kk), db + (uint64_t)(2 * kk), idesc, (kb | kk) ? 1u : 0u);
                tc_commit(&empty[s]);
            }
            tc_commit(&acc_full);
        }
    } else {
        // ---- epilogue: thread = token (TMEM lane); 32 columns at a time
        const int q = warp & 3;
        const int tok = 32 * q + lane;
        const int t = t0 + tok;
        mbar_wait(&acc_full, 0, abortp, &g_gate_status);
        tc_fence_after();
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        if (rank > 0) {
            // partial sums of this rank's K steps go to rank 0
            const uint32_t dst_row = map_to_cta(smem_u32(red + ((size_t)(rank - 1) * GP_M + tok) * p.n_out * 4), 0);
            const uint32_t dst_bar = map_to_cta(smem_u32(&red_full), 0);
            for (int c0 = 0; c0 < p.n_out; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(lane_addr + c0, r);
                tc_wait_ld();
#pragma unroll
                for (int g4 = 0; g4 < 8; ++g4) {
                    const int piece = c0 / 4 + g4;
                    if (piece < npieces)
                        st_async_f32x4(dst_row + (uint32_t)(((piece + tok) % npieces) * 16), __uint_as_float(r[4 * g4]), __uint_as_float(r[4 * g4 + 1]),
                                       __uint_as_float(r[4 * g4 + 2]), __uint_as_float(r[4 * g4 + 3]), dst_bar);
                }
            }
        } else {
            if (split > 1) mbar_wait(&red_full, 0, abortp, &g_gate_status);      // the other ranks' tiles have landed
            for (int c0 = 0; c0 < p.n_out; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(lane_addr + c0, r);
                tc_wait_ld();
                if (t < p.T) {
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const int col = c0 + c;                                           // H is a multiple of 4: a group of four never straddles
                        if (col < p.n_out) {
                            float z[4] = {__uint_as_float(r[c]), __uint_as_float(r[c + 1]), __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3])};
                            for (int sr = 0; sr + 1 < split; ++sr) {
                                const float4 x = *reinterpret_cast<const float4*>(red + ((size_t)sr * GP_M + tok) * p.n_out * 4 + ((col / 4 + tok) % npieces) * 16);
                                z[0] += x.x; z[1] += x.y; z[2] += x.z; z[3] += x.w;
                            }
                            float y[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                if (p.bias) z[e] += __ldg(p.bias + col + e);
                                y[e] = 1.f / (1.f + ex2(-1.4426950408889634f * z[e]));      // logistic(z); ex2 of a large argument is inf: 1 / inf = 0
                            }
                            float* dst = col < p.H ? p.g_hist + (size_t)t * p.H + col : p.g_rec + (size_t)t * p.H + (col - p.H);
                            *reinterpret_cast<float4*>(dst) = make_float4(y[0], y[1], y[2], y[3]);
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    if (split > 1) cluster_sync_all();      // rank 0's shared memory stays up until every rank has sent its tile
    else __syncthreads();
    if (warp == 1) tmem_dealloc(tb, ncols);
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows, cols] bf16 row-major seen as (cols, rows); a box is 64 columns (128 bytes, swizzled) x box_rows rows.
bool make_map_2d(CUtensorMap* m, const void* base, int rows, int cols, int box_rows) {
    static EncodeFn encode = [] {      // looked up once
        cudaDriverEntryPointQueryResult qr;
        void* ptr = nullptr;
        EncodeFn f = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
            f = reinterpret_cast<EncodeFn>(ptr);
        (void)cudaGetLastError();
        return f;
    }();
    if (!encode) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    return encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

dsla_status launch_gate_project(const dsla_gate_project_args* a, cudaStream_t s) {
    const int n_out = 2 * a->H;
    CUtensorMap mx, mw;
    if (!make_map_2d(&mx, a->x, a->T, a->D_model, GP_M) || !make_map_2d(&mw, a->w, n_out, a->D_model, n_out)) return DSLA_ERR_CUDA;
    const int a_bytes = GP_M * GP_KB * 2, b_bytes = n_out * GP_KB * 2;
    const int stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);
    const int tiles_m = (a->T + GP_M - 1) / GP_M, nk = a->D_model / GP_KB;
    // split K over a cluster while the token tiles alone leave SMs idle, each rank keeps at least four K steps and the
    // partial tiles fit behind the stages
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    int split = 1;
    for (int c = 4; c >= 2; c >>= 1) {
        const size_t red = (size_t)(c - 1) * GP_M * n_out * 4;
        if ((long long)tiles_m * c <= sms && nk % c == 0 && nk / c >= 4 && GP_STAGES * (size_t)stage_bytes + red <= 200 * 1024) { split = c; break; }
    }
    const int smem = GP_STAGES * stage_bytes + (split - 1) * GP_M * n_out * 4 + 1024;
    if (cudaFuncSetAttribute(gate_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return DSLA_ERR_CUDA;
    GateProjectParams p{a->bias, a->g_hist, a->g_rec, a->T, a->H, a->D_model, n_out, split};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles_m * split));
    cfg.blockDim = dim3(GP_NTHREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = split > 1 ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, gate_project_kernel, mx, mw, p) != cudaSuccess) return DSLA_ERR_CUDA;
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

dsla_status gate_project_last_error() {
    int host = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return DSLA_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&host, g_gate_status, sizeof(int)) != cudaSuccess) return DSLA_ERR_CUDA;
    if (host != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_gate_status, &zero, sizeof(int)) != cudaSuccess) return DSLA_ERR_CUDA;
    }
    return host == 0 ? DSLA_OK : DSLA_ERR_TIMEOUT;
}

}  // namespace dsla
