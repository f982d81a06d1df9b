// Gate producer of the dual-state layer: the activated gates come from single linear layers on the layer input
// (Sec. 5.3; zero bias at initialisation, App. B),
//     [g_hist | g_rec][t, :] = logistic(x[t, :] W^T + b),        x: [T, D_model] bf16,  W: [2 H, D_model] bf16,
// written straight in the [T, H] fp32 layout the prefill and decode kernels read, so no pre-activation tensor
// crosses HBM.  A tcgen05 GEMM: CTA = 128 tokens, M = 128 (tokens on the TMEM lanes), N = 2 H, K = D_model in
// steps of 64; TMA lands the x and W tiles (128-byte swizzle) in a four-stage ring; the epilogue reads the fp32
// accumulator from TMEM (one token per thread), adds the bias, applies the logistic and stores 128 contiguous bytes
// per thread and gate tensor.  Bound by reading x once from HBM (T * D_model * 2 bytes).
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
};

__global__ void __launch_bounds__(GP_NTHREADS, 1)
gate_project_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const GateProjectParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full[GP_STAGES], empty[GP_STAGES], acc_full;
    __shared__ uint32_t tmem_base;
    __shared__ int abort_flag;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int t0 = blockIdx.x * GP_M;
    const int nk = p.D_model / GP_KB;
    const int a_bytes = GP_M * GP_KB * 2, b_bytes = p.n_out * GP_KB * 2;
    const int stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);
    uint32_t ncols = 32;
    while ((int)ncols < p.n_out) ncols <<= 1;       // TMEM allocations are powers of two >= 32 columns

    if (tid == 0) {
        for (int s = 0; s < GP_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(&acc_full, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) { tmem_alloc(&tmem_base, ncols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base;
    volatile int* abortp = &abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&map_x); prefetch_tensormap(&map_w);
            for (int kb = 0; kb < nk; ++kb) {
                const int s = kb % GP_STAGES, u = kb / GP_STAGES;
                if (u >= 1) mbar_wait(&empty[s], (u - 1) & 1, abortp, &g_gate_status);
                uint8_t* st = tiles + s * stage_bytes;
                mbar_arrive_expect_tx(&full[s], (uint32_t)(a_bytes + b_bytes));
                tma_load_2d(st, &map_x, &full[s], kb * GP_KB, t0);                 // rows past T are filled with zeros
                tma_load_2d(st + a_bytes, &map_w, &full[s], kb * GP_KB, 0);
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
        const int t = t0 + 32 * q + lane;
        mbar_wait(&acc_full, 0, abortp, &g_gate_status);
        tc_fence_after();
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        for (int c0 = 0; c0 < p.n_out; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(lane_addr + c0, r);
            tc_wait_ld();
            if (t < p.T) {
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    float y[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int col = c0 + c + e;
                        float z = __uint_as_float(r[c + e]);
                        if (p.bias && col < p.n_out) z += __ldg(p.bias + col);
                        y[e] = 1.f / (1.f + ex2(-1.4426950408889634f * z));          // logistic(z); ex2 of a large argument is inf: 1 / inf = 0
                    }
                    const int col = c0 + c;                                           // H is a multiple of 4: a group of four never straddles
                    if (col < p.n_out) {
                        float* dst = col < p.H ? p.g_hist + (size_t)t * p.H + col : p.g_rec + (size_t)t * p.H + (col - p.H);
                        *reinterpret_cast<float4*>(dst) = make_float4(y[0], y[1], y[2], y[3]);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tb, ncols);
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows, cols] bf16 row-major seen as (cols, rows); a box is 64 columns (128 bytes, swizzled) x box_rows rows.
bool make_map_2d(CUtensorMap* m, const void* base, int rows, int cols, int box_rows) {
    cudaDriverEntryPointQueryResult qr;
    void* ptr = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) != cudaSuccess || qr != cudaDriverEntryPointSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    return reinterpret_cast<EncodeFn>(ptr)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
                                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

dsla_status launch_gate_project(const dsla_gate_project_args* a, cudaStream_t s) {
    const int n_out = 2 * a->H;
    CUtensorMap mx, mw;
    if (!make_map_2d(&mx, a->x, a->T, a->D_model, GP_M) || !make_map_2d(&mw, a->w, n_out, a->D_model, n_out)) return DSLA_ERR_CUDA;
    const int a_bytes = GP_M * GP_KB * 2, b_bytes = n_out * GP_KB * 2;
    const int smem = GP_STAGES * (a_bytes + ((b_bytes + 1023) & ~1023)) + 1024;
    if (cudaFuncSetAttribute(gate_project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return DSLA_ERR_CUDA;
    GateProjectParams p{a->bias, a->g_hist, a->g_rec, a->T, a->H, a->D_model, n_out};
    gate_project_kernel<<<dim3((unsigned)((a->T + GP_M - 1) / GP_M)), dim3(GP_NTHREADS), smem, s>>>(mx, mw, p);
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
