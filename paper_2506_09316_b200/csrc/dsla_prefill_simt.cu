// Chunkwise prefill of the dual-state linear attention layer on CUDA cores, fp32 arithmetic.
// Serves the fp32 configuration (1e-4 tolerance rules out bf16/tf32 tensor-core products) and any
// shape the tensor-core kernel does not cover.  Mathematics (derived from the recurrence of
// Sec. 4.1 and its unrolled score form): inside a chunk with inclusive cumulative log-gates b^i_j,
//     o_j = sum_{s<=j} (q_j.k_s) [gamma e^{b1_j-b1_s} + (1-gamma) e^{b2_j-b2_s}] v_s
//           + gamma e^{b1_j} q_j S^1 + (1-gamma) e^{b2_j} q_j S^2
//     S^i <- e^{b^i_last} S^i + sum_s e^{b^i_last - b^i_s} k_s^T v_s
// Exponents are always differences b_j - b_s <= 0, so nothing overflows.  A gate that is exactly 0
// is not pushed through log(): zero gates are counted (zc) and a factor is 0 whenever a zero gate
// lies between the two tokens, which keeps tokens after the zero exact.
#include "dsla_internal.cuh"

namespace dsla {

namespace {

template <typename T> struct Vec4;
template <> struct Vec4<float> {
    static __device__ __forceinline__ float4 load(const float* p) { return *reinterpret_cast<const float4*>(p); }
};
template <> struct Vec4<__nv_bfloat16> {
    static __device__ __forceinline__ float4 load(const __nv_bfloat16* p) {
        const uint2 u = *reinterpret_cast<const uint2*>(p);
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&u.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&u.y);
        return make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
    }
};

__device__ __forceinline__ void store2(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16* p, float a, float b) {
    *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b);
}

}  // namespace

// CTA = (sequence, head, 32-column slab of d_v); 256 threads.  The slab's two state slices live in
// registers (4x4 tile per thread per state) across the chunk loop, with a copy in shared memory for
// the readout.  Q K^T is recomputed per slab (D/32 times); acceptable for this fallback path.
template <int D, int C, typename T>
__global__ void __launch_bounds__(256) prefill_simt_kernel(const PrefillParams p) {
    constexpr int DVS = 32, SLABS = D / DVS, DP = D + 4, VP = DVS + 4, CP = C + 4, NT = 256;
    extern __shared__ __align__(16) float smem[];
    float* Qs = smem;                 // [C][DP]
    float* Ks = Qs + C * DP;          // [C][DP]
    float* Vs = Ks + C * DP;          // [C][VP]
    float* Ps = Vs + C * VP;          // [C][CP]  masked scores
    float* Ss = Ps + C * CP;          // [2][D][VP]
    float* bb = Ss + 2 * D * VP;      // [2][C] cumulative log-gate (zeros skipped)
    float* rowf = bb + 2 * C;         // [2][C] weight_i * e^{b_j} (0 behind a zero gate)
    float* ww = rowf + 2 * C;         // [2][C] e^{b_last - b_s}
    int* zc = reinterpret_cast<int*>(ww + 2 * C);  // [2][C] zero-gate count, inclusive
    __shared__ float a_dec[2];

    const int tid = threadIdx.x;
    const int slab = blockIdx.x % SLABS;
    const int h = (blockIdx.x / SLABS) % p.H;
    const int n = blockIdx.x / (SLABS * p.H);
    const int t_begin = p.cu_seqlens ? p.cu_seqlens[n] : n * p.T;
    const int t_end = p.cu_seqlens ? p.cu_seqlens[n + 1] : (n + 1) * p.T;
    const int len = t_end - t_begin;
    const int slot = p.slots ? p.slots[n] : n;
    if (slot < 0 || slot >= p.num_slots) return;
    const int col0 = slab * DVS;

    float* G1 = p.state + (((size_t)slot * 2 + 0) * p.H + h) * (size_t)(D * D);
    float* G2 = G1 + (size_t)p.H * D * D;

    // state tile of this thread: rows k0..k0+3, columns n0..n0+3 of the slab
    const bool own = tid < (D / 4) * 8;
    const int k0 = (tid >> 3) * 4, n0 = (tid & 7) * 4;
    float s1[4][4], s2[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) s1[a][b] = s2[a][b] = 0.f;
    if (own && p.use_initial_state) {
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const float4 x = *reinterpret_cast<const float4*>(G1 + (size_t)(k0 + a) * D + col0 + n0);
            const float4 y = *reinterpret_cast<const float4*>(G2 + (size_t)(k0 + a) * D + col0 + n0);
            s1[a][0] = x.x; s1[a][1] = x.y; s1[a][2] = x.z; s1[a][3] = x.w;
            s2[a][0] = y.x; s2[a][1] = y.y; s2[a][2] = y.z; s2[a][3] = y.w;
        }
    }
    if (len <= 0 && p.use_initial_state) return;  // nothing to do, slot untouched
    if (own) {
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            *reinterpret_cast<float4*>(Ss + (k0 + a) * VP + n0) = make_float4(s1[a][0], s1[a][1], s1[a][2], s1[a][3]);
            *reinterpret_cast<float4*>(Ss + D * VP + (k0 + a) * VP + n0) = make_float4(s2[a][0], s2[a][1], s2[a][2], s2[a][3]);
        }
    }
    const float gam = p.gamma[h];
    const float W1 = gam * p.scale, W2 = (1.f - gam) * p.scale;
    const T* qg = reinterpret_cast<const T*>(p.q);
    const T* kg = reinterpret_cast<const T*>(p.k);
    const T* vg = reinterpret_cast<const T*>(p.v);
    T* og = reinterpret_cast<T*>(p.o);

    for (int c0 = 0; c0 < len; c0 += C) {
        const int valid = min(C, len - c0);
        __syncthreads();
        // ---- stage Q, K, V (rows past the end of the sequence become zeros)
        for (int idx = tid; idx < C * (D / 4); idx += NT) {
            const int row = idx / (D / 4), c = idx % (D / 4);
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
            if (row < valid) {
                const size_t off = ((size_t)(t_begin + c0 + row) * p.H + h) * D + c * 4;
                x = Vec4<T>::load(qg + off);
                y = Vec4<T>::load(kg + off);
            }
            *reinterpret_cast<float4*>(Qs + row * DP + c * 4) = x;
            *reinterpret_cast<float4*>(Ks + row * DP + c * 4) = y;
        }
        for (int idx = tid; idx < C * (DVS / 4); idx += NT) {
            const int row = idx / (DVS / 4), c = idx % (DVS / 4);
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row < valid) x = Vec4<T>::load(vg + ((size_t)(t_begin + c0 + row) * p.H + h) * D + col0 + c * 4);
            *reinterpret_cast<float4*>(Vs + row * VP + c * 4) = x;
        }
        // ---- inclusive scan of log-gates (fp64 accumulation) and of the zero-gate count
        if (tid < 64) {
            constexpr int PER = C >= 32 ? C / 32 : 1;
            const int i = tid >> 5, lane = tid & 31;
            const float* gp = i == 0 ? p.g_hist : p.g_rec;
            double lg[PER];
            int zz[PER];
            double run = 0.0;
            int zrun = 0;
#pragma unroll
            for (int e = 0; e < PER; ++e) {
                const int j = lane * PER + e;
                float g = 1.f;
                if (j < valid) g = gp[(size_t)(t_begin + c0 + j) * p.H + h];
                const bool zero = !(g > 0.f);
                run += zero ? 0.0 : (double)logf(g);
                zrun += zero ? 1 : 0;
                lg[e] = run;
                zz[e] = zrun;
            }
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const double up = __shfl_up_sync(0xffffffffu, run, off);
                const int zup = __shfl_up_sync(0xffffffffu, zrun, off);
                if (lane >= off) { run += up; zrun += zup; }
            }
            const double excl = run - lg[PER - 1];
            const int zexcl = zrun - zz[PER - 1];
#pragma unroll
            for (int e = 0; e < PER; ++e) {
                const int j = lane * PER + e;
                if (j < C) {
                    bb[i * C + j] = (float)(excl + lg[e]);
                    zc[i * C + j] = zexcl + zz[e];
                }
            }
        }
        __syncthreads();
        if (tid < 2 * C) {
            const int i = tid / C, j = tid % C;
            const float bl = bb[i * C + C - 1];
            const int zl = zc[i * C + C - 1];
            const float b = bb[i * C + j];
            const int z = zc[i * C + j];
            rowf[i * C + j] = (z == 0) ? (i == 0 ? W1 : W2) * expf(b) : 0.f;
            ww[i * C + j] = (z == zl) ? expf(bl - b) : 0.f;
            if (j == 0) a_dec[i] = (zl == 0) ? expf(bl) : 0.f;
        }
        __syncthreads();
        // ---- masked scores: 4x4 tiles of the lower triangle
        for (int tile = tid; tile < (C / 4) * (C / 4); tile += NT) {
            const int j0 = (tile / (C / 4)) * 4, s0 = (tile % (C / 4)) * 4;
            float acc[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
            if (s0 <= j0) {
                for (int kk = 0; kk < D; kk += 4) {
                    float4 qv[4], kv[4];
#pragma unroll
                    for (int a = 0; a < 4; ++a) qv[a] = *reinterpret_cast<const float4*>(Qs + (j0 + a) * DP + kk);
#pragma unroll
                    for (int b = 0; b < 4; ++b) kv[b] = *reinterpret_cast<const float4*>(Ks + (s0 + b) * DP + kk);
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            acc[a][b] = fmaf(qv[a].x, kv[b].x, acc[a][b]);
                            acc[a][b] = fmaf(qv[a].y, kv[b].y, acc[a][b]);
                            acc[a][b] = fmaf(qv[a].z, kv[b].z, acc[a][b]);
                            acc[a][b] = fmaf(qv[a].w, kv[b].w, acc[a][b]);
                        }
                }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const int j = j0 + a, s = s0 + b;
                        float m = 0.f;
                        if (s <= j) {
                            const float d1 = (zc[j] == zc[s]) ? expf(bb[j] - bb[s]) : 0.f;
                            const float d2 = (zc[C + j] == zc[C + s]) ? expf(bb[C + j] - bb[C + s]) : 0.f;
                            m = W1 * d1 + W2 * d2;
                        }
                        acc[a][b] *= m;
                    }
            }
#pragma unroll
            for (int a = 0; a < 4; ++a)
                *reinterpret_cast<float4*>(Ps + (j0 + a) * CP + s0) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
        }
        __syncthreads();
        // ---- outputs: 4 rows x 2 columns per thread
        for (int tile = tid; tile < (C / 4) * (DVS / 2); tile += NT) {
            const int j0 = (tile / (DVS / 2)) * 4, m0 = (tile % (DVS / 2)) * 2;
            float acc[4][2], r1[4][2], r2[4][2];
#pragma unroll
            for (int a = 0; a < 4; ++a) { acc[a][0] = acc[a][1] = r1[a][0] = r1[a][1] = r2[a][0] = r2[a][1] = 0.f; }
            for (int s = 0; s < j0 + 4; s += 4) {  // masked scores are 0 beyond the diagonal tile
                float4 pv[4];
                float2 vv[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) pv[a] = *reinterpret_cast<const float4*>(Ps + (j0 + a) * CP + s);
#pragma unroll
                for (int e = 0; e < 4; ++e) vv[e] = *reinterpret_cast<const float2*>(Vs + (s + e) * VP + m0);
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    acc[a][0] = fmaf(pv[a].x, vv[0].x, acc[a][0]); acc[a][1] = fmaf(pv[a].x, vv[0].y, acc[a][1]);
                    acc[a][0] = fmaf(pv[a].y, vv[1].x, acc[a][0]); acc[a][1] = fmaf(pv[a].y, vv[1].y, acc[a][1]);
                    acc[a][0] = fmaf(pv[a].z, vv[2].x, acc[a][0]); acc[a][1] = fmaf(pv[a].z, vv[2].y, acc[a][1]);
                    acc[a][0] = fmaf(pv[a].w, vv[3].x, acc[a][0]); acc[a][1] = fmaf(pv[a].w, vv[3].y, acc[a][1]);
                }
            }
            for (int kk = 0; kk < D; kk += 4) {
                float4 qv[4];
                float2 x1[4], x2[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) qv[a] = *reinterpret_cast<const float4*>(Qs + (j0 + a) * DP + kk);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    x1[e] = *reinterpret_cast<const float2*>(Ss + (kk + e) * VP + m0);
                    x2[e] = *reinterpret_cast<const float2*>(Ss + D * VP + (kk + e) * VP + m0);
                }
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    r1[a][0] = fmaf(qv[a].x, x1[0].x, r1[a][0]); r1[a][1] = fmaf(qv[a].x, x1[0].y, r1[a][1]);
                    r1[a][0] = fmaf(qv[a].y, x1[1].x, r1[a][0]); r1[a][1] = fmaf(qv[a].y, x1[1].y, r1[a][1]);
                    r1[a][0] = fmaf(qv[a].z, x1[2].x, r1[a][0]); r1[a][1] = fmaf(qv[a].z, x1[2].y, r1[a][1]);
                    r1[a][0] = fmaf(qv[a].w, x1[3].x, r1[a][0]); r1[a][1] = fmaf(qv[a].w, x1[3].y, r1[a][1]);
                    r2[a][0] = fmaf(qv[a].x, x2[0].x, r2[a][0]); r2[a][1] = fmaf(qv[a].x, x2[0].y, r2[a][1]);
                    r2[a][0] = fmaf(qv[a].y, x2[1].x, r2[a][0]); r2[a][1] = fmaf(qv[a].y, x2[1].y, r2[a][1]);
                    r2[a][0] = fmaf(qv[a].z, x2[2].x, r2[a][0]); r2[a][1] = fmaf(qv[a].z, x2[2].y, r2[a][1]);
                    r2[a][0] = fmaf(qv[a].w, x2[3].x, r2[a][0]); r2[a][1] = fmaf(qv[a].w, x2[3].y, r2[a][1]);
                }
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int j = j0 + a;
                if (j < valid) {
                    const float f1 = rowf[j], f2 = rowf[C + j];
                    const float o0 = acc[a][0] + f1 * r1[a][0] + f2 * r2[a][0];
                    const float o1 = acc[a][1] + f1 * r1[a][1] + f2 * r2[a][1];
                    store2(og + ((size_t)(t_begin + c0 + j) * p.H + h) * D + col0 + m0, o0, o1);
                }
            }
        }
        // ---- state carry in registers: S <- a S + (K (.) w)^T V
        if (own) {
            float u1[4][4], u2[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) u1[a][b] = u2[a][b] = 0.f;
            for (int s = 0; s < C; ++s) {
                const float4 kv = *reinterpret_cast<const float4*>(Ks + s * DP + k0);
                const float4 vv = *reinterpret_cast<const float4*>(Vs + s * VP + n0);
                const float w1 = ww[s], w2 = ww[C + s];
                const float ka[4] = {kv.x, kv.y, kv.z, kv.w};
                const float va[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    const float k1 = ka[a] * w1, k2 = ka[a] * w2;
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        u1[a][b] = fmaf(k1, va[b], u1[a][b]);
                        u2[a][b] = fmaf(k2, va[b], u2[a][b]);
                    }
                }
            }
            const float a1 = a_dec[0], a2 = a_dec[1];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    s1[a][b] = fmaf(a1, s1[a][b], u1[a][b]);
                    s2[a][b] = fmaf(a2, s2[a][b], u2[a][b]);
                }
        }
        __syncthreads();  // every readout of the old state copy is done
        if (own) {
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                *reinterpret_cast<float4*>(Ss + (k0 + a) * VP + n0) = make_float4(s1[a][0], s1[a][1], s1[a][2], s1[a][3]);
                *reinterpret_cast<float4*>(Ss + D * VP + (k0 + a) * VP + n0) = make_float4(s2[a][0], s2[a][1], s2[a][2], s2[a][3]);
            }
        }
    }
    if (own) {
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            *reinterpret_cast<float4*>(G1 + (size_t)(k0 + a) * D + col0 + n0) = make_float4(s1[a][0], s1[a][1], s1[a][2], s1[a][3]);
            *reinterpret_cast<float4*>(G2 + (size_t)(k0 + a) * D + col0 + n0) = make_float4(s2[a][0], s2[a][1], s2[a][2], s2[a][3]);
        }
    }
}

template <int D, int C, typename T>
static dsla_status launch_one(const PrefillParams& p, cudaStream_t s) {
    constexpr int DVS = 32, DP = D + 4, VP = DVS + 4, CP = C + 4;
    constexpr size_t smem = sizeof(float) * (2 * C * DP + C * VP + C * CP + 2 * D * VP + 6 * C) + sizeof(int) * 2 * C;
    static bool configured = false;  // per process; the attribute is per function and device-wide enough here
    cudaError_t e = cudaFuncSetAttribute(prefill_simt_kernel<D, C, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    (void)configured;
    if (e != cudaSuccess) return DSLA_ERR_CUDA;
    const long long blocks = (long long)p.N * p.H * (D / DVS);
    if (blocks > 0x7fffffffLL) return DSLA_ERR_UNSUPPORTED;
    prefill_simt_kernel<D, C, T><<<dim3((unsigned)blocks), dim3(256), smem, s>>>(p);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

template <int D, typename T>
static dsla_status launch_chunk(const PrefillParams& p, int chunk, cudaStream_t s) {
    switch (chunk) {
        case 16: return launch_one<D, 16, T>(p, s);
        case 32: return launch_one<D, 32, T>(p, s);
        case 64: return launch_one<D, 64, T>(p, s);
        default: return DSLA_ERR_UNSUPPORTED;
    }
}

dsla_status launch_prefill_simt(const PrefillParams& p, int d, int chunk, dsla_dtype dt, cudaStream_t s) {
    if (p.N == 0) return DSLA_OK;
    if (d == 128 && dt == DSLA_BF16) return launch_chunk<128, __nv_bfloat16>(p, chunk, s);
    if (d == 128 && dt == DSLA_F32) return launch_chunk<128, float>(p, chunk, s);
    if (d == 64 && dt == DSLA_BF16) return launch_chunk<64, __nv_bfloat16>(p, chunk, s);
    if (d == 64 && dt == DSLA_F32) return launch_chunk<64, float>(p, chunk, s);
    return DSLA_ERR_UNSUPPORTED;
}

}  // namespace dsla
