// Decode step of the dual-state linear attention layer (Sec. 4.1 applied to one new token):
//     S^i <- g^i S^i + k^T v  (i = history, recency),   o = scale * q (gamma S^1 + (1-gamma) S^2)
// One pass over the fp32 states: every element is loaded once, updated, used for the readout and
// stored back in place.  HBM-bound: 4*d*d*4 bytes of state traffic per (row, head).
#include "dsla_internal.cuh"

namespace dsla {

// A CTA owns (batch row, head, 32-column slab of d_v): all D rows of both states for those
// columns.  A row segment is 128 bytes, so each warp load instruction covers four full lines.
// The readout sum over d_k stays inside the CTA; no atomics, one writer per state element.
template <int D, typename T>
__global__ void __launch_bounds__(128) decode_kernel(const DecodeParams p) {
    constexpr int SLABS = D / 32;
    constexpr int RPT = D / 16;  // rows per thread
    const int slab = blockIdx.x % SLABS;
    const int h = (blockIdx.x / SLABS) % p.H;
    const int b = blockIdx.x / (SLABS * p.H);
    const int tid = threadIdx.x;
    const int c4 = tid & 7;   // float4 column group inside the slab
    const int r0 = tid >> 3;  // 0..15
    const int col = slab * 32 + c4 * 4;

    // The kernel is launched as a programmatic dependent of whatever precedes it in the stream: it may become
    // resident while that grid drains (hiding the launch latency), reads or writes nothing before this wait, and
    // lets its own successor do the same.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int slot = p.slots ? p.slots[b] : b;
    T* o = reinterpret_cast<T*>(p.o) + ((size_t)b * p.H + h) * D;
    if (slot < 0 || slot >= p.num_slots) {
        if (tid < 32) o[slab * 32 + tid] = from_f32<T>(0.f);
        return;
    }

    float* S1 = p.state + (((size_t)slot * 2 + 0) * p.H + h) * (size_t)(D * D);
    float* S2 = S1 + (size_t)p.H * D * D;

    // issue every state load first: 2 * RPT independent 16-byte loads per thread
    float4 s1[RPT], s2[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = r0 + 16 * i;
        s1[i] = __ldcs(reinterpret_cast<const float4*>(S1 + (size_t)r * D + col));
        s2[i] = __ldcs(reinterpret_cast<const float4*>(S2 + (size_t)r * D + col));
    }

    __shared__ float sq[D], sk[D];
    __shared__ float red[4][32];
    const size_t base = ((size_t)b * p.H + h) * D;
    for (int i = tid; i < D; i += 128) {
        sq[i] = to_f32(reinterpret_cast<const T*>(p.q)[base + i]) * p.scale;
        sk[i] = to_f32(reinterpret_cast<const T*>(p.k)[base + i]);
    }
    const T* vp = reinterpret_cast<const T*>(p.v) + base + col;
    const float v0 = to_f32(vp[0]), v1 = to_f32(vp[1]), v2 = to_f32(vp[2]), v3 = to_f32(vp[3]);
    const float g1 = p.g_hist[(size_t)b * p.H + h], g2 = p.g_rec[(size_t)b * p.H + h];
    const float gam = p.gamma[h], gam2 = 1.f - gam;
    __syncthreads();

    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = r0 + 16 * i;
        const float kk = sk[r], qq = sq[r];
        float4 x = s1[i], y = s2[i];
        x.x = fmaf(g1, x.x, kk * v0); x.y = fmaf(g1, x.y, kk * v1);
        x.z = fmaf(g1, x.z, kk * v2); x.w = fmaf(g1, x.w, kk * v3);
        y.x = fmaf(g2, y.x, kk * v0); y.y = fmaf(g2, y.y, kk * v1);
        y.z = fmaf(g2, y.z, kk * v2); y.w = fmaf(g2, y.w, kk * v3);
        __stcs(reinterpret_cast<float4*>(S1 + (size_t)r * D + col), x);
        __stcs(reinterpret_cast<float4*>(S2 + (size_t)r * D + col), y);
        a0 = fmaf(qq, gam * x.x + gam2 * y.x, a0);
        a1 = fmaf(qq, gam * x.y + gam2 * y.y, a1);
        a2 = fmaf(qq, gam * x.z + gam2 * y.z, a2);
        a3 = fmaf(qq, gam * x.w + gam2 * y.w, a3);
    }
    // sum over the 16 row groups: lanes differing in bits 3,4, then the four warps
#pragma unroll
    for (int m = 8; m <= 16; m <<= 1) {
        a0 += __shfl_xor_sync(0xffffffffu, a0, m);
        a1 += __shfl_xor_sync(0xffffffffu, a1, m);
        a2 += __shfl_xor_sync(0xffffffffu, a2, m);
        a3 += __shfl_xor_sync(0xffffffffu, a3, m);
    }
    const int lane = tid & 31, warp = tid >> 5;
    if (lane < 8) {
        red[warp][lane * 4 + 0] = a0; red[warp][lane * 4 + 1] = a1;
        red[warp][lane * 4 + 2] = a2; red[warp][lane * 4 + 3] = a3;
    }
    __syncthreads();
    if (tid < 32) {
        const float r = red[0][tid] + red[1][tid] + red[2][tid] + red[3][tid];
        o[slab * 32 + tid] = from_f32<T>(r);
    }
}

dsla_status launch_decode(const DecodeParams& p, int d, dsla_dtype dt, cudaStream_t s) {
    if (p.B == 0) return DSLA_OK;
    const long long blocks = (long long)p.B * p.H * (d / 32);
    if (blocks > 0x7fffffffLL) return DSLA_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t rc;
    if (d == 128 && dt == DSLA_BF16) rc = cudaLaunchKernelEx(&cfg, decode_kernel<128, __nv_bfloat16>, p);
    else if (d == 128 && dt == DSLA_F32) rc = cudaLaunchKernelEx(&cfg, decode_kernel<128, float>, p);
    else if (d == 64 && dt == DSLA_BF16) rc = cudaLaunchKernelEx(&cfg, decode_kernel<64, __nv_bfloat16>, p);
    else if (d == 64 && dt == DSLA_F32) rc = cudaLaunchKernelEx(&cfg, decode_kernel<64, float>, p);
    else return DSLA_ERR_UNSUPPORTED;
    if (rc != cudaSuccess) return DSLA_ERR_CUDA;
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // namespace dsla
