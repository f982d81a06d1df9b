// Decode step of the dual-state linear attention layer (Sec. 4.1 applied to one new token):
//     S^i <- g^i S^i + k^T v  (i = history, recency),   o = scale * q (gamma S^1 + (1-gamma) S^2)
// One pass over the fp32 states: every element is loaded once, updated, used for the readout and
// stored back in place.  HBM-bound: 4*d*d*4 bytes of state traffic per (row, head) and state pair.
// The same kernel serves the n-state form (Sec. 4.2; 1, 2, 4 or 8 states with one blend weight each,
// o = scale * q sum_i w_i S^i), gates per key channel (the gated-linear-attention form of Sec. 2: one
// gate per state ROW), and batches in which only some rows belong to a DSLA layer (Sec. 4.5, App. D).
#include "dsla_internal.cuh"

namespace dsla {

// A CTA owns (batch row, head, 32-column slab of d_v): all D rows of every state for those
// columns.  A row segment is 128 bytes, so each warp load instruction covers four full lines.
// The readout sum over d_k stays inside the CTA; no atomics, one writer per state element.
// NS = number of states, VG = gates are vectors over the key channels.
template <int D, typename T, int NS, bool VG>
__global__ void __launch_bounds__(128) decode_kernel(const DecodeParams p) {
    constexpr int SLABS = D / 32;
    constexpr int RPT = D / 16;  // rows per thread
    constexpr int GRP = NS >= 2 ? 2 : 1;   // states streamed together (their loads are all issued before the first use)
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
    if (p.row_mask && p.row_mask[b] == 0) return;      // not a DSLA row in this layer: state and output stay as they are
    const int slot = p.slots ? p.slots[b] : b;
    T* o = reinterpret_cast<T*>(p.o) + ((size_t)b * p.H + h) * D;
    if (slot < 0 || slot >= p.num_slots) {
        if (tid < 32) o[slab * 32 + tid] = from_f32<T>(0.f);
        return;
    }

    const size_t sstride = (size_t)p.H * D * D;      // between the states of a slot
    float* S0 = p.state + (((size_t)slot * NS) * p.H + h) * (size_t)(D * D);

    // issue the loads of the first group first: GRP * RPT independent 16-byte loads per thread
    float4 s[GRP][RPT];
#pragma unroll
    for (int g = 0; g < GRP; ++g)
#pragma unroll
        for (int i = 0; i < RPT; ++i) s[g][i] = __ldcs(reinterpret_cast<const float4*>(S0 + g * sstride + (size_t)(r0 + 16 * i) * D + col));

    __shared__ float sq[D], sk[D];
    __shared__ float sg[VG ? NS : 1][VG ? D : 1];
    __shared__ float red[4][32];
    const size_t base = ((size_t)b * p.H + h) * D;
    for (int i = tid; i < D; i += 128) {
        sq[i] = to_f32(reinterpret_cast<const T*>(p.q)[base + i]) * p.scale;
        sk[i] = to_f32(reinterpret_cast<const T*>(p.k)[base + i]);
        if (VG) {
#pragma unroll
            for (int n = 0; n < NS; ++n) sg[n][i] = p.g[n][base + i];
        }
    }
    const T* vp = reinterpret_cast<const T*>(p.v) + base + col;
    const float v0 = to_f32(vp[0]), v1 = to_f32(vp[1]), v2 = to_f32(vp[2]), v3 = to_f32(vp[3]);
    float gs[NS], w[NS];
#pragma unroll
    for (int n = 0; n < NS; ++n) {
        gs[n] = VG ? 0.f : p.g[n][(size_t)b * p.H + h];
        w[n] = p.weights ? p.weights[(size_t)h * NS + n] : (n == 0 ? p.gamma[h] : 1.f - p.gamma[h]);
    }
    __syncthreads();

    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int n0 = 0; n0 < NS; n0 += GRP) {
        if (n0 > 0) {
#pragma unroll
            for (int g = 0; g < GRP; ++g)
#pragma unroll
                for (int i = 0; i < RPT; ++i)
                    s[g][i] = __ldcs(reinterpret_cast<const float4*>(S0 + (n0 + g) * sstride + (size_t)(r0 + 16 * i) * D + col));
        }
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const int r = r0 + 16 * i;
            const float kk = sk[r], qq = sq[r];
#pragma unroll
            for (int g = 0; g < GRP; ++g) {
                const float gg = VG ? sg[n0 + g][r] : gs[n0 + g];
                float4 x = s[g][i];
                x.x = fmaf(gg, x.x, kk * v0); x.y = fmaf(gg, x.y, kk * v1);
                x.z = fmaf(gg, x.z, kk * v2); x.w = fmaf(gg, x.w, kk * v3);
                __stcs(reinterpret_cast<float4*>(S0 + (n0 + g) * sstride + (size_t)r * D + col), x);
                const float qw = qq * w[n0 + g];
                a0 = fmaf(qw, x.x, a0); a1 = fmaf(qw, x.y, a1); a2 = fmaf(qw, x.z, a2); a3 = fmaf(qw, x.w, a3);
            }
        }
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

namespace {

template <int D, typename T, int NS, bool VG>
cudaError_t launch_variant(const cudaLaunchConfig_t* cfg, const DecodeParams& p) {
    return cudaLaunchKernelEx(cfg, decode_kernel<D, T, NS, VG>, p);
}

template <int D, typename T>
cudaError_t launch_states(const cudaLaunchConfig_t* cfg, const DecodeParams& p) {
    const bool vg = p.per_channel != 0;
    switch (p.n_states) {
        case 1: return vg ? launch_variant<D, T, 1, true>(cfg, p) : launch_variant<D, T, 1, false>(cfg, p);
        case 2: return vg ? launch_variant<D, T, 2, true>(cfg, p) : launch_variant<D, T, 2, false>(cfg, p);
        case 4: return vg ? launch_variant<D, T, 4, true>(cfg, p) : launch_variant<D, T, 4, false>(cfg, p);
        case 8: return vg ? launch_variant<D, T, 8, true>(cfg, p) : launch_variant<D, T, 8, false>(cfg, p);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

dsla_status launch_decode(const DecodeParams& p, int d, dsla_dtype dt, cudaStream_t s) {
    if (p.B == 0) return DSLA_OK;
    if (p.n_states != 1 && p.n_states != 2 && p.n_states != 4 && p.n_states != 8) return DSLA_ERR_UNSUPPORTED;
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
    if (d == 128 && dt == DSLA_BF16) rc = launch_states<128, __nv_bfloat16>(&cfg, p);
    else if (d == 128 && dt == DSLA_F32) rc = launch_states<128, float>(&cfg, p);
    else if (d == 64 && dt == DSLA_BF16) rc = launch_states<64, __nv_bfloat16>(&cfg, p);
    else if (d == 64 && dt == DSLA_F32) rc = launch_states<64, float>(&cfg, p);
    else return DSLA_ERR_UNSUPPORTED;
    if (rc != cudaSuccess) return DSLA_ERR_CUDA;
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // namespace dsla
