// Token-by-token prefill on CUDA cores, fp32 arithmetic, for the forms of the layer the chunkwise kernels do not
// cover: gates per key channel (the gated-linear-attention form of Sec. 2, G = alpha^T 1: one gate per state ROW) and
// n states with one blend weight each (Sec. 4.2; 1, 2, 4 or 8 states in the ablation of Sec. 5.5):
//     S^i_t = g^i_t (.) S^i_{t-1} + k_t^T v_t,        o_t = scale * q_t sum_i w_i S^i_t .
// This is the recurrence itself, not a chunked form: with one gate per row there is no single decay factor per token
// pair to mask a score matrix with, and the plain loop has no range problem for any gate value.  It is a correctness
// path (a few million tokens per second per layer), not a tuned one.
//
// CTA = (sequence, head, 32-column slab of d_v), 8 warps.  Warp w owns the four d_v columns 4 w .. 4 w + 3 of the
// slab; lane l owns the d_k rows l, l + 32, ..: the state slices of up to four states stay in registers for the whole
// sequence, the sum over d_k of the readout is a warp shuffle reduction, and the CTA synchronises only once per
// block of 16 tokens (to stage q, k, v and the gates in shared memory).  More than four states run as several
// launches that add to the output.
#include "dsla_internal.cuh"

namespace dsla {

namespace {

constexpr int TB = 16;      // tokens staged per round

template <int D, typename T, int NSG, bool VG>
__global__ void __launch_bounds__(256) prefill_recurrent_kernel(const RecurrentParams p) {
    constexpr int RPL = D / 32;     // d_k rows per lane
    __shared__ float sq[TB][D], sk[TB][D], sv[TB][32];
    __shared__ float sg[NSG][TB][VG ? D : 1];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slab = blockIdx.x % (D / 32);
    const int h = (blockIdx.x / (D / 32)) % p.H;
    const int n = blockIdx.x / ((D / 32) * p.H);
    const int t_begin = p.cu_seqlens ? p.cu_seqlens[n] : n * p.T;
    const int t_end = p.cu_seqlens ? p.cu_seqlens[n + 1] : (n + 1) * p.T;
    const int len = t_end - t_begin;
    const int slot = p.slots ? p.slots[n] : n;
    if (slot < 0 || slot >= p.num_slots) return;
    if (len <= 0 && p.use_initial_state) return;      // nothing to do, slot untouched
    const int col0 = slab * 32 + 4 * warp;            // this warp's first d_v column
    const size_t sstride = (size_t)p.H * D * D;
    float* S0 = p.state + (((size_t)slot * p.n_states_total + p.state_first) * p.H + h) * (size_t)(D * D);

    float s[NSG][RPL][4], w[NSG];
#pragma unroll
    for (int i = 0; i < NSG; ++i) {
        w[i] = (p.weights ? p.weights[(size_t)h * p.n_states_total + p.state_first + i]
                          : (p.state_first + i == 0 ? p.gamma[h] : 1.f - p.gamma[h])) * p.scale;
#pragma unroll
        for (int r = 0; r < RPL; ++r) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (p.use_initial_state) x = *reinterpret_cast<const float4*>(S0 + i * sstride + (size_t)(lane + 32 * r) * D + col0);
            s[i][r][0] = x.x; s[i][r][1] = x.y; s[i][r][2] = x.z; s[i][r][3] = x.w;
        }
    }
    const T* qg = reinterpret_cast<const T*>(p.q);
    const T* kg = reinterpret_cast<const T*>(p.k);
    const T* vg = reinterpret_cast<const T*>(p.v);
    T* og = reinterpret_cast<T*>(p.o);

    for (int c0 = 0; c0 < len; c0 += TB) {
        const int nt = min(TB, len - c0);
        __syncthreads();
        for (int idx = tid; idx < nt * D; idx += 256) {
            const int j = idx / D, c = idx % D;
            const size_t off = ((size_t)(t_begin + c0 + j) * p.H + h) * D + c;
            sq[j][c] = to_f32(qg[off]);
            sk[j][c] = to_f32(kg[off]);
            if (VG) {
#pragma unroll
                for (int i = 0; i < NSG; ++i) sg[i][j][c] = fmaxf(p.g[i][off], 0.f);
            }
        }
        for (int idx = tid; idx < nt * 32; idx += 256) {
            const int j = idx / 32, c = idx % 32;
            sv[j][c] = to_f32(vg[((size_t)(t_begin + c0 + j) * p.H + h) * D + slab * 32 + c]);
            if (!VG && c < NSG) sg[c][j][0] = fmaxf(p.g[c][(size_t)(t_begin + c0 + j) * p.H + h], 0.f);
        }
        __syncthreads();
#pragma unroll 4      // four tokens in flight: their shuffle reductions overlap (8 spills with vector gates)
        for (int j = 0; j < nt; ++j) {
            const float4 vv = *reinterpret_cast<const float4*>(&sv[j][4 * warp]);
            float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll
            for (int r = 0; r < RPL; ++r) {
                const int row = lane + 32 * r;
                const float kk = sk[j][row], qq = sq[j][row];
#pragma unroll
                for (int i = 0; i < NSG; ++i) {
                    const float g = VG ? sg[i][j][row] : sg[i][j][0];
                    s[i][r][0] = fmaf(g, s[i][r][0], kk * vv.x); s[i][r][1] = fmaf(g, s[i][r][1], kk * vv.y);
                    s[i][r][2] = fmaf(g, s[i][r][2], kk * vv.z); s[i][r][3] = fmaf(g, s[i][r][3], kk * vv.w);
                    const float qw = qq * w[i];
                    o0 = fmaf(qw, s[i][r][0], o0); o1 = fmaf(qw, s[i][r][1], o1);
                    o2 = fmaf(qw, s[i][r][2], o2); o3 = fmaf(qw, s[i][r][3], o3);
                }
            }
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) {
                o0 += __shfl_xor_sync(0xffffffffu, o0, m); o1 += __shfl_xor_sync(0xffffffffu, o1, m);
                o2 += __shfl_xor_sync(0xffffffffu, o2, m); o3 += __shfl_xor_sync(0xffffffffu, o3, m);
            }
            if (lane < 4) {
                T* dst = og + ((size_t)(t_begin + c0 + j) * p.H + h) * D + col0 + lane;
                float val = lane == 0 ? o0 : lane == 1 ? o1 : lane == 2 ? o2 : o3;
                if (p.accumulate) val += to_f32(*dst);
                *dst = from_f32<T>(val);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < NSG; ++i)
#pragma unroll
        for (int r = 0; r < RPL; ++r)
            *reinterpret_cast<float4*>(S0 + i * sstride + (size_t)(lane + 32 * r) * D + col0) =
                make_float4(s[i][r][0], s[i][r][1], s[i][r][2], s[i][r][3]);
}

template <int D, typename T, int NSG>
dsla_status launch_group(const RecurrentParams& p, cudaStream_t s) {
    const long long blocks = (long long)p.N * p.H * (D / 32);
    if (blocks > 0x7fffffffLL) return DSLA_ERR_UNSUPPORTED;
    if (p.per_channel) {
        if constexpr (NSG * D <= 256) prefill_recurrent_kernel<D, T, NSG, true><<<dim3((unsigned)blocks), dim3(256), 0, s>>>(p);
        else return DSLA_ERR_UNSUPPORTED;      // (never chosen: such groups would not fit the static shared memory)
    } else {
        prefill_recurrent_kernel<D, T, NSG, false><<<dim3((unsigned)blocks), dim3(256), 0, s>>>(p);
    }
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

template <int D, typename T>
dsla_status launch_all(RecurrentParams p, const float* const* gates, int n_states, cudaStream_t s) {
    // groups of up to four states (two when the gates are vectors and d = 128: shared memory); later groups add to the output
    const int grp = n_states >= 4 ? ((p.per_channel && D == 128) ? 2 : 4) : n_states;
    for (int first = 0; first < n_states; first += grp) {
        p.state_first = first;
        p.accumulate = first > 0;
        for (int i = 0; i < grp; ++i) p.g[i] = gates[first + i];
        dsla_status rc;
        switch (grp) {
            case 1: rc = launch_group<D, T, 1>(p, s); break;
            case 2: rc = launch_group<D, T, 2>(p, s); break;
            default: rc = launch_group<D, T, 4>(p, s); break;
        }
        if (rc != DSLA_OK) return rc;
    }
    return DSLA_OK;
}

}  // namespace

dsla_status launch_prefill_recurrent(const RecurrentParams& p, const float* const* gates, int n_states, int d, dsla_dtype dt,
                                     cudaStream_t s) {
    if (p.N == 0) return DSLA_OK;
    if (n_states != 1 && n_states != 2 && n_states != 4 && n_states != 8) return DSLA_ERR_UNSUPPORTED;
    if (d == 128 && dt == DSLA_BF16) return launch_all<128, __nv_bfloat16>(p, gates, n_states, s);
    if (d == 128 && dt == DSLA_F32) return launch_all<128, float>(p, gates, n_states, s);
    if (d == 64 && dt == DSLA_BF16) return launch_all<64, __nv_bfloat16>(p, gates, n_states, s);
    if (d == 64 && dt == DSLA_F32) return launch_all<64, float>(p, gates, n_states, s);
    return DSLA_ERR_UNSUPPORTED;
}

}  // namespace dsla
