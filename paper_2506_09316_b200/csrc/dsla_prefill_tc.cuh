// Pieces shared by the translation units of the tensor-core prefill (bf16, d = 128, chunk C = 64):
// launch parameters, the split of a sequence into segments along T, the layout of the segment
// summaries in the workspace, and the cold-path helpers that move a state between global memory and
// TMEM.  Functions here are inline or static.
#pragma once
#include "dsla_internal.cuh"
#include "tc_utils.cuh"

namespace dsla {

using namespace tc;

constexpr int C = 64;                 // tokens per chunk
constexpr int D = 128;                // head size
// One summary per (sequence, head, segment): U (both states, fp32 [2][D][D]) followed by the two
// segment decays A[2], padded to a multiple of 256 bytes.
constexpr size_t SUMMARY_STRIDE = 2 * D * D * sizeof(float) + 256;
constexpr int ORDER_MAX_N = 8192;     // packed batches up to this many sequences are visited longest first

struct TcParams {
    PrefillParams p;
    float* ws;          // summaries: [(n*H + h)*nseg + g] -> {U[2][D][D], A[2]}
    const float* init;  // initial states the segments start from: the slots themselves, or a snapshot of them
                        // [(n*H + h)][2][D][D] taken before the main grid when a sequence is split (the CTA of the
                        // last segment overwrites the slot while CTAs of earlier segments may not have read it yet)
    int nseg;           // segments per sequence (grid dimension)
    int cps;            // chunks per segment (mean)
    int skew8;          // eighths of a chunk by which consecutive segments get shorter (later segments start later: they
                        // first fold the summaries of all earlier segments into their initial state)
    const int* order;   // sequences by descending length (longest first), or nullptr for index order
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
// 32 bt_begin .. 32 bt_end - 1.  The fold is a chain of dependent rounds of loads.
static __device__ __noinline__ void init_state_pass(const float* base, int use_initial_state, const float* wsu, int g, int hi, int v,
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

// Final fp32 state of one (state, d_v lane) from TMEM to global memory [d_k][d_v], d_k rows 32 bt_begin .. 32 bt_end - 1
// (cold path, out of line).
static __device__ __noinline__ void store_state(float* dst, int v, uint32_t s_addr, int bt_begin, int bt_end) {
#pragma unroll 1
    for (int bt = bt_begin; bt < bt_end; ++bt) {
        uint32_t r[32];
        tmem_ld32(s_addr + 32 * bt, r);
        tc_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) dst[(size_t)(32 * bt + k) * D + v] = __uint_as_float(r[k]);
    }
}

// dsla_prefill_summary.cu: helper launches of the tensor-core prefill (all enqueue on s and count themselves)
bool make_tile_map(CUtensorMap* m, const void* base, int T_total, int H);
void launch_seq_order(const int32_t* cu, int N, int* order, cudaStream_t s);
void launch_state_snapshot(const PrefillParams& p, float* snap, cudaStream_t s);
dsla_status launch_summary(const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& tp, cudaStream_t s);
// dsla_prefill_tc_pair.cu: the cluster variant's main grid, and how many of its clusters fit on the device at once
dsla_status launch_main_pair(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& tp, bool dependent,
                             cudaStream_t s);
int pair_resident_clusters();

}  // namespace dsla
