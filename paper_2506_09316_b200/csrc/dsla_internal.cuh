// Internal declarations shared by the translation units of libdsla (never installed).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dsla.h"

struct dsla_state {
    float* data;          // [num_slots][n_states][H][d_k][d_v]
    int* status;          // device status word (0 = ok)
    int num_slots, n_states, H, d_k, d_v;
    int owns_data;
    int device;
};

namespace dsla {

// Launch parameters of the prefill kernels (all pointers device).
struct PrefillParams {
    const void *q, *k, *v;
    void* o;
    const float *g_hist, *g_rec, *gamma;
    const int32_t* cu_seqlens;  // may be null (dense)
    const int32_t* slots;       // may be null
    float* state;               // [num_slots][n_total][H][D][D]; this call works on states state_first, state_first + 1
    int* status;
    int N, T, H, num_slots;
    int max_chunks;             // ceil(max_seqlen / C)
    float scale;
    int use_initial_state;
    // n-state form run two states at a time (tensor-core kernel only; the dual-state path leaves the defaults)
    const float* weights;       // [H, n_total] blend weights, or nullptr: (gamma, 1 - gamma)
    int n_total;                // states per slot (2 for the dual-state layer)
    int state_first;            // index of the first of the two states of this call
    int single;                 // only state_first exists (n = 1): the second state of the kernel runs with weight 0 on the first
                                // state's gates, starts from zero and is never loaded from or stored to the slot
};

struct DecodeParams {
    const void *q, *k, *v;
    void* o;
    const float* g[8];          // gate of every state: [B, H], or [B, H, d_k] when per_channel
    const float* gamma;         // [H] (dual state: weights gamma, 1 - gamma) when weights == nullptr
    const float* weights;       // [H, n_states] or nullptr
    const int32_t* slots;
    const uint8_t* row_mask;    // [B] or nullptr: rows with 0 are left untouched
    float* state;               // [num_slots][n_states][H][D][D]
    int B, H, num_slots, n_states, per_channel;
    float scale;
};

// Launch parameters of the token-by-token prefill (one group of up to four states per launch).
struct RecurrentParams {
    const void *q, *k, *v;
    void* o;
    const float* g[4];          // gates of this launch's states: [T_total, H], or [T_total, H, d_k] when per_channel
    const float* weights;       // [H, n_states_total], or nullptr: two states weighted (gamma, 1 - gamma)
    const float* gamma;         // [H], used when weights == nullptr
    const int32_t *cu_seqlens, *slots;
    float* state;               // [num_slots][n_states_total][H][D][D]
    int N, T, H, num_slots, n_states_total, state_first, per_channel, use_initial_state, accumulate;
    float scale;
};

void count_launch(int n = 1);

// dsla_api.cu: argument checks + dispatch shared by the prefill entry points
dsla_status prefill_checked(const dsla_prefill_args* a, dsla_state* st, cudaStream_t s);
// dsla_decode.cu
dsla_status launch_decode(const DecodeParams& p, int d, dsla_dtype dt, cudaStream_t s);
// dsla_gate_project.cu
dsla_status launch_gate_project(const dsla_gate_project_args* a, cudaStream_t s);
dsla_status gate_project_last_error();
// dsla_prefill_recurrent.cu: gates[i] is the gate tensor of state i (n_states of them)
dsla_status launch_prefill_recurrent(const RecurrentParams& p, const float* const* gates, int n_states, int d, dsla_dtype dt,
                                     cudaStream_t s);
// dsla_prefill_simt.cu
dsla_status launch_prefill_simt(const PrefillParams& p, int d, int chunk, dsla_dtype dt, cudaStream_t s);
// dsla_prefill_summary.cu: one warp waits, with the given poll limit, on a barrier nobody arrives at
void launch_bounded_wait_selftest(int* status, unsigned max_polls, cudaStream_t s);
// dsla_prefill_tc.cu (pair = the cluster variant of dsla_prefill_tc_pair.cu)
bool prefill_tc_available();
size_t prefill_tc_workspace_bytes(const dsla_prefill_args* a, bool pair);
dsla_status launch_prefill_tc(const PrefillParams& p, const dsla_prefill_args* a, bool pair, cudaStream_t s);

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

}  // namespace dsla
