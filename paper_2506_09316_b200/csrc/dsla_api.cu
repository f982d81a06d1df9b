// C-ABI entry points of libdsla: argument checks, state store management, kernel dispatch.
#include <atomic>
#include <mutex>
#include <cstdio>
#include <cstdlib>
#include <new>

#include "dsla_internal.cuh"

namespace dsla {
static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

__global__ void zero_slots_kernel(float* data, const int32_t* slots, int num_slots, size_t slot_elems) {
    const int s = slots[blockIdx.y];
    if (s < 0 || s >= num_slots) return;
    float4* base = reinterpret_cast<float4*>(data + (size_t)s * slot_elems);
    const size_t n4 = slot_elems / 4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x)
        base[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// o += t over n8 pieces of eight bf16 (fp32 sum, one rounding): the share of a later pair of states of the n-state prefill
__global__ void __launch_bounds__(256) add_bf16_kernel(uint4* __restrict__ o, const uint4* __restrict__ t, size_t n8) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
        uint4 a = o[i];
        const uint4 b = __ldcs(t + i);
        __nv_bfloat162* pa = reinterpret_cast<__nv_bfloat162*>(&a);
        const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 x = __bfloat1622float2(pa[e]), y = __bfloat1622float2(pb[e]);
            pa[e] = __floats2bfloat162_rn(x.x + y.x, x.y + y.y);
        }
        o[i] = a;
    }
}
}  // namespace dsla

using namespace dsla;

// A store belongs to the device that was current when it was created; kernels for it must be launched there.
static bool on_store_device(const dsla_state* st) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == st->device;
}
static bool supported_d(int dk, int dv) { return dk == dv && (dk == 64 || dk == 128); }
static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
static size_t esize(dsla_dtype dt) { return dt == DSLA_F32 ? 4 : 2; }

extern "C" {

const char* dsla_status_string(dsla_status s) {
    switch (s) {
        case DSLA_OK: return "DSLA_OK";
        case DSLA_ERR_INVALID_ARG: return "DSLA_ERR_INVALID_ARG";
        case DSLA_ERR_UNSUPPORTED: return "DSLA_ERR_UNSUPPORTED";
        case DSLA_ERR_CUDA: return "DSLA_ERR_CUDA";
        case DSLA_ERR_OOM: return "DSLA_ERR_OOM";
        case DSLA_ERR_TIMEOUT: return "DSLA_ERR_TIMEOUT";
        case DSLA_ERR_SCRATCH_LIMIT: return "DSLA_ERR_SCRATCH_LIMIT";
    }
    return "DSLA_ERR_UNKNOWN";
}

uint64_t dsla_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

static bool supported_n(int n) { return n == 1 || n == 2 || n == 4 || n == 8; }

size_t dsla_state_bytes_n(int num_slots, int n_states, int H, int d_k, int d_v) {
    if (num_slots <= 0 || n_states <= 0 || H <= 0 || d_k <= 0 || d_v <= 0) return 0;
    return (size_t)num_slots * (size_t)n_states * (size_t)H * (size_t)d_k * (size_t)d_v * sizeof(float);
}

size_t dsla_state_bytes(int num_slots, int H, int d_k, int d_v) { return dsla_state_bytes_n(num_slots, 2, H, d_k, d_v); }

dsla_status dsla_state_alloc(dsla_state** out, int num_slots, int H, int d_k, int d_v, void* ext_buf, size_t ext_bytes) {
    return dsla_state_alloc_n(out, num_slots, 2, H, d_k, d_v, ext_buf, ext_bytes);
}

dsla_status dsla_state_alloc_n(dsla_state** out, int num_slots, int n_states, int H, int d_k, int d_v, void* ext_buf,
                               size_t ext_bytes) {
    if (!out) return DSLA_ERR_INVALID_ARG;
    *out = nullptr;
    if (num_slots <= 0 || n_states <= 0 || H <= 0 || d_k <= 0 || d_v <= 0) return DSLA_ERR_INVALID_ARG;
    if (!supported_d(d_k, d_v) || !supported_n(n_states)) return DSLA_ERR_UNSUPPORTED;
    const size_t bytes = dsla_state_bytes_n(num_slots, n_states, H, d_k, d_v);
    if (ext_buf && (ext_bytes < bytes || !aligned(ext_buf, 256))) return DSLA_ERR_INVALID_ARG;
    dsla_state* st = new (std::nothrow) dsla_state();
    if (!st) return DSLA_ERR_OOM;
    st->num_slots = num_slots; st->n_states = n_states; st->H = H; st->d_k = d_k; st->d_v = d_v;
    st->owns_data = ext_buf ? 0 : 1;
    st->data = static_cast<float*>(ext_buf);
    st->status = nullptr;
    if (cudaGetDevice(&st->device) != cudaSuccess) { delete st; return DSLA_ERR_CUDA; }
    if (!ext_buf) {
        cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&st->data), bytes);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            delete st;
            return e == cudaErrorMemoryAllocation ? DSLA_ERR_OOM : DSLA_ERR_CUDA;
        }
    }
    if (cudaMalloc(reinterpret_cast<void**>(&st->status), 256) != cudaSuccess ||
        cudaMemset(st->status, 0, 256) != cudaSuccess) {
        (void)cudaGetLastError();
        if (st->owns_data) cudaFree(st->data);
        if (st->status) cudaFree(st->status);
        delete st;
        return DSLA_ERR_CUDA;
    }
    *out = st;
    return DSLA_OK;
}

dsla_status dsla_state_free(dsla_state* st) {
    if (!st) return DSLA_OK;
    dsla_status rc = DSLA_OK;
    if (st->owns_data && st->data && cudaFree(st->data) != cudaSuccess) rc = DSLA_ERR_CUDA;
    if (st->status && cudaFree(st->status) != cudaSuccess) rc = DSLA_ERR_CUDA;
    delete st;
    return rc;
}

void* dsla_state_data(dsla_state* st) { return st ? st->data : nullptr; }

dsla_status dsla_state_zero(dsla_state* st, const int32_t* slots_dev, int n, void* cuda_stream) {
    if (!st) return DSLA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t slot_elems = (size_t)st->n_states * st->H * st->d_k * st->d_v;
    if (!slots_dev) {
        return cudaMemsetAsync(st->data, 0, slot_elems * sizeof(float) * st->num_slots, s) == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
    }
    if (n < 0 || n > 65535) return DSLA_ERR_INVALID_ARG;
    if (n == 0) return DSLA_OK;
    zero_slots_kernel<<<dim3(32, n), 256, 0, s>>>(st->data, slots_dev, st->num_slots, slot_elems);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

dsla_status dsla_state_last_error(dsla_state* st) {
    if (!st) return DSLA_ERR_INVALID_ARG;
    int host = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return DSLA_ERR_CUDA;
    if (cudaMemcpy(&host, st->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return DSLA_ERR_CUDA;
    if (host != 0 && cudaMemset(st->status, 0, sizeof(int)) != cudaSuccess) return DSLA_ERR_CUDA;
    if (host == 0) return DSLA_OK;
    return host == (int)DSLA_ERR_INVALID_ARG ? DSLA_ERR_INVALID_ARG : DSLA_ERR_TIMEOUT;
}

dsla_status dsla_selftest_bounded_wait(dsla_state* st, unsigned max_polls, void* cuda_stream) {
    if (!st || max_polls == 0 || max_polls > 1000000u) return DSLA_ERR_INVALID_ARG;
    launch_bounded_wait_selftest(st->status, max_polls, static_cast<cudaStream_t>(cuda_stream));
    return cudaGetLastError() == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

// ---- prefill ------------------------------------------------------------------------------
static dsla_impl resolve_impl(const dsla_prefill_args* a) {
    if (a->gate_layout == DSLA_GATE_PER_KEY_CHANNEL) return DSLA_IMPL_SIMT;
    if (a->impl == DSLA_IMPL_SIMT || a->impl == DSLA_IMPL_TENSOR || a->impl == DSLA_IMPL_TENSOR_PAIR) return a->impl;
    return (a->dtype == DSLA_BF16 && a->d_k == 128 && prefill_tc_available()) ? DSLA_IMPL_TENSOR : DSLA_IMPL_SIMT;
}

static dsla_status check_prefill_sizes(const dsla_prefill_args* a) {
    if (!a) return DSLA_ERR_INVALID_ARG;
    if (a->N < 0 || a->T_total < 0 || a->H <= 0 || a->max_seqlen < 0) return DSLA_ERR_INVALID_ARG;
    if (a->dtype != DSLA_F32 && a->dtype != DSLA_BF16) return DSLA_ERR_INVALID_ARG;
    if (a->d_k <= 0 || a->d_v <= 0) return DSLA_ERR_INVALID_ARG;
    if (!supported_d(a->d_k, a->d_v)) return DSLA_ERR_UNSUPPORTED;
    if (!a->cu_seqlens) {
        if (a->T < 0 || (long long)a->N * a->T != a->T_total || a->max_seqlen < a->T) return DSLA_ERR_INVALID_ARG;
    } else if (a->max_seqlen > a->T_total) {
        return DSLA_ERR_INVALID_ARG;
    }
    if (a->impl != DSLA_IMPL_AUTO && a->impl != DSLA_IMPL_SIMT && a->impl != DSLA_IMPL_TENSOR && a->impl != DSLA_IMPL_TENSOR_PAIR)
        return DSLA_ERR_INVALID_ARG;
    if (a->gate_layout != DSLA_GATE_SCALAR && a->gate_layout != DSLA_GATE_PER_KEY_CHANNEL) return DSLA_ERR_INVALID_ARG;
    if (a->gate_layout == DSLA_GATE_PER_KEY_CHANNEL) {      // the token-by-token CUDA-core kernel; chunk is ignored
        return (a->impl == DSLA_IMPL_TENSOR || a->impl == DSLA_IMPL_TENSOR_PAIR) ? DSLA_ERR_UNSUPPORTED : DSLA_OK;
    }
    const dsla_impl impl = resolve_impl(a);
    const int chunk = a->chunk == 0 ? 64 : a->chunk;
    if (impl == DSLA_IMPL_SIMT) {
        if (chunk != 16 && chunk != 32 && chunk != 64) return DSLA_ERR_UNSUPPORTED;
    } else {
        if (a->dtype != DSLA_BF16 || a->d_k != 128 || chunk != 64 || !prefill_tc_available()) return DSLA_ERR_UNSUPPORTED;
    }
    return DSLA_OK;
}

size_t dsla_prefill_workspace_bytes(const dsla_prefill_args* a) {
    if (check_prefill_sizes(a) != DSLA_OK) return 0;
    const dsla_impl impl = resolve_impl(a);
    return impl == DSLA_IMPL_SIMT ? 0 : prefill_tc_workspace_bytes(a, impl == DSLA_IMPL_TENSOR_PAIR);
}

static dsla_status prefill_device(const dsla_prefill_args* a, dsla_state* st, cudaStream_t s) {
    dsla_status rc = check_prefill_sizes(a);
    if (rc != DSLA_OK) return rc;
    if (!st) return DSLA_ERR_INVALID_ARG;
    if (st->n_states != 2 || st->H != a->H || st->d_k != a->d_k || st->d_v != a->d_v) return DSLA_ERR_INVALID_ARG;
    if (!a->slots && a->N > st->num_slots) return DSLA_ERR_INVALID_ARG;
    if (!on_store_device(st)) return DSLA_ERR_INVALID_ARG;
    if (a->N == 0) return DSLA_OK;
    if (!a->gamma) return DSLA_ERR_INVALID_ARG;
    if (a->T_total > 0) {
        if (!a->q || !a->k || !a->v || !a->o || !a->g_hist || !a->g_rec) return DSLA_ERR_INVALID_ARG;
        if (!aligned(a->q, 16) || !aligned(a->k, 16) || !aligned(a->v, 16) || !aligned(a->o, 16)) return DSLA_ERR_INVALID_ARG;
        if (!aligned(a->g_hist, 4) || !aligned(a->g_rec, 4)) return DSLA_ERR_INVALID_ARG;
    }
    const size_t need = dsla_prefill_workspace_bytes(a);
    if (need > 0 && (!a->workspace || a->workspace_bytes < need || !aligned(a->workspace, 256))) return DSLA_ERR_INVALID_ARG;
    if (!(a->scale == a->scale)) return DSLA_ERR_INVALID_ARG;

    PrefillParams p{};
    p.q = a->q; p.k = a->k; p.v = a->v; p.o = a->o;
    p.g_hist = a->g_hist; p.g_rec = a->g_rec; p.gamma = a->gamma;
    p.cu_seqlens = a->cu_seqlens; p.slots = a->slots;
    p.state = st->data; p.status = st->status;
    p.N = a->N; p.T = a->T; p.H = a->H; p.num_slots = st->num_slots;
    const int chunk = a->chunk == 0 ? 64 : a->chunk;
    p.max_chunks = (a->max_seqlen + chunk - 1) / chunk;
    p.scale = a->scale; p.use_initial_state = a->use_initial_state ? 1 : 0;
    p.weights = nullptr; p.n_total = 2; p.state_first = 0; p.single = 0;
    if (a->gate_layout == DSLA_GATE_PER_KEY_CHANNEL) {
        // the dual state as two states whose weights the kernel derives from gamma: (gamma, 1 - gamma)
        RecurrentParams r{};
        r.q = a->q; r.k = a->k; r.v = a->v; r.o = a->o;
        r.weights = nullptr; r.cu_seqlens = a->cu_seqlens; r.slots = a->slots; r.state = st->data;
        r.N = a->N; r.T = a->T; r.H = a->H; r.num_slots = st->num_slots; r.n_states_total = 2;
        r.per_channel = 1; r.use_initial_state = a->use_initial_state ? 1 : 0; r.scale = a->scale;
        r.gamma = a->gamma;
        const float* gates[2] = {a->g_hist, a->g_rec};
        return launch_prefill_recurrent(r, gates, 2, a->d_k, a->dtype, s);
    }
    const dsla_impl impl = resolve_impl(a);
    if (impl != DSLA_IMPL_SIMT) return launch_prefill_tc(p, a, impl == DSLA_IMPL_TENSOR_PAIR, s);
    return launch_prefill_simt(p, a->d_k, chunk, a->dtype, s);
}

}  // extern "C"
namespace dsla {
dsla_status prefill_checked(const dsla_prefill_args* a, dsla_state* st, cudaStream_t s) { return prefill_device(a, st, s); }
}
extern "C" {

dsla_status dsla_prefill(const dsla_prefill_args* a, dsla_state* st, void* cuda_stream) {
    return prefill_device(a, st, static_cast<cudaStream_t>(cuda_stream));
}

// ---- decode -------------------------------------------------------------------------------
static dsla_status check_decode(const dsla_decode_args* a, dsla_state* st) {
    if (!a || !st) return DSLA_ERR_INVALID_ARG;
    if (a->B < 0 || a->H <= 0 || a->d_k <= 0 || a->d_v <= 0) return DSLA_ERR_INVALID_ARG;
    if (a->dtype != DSLA_F32 && a->dtype != DSLA_BF16) return DSLA_ERR_INVALID_ARG;
    if (!supported_d(a->d_k, a->d_v)) return DSLA_ERR_UNSUPPORTED;
    if (st->n_states != 2 || st->H != a->H || st->d_k != a->d_k || st->d_v != a->d_v) return DSLA_ERR_INVALID_ARG;
    if (!a->slots && a->B > st->num_slots) return DSLA_ERR_INVALID_ARG;
    if (!(a->scale == a->scale)) return DSLA_ERR_INVALID_ARG;
    if (a->gate_layout != DSLA_GATE_SCALAR && a->gate_layout != DSLA_GATE_PER_KEY_CHANNEL) return DSLA_ERR_INVALID_ARG;
    if (!on_store_device(st)) return DSLA_ERR_INVALID_ARG;
    return DSLA_OK;
}

static dsla_status decode_device(const dsla_decode_args* a, dsla_state* st, cudaStream_t s) {
    dsla_status rc = check_decode(a, st);
    if (rc != DSLA_OK) return rc;
    if (a->B == 0) return DSLA_OK;
    if (!a->q || !a->k || !a->v || !a->o || !a->g_hist || !a->g_rec || !a->gamma) return DSLA_ERR_INVALID_ARG;
    if (!aligned(a->q, 16) || !aligned(a->k, 16) || !aligned(a->v, 16) || !aligned(a->o, 16)) return DSLA_ERR_INVALID_ARG;
    DecodeParams p{};
    p.q = a->q; p.k = a->k; p.v = a->v; p.o = a->o;
    p.g[0] = a->g_hist; p.g[1] = a->g_rec; p.gamma = a->gamma; p.weights = nullptr; p.slots = a->slots;
    p.row_mask = a->row_mask; p.n_states = 2; p.per_channel = a->gate_layout == DSLA_GATE_PER_KEY_CHANNEL;
    p.state = st->data; p.B = a->B; p.H = a->H; p.num_slots = st->num_slots; p.scale = a->scale;
    return launch_decode(p, a->d_k, a->dtype, s);
}

// ---- n states -----------------------------------------------------------------------------
dsla_status dsla_nstate_decode_step(const dsla_nstate_decode_args* a, dsla_state* st, void* cuda_stream) {
    if (!a || !st) return DSLA_ERR_INVALID_ARG;
    if (a->B < 0 || a->H <= 0 || a->d_k <= 0 || a->d_v <= 0 || a->n_states <= 0) return DSLA_ERR_INVALID_ARG;
    if (a->dtype != DSLA_F32 && a->dtype != DSLA_BF16) return DSLA_ERR_INVALID_ARG;
    if (a->gate_layout != DSLA_GATE_SCALAR && a->gate_layout != DSLA_GATE_PER_KEY_CHANNEL) return DSLA_ERR_INVALID_ARG;
    if (!supported_d(a->d_k, a->d_v) || !supported_n(a->n_states)) return DSLA_ERR_UNSUPPORTED;
    if (st->n_states != a->n_states || st->H != a->H || st->d_k != a->d_k || st->d_v != a->d_v) return DSLA_ERR_INVALID_ARG;
    if (!a->slots && a->B > st->num_slots) return DSLA_ERR_INVALID_ARG;
    if (!(a->scale == a->scale) || !on_store_device(st)) return DSLA_ERR_INVALID_ARG;
    if (a->B == 0) return DSLA_OK;
    if (!a->q || !a->k || !a->v || !a->o || !a->gates || !a->weights) return DSLA_ERR_INVALID_ARG;
    if (!aligned(a->q, 16) || !aligned(a->k, 16) || !aligned(a->v, 16) || !aligned(a->o, 16)) return DSLA_ERR_INVALID_ARG;
    DecodeParams p{};
    p.q = a->q; p.k = a->k; p.v = a->v; p.o = a->o;
    const bool pc = a->gate_layout == DSLA_GATE_PER_KEY_CHANNEL;
    const size_t gstride = (size_t)a->B * a->H * (pc ? a->d_k : 1);
    for (int i = 0; i < a->n_states; ++i) p.g[i] = a->gates + (size_t)i * gstride;
    p.gamma = nullptr; p.weights = a->weights; p.slots = a->slots; p.row_mask = a->row_mask;
    p.n_states = a->n_states; p.per_channel = pc ? 1 : 0;
    p.state = st->data; p.B = a->B; p.H = a->H; p.num_slots = st->num_slots; p.scale = a->scale;
    return launch_decode(p, a->d_k, a->dtype, static_cast<cudaStream_t>(cuda_stream));
}

// the n-state prefill as a dual-state prefill problem of the same sizes (what the segment plan and the workspace depend on)
static dsla_prefill_args nstate_as_prefill_args(const dsla_nstate_prefill_args* a) {
    dsla_prefill_args b{};
    b.q = a->q; b.k = a->k; b.v = a->v; b.o = a->o;
    b.cu_seqlens = a->cu_seqlens; b.slots = a->slots;
    b.N = a->N; b.T = a->T; b.T_total = a->T_total; b.max_seqlen = a->max_seqlen; b.H = a->H; b.d_k = a->d_k; b.d_v = a->d_v;
    b.chunk = 64; b.dtype = a->dtype; b.scale = a->scale; b.use_initial_state = a->use_initial_state;
    b.impl = DSLA_IMPL_TENSOR; b.gate_layout = DSLA_GATE_SCALAR;
    b.workspace = a->workspace; b.workspace_bytes = a->workspace_bytes;
    return b;
}

static dsla_status check_nstate_prefill_sizes(const dsla_nstate_prefill_args* a) {
    if (!a) return DSLA_ERR_INVALID_ARG;
    if (a->N < 0 || a->T_total < 0 || a->H <= 0 || a->d_k <= 0 || a->d_v <= 0 || a->n_states <= 0 || a->max_seqlen < 0) return DSLA_ERR_INVALID_ARG;
    if (a->dtype != DSLA_F32 && a->dtype != DSLA_BF16) return DSLA_ERR_INVALID_ARG;
    if (a->gate_layout != DSLA_GATE_SCALAR && a->gate_layout != DSLA_GATE_PER_KEY_CHANNEL) return DSLA_ERR_INVALID_ARG;
    if (a->impl != DSLA_IMPL_AUTO && a->impl != DSLA_IMPL_SIMT && a->impl != DSLA_IMPL_TENSOR) return DSLA_ERR_INVALID_ARG;
    if (!supported_d(a->d_k, a->d_v) || !supported_n(a->n_states)) return DSLA_ERR_UNSUPPORTED;
    if (!a->cu_seqlens) {
        if (a->T < 0 || (long long)a->N * a->T != a->T_total || a->max_seqlen < a->T) return DSLA_ERR_INVALID_ARG;
    } else if (a->max_seqlen > a->T_total) {
        return DSLA_ERR_INVALID_ARG;
    }
    return DSLA_OK;
}

// pairs of states (or the single state) through the chunkwise tensor-core kernel: bf16, d = 128, scalar gates
static bool nstate_tensor_applies(const dsla_nstate_prefill_args* a) {
    return a->dtype == DSLA_BF16 && a->d_k == 128 && a->gate_layout == DSLA_GATE_SCALAR && prefill_tc_available();
}

// pairs after the first write their share of o to a scratch tensor that is then added to o
static size_t nstate_o_scratch_bytes(const dsla_nstate_prefill_args* a) {
    return a->n_states > 2 ? (((size_t)a->T_total * a->H * a->d_v * 2 + 255) & ~(size_t)255) : 0;
}

size_t dsla_nstate_prefill_workspace_bytes(const dsla_nstate_prefill_args* a) {
    if (check_nstate_prefill_sizes(a) != DSLA_OK || a->impl == DSLA_IMPL_SIMT || !nstate_tensor_applies(a)) return 0;
    const dsla_prefill_args b = nstate_as_prefill_args(a);
    return prefill_tc_workspace_bytes(&b, false) + nstate_o_scratch_bytes(a);
}

dsla_status dsla_nstate_prefill(const dsla_nstate_prefill_args* a, dsla_state* st, void* cuda_stream) {
    if (!a || !st) return DSLA_ERR_INVALID_ARG;
    const dsla_status rc0 = check_nstate_prefill_sizes(a);
    if (rc0 != DSLA_OK) return rc0;
    if (a->impl == DSLA_IMPL_TENSOR && !nstate_tensor_applies(a)) return DSLA_ERR_UNSUPPORTED;
    if (st->n_states != a->n_states || st->H != a->H || st->d_k != a->d_k || st->d_v != a->d_v) return DSLA_ERR_INVALID_ARG;
    if (!a->slots && a->N > st->num_slots) return DSLA_ERR_INVALID_ARG;
    if (!(a->scale == a->scale) || !on_store_device(st)) return DSLA_ERR_INVALID_ARG;
    if (a->N == 0) return DSLA_OK;
    if (!a->weights) return DSLA_ERR_INVALID_ARG;
    if (a->T_total > 0) {
        if (!a->q || !a->k || !a->v || !a->o || !a->gates) return DSLA_ERR_INVALID_ARG;
        if (!aligned(a->q, 16) || !aligned(a->k, 16) || !aligned(a->v, 16) || !aligned(a->o, 16)) return DSLA_ERR_INVALID_ARG;
    }
    if (a->impl != DSLA_IMPL_SIMT && nstate_tensor_applies(a) && a->T_total > 0) {
        const dsla_prefill_args b = nstate_as_prefill_args(a);
        const size_t need_tc = prefill_tc_workspace_bytes(&b, false), need = need_tc + nstate_o_scratch_bytes(a);
        if (need > 0 && (!a->workspace || a->workspace_bytes < need || !aligned(a->workspace, 256))) return DSLA_ERR_INVALID_ARG;
        if (!aligned(a->gates, 4)) return DSLA_ERR_INVALID_ARG;
        void* o_scratch = static_cast<char*>(a->workspace) + need_tc;
        const size_t n8 = (size_t)a->T_total * a->H * a->d_v / 8;
        cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
        PrefillParams p{};
        p.q = a->q; p.k = a->k; p.v = a->v; p.o = a->o;
        p.gamma = nullptr; p.cu_seqlens = a->cu_seqlens; p.slots = a->slots;
        p.state = st->data; p.status = st->status;
        p.N = a->N; p.T = a->T; p.H = a->H; p.num_slots = st->num_slots;
        p.max_chunks = (a->max_seqlen + 63) / 64;
        p.scale = a->scale; p.use_initial_state = a->use_initial_state ? 1 : 0;
        p.weights = a->weights; p.n_total = a->n_states;
        const size_t gs = (size_t)a->T_total * a->H;
        for (int first = 0; first < a->n_states; first += 2) {      // one pass of the dual-state kernel per pair of states
            p.g_hist = a->gates + (size_t)first * gs;
            p.single = a->n_states == 1;
            p.g_rec = a->gates + (size_t)(p.single ? first : first + 1) * gs;
            p.state_first = first;
            p.o = first == 0 ? a->o : o_scratch;
            const dsla_status rc = launch_prefill_tc(p, &b, false, s);
            if (rc != DSLA_OK) return rc;
            if (first > 0) {
                const size_t blocks = (n8 + 255) / 256;
                add_bf16_kernel<<<dim3((unsigned)(blocks < 148 * 8 ? blocks : 148 * 8)), dim3(256), 0, s>>>(
                    static_cast<uint4*>(a->o), static_cast<const uint4*>(o_scratch), n8);
                count_launch();
                if (cudaGetLastError() != cudaSuccess) return DSLA_ERR_CUDA;
            }
        }
        return DSLA_OK;
    }
    RecurrentParams r{};
    r.q = a->q; r.k = a->k; r.v = a->v; r.o = a->o;
    r.weights = a->weights; r.gamma = nullptr; r.cu_seqlens = a->cu_seqlens; r.slots = a->slots; r.state = st->data;
    r.N = a->N; r.T = a->T; r.H = a->H; r.num_slots = st->num_slots; r.n_states_total = a->n_states;
    const bool pc = a->gate_layout == DSLA_GATE_PER_KEY_CHANNEL;
    r.per_channel = pc ? 1 : 0; r.use_initial_state = a->use_initial_state ? 1 : 0; r.scale = a->scale;
    const size_t gstride = (size_t)a->T_total * a->H * (pc ? a->d_k : 1);
    const float* gates[8];
    for (int i = 0; i < a->n_states; ++i) gates[i] = a->gates + (size_t)i * gstride;
    return launch_prefill_recurrent(r, gates, a->n_states, a->d_k, a->dtype, static_cast<cudaStream_t>(cuda_stream));
}

dsla_status dsla_decode_step(const dsla_decode_args* a, dsla_state* st, void* cuda_stream) {
    return decode_device(a, st, static_cast<cudaStream_t>(cuda_stream));
}

// ---- gate producer ------------------------------------------------------------------------
dsla_status dsla_gate_project(const dsla_gate_project_args* a, void* cuda_stream) {
    if (!a || a->T < 0 || a->H <= 0 || a->D_model <= 0) return DSLA_ERR_INVALID_ARG;
    if (a->H % 8 != 0 || 2 * a->H > 256 || a->D_model % 64 != 0) return DSLA_ERR_UNSUPPORTED;
    if (a->T == 0) return DSLA_OK;
    if (!a->x || !a->w || !a->g_hist || !a->g_rec) return DSLA_ERR_INVALID_ARG;
    if (!aligned(a->x, 16) || !aligned(a->w, 16) || !aligned(a->g_hist, 16) || !aligned(a->g_rec, 16)) return DSLA_ERR_INVALID_ARG;
    return launch_gate_project(a, static_cast<cudaStream_t>(cuda_stream));
}

dsla_status dsla_gate_project_last_error(void) { return gate_project_last_error(); }

// ---- host-buffer variants -----------------------------------------------------------------
static size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

size_t dsla_prefill_staging_bytes(const dsla_prefill_args* a) {
    if (check_prefill_sizes(a) != DSLA_OK) return 0;
    const size_t t = up256((size_t)a->T_total * a->H * a->d_k * esize(a->dtype));
    const size_t g = up256((size_t)a->T_total * a->H * sizeof(float));
    return 4 * t + 2 * g;
}

// Side streams and events of the host-buffer prefill pipeline, one set per device, created on first use and kept.
namespace {
constexpr int HOST_MAX_SLICES = 8;
struct HostPipe {
    bool ready = false;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t start = nullptr, end = nullptr, copied[HOST_MAX_SLICES] = {}, done[HOST_MAX_SLICES] = {};
};
std::mutex g_pipe_mutex;
HostPipe g_pipes[64];

HostPipe* host_pipe() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe& hp = g_pipes[dev];
    if (!hp.ready) {
        bool ok = cudaStreamCreateWithFlags(&hp.h2d, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.end, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < HOST_MAX_SLICES; ++i)
            ok = cudaEventCreateWithFlags(&hp.copied[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { (void)cudaGetLastError(); return nullptr; }
        hp.ready = true;
    }
    return &hp;
}

// One long sequence from host buffers: the tokens are cut into slices, and while slice i is being computed (continuing
// from the states slice i-1 left in the slot) slice i+1 is on its way to the device and the outputs of slice i-1 are on
// their way back, on two side streams that are forked from and joined back into the caller's stream with events.
dsla_status prefill_host_sliced(const dsla_prefill_args* a, const dsla_prefill_args& d, dsla_state* st, cudaStream_t s) {
    HostPipe* hp = host_pipe();
    if (!hp) return DSLA_ERR_CUDA;
    // The side streams and events are one set per device: calls from several host threads enqueue one after the other.
    static std::mutex enqueue_mutex;
    std::lock_guard<std::mutex> enqueue_lock(enqueue_mutex);
    const int T = a->T_total;
    int nsl = T / 1024;
    if (nsl > HOST_MAX_SLICES) nsl = HOST_MAX_SLICES;
    const int per = ((T + nsl - 1) / nsl + 63) / 64 * 64;          // whole chunks per slice
    const size_t row = (size_t)a->H * a->d_k * esize(a->dtype), grow = (size_t)a->H * sizeof(float);
    bool ok = cudaEventRecord(hp->start, s) == cudaSuccess && cudaStreamWaitEvent(hp->h2d, hp->start, 0) == cudaSuccess &&
              cudaStreamWaitEvent(hp->d2h, hp->start, 0) == cudaSuccess;
    int used = 0;
    for (int i = 0, t0 = 0; ok && t0 < T; ++i, t0 += per, ++used) {
        const int len = T - t0 < per ? T - t0 : per;
        const size_t off = (size_t)t0 * row, goff = (size_t)t0 * grow, nb = (size_t)len * row, ngb = (size_t)len * grow;
        auto dev = [&](const void* p, size_t o) { return const_cast<char*>(static_cast<const char*>(p)) + o; };
        ok = cudaMemcpyAsync(dev(d.q, off), dev(a->q, off), nb, cudaMemcpyHostToDevice, hp->h2d) == cudaSuccess &&
             cudaMemcpyAsync(dev(d.k, off), dev(a->k, off), nb, cudaMemcpyHostToDevice, hp->h2d) == cudaSuccess &&
             cudaMemcpyAsync(dev(d.v, off), dev(a->v, off), nb, cudaMemcpyHostToDevice, hp->h2d) == cudaSuccess &&
             cudaMemcpyAsync(dev(d.g_hist, goff), dev(a->g_hist, goff), ngb, cudaMemcpyHostToDevice, hp->h2d) == cudaSuccess &&
             cudaMemcpyAsync(dev(d.g_rec, goff), dev(a->g_rec, goff), ngb, cudaMemcpyHostToDevice, hp->h2d) == cudaSuccess &&
             cudaEventRecord(hp->copied[i], hp->h2d) == cudaSuccess && cudaStreamWaitEvent(s, hp->copied[i], 0) == cudaSuccess;
        if (!ok) break;
        dsla_prefill_args sl = d;
        sl.q = dev(d.q, off); sl.k = dev(d.k, off); sl.v = dev(d.v, off); sl.o = dev(d.o, off);
        sl.g_hist = reinterpret_cast<const float*>(dev(d.g_hist, goff));
        sl.g_rec = reinterpret_cast<const float*>(dev(d.g_rec, goff));
        sl.T = len; sl.T_total = len; sl.max_seqlen = len;
        sl.use_initial_state = i > 0 ? 1 : a->use_initial_state;
        const dsla_status rc = prefill_device(&sl, st, s);
        if (rc != DSLA_OK) {
            // join the forked side streams back into the caller's stream before reporting the failure
            if (cudaEventRecord(hp->end, hp->h2d) == cudaSuccess) (void)cudaStreamWaitEvent(s, hp->end, 0);
            if (cudaEventRecord(hp->end, hp->d2h) == cudaSuccess) (void)cudaStreamWaitEvent(s, hp->end, 0);
            return rc;
        }
        ok = cudaEventRecord(hp->done[i], s) == cudaSuccess && cudaStreamWaitEvent(hp->d2h, hp->done[i], 0) == cudaSuccess &&
             cudaMemcpyAsync(dev(a->o, off), dev(d.o, off), nb, cudaMemcpyDeviceToHost, hp->d2h) == cudaSuccess;
    }
    ok = ok && cudaEventRecord(hp->end, hp->d2h) == cudaSuccess && cudaStreamWaitEvent(s, hp->end, 0) == cudaSuccess;
    return ok ? DSLA_OK : DSLA_ERR_CUDA;
}
}  // namespace

dsla_status dsla_prefill_host(const dsla_prefill_args* a, dsla_state* st, void* staging, size_t staging_bytes, void* cuda_stream) {
    dsla_status rc = check_prefill_sizes(a);
    if (rc != DSLA_OK) return rc;
    if (a->T_total == 0) return prefill_device(a, st, static_cast<cudaStream_t>(cuda_stream));
    const size_t need = dsla_prefill_staging_bytes(a);
    if (!staging || staging_bytes < need || !aligned(staging, 256)) return DSLA_ERR_INVALID_ARG;
    if (!a->q || !a->k || !a->v || !a->o || !a->g_hist || !a->g_rec) return DSLA_ERR_INVALID_ARG;
    if (a->gate_layout != DSLA_GATE_SCALAR) return DSLA_ERR_UNSUPPORTED;      // host-buffer variants stage scalar gates only
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t tb = (size_t)a->T_total * a->H * a->d_k * esize(a->dtype), t = up256(tb);
    const size_t gb = (size_t)a->T_total * a->H * sizeof(float), g = up256(gb);
    char* base = static_cast<char*>(staging);
    dsla_prefill_args d = *a;
    d.q = base; d.k = base + t; d.v = base + 2 * t; d.o = base + 3 * t;
    d.g_hist = reinterpret_cast<float*>(base + 4 * t);
    d.g_rec = reinterpret_cast<float*>(base + 4 * t + g);
    if (a->cu_seqlens == nullptr && a->N == 1 && a->T_total >= 2048) return prefill_host_sliced(a, d, st, s);
    bool ok = cudaMemcpyAsync(const_cast<void*>(d.q), a->q, tb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<void*>(d.k), a->k, tb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<void*>(d.v), a->v, tb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<float*>(d.g_hist), a->g_hist, gb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<float*>(d.g_rec), a->g_rec, gb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (!ok) return DSLA_ERR_CUDA;
    rc = prefill_device(&d, st, s);
    if (rc != DSLA_OK) return rc;
    return cudaMemcpyAsync(a->o, d.o, tb, cudaMemcpyDeviceToHost, s) == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

size_t dsla_decode_staging_bytes(const dsla_decode_args* a) {
    if (!a || a->B < 0 || a->H <= 0 || a->d_k <= 0 || a->d_v <= 0) return 0;
    const size_t t = up256((size_t)a->B * a->H * a->d_k * esize(a->dtype));
    const size_t g = up256((size_t)a->B * a->H * sizeof(float));
    return 4 * t + 2 * g;
}

dsla_status dsla_decode_step_host(const dsla_decode_args* a, dsla_state* st, void* staging, size_t staging_bytes, void* cuda_stream) {
    dsla_status rc = check_decode(a, st);
    if (rc != DSLA_OK) return rc;
    if (a->B == 0) return DSLA_OK;
    const size_t need = dsla_decode_staging_bytes(a);
    if (!staging || staging_bytes < need || !aligned(staging, 256)) return DSLA_ERR_INVALID_ARG;
    if (!a->q || !a->k || !a->v || !a->o || !a->g_hist || !a->g_rec) return DSLA_ERR_INVALID_ARG;
    if (a->gate_layout != DSLA_GATE_SCALAR || a->row_mask) return DSLA_ERR_UNSUPPORTED;      // host-buffer variant: scalar gates, every row
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t tb = (size_t)a->B * a->H * a->d_k * esize(a->dtype), t = up256(tb);
    const size_t gb = (size_t)a->B * a->H * sizeof(float), g = up256(gb);
    char* base = static_cast<char*>(staging);
    dsla_decode_args d = *a;
    d.q = base; d.k = base + t; d.v = base + 2 * t; d.o = base + 3 * t;
    d.g_hist = reinterpret_cast<float*>(base + 4 * t);
    d.g_rec = reinterpret_cast<float*>(base + 4 * t + g);
    bool ok = cudaMemcpyAsync(const_cast<void*>(d.q), a->q, tb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<void*>(d.k), a->k, tb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<void*>(d.v), a->v, tb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<float*>(d.g_hist), a->g_hist, gb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(const_cast<float*>(d.g_rec), a->g_rec, gb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (!ok) return DSLA_ERR_CUDA;
    rc = decode_device(&d, st, s);
    if (rc != DSLA_OK) return rc;
    return cudaMemcpyAsync(a->o, d.o, tb, cudaMemcpyDeviceToHost, s) == cudaSuccess ? DSLA_OK : DSLA_ERR_CUDA;
}

}  // extern "C"
