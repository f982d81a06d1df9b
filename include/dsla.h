/*
 * libdsla -- dual-state linear attention (DSLA) layer for NVIDIA B200 (sm_100a).
 *
 * The layer replaces softmax self-attention at inference time.  Per (sequence, head) it keeps two
 * recurrent states, "history" (i = 1, slow decay) and "recency" (i = 2, fast decay):
 *
 *     S^i_t = g^i_t * S^i_{t-1} + k_t^T v_t                      (Sec. 4.1, dual-state update)
 *     o_t   = scale * q_t ( gamma S^1_t + (1 - gamma) S^2_t )    (Sec. 4.1, blended readout)
 *
 * g^i_t in [0,1] is an already-activated scalar gate per (token, head, state); gamma is a blend
 * weight per head (a per-layer gamma is the same value in every entry).  The feature map is the
 * identity and there is no normaliser (none is defined in Sec. 4.1).
 *
 * Conventions for every entry point
 *   - plain C ABI; every pointer is a DEVICE pointer unless its comment says "host";
 *   - the caller owns all tensors; prefill and decode allocate nothing;
 *   - work is enqueued on the CUDA stream passed as `cuda_stream` (a cudaStream_t; NULL = default
 *     stream) and the call returns without waiting for it;
 *   - argument errors are detected on the host before anything is launched and reported through
 *     the return value; nothing is thrown, nothing aborts, there is no CPU fallback;
 *   - supported head sizes: d_k == d_v in {64, 128}; everything else is DSLA_ERR_UNSUPPORTED;
 *   - a state store belongs to the device that was current in dsla_state_alloc; prefill and decode calls for it must be
 *     made with that device current (DSLA_ERR_INVALID_ARG otherwise).
 */
#ifndef DSLA_H_
#define DSLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DSLA_OK = 0,
    DSLA_ERR_INVALID_ARG = 1, /* NULL pointer, negative size, misaligned pointer, slot out of range ... */
    DSLA_ERR_UNSUPPORTED = 2, /* head size / chunk / dtype combination that no kernel covers */
    DSLA_ERR_CUDA = 3,        /* a CUDA runtime call failed (no device, launch error, ...) */
    DSLA_ERR_OOM = 4,         /* device allocation failed (dsla_state_alloc only) */
    DSLA_ERR_TIMEOUT = 5,     /* a bounded on-device wait ran out; see dsla_state_last_error */
    DSLA_ERR_SCRATCH_LIMIT = 6 /* dsla_prefill_static_ws only: the call needs more scratch than the built-in array holds */
} dsla_status;

typedef enum { DSLA_F32 = 0, DSLA_BF16 = 1 } dsla_dtype;

/* Shape of a gate tensor.  SCALAR: one activated gate per (token, head, state), G = g 11^T, shape [T, H].
 * PER_KEY_CHANNEL: one gate per key channel, G = alpha^T 1 (the gated-linear-attention parameterisation of Sec. 2,
 * which Sec. 4.1 carries over to G^1_t, G^2_t): shape [T, H, d_k]; row a of a state decays with alpha_a. */
typedef enum { DSLA_GATE_SCALAR = 0, DSLA_GATE_PER_KEY_CHANNEL = 1 } dsla_gate_layout;

/* Which prefill kernel runs.
 *   SIMT        : CUDA cores, fp32 arithmetic; any supported dtype and head size, chunk 16 / 32 / 64.
 *   TENSOR      : tcgen05 tensor cores, bf16 with d = 128, chunk 64; one CTA holds both states of a (sequence, head) pair.
 *   TENSOR_PAIR : same mathematics and limits, one state per CTA in a cluster of two CTAs that exchange partial
 *                 outputs through distributed shared memory.
 *   AUTO        : TENSOR for bf16 with d = 128 (the faster of the two tensor variants on the measured shapes), else SIMT
 *                 -- in particular bf16 with d = 64 and everything fp32 run on CUDA cores, an order of magnitude slower. */
typedef enum { DSLA_IMPL_AUTO = 0, DSLA_IMPL_SIMT = 1, DSLA_IMPL_TENSOR = 2, DSLA_IMPL_TENSOR_PAIR = 3 } dsla_impl;

/* ------------------------------------------------------------------------------------------
 * Dual-state store.  One "slot" holds the two states of every head of one sequence of one layer:
 * fp32 [num_slots][2][H][d_k][d_v], d_v contiguous; index 0 of the second axis is the history
 * state S^1, index 1 the recency state S^2 (the two states of Sec. 4.1).  Its size does not depend
 * on the context length (Sec. 5.3: decoding updates only two states).
 * ------------------------------------------------------------------------------------------ */
typedef struct dsla_state dsla_state;

/* Bytes needed for the store above (0 on invalid sizes). */
size_t dsla_state_bytes(int num_slots, int H, int d_k, int d_v);

/* Creates a store on the current device.
 *   ext_buf == NULL : the library cudaMalloc's dsla_state_bytes() once (DSLA_ERR_OOM on failure);
 *   ext_buf != NULL : the store borrows caller memory (256-byte aligned, ext_bytes >= the size
 *                     above, else DSLA_ERR_INVALID_ARG); the caller keeps ownership.
 * The contents are NOT initialised; call dsla_state_zero or run a prefill with
 * use_initial_state = 0.  A 4-byte device status word is allocated alongside. */
dsla_status dsla_state_alloc(dsla_state** out, int num_slots, int H, int d_k, int d_v,
                             void* ext_buf, size_t ext_bytes);

/* Frees the handle and only the memory the library allocated.  NULL is accepted. */
dsla_status dsla_state_free(dsla_state* st);

/* Device pointer to the fp32 store (for copy-out, checkpointing, parity checks). */
void* dsla_state_data(dsla_state* st);

/* Zeroes n slots listed in slots_dev (device int32[n]; entries < 0 are ignored), or the whole
 * store when slots_dev == NULL (n is then ignored). */
dsla_status dsla_state_zero(dsla_state* st, const int32_t* slots_dev, int n, void* cuda_stream);

/* Reads back (synchronising the whole device) and clears the status word that kernels raise for problems only the
 * device can see: DSLA_OK; DSLA_ERR_TIMEOUT when a bounded on-device wait gave up (the kernel then ran to its end
 * without hanging, its results are invalid); DSLA_ERR_INVALID_ARG when a packed sequence turned out longer than
 * max_seqlen (the tensor-core prefill sizes its segments from max_seqlen, so the tail of that sequence was not
 * computed). */
dsla_status dsla_state_last_error(dsla_state* st);

/* Diagnostic: exercises the give-up path of the bounded waits without hanging anything.  A one-warp kernel waits,
 * for at most max_polls polls (1 .. 1,000,000; a poll takes about 0.1 us), on a barrier that nobody arrives at; the
 * wait runs out, the kernel raises the status word of `st` and returns.  dsla_state_last_error(st) then reports
 * DSLA_ERR_TIMEOUT and the device stays usable.  (No counterpart in the paper.) */
dsla_status dsla_selftest_bounded_wait(dsla_state* st, unsigned max_polls, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Prefill: the chunkwise-parallel form of the recurrence.  Inside a chunk of C tokens the output
 * is the masked quadratic form of the unrolled scores (Sec. 4.1: sigma^i_t = (q_T . k_t) times the
 * product of the gates t+1..T, blended by gamma); between chunks the two states are carried as
 *     S^i <- (prod of the chunk's gates) S^i + sum_s (prod of gates s+1..end) k_s^T v_s .
 * The result equals the token-by-token recurrence up to floating-point summation order and does
 * not depend on `chunk`.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    const void* q;              /* [T_total, H, d_k]  dtype, row-major, 16-byte aligned           */
    const void* k;              /* [T_total, H, d_k]                                              */
    const void* v;              /* [T_total, H, d_v]                                              */
    void* o;                    /* [T_total, H, d_v]  dtype (output)                              */
    const float* g_hist;        /* [T_total, H] fp32 in [0,1]: gate of the history state          */
    const float* g_rec;         /* [T_total, H] fp32 in [0,1]: gate of the recency state          */
    const float* gamma;         /* [H] fp32: weight of the history branch; recency gets 1 - gamma */
    const int32_t* cu_seqlens;  /* [N + 1] int32, cu[0] = 0, cu[N] = T_total (packed sequences);
                                   NULL means N sequences of exactly T tokens each               */
    const int32_t* slots;       /* [N] int32 slot of each sequence; NULL means slot n = n.  Entries
                                   must be distinct and in [0, num_slots) (not checked on host)  */
    int N;                      /* number of sequences                                           */
    int T;                      /* tokens per sequence when cu_seqlens == NULL, else ignored      */
    int T_total;                /* rows of q/k/v/o                                               */
    int max_seqlen;             /* upper bound on any sequence length (sizes the grid)           */
    int H, d_k, d_v;
    int chunk;                  /* C: 16, 32 or 64 for the CUDA-core kernel; 64 (or 0 = default) for
                                   the tensor-core kernel                                        */
    dsla_dtype dtype;           /* dtype of q, k, v, o; the states are always fp32               */
    float scale;                /* multiplies o (1.0f for the plain definition)                  */
    int use_initial_state;      /* 0: start every sequence from zero states; 1: continue from the
                                   contents of its slot (chunked prefill / resume)               */
    dsla_impl impl;
    void* workspace;            /* scratch of dsla_prefill_workspace_bytes(); may be NULL if 0    */
    size_t workspace_bytes;
    dsla_gate_layout gate_layout; /* SCALAR (0): g_hist, g_rec are [T_total, H].  PER_KEY_CHANNEL: [T_total, H, d_k];
                                   served by a token-by-token CUDA-core kernel (impl AUTO or SIMT; the tensor-core
                                   kernels take scalar gates only: DSLA_ERR_UNSUPPORTED)                        */
} dsla_prefill_args;

/* Scratch the chosen kernel needs for these sizes (0 for the SIMT kernel): the segment summaries of
 * sequences that are split along T, plus, for packed batches (cu_seqlens != NULL, N > 1), one int32 per
 * sequence for the longest-first visiting order.  Pointers in `a` are not dereferenced (cu_seqlens is
 * only compared with NULL). */
size_t dsla_prefill_workspace_bytes(const dsla_prefill_args* a);

/* Writes o for every token and the final states of every sequence into its slot.  A sequence of
 * length 0 writes no output; its slot is zeroed when use_initial_state == 0 and left as is
 * otherwise.  `a` is a host pointer and is read before the call returns. */
dsla_status dsla_prefill(const dsla_prefill_args* a, dsla_state* st, void* cuda_stream);

/* Prefill for callers that cannot hand the library a scratch buffer.  (No counterpart in the paper: this
 * is a deployment convenience, not part of the method.)
 *
 * Who needs it: code that runs where device memory cannot be allocated at the time of the call -- for
 * example a serving loop whose allocator is frozen after start-up, a plug-in that is only handed its
 * input and output tensors, or a latency-critical path that must never reach cudaMalloc (an allocation
 * can stall a step for hundreds of milliseconds).  dsla_prefill needs a caller-owned workspace whenever
 * it splits sequences into segments; this variant uses a fixed array inside the library instead:
 *
 *     static __device__ array of DSLA_STATIC_SCRATCH_BYTES bytes, one per GPU that loads the library,
 *     held until the process exits.
 *
 * It computes exactly what dsla_prefill computes for the same arguments (a->workspace and
 * a->workspace_bytes are ignored) and allocates nothing: no cudaMalloc, no cudaFree, no allocating
 * library call.  If the arguments would need more scratch than the array holds
 * (dsla_prefill_workspace_bytes(a) > DSLA_STATIC_SCRATCH_BYTES) nothing is launched and
 * DSLA_ERR_SCRATCH_LIMIT is returned; use dsla_prefill with your own workspace then.
 *
 * The first call on each device looks up the array's device address (one cudaGetSymbolAddress with that
 * device current); make that first call outside any CUDA stream capture.  Every call on a device shares the
 * one array and the array keeps whatever the previous call left in it: each call overwrites every entry it
 * later reads, so nothing has to be cleared, but two calls that overlap on the GPU (different streams,
 * or different host threads without ordering) race on it.  Run them on one stream or order them with
 * events. */
#define DSLA_STATIC_SCRATCH_BYTES (18u << 20)
dsla_status dsla_prefill_static_ws(const dsla_prefill_args* a, dsla_state* st, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Decode: one step of the recurrence per batch row, fused with the readout and the blend
 * (Sec. 4.1 equations applied to one new token; Sec. 5.3: constant cost per token).  Each state
 * element is read once and written once, in place.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    const void* q;          /* [B, H, d_k] dtype                                                  */
    const void* k;          /* [B, H, d_k]                                                        */
    const void* v;          /* [B, H, d_v]                                                        */
    void* o;                /* [B, H, d_v] dtype (output); rows with slot < 0 are written as 0    */
    const float* g_hist;    /* [B, H] fp32                                                        */
    const float* g_rec;     /* [B, H] fp32                                                        */
    const float* gamma;     /* [H] fp32                                                           */
    const int32_t* slots;   /* [B] int32 slot per row; < 0 skips the row (padding in a continuous
                               batch); NULL means slot b = b.  Live entries must be distinct     */
    int B, H, d_k, d_v;
    dsla_dtype dtype;
    float scale;
    dsla_gate_layout gate_layout; /* SCALAR (0): g_hist, g_rec are [B, H]; PER_KEY_CHANNEL: [B, H, d_k]          */
    const uint8_t* row_mask;    /* [B] bytes or NULL.  A batch may mix requests whose layer at this depth is a DSLA
                                   layer with requests that still run softmax attention there (Sec. 4.5, App. D):
                                   rows with 0 are not touched at all -- neither their slot nor their row of o, which
                                   the attention kernel of the same step writes; NULL = every row is a DSLA row      */
} dsla_decode_args;

dsla_status dsla_decode_step(const dsla_decode_args* a, dsla_state* st, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * n states.  Sec. 4.2 argues that two states suffice; the number-of-states ablation of Sec. 5.5 runs the layer with
 * 1, 2, 4 and 8 states.  The general form keeps n recurrent states per (sequence, head), each with its own gate, and
 * blends them with one weight per state:
 *     S^i_t = g^i_t * S^i_{t-1} + k_t^T v_t   (i = 0 .. n-1),      o_t = scale * q_t sum_i w_i S^i_t .
 * n = 2 with w = (gamma, 1 - gamma) is the dual-state layer above.  Supported n: 1, 2, 4, 8.
 * The store is fp32 [num_slots][n_states][H][d_k][d_v]; dsla_state_alloc is dsla_state_alloc_n with n_states = 2, and
 * the dual-state entry points accept only such stores (DSLA_ERR_INVALID_ARG otherwise).
 * ------------------------------------------------------------------------------------------ */
size_t dsla_state_bytes_n(int num_slots, int n_states, int H, int d_k, int d_v);
dsla_status dsla_state_alloc_n(dsla_state** out, int num_slots, int n_states, int H, int d_k, int d_v,
                               void* ext_buf, size_t ext_bytes);

typedef struct {
    const void* q;              /* [B, H, d_k] dtype                                                          */
    const void* k;              /* [B, H, d_k]                                                                */
    const void* v;              /* [B, H, d_v]                                                                */
    void* o;                    /* [B, H, d_v] dtype (output)                                                 */
    const float* gates;         /* [n_states, B, H] fp32 (or [n_states, B, H, d_k] per key channel)           */
    const float* weights;       /* [H, n_states] fp32 blend weight of every state                             */
    const int32_t* slots;       /* as in dsla_decode_args                                                     */
    const uint8_t* row_mask;    /* as in dsla_decode_args                                                     */
    int B, H, d_k, d_v, n_states;
    dsla_dtype dtype;
    float scale;
    dsla_gate_layout gate_layout;
} dsla_nstate_decode_args;

/* One recurrence step of the n-state form, in place, one pass over the states (HBM traffic n_states/2 times that of
 * the dual-state step). */
dsla_status dsla_nstate_decode_step(const dsla_nstate_decode_args* a, dsla_state* st, void* cuda_stream);

typedef struct {
    const void *q, *k, *v;      /* [T_total, H, d] dtype, 16-byte aligned                                      */
    void* o;                    /* [T_total, H, d_v] dtype (output)                                           */
    const float* gates;         /* [n_states, T_total, H] fp32 (or [n_states, T_total, H, d_k])               */
    const float* weights;       /* [H, n_states]                                                              */
    const int32_t* cu_seqlens;  /* as in dsla_prefill_args                                                    */
    const int32_t* slots;
    int N, T, T_total, H, d_k, d_v, n_states;
    dsla_dtype dtype;
    float scale;
    int use_initial_state;
    dsla_gate_layout gate_layout;
    int max_seqlen;             /* as in dsla_prefill_args (dense batches: T)                                  */
    dsla_impl impl;             /* AUTO, SIMT (the token-by-token kernel) or TENSOR                           */
    void* workspace;            /* device scratch of dsla_nstate_prefill_workspace_bytes(a) bytes, 256-byte    */
    size_t workspace_bytes;     /* aligned; may be NULL / 0 when that function returns 0                       */
} dsla_nstate_prefill_args;

/* Prefill of the n-state form.  Two kernels:
 *  - SIMT: the recurrence itself on CUDA cores, token by token (fp32 arithmetic, no workspace), for every supported
 *    n, dtype, d and gate layout.  With more than four states (more than two when the gates are per key channel and
 *    d = 128) the states are processed in groups, each group adding its share to o.
 *  - TENSOR (what AUTO picks when it applies): bf16, d = 128, scalar gates (n = 1 runs as a pair whose second state
 *    has weight 0 and is never stored): the chunkwise tensor-core
 *    kernel of dsla_prefill run once per pair of states (2i, 2i + 1) with the weights (w_2i, w_2i+1); pairs after the
 *    first write their share to a scratch tensor in the workspace that is then added to o, so o is rounded to bf16 once
 *    per pair.  Needs the workspace below.
 * Errors as dsla_prefill; time-outs and a too small max_seqlen are reported through dsla_state_last_error. */
size_t dsla_nstate_prefill_workspace_bytes(const dsla_nstate_prefill_args* a);
dsla_status dsla_nstate_prefill(const dsla_nstate_prefill_args* a, dsla_state* st, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Gate producer.  The gates of the two states come from single linear layers on the layer's input (Sec. 5.3; App. B:
 * zero bias, history layer near identity, recency layer random at initialisation).  This entry point computes
 *     [g_hist | g_rec][t, :] = logistic(x[t, :] W^T + bias)
 * on the tensor cores and writes the two [T, H] fp32 tensors dsla_prefill / dsla_decode_step read, so the
 * pre-activations never exist in memory.  Rows 0 .. H-1 of W (and of bias) produce the history gates, rows H .. 2H-1
 * the recency gates.  Requirements: H a multiple of 8 with 2 H <= 256; D_model a multiple of 64; x, w 16-byte aligned,
 * g_hist, g_rec 16-byte aligned; else DSLA_ERR_INVALID_ARG / DSLA_ERR_UNSUPPORTED.  dsla_gate_project_last_error reads
 * (synchronising the device) and clears the kernel's time-out flag: DSLA_OK or DSLA_ERR_TIMEOUT.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    const void* x;          /* [T, D_model] bf16, row-major                                               */
    const void* w;          /* [2 H, D_model] bf16, row-major (one row per output)                        */
    const float* bias;      /* [2 H] fp32 or NULL                                                         */
    float* g_hist;          /* [T, H] fp32 (output)                                                       */
    float* g_rec;           /* [T, H] fp32 (output)                                                       */
    int T, H, D_model;
} dsla_gate_project_args;
dsla_status dsla_gate_project(const dsla_gate_project_args* a, void* cuda_stream);
dsla_status dsla_gate_project_last_error(void);

/* ------------------------------------------------------------------------------------------
 * Host-buffer variants (end-to-end path): q, k, v, o, g_hist, g_rec in `a` are HOST pointers
 * (pinned memory gives asynchronous copies); gamma, cu_seqlens, slots and the workspace stay
 * device pointers.  `staging` is caller-owned device memory of at least
 * dsla_*_staging_bytes(a); inputs are copied into it, the kernels run on it, and o is copied back,
 * all ordered on `cuda_stream`.  The caller synchronises the stream before reading o.  A single dense sequence of
 * 2048 tokens or more (cu_seqlens == NULL, N == 1) is cut into slices of about 1024 tokens: while slice i is computed,
 * continuing from the states slice i-1 left in the slot, the inputs of slice i+1 and the outputs of slice i-1 are copied
 * on two internal streams (created once per device) that are forked from and joined back into `cuda_stream` with
 * events; the result equals the unsliced one up to floating-point summation order.  Those streams and events are one set
 * per device: host threads that call dsla_prefill_host at the same time are enqueued one after the other (a mutex), and two
 * calls on different caller streams must not be in flight on the GPU together (the second would wait on events the first recorded).
 * ------------------------------------------------------------------------------------------ */
size_t dsla_prefill_staging_bytes(const dsla_prefill_args* a);
dsla_status dsla_prefill_host(const dsla_prefill_args* a, dsla_state* st, void* staging,
                              size_t staging_bytes, void* cuda_stream);
size_t dsla_decode_staging_bytes(const dsla_decode_args* a);
dsla_status dsla_decode_step_host(const dsla_decode_args* a, dsla_state* st, void* staging,
                                  size_t staging_bytes, void* cuda_stream);

/* Static, human-readable name of a status code. */
const char* dsla_status_string(dsla_status s);

/* Number of kernels this library has launched in this process (for launch accounting). */
uint64_t dsla_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DSLA_H_ */
