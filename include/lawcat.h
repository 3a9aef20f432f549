/*
 * lawcat.h -- C ABI of the LAWCAT linearized-attention layer for NVIDIA B200 (sm_100a).
 *
 * The layer (paper Section 4, Fig. 1):
 *   1. causal depthwise Conv1D across tokens, width conv_k = r+1, on the query and on the key stream,
 *      separate weights per stream (Section 4.1; appendix "share the linear and Conv layers");
 *   2. one shared per-head linear layer followed by a nonlinearity -- the feature map phi -- applied to both
 *      conv outputs, giving qdot and kdot (Section 4.1, Section 4.2 first paragraph);
 *   3. normalized gated linear attention: S_t = G_t (.) S_{t-1} + kdot_t^T v_t (Eq. 4), output
 *      o_t = qdot_t S_t / (qdot_t . z_t) with z_t the same recurrence on kdot_t alone (Eq. 8).
 *
 * Conventions shared by every entry point
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, contiguous in the stated shape with the
 *     last index fastest, and 16-byte aligned. The library never allocates, frees or synchronizes; work is
 *     enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - `p->dtype` is the storage type of q, k, v, gate, the conv and mix weights, the conv caches, qdot, kdot,
 *     o and the input gradients: float (LAWCAT_F32) or bfloat16 (LAWCAT_BF16). All arithmetic accumulates
 *     in fp32. States S, z, the denominator `den` and all weight gradients are always fp32.
 *   - Heads: H query heads, H_kv key/value heads, H % H_kv == 0, G = H / H_kv. Query head h reads key and
 *     value head h / G. kdot, the gate and the state are per QUERY head because the mix weights are.
 *   - Gate: gate[b,t,h,:] has gate_dim = d_k entries (one decay per key channel) or 1 (one per head).
 *     LAWCAT_GATE_LOGITS: log-decay g = logsigmoid(gate) / gate_tau ("sigmoid" gate of Section 4.2);
 *     LAWCAT_GATE_LOGDECAY: g = gate itself, which must be <= 0. The decay is alpha = exp(g) in (0, 1].
 *     Token t's decay multiplies S_{t-1}; it never touches token t's own kdot_t^T v_t (J_{t,t} = 1, Eq. 6).
 *   - Conv taps: w[(head*d_k + c)*conv_k + delta] multiplies x[t - delta], delta = 0 is the current token.
 *     Rows with t - delta < 0 come from the conv cache when one is given, otherwise they are zero.
 *     A conv cache holds the conv_k-1 raw (pre-conv) tokens that precede t = 0, oldest first.
 *   - Mix: y[e] = sum_c u[c] * W[h][c][e]; the same W[h] serves the query stream and the key stream.
 *   - A NULL optional input means "absent" (zero state, zero cache); a NULL optional output is not written.
 *   - `ws` is caller-provided scratch of at least lawcat_workspace_bytes(p, op) bytes (may be NULL when 0).
 *   - Return value: a lawcat_status. Argument problems are detected on the host before anything is enqueued.
 *     `dev_status` (optional device int, caller-zeroed) receives a nonzero lawcat_status if a kernel had to
 *     give up asynchronously (a bounded wait that ran out); kernels never trap.
 *   - Supported shapes: d_k and d_v in {16, 32, 64, 128}; 1 <= conv_k <= 8; gate_dim in {1, d_k}.
 *     Anything else returns LAWCAT_ERR_UNSUPPORTED; nothing falls back to the host.
 */
#ifndef LAWCAT_H_
#define LAWCAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LAWCAT_OK = 0,
  LAWCAT_ERR_INVALID_ARG = 1,
  LAWCAT_ERR_UNSUPPORTED = 2,
  LAWCAT_ERR_CUDA = 3,
  LAWCAT_ERR_WORKSPACE_TOO_SMALL = 4,
  LAWCAT_ERR_TIMEOUT = 5,
  LAWCAT_ERR_NUMERIC = 6,
  LAWCAT_ERR_TOO_LARGE = 7 /* the problem exceeds a fixed built-in limit (see lawcat_layer_fwd_noalloc) */
} lawcat_status;

enum { LAWCAT_F32 = 0, LAWCAT_BF16 = 1 };
enum { LAWCAT_PHI_SOFTMAX = 0, LAWCAT_PHI_ELU1 = 1, LAWCAT_PHI_IDENTITY = 2 };
enum { LAWCAT_GATE_LOGITS = 0, LAWCAT_GATE_LOGDECAY = 1 };
enum {
  LAWCAT_OP_CONV_FWD = 0,
  LAWCAT_OP_CONV_BWD = 1,
  LAWCAT_OP_GLA_FWD = 2,
  LAWCAT_OP_GLA_BWD = 3,
  LAWCAT_OP_LAYER_FWD = 4,
  LAWCAT_OP_DECODE_STEP = 5,
  LAWCAT_OP_LAYER_BWD = 6
};

typedef struct {
  int32_t B, T, H, H_kv, d_k, d_v;
  int32_t conv_k;    /* conv width r+1 (the paper uses 4, Section 4.1) */
  int32_t gate_dim;  /* d_k or 1 */
  int32_t chunk;     /* tokens per chunk of the chunkwise-parallel form; 0 = library chooses */
  int32_t dtype;     /* LAWCAT_F32 | LAWCAT_BF16 */
  int32_t phi;       /* LAWCAT_PHI_* : softmax over the d_k mix outputs, 1+ELU (Section 2), identity */
  int32_t gate_mode; /* LAWCAT_GATE_* */
  float gate_tau;    /* divisor of logsigmoid in LOGITS mode; 1 = the plain sigmoid gate */
  float eps;         /* added to the denominator of Eq. 8 */
  int32_t normalize; /* 1 = Eq. 8; 0 = numerator only (the "NN" ablation, Table 2) */
  int32_t mix_unshared; /* 0 = one linear layer W[h] for the query and the key stream (Section 4.1, the paper's choice);
                           1 = a separate one per stream (the "unshared linear" rows of the appendix table on sharing):
                           W is then [2,H,d_k,d_k], query matrices first, and dW likewise */
} lawcat_params;

/* Scratch bytes entry point `op` (LAWCAT_OP_*) needs for these parameters; 0 on invalid parameters. */
size_t lawcat_workspace_bytes(const lawcat_params* p, int op);

/* Static, human-readable name of a status code. */
const char* lawcat_status_string(int status);

/*
 * Detail of the last LAWCAT_ERR_CUDA this host thread got from a kernel launch: the CUDA runtime's message and the
 * place in the library that saw it ("" when there was none). The string belongs to the library and is overwritten by
 * the thread's next such error.
 */
const char* lawcat_last_cuda_error(void);

/* Library version, major*10000 + minor*100 + patch. */
int lawcat_version(void);

/*
 * Profiling aids (the paper has no counterpart; its only timing is an end-to-end latency plot, Section 5.5).
 * lawcat_launch_count: kernels this library has launched in this process so far (monotonic, host counter).
 * lawcat_trace_begin:  from now on bracket every kernel launch with a pair of CUDA events on its stream.
 * lawcat_trace_end:    stop tracing, wait for the recorded events (this call synchronizes on them) and write one line
 *                      per kernel, "<name> <launches> <total milliseconds>\n", into the HOST buffer buf (NUL-terminated,
 *                      truncated to buf_bytes). Tracing creates CUDA events; it is meant for benchmarks, not serving.
 */
unsigned long long lawcat_launch_count(void);
int lawcat_trace_begin(void);
int lawcat_trace_end(char* buf, size_t buf_bytes);

/*
 * Test hook (no counterpart in the paper). Every device-side wait of the tensor-core layer kernels is bounded: after
 * `cycles` clock cycles (default about two seconds) a waiting role gives up, the block leaves its loops, lets its
 * copies land, frees its tensor memory and returns, and dev_status receives LAWCAT_ERR_TIMEOUT. This call sets the bound
 * for the launches that follow (0 restores the default), so that a test can make a wait run out without faulting or
 * hanging anything. Host-side, process-wide, not meant for production code.
 */
void lawcat_test_set_wait_limit(long long cycles);

/*
 * Causal depthwise conv on q and k (Section 4.1: qtilde_t = sum_delta w_delta q_{t-delta}), then, when W is not
 * NULL, the shared per-head linear layer and phi (Section 4.1; Section 4.2 defines qdot, kdot).
 *   q [B,T,H,d_k]  k [B,T,H_kv,d_k]  w_q [H*d_k,conv_k]  w_k [H_kv*d_k,conv_k]  W [H,d_k,d_k] or NULL
 *   (p->mix_unshared = 1: W [2,H,d_k,d_k], the key stream mixes with W[1][h]; the same holds wherever W appears below)
 *   cache_q [B,conv_k-1,H*d_k], cache_k [B,conv_k-1,H_kv*d_k]  (nullable)
 *   out, W != NULL: qdot [B,T,H,d_k], kdot [B,T,H,d_k]   (kdot per query head: phi uses W[h])
 *   out, W == NULL: qdot = conv(q) [B,T,H,d_k], kdot = conv(k) [B,T,H_kv,d_k]
 * Kernels: bf16 storage with W, d_k = 64 or 128 and conv_k <= 4 runs the mix on the tensor cores (fp16 operands, fp32
 * accumulation, results within the bf16 tolerance of 1e-2 of the RMS); every other case, and chunk = 1, runs exact
 * fp32 kernels.
 */
int lawcat_conv_fwd(const lawcat_params* p, const void* q, const void* k, const void* w_q, const void* w_k,
                    const void* W, const void* cache_q, const void* cache_k, void* qdot, void* kdot, void* ws,
                    size_t ws_bytes, void* stream, int* dev_status);

/*
 * The gate function in front of the layer (Section 4.2: additional linear layers whose output goes through a sigmoid;
 * appendix, ablation on the rank of the gate function: two consecutive low-rank linear layers, rank 16 ... 128 or full):
 *   a_t = A2 (A1 x_t) + bias
 *   x [B,T,d_model] hidden states, A1 [rank,d_model] first layer, A2 [H*gate_dim,rank] second layer,
 *   bias [H*gate_dim] (nullable), all in p->dtype
 *   out: gate [B,T,H,gate_dim] in p->dtype: the logits, i.e. the `gate` input of the entry points below with
 *        gate_mode = LAWCAT_GATE_LOGITS, which apply the sigmoid and the power 1/gate_tau where they read them.
 * Only B, T, H, gate_dim, dtype and chunk of *p are used. d_model <= 16384, rank <= 1024.
 * Kernels: bf16 storage with rank 16, 32, 64 or 128, d_model and H*gate_dim multiples of 8 runs both layers in one
 * tensor-core kernel (bf16 operands, the bottleneck activations as a two-term bf16 pair, fp32 accumulation; one rounding
 * to bf16 at the end). Calls of up to 1024 tokens (a decode step, a short prompt; bf16, rank, d_model and H*gate_dim
 * multiples of 8) run a latency-oriented fp32 CUDA-core kernel instead (about 18 us for a decode step of 64 sequences at
 * the 7B widths, where one block of the tensor-core kernel takes 50). Every other case, and chunk = 1, runs exact fp32
 * kernels with the bottleneck activations [B*T,rank] in fp32 scratch (lawcat_gate_fn_workspace_bytes; 0 for the other two
 * kernels).
 * Errors: as for every entry point (see the top of this header); the tensor-core kernel's waits are bounded
 * (LAWCAT_ERR_TIMEOUT through dev_status).
 */
size_t lawcat_gate_fn_workspace_bytes(const lawcat_params* p, int32_t d_model, int32_t rank);
int lawcat_gate_fn_fwd(const lawcat_params* p, int32_t d_model, int32_t rank, const void* x, const void* A1,
                       const void* A2, const void* bias, void* gate, void* ws, size_t ws_bytes, void* stream,
                       int* dev_status);

/*
 * Backward of lawcat_conv_fwd (needed by the layer-wise distillation of Section 5.1; the paper prints no formulas,
 * this is the chain rule on conv -> mix -> phi). d_qdot, d_kdot have the shapes of the forward outputs.
 *   out: dq [B,T,H,d_k], dk [B,T,H_kv,d_k] in p->dtype; dw_q, dw_k, dW in fp32, shaped like w_q, w_k, W.
 * Weight gradients are overwritten, not accumulated. dW must be NULL when W is NULL. Any output may be NULL.
 * Kernels: bf16 storage with W, d_k = 64 and the softmax feature map runs the mix, the softmax Jacobian and dW on the
 * tensor cores (two-term fp16 operands); every other case, and chunk = 1, runs exact fp32 kernels.
 */
int lawcat_conv_bwd(const lawcat_params* p, const void* q, const void* k, const void* w_q, const void* w_k,
                    const void* W, const void* cache_q, const void* cache_k, const void* d_qdot,
                    const void* d_kdot, void* dq, void* dk, float* dw_q, float* dw_k, float* dW, void* ws,
                    size_t ws_bytes, void* stream, int* dev_status);

/*
 * Normalized gated linear attention on given feature-mapped streams (Eq. 4 - Eq. 8).
 *   qdot, kdot [B,T,H,d_k]  v [B,T,H_kv,d_v]  gate [B,T,H,gate_dim]
 *   S0 [B,H,d_k,d_v] fp32, z0 [B,H,d_k] fp32: state before token 0 (nullable = zero, Eq. 5)
 *   out: o [B,T,H,d_v]; den [B,T,H] fp32 = qdot_t . z_t + eps (nullable; gla_bwd needs it);
 *        S_T, z_T = state after the last token (nullable)
 * Kernels: bf16 storage with d_k = d_v = 64 runs chunkwise (64 tokens) on the tensor cores, with the same two exceptions
 * and the same LAWCAT_ERR_NUMERIC report as lawcat_layer_fwd (sharp sigmoid gates, calls of fewer than 16 tokens); every
 * other case, and chunk = 1, runs the exact recurrence. ws: lawcat_workspace_bytes(p, LAWCAT_OP_GLA_FWD).
 */
int lawcat_gla_fwd(const lawcat_params* p, const void* qdot, const void* kdot, const void* v, const void* gate,
                   const float* S0, const float* z0, void* o, float* den, float* S_T, float* z_T, void* ws,
                   size_t ws_bytes, void* stream, int* dev_status);

/*
 * Backward of lawcat_gla_fwd for an upstream gradient dO [B,T,H,d_v] (distillation step, Section 5.1; chain rule
 * on Eq. 4 and Eq. 8). o and den (the forward outputs) are accepted for symmetry and may be NULL: the backward
 * recomputes the denominator and dO.o in fp32, because the stored o is rounded to the storage type.
 *   out: d_qdot, d_kdot [B,T,H,d_k]; dv [B,T,H_kv,d_v] (summed over the G query heads of a group);
 *        dgate [B,T,H,gate_dim] -- the gradient with respect to the `gate` input (logits or log-decays).
 * No gradient flows into S0, z0 and none is taken from S_T, z_T.
 * Kernels: bf16 storage with d_k = d_v = 64, log-decay gates or sigmoid gates with gate_tau >= 8, and at least 16
 * tokens runs the chunkwise tensor-core backward (two-term fp16 operands: gradients within 1e-2 of their RMS); sharper
 * gates, shorter calls, other shapes and chunk = 1 run the exact three-sweep backward. ws: lawcat_workspace_bytes(p, LAWCAT_OP_GLA_BWD).
 */
int lawcat_gla_bwd(const lawcat_params* p, const void* qdot, const void* kdot, const void* v, const void* gate,
                   const float* S0, const float* z0, const void* o, const float* den, const void* dO,
                   void* d_qdot, void* d_kdot, void* dv, void* dgate, void* ws, size_t ws_bytes, void* stream,
                   int* dev_status);

/*
 * The whole layer forward, fused: conv -> mix -> phi -> normalized GLA (Fig. 1); the prefill path of Section 5.5.
 * Inputs as in lawcat_conv_fwd (W required) and lawcat_gla_fwd. The conv caches and the state allow a long
 * sequence to be processed in pieces (Section 4.1 on caching; streaming use in Section 6):
 *   cache_q_out [B,conv_k-1,H*d_k], cache_k_out [B,conv_k-1,H_kv*d_k] = the last conv_k-1 raw tokens seen
 *   (taken from the input caches when T < conv_k-1); S_T, z_T = the state after the last token. All nullable.
 * The *_out buffers must not alias the *_in buffers.
 * bf16 storage with d_k = d_v in {64, 128}, the softmax feature map, conv_k <= 4 and chunk in {0, 64} run on the
 * chunkwise tensor-core kernel (chunks of 64 tokens, 16-bit operands, fp32 accumulation: results within the bf16
 * tolerance of the exact recurrence); chunk = 1 selects the exact fp32 recurrence for any supported shape. Inside that
 * set two cases also take the exact recurrence: sharp sigmoid gates (LAWCAT_GATE_LOGITS with gate_tau < 8: the decay
 * factors of half a chunk then leave the fp16 range, and 8-bit-mantissa operands miss the tolerance), and calls of fewer
 * than 16 tokens (a state of so few terms shows the rounding of single operands). With LAWCAT_GATE_LOGDECAY the caller
 * chooses the decays and the kernel cannot know them in advance: when a half chunk's accumulated log2-decay exceeds 8 in
 * magnitude (a state that loses about a sixth or more at every token), or a state entry exceeds 3e4, the affected chunks run
 * on 8-bit-mantissa operands, the result is delivered, and dev_status reports LAWCAT_ERR_NUMERIC: the result may miss
 * the tolerance; chunk = 1 has no such limit.
 * Asynchronous conditions arrive through dev_status (largest code wins): LAWCAT_ERR_NUMERIC, as above, or a decay
 * exponent within half a chunk left the range +-120 and was clamped; LAWCAT_ERR_TIMEOUT, a bounded device-side wait ran
 * out (the kernel has released its resources and returned; the outputs are undefined).
 */
int lawcat_layer_fwd(const lawcat_params* p, const void* q, const void* k, const void* v, const void* gate,
                     const void* w_q, const void* w_k, const void* W, const void* cache_q_in,
                     const void* cache_k_in, const float* S0, const float* z0, void* o, void* cache_q_out,
                     void* cache_k_out, float* S_T, float* z_T, void* ws, size_t ws_bytes, void* stream,
                     int* dev_status);

/*
 * lawcat_layer_fwd over PACKED sequences of different lengths (batched and chunked prefill of a serving loop; the paper
 * points to the streaming use of the constant-size state in Section 6). The tokens of nseq sequences lie back to back
 * along T: p->B must be 1, p->T is the total, and sequence i covers tokens [cu_seqlens[i], cu_seqlens[i+1]).
 *   cu_seqlens: HOST array of nseq + 1 non-decreasing ints, cu_seqlens[0] = 0, cu_seqlens[nseq] = p->T
 *   q, k, v, gate, o: as in lawcat_layer_fwd with B = 1
 *   S0 [nseq,H,d_k,d_v], z0 [nseq,H,d_k], cache_q_in [nseq,conv_k-1,H*d_k], cache_k_in [nseq,conv_k-1,H_kv*d_k]:
 *     what each sequence starts from (nullable: every sequence starts from nothing, i.e. the state is reset at every
 *     boundary; a chunk of a longer sequence passes the state and caches its previous chunk returned)
 *   S_T, z_T, cache_q_out, cache_k_out: the same per sequence after its last token (nullable)
 * No token of one sequence reaches another: neither through the conv (its first conv_k - 1 tokens see the sequence's own
 * cache or zeros) nor through the state. An empty sequence hands its state and caches through. The sequences are
 * enqueued one after the other on `stream`, sharing `ws` (lawcat_layer_fwd_varlen_workspace_bytes: the largest need).
 */
size_t lawcat_layer_fwd_varlen_workspace_bytes(const lawcat_params* p, const int32_t* cu_seqlens, int nseq);
int lawcat_layer_fwd_varlen(const lawcat_params* p, const int32_t* cu_seqlens, int nseq, const void* q, const void* k,
                            const void* v, const void* gate, const void* w_q, const void* w_k, const void* W,
                            const void* cache_q_in, const void* cache_k_in, const float* S0, const float* z0, void* o,
                            void* cache_q_out, void* cache_k_out, float* S_T, float* z_T, void* ws, size_t ws_bytes,
                            void* stream, int* dev_status);

/*
 * Backward of the whole layer (Fig. 1) for an upstream gradient dO [B,T,H,d_v]: the layer-wise distillation step of
 * Section 5.1 in one call (chain rule on conv -> mix -> phi -> Eq. 4, Eq. 8; the paper prints no formulas). The features
 * qdot, kdot are recomputed from q, k and never stored in the storage type: on the tensor-core path (bf16, d_k = d_v =
 * 64, softmax feature map, conv_k <= 4, gate_tau >= 8 in LOGITS mode, chunk != 1) they
 * and their gradients pass between the stages in fp32 scratch; every other shape runs the exact kernels as the chain
 * conv -> attention -> attention backward -> conv backward entirely in fp32 (bf16 tensors are widened into scratch
 * first and the four activation gradients narrowed at the end).
 *   in:  the inputs of lawcat_layer_fwd (caches and initial state nullable) and dO
 *   out: dq [B,T,H,d_k], dk [B,T,H_kv,d_k], dv [B,T,H_kv,d_v], dgate [B,T,H,gate_dim] in p->dtype;
 *        dw_q, dw_k, dW in fp32, shaped like w_q, w_k, W, overwritten. All outputs are required.
 * No gradient flows into the conv caches or the initial state.
 */
int lawcat_layer_bwd(const lawcat_params* p, const void* q, const void* k, const void* v, const void* gate,
                     const void* w_q, const void* w_k, const void* W, const void* cache_q, const void* cache_k,
                     const float* S0, const float* z0, const void* dO, void* dq, void* dk, void* dv, void* dgate,
                     float* dw_q, float* dw_k, float* dW, void* ws, size_t ws_bytes, void* stream, int* dev_status);

/*
 * One recurrent decode step for B sequences (p->T is ignored): the layer at a single token, using the conv cache
 * of Section 4.1 and the constant-size state of Eq. 4.
 *   q_t [B,H,d_k]  k_t [B,H_kv,d_k]  v_t [B,H_kv,d_v]  gate_t [B,H,gate_dim]
 *   S [B,H,d_k,d_v], z [B,H,d_k] fp32 and cache_q, cache_k (layout as above) are REQUIRED and updated IN PLACE:
 *   the state advances by one token, the caches drop their oldest row and append q_t, k_t.
 *   out: o_t [B,H,d_v]
 *   ws: device scratch of lawcat_workspace_bytes(p, LAWCAT_OP_DECODE_STEP) bytes (the token's features, decays and
 *   denominators, handed from the first launch of the step to the second); LAWCAT_ERR_WORKSPACE_TOO_SMALL otherwise.
 */
int lawcat_decode_step(const lawcat_params* p, const void* q_t, const void* k_t, const void* v_t,
                       const void* gate_t, const void* w_q, const void* w_k, const void* W, float* S, float* z,
                       void* cache_q, void* cache_k, void* o_t, void* ws, size_t ws_bytes, void* stream,
                       int* dev_status);

/*
 * The layer forward of Fig. 1 for callers whose tensors live in HOST memory (pinned memory makes the copies
 * asynchronous). h_* are host pointers laid out like the device tensors of lawcat_layer_fwd (no caches, zero initial
 * state); `arena` is caller-owned DEVICE scratch of at least lawcat_layer_fwd_host_arena_bytes(p) bytes that receives
 * the inputs, the output, the workspace and the state handed from slice to slice. The sequence is processed in slices
 * of 2048 tokens (the state of Eq. 4 and the conv cache of Section 4.1 carry over, as in chunked prefill): the
 * host-to-device copies of the next slice, the layer on the current slice and the copy of the previous slice's output
 * back to h_o run on three streams. The two copy streams belong to the library (one pair per device, created on the
 * first call); they start behind everything already enqueued on `stream`, and `stream` ends behind the last copy, so
 * that the caller orders and synchronizes on `stream` alone. Returns without synchronizing; h_o is valid once
 * `stream` has drained. Calls that share an arena must be enqueued on the same stream.
 */
size_t lawcat_layer_fwd_host_arena_bytes(const lawcat_params* p);
int lawcat_layer_fwd_host(const lawcat_params* p, const void* h_q, const void* h_k, const void* h_v,
                          const void* h_gate, const void* h_w_q, const void* h_w_k, const void* h_W, void* h_o,
                          void* arena, size_t arena_bytes, void* stream);

/*
 * lawcat_layer_fwd without any caller-provided workspace (the paper has no counterpart; this exists for deployment).
 *
 * Who needs it: code that must not, or cannot, allocate device memory at the point of the call -- a serving loop whose
 * memory pool is frozen after start-up, a plugin running inside a host application that owns the allocator, a callback
 * that runs where cudaMalloc is forbidden. Such callers cannot size and provide `ws`. Here the scratch (the fp32
 * conv+mix+phi outputs qdot and kdot of the exact CUDA-core path) lives in a fixed device array inside the library
 * image, LAWCAT_NOALLOC_SCRATCH_BYTES large; every GPU that loads the library holds that memory until the process ends.
 *
 * Arguments and results are those of lawcat_layer_fwd minus ws/ws_bytes; the computation is the exact (fp32
 * accumulate, CUDA-core) path for every dtype. The call allocates nothing and frees nothing.
 *   - Limit: 2 * roundup256(4 * B*T*H*d_k) bytes must fit the array, i.e. B*T*H*d_k <= 4 Mi elements with the default
 *     32 MiB. Larger problems return LAWCAT_ERR_TOO_LARGE before anything is enqueued: split the sequence and carry the
 *     state and the conv caches from call to call.
 *   - The first call on each device looks up the device address of the array (cudaGetSymbolAddress, with that device
 *     current); make that first call outside of any stream capture.
 *   - All calls on one device share the one array, and it keeps whatever the previous call left in it. Nothing in it
 *     has to start at zero (both tensors are fully written before they are read), but two calls whose kernels overlap
 *     on the GPU -- different streams, no ordering between them -- race on it. Keep calls on one stream or order them.
 */
#define LAWCAT_NOALLOC_SCRATCH_BYTES (32u << 20)
size_t lawcat_noalloc_scratch_bytes(void);
int lawcat_layer_fwd_noalloc(const lawcat_params* p, const void* q, const void* k, const void* v, const void* gate,
                             const void* w_q, const void* w_k, const void* W, const void* cache_q_in,
                             const void* cache_k_in, const float* S0, const float* z0, void* o, void* cache_q_out,
                             void* cache_k_out, float* S_T, float* z_T, void* stream, int* dev_status);

#ifdef __cplusplus
}
#endif
#endif /* LAWCAT_H_ */
