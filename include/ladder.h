/* libladder -- bf16 forward (prefill + autoregressive decode) of a Ladder-Residual /
 * standard-residual / hybrid Llama-shaped transformer on ONE NVIDIA B200 (sm_100a).
 *
 * Plain C ABI: no C++ or torch types cross this boundary.  Unless a parameter says
 * HOST, every data pointer is a DEVICE pointer on the current CUDA device.  All work is
 * enqueued stream-ordered on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 * legacy default stream); an internal second stream, when enabled, is forked from and
 * joined back to it with events, so callers see ordinary stream semantics.  No call
 * synchronises the device unless its comment says so.
 *
 * Residual rules implemented (m = 1..2N indexes modules, odd = attention, even = MLP):
 *   standard layer :  x_m = x_{m-1} + h_m(x_{m-1})                      (paper Sec. 2, Eq. 1)
 *   ladder layer   :  x_m = x_{m-1} + h_m(x_{m-2})                      (paper Sec. 3.1, Eq. 2)
 * in the pending-output form of the paper's Algorithm 1 with the all-reduce removed:
 * initial pending outputs are zero (modules 1 and 2 both read x_0), outputs still pending
 * after the last layer are added before the final norm, and a standard layer first adds
 * whatever is pending and leaves nothing pending.  Each module h_m is pre-norm RMSNorm
 * followed by grouped-query causal attention with rotary embedding on interleaved pairs,
 * or by a SwiGLU MLP ("Llama-3's model architecture", paper Sec. 3.3.1).
 *
 * Numerics: bf16 weights, 16-bit KV cache in IEEE binary16 (same bytes as bf16, three more significant bits:
 * with bf16 keys and values the cache alone puts deep models outside a 2e-2 hidden-state bound), fp32
 * accumulation, fp32 softmax, fp32 residual stream, fp32 logits.  In the decode path activations enter the
 * tensor cores as a bf16 high + low pair (about 16 mantissa bits; free in a bandwidth-bound
 * kernel) for batch <= 16, and so do the prefill GEMMs; queries enter the attention as a binary16 high + low pair.
 * Greedy argmax picks the lowest index on ties.
 *
 * Errors: every function returns a ladder_status_t; argument errors are detected on the
 * host before anything is launched; nothing aborts, traps or hangs the device.
 * A model object is not thread-safe; distinct objects are independent.
 */
#ifndef LADDER_H_
#define LADDER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ladder_model ladder_model_t; /* opaque, owned by the library */

typedef enum {
  LADDER_OK = 0,
  LADDER_ERR_INVALID_ARG = 1, /* NULL / out-of-range argument                          */
  LADDER_ERR_UNSUPPORTED = 2, /* shape outside what the kernels handle (see create)    */
  LADDER_ERR_OOM = 3,         /* workspace allocation failed                           */
  LADDER_ERR_CUDA = 4,        /* a CUDA call failed (sticky; see ladder_last_error)    */
  LADDER_ERR_STATE = 5,       /* cache overflow, batch > max_batch, prefill on a non-empty position */
  LADDER_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out in an earlier step (see ladder_device_status) */
} ladder_status_t;

/* Bits of the device status word (ladder_device_status). */
#define LADDER_DEV_BAD_TOKEN 1      /* a token id was outside [0, vocab): row treated as id 0 */
#define LADDER_DEV_CACHE_OVERFLOW 2 /* a position >= max_seq_len reached a kernel: store skipped */
#define LADDER_DEV_TIMEOUT 4        /* a bounded wait inside the persistent decode kernel gave up (about 0.3 s): that
                                       step's outputs are invalid; later launches end at once until the word is read */

/* Per-layer architecture (ladder_config_t.layer_mode), paper Sec. 3.3.1. */
#define LADDER_LAYER_STANDARD 0    /* x_m = x_{m-1} + h_m(x_{m-1})                           (Sec. 2, Eq. 1)   */
#define LADDER_LAYER_LADDER 1      /* x_m = x_{m-1} + h_m(x_{m-2})                           (Sec. 3.1, Eq. 2) */
#define LADDER_LAYER_PARALLEL 2    /* parallel attention and MLP: both modules read the layer's input through ONE
                                      RMSNorm (the attention gain; mlp_norm of the layer is unused) and both
                                      outputs are added: x_l = x_{l-1} + Attn(n) + MLP(n), n = Norm(x_{l-1})     */
#define LADDER_LAYER_UPPER_BOUND 3 /* the communication-free upper bound: the standard model with the all-reduce
                                      deleted, which on one device is the standard model (alias of 0)           */

typedef struct {
  uint32_t struct_size; /* sizeof(ladder_config_t), for ABI versioning */
  int32_t d_model, n_layers, n_q_heads, n_kv_heads, head_dim, d_ff, vocab_size;
  float rms_eps, rope_theta;
  int32_t max_batch;        /* largest batch of any call (decode kernels: <= 64)          */
  int32_t max_seq_len;      /* cache capacity per sequence (prompt + generated)           */
  int32_t max_prefill_tokens; /* largest batch*seq_len of a prefill call; 0 = max_batch*max_seq_len */
  const uint8_t* layer_is_ladder; /* HOST, n_layers bytes, copied. NULL = all ladder; 0 = standard layer */
  /* -- appended fields: a caller may pass struct_size = offsetof(ladder_config_t, layer_mode) and omit them -- */
  const uint8_t* layer_mode;      /* HOST, n_layers bytes of LADDER_LAYER_*, copied; NULL = use layer_is_ladder */
  const uint8_t* module_stale;    /* HOST, 2*n_layers bytes, copied; NULL = what the layer modes imply.  Entry m-1
                                     non-zero: module m (1-based; odd = attention, even = MLP) reads x_{m-2}
                                     instead of x_{m-1}.  Module 1 reads x_0 whatever its entry.  Implied rule:
                                     ladder layer 1,1 except that the attention of a ladder layer directly after
                                     a non-ladder layer reads the complete stream (0); standard 0,0; parallel 0,1.
                                     States any other rule module by module, e.g. the hybrid in which the first
                                     ladder attention also skips the preceding MLP's output. */
} ladder_config_t;
/* Shape limits (else LADDER_ERR_UNSUPPORTED): max_seq_len <= 65536 (the decode attention merges at most 1024
 * splits of 64 keys); head_dim 64 or 128; n_q_heads % n_kv_heads == 0;
 * d_model, n_q_heads*head_dim and d_ff multiples of 8; (n_q_heads+2 n_kv_heads)*head_dim,
 * 2*d_ff, d_model and vocab_size multiples of 8. */

/* Weights: bf16, row-major with the input (K) dimension contiguous, 16-byte aligned.
 * BORROWED: the caller owns them and keeps them alive and unchanged until ladder_destroy;
 * the library never writes, frees or copies them (a 70B model is ~141 GB). */
typedef struct {
  const void* tok_embedding;    /* [vocab, d_model]                                        */
  const void* final_norm;       /* [d_model]                                               */
  const void* lm_head;          /* [vocab, d_model] (untied)                               */
  const void* const* attn_norm; /* HOST array[n_layers] of device ptrs, each [d_model]     */
  const void* const* w_qkv;     /* [(Hq+2Hkv)*Dh, d_model]: Q heads, then K heads, then V  */
  const void* const* w_o;       /* [d_model, Hq*Dh]                                        */
  const void* const* mlp_norm;  /* [d_model]                                               */
  const void* const* w_gate_up; /* [2*d_ff, d_model]: row 2j = gate_j, row 2j+1 = up_j      */
  const void* const* w_down;    /* [d_model, d_ff]                                         */
} ladder_weights_t;

/* KV cache: caller-allocated, library reads and writes.  K holds post-rotation keys.  Elements are IEEE binary16
 * (fp16), 2 bytes each; values beyond +-65504 saturate (keys and values are projections of RMS-normalised
 * activations and stay far inside that range). */
typedef struct {
  void* k;           /* binary16 [n_layers][max_batch][n_kv_heads][max_seq_len][head_dim] */
  void* v;           /* same shape                                                    */
  int32_t* seq_lens; /* int32 [max_batch]: tokens cached per sequence; prefill sets it,
                        each decode step reads the position from it and adds one        */
} ladder_kv_cache_t;

/* Outputs: all optional (NULL = not wanted), caller-owned device buffers. */
typedef struct {
  int32_t* next_tokens; /* [batch] greedy token                                            */
  float* final_hidden;  /* [batch, d_model] final RMSNorm output at the last/current position */
  float* logits;        /* [batch, vocab]                                                  */
  float* all_hidden;    /* prefill only: [batch, seq_len, d_model] final RMSNorm at every position */
} ladder_outputs_t;

/* Bytes of ONE of the two cache buffers (k or v) for this configuration.  The paper never names the cache; it is
 * implied by its "prefill and decode phase" (Sec. 3.2): keys (after rotation) and values of every layer, kept so
 * that a decode step attends to all earlier positions without recomputing them. */
size_t ladder_kv_cache_bytes(const ladder_config_t* cfg);

/* Validates the configuration, allocates the workspace (two fp32 residual buffers of
 * max(max_batch, max_prefill_tokens) rows, activation scratch, split-KV partials, the
 * rotary table), creates the second stream and events.  Allocates device memory and may
 * synchronise.  On failure *out is NULL. */
ladder_status_t ladder_model_create(const ladder_config_t* cfg, const ladder_weights_t* weights,
                                    ladder_model_t** out);

/* Decode scheduling (paper Sec. 3.2: side stream, CUDA graphs).
 *   n_streams 1|2 : with 2, attention modules and MLP modules of ladder layers run on two
 *                   streams with the event edges the ladder rule allows (module m's last GEMM
 *                   waits for module m-1; everything before it does not); standard layers serialise.
 *   use_graph 0|1 : capture one decode step as a CUDA graph and replay it.
 *   use_pdl   0|1 : launch consecutive kernels of a stream with programmatic dependent launch so a
 *                   kernel's weight prefetch starts before its predecessor has drained.
 * Defaults: 2, 1, 1.  Results are bit-identical across all settings. */
ladder_status_t ladder_model_set_schedule(ladder_model_t* m, int32_t n_streams, int32_t use_graph, int32_t use_pdl);

/* Persistent decode step (default on; batch <= 4: there the bf16 hi + lo activation pair fits one MMA tile;
 * larger batches take the tcgen05 kernels, one kernel per GEMM).  The ladder layers at the top of the model (all layers of
 * an all-ladder model) and the LM head of a decode step run as ONE cooperative kernel launch.  Standard-residual
 * layers below them run one kernel per GEMM when a layer's weights exceed 300 MB (measured faster there) and go
 * into the same launch otherwise; on = 2 puts every layer into the launch whatever its size.  A large-layer
 * model whose top layer is standard does not use the launch at all.  Every weight-streaming GEMM is a phase of
 * that kernel,
 * attention runs on dedicated warps of the same CTAs, and a grid-wide hand-over is a counter in global
 * memory that is polled only where data crosses SMs.  With the ladder rule (Eq. 2: module m reads
 * x_{m-2}) every such dependency points two phases back, so the weight stream never stops between
 * modules; with the standard rule (Eq. 1) each phase waits for the one before.  on = 0 selects the
 * multi-kernel schedule configured by ladder_model_set_schedule (also used automatically for batch > 4
 * and on devices where the kernel cannot be made resident).  Results are bit-identical either way.
 * A fresh model (before any call of this function) takes this path for batch <= 4 except for all-ladder models with layers below 300 MB whose attention module is at most a
 * quarter as wide as the hidden size (one tensor-parallel rank's slice), where the pending-output form on the tcgen05
 * GEMMs measured 4-6 % faster; on != 0 insists on the persistent kernel.
 * ladder_model_persistent_active returns 1 when decode steps of batch <= 4 take this path. */
ladder_status_t ladder_model_set_persistent(ladder_model_t* m, int32_t on);
int32_t ladder_model_persistent_active(const ladder_model_t* m);

/* Test hook for the bounded waits of the persistent kernel: with on = 1 the LM-head phase of the next decode
 * steps waits for one more finished unit than its producer phase has, i.e. for a count that is never reached.
 * Nothing faults or spins forever: the wait gives up after about 0.3 s, sets the LADDER_DEV_TIMEOUT bit of the
 * device status word, every other wait in the launch gives up as soon as it sees the bit, and the launch ends.
 * Later launches return at once until ladder_device_status has read and cleared the word.  on = 0 restores
 * the real dependency. */
ladder_status_t ladder_debug_stall_last_phase(ladder_model_t* m, int32_t on);

/* Host only (no GPU needed): describes the phase list the persistent kernel would execute for this
 * configuration, batch and SM count, as int32 words, for inspection and tests.
 *   header: n_phases, n_attention_nodes, n_counters, first_layer_in_kernel, ok
 *   per phase (56 words): kind (0 QKV, 1 gate/up, 2 Wo, 3 down, 4 LM head), layer, N, K, n_units, n_static, n_claims,
 *     claim_counter, done_counter, n_rounds, count[10], size[10], n_act_deps, act_dep[6], act_need[6],
 *     n_epi_deps, epi_dep[6], epi_need[6]
 *   per attention node (29 words): layer, split_counter, merge_counter, n_deps, dep[6], need[6], n_merge_deps,
 *     merge_dep[6], merge_need[6]
 * Returns the number of words written, -(words needed) if cap is too small, -1 on a bad argument. */
int32_t ladder_stack_plan(const ladder_config_t* cfg, int32_t batch, int32_t sm_count, int32_t* out, int32_t cap);

/* With two streams, the GEMMs of a ladder layer's attention module and MLP module can be run side by side on
 * disjoint sets of SMs (each GEMM is a persistent kernel that claims its work dynamically, so it runs
 * on any number of CTAs).  sms_attention_stream: -1 = the library's choice (default): no split, every GEMM on all
 * SMs, which measured fastest everywhere except for batch 5..64 with layers below 300 MB, where 56 of 148 SMs (44 above batch 32) go
 * to the attention stream; -2 = never split; 0 = in proportion to the bytes each module streams; n > 0 = that many
 * SMs (at most half of them) for the attention module's GEMMs and the rest for the MLP's.  Batch <= 4: results are
 * bit-identical for every setting.  Batch 5..64: every CTA accumulates one contiguous K range in fp32, so the number
 * of CTAs a GEMM runs on decides where the sums are cut: settings that give a GEMM different shares differ in
 * rounding (~1e-4 of the hidden state), each of them reproducible from run to run.
 * Whenever the split is on, every module reads x_{m-2} (all layers ladder) and batch is 5..64 (any batch when the
 * split was asked for explicitly), the step also runs
 * in the pending-output form of Algorithm 1: a module's output stays in a buffer of its own and is added to the
 * residual when the next module's input is normalised, so the attention chain and the MLP chain wait for each
 * other's normalised-input kernel only, never for a GEMM.  The additions are the same fp32 additions in the same
 * order (bit-identical to -3 on the same shares).  -3 = the library's choice of split without that form (each output
 * added by its GEMM's epilogue). */
ladder_status_t ladder_model_set_sm_split(ladder_model_t* m, int32_t sms_attention_stream);

/* Tensor parallelism (paper Sec. 2, Eq. 1: x_i = AllReduce(h_i(x_{i-1})) + x_{i-1}; Sec. 3.1, Eq. 2 and Algorithm 1:
 * with ladder residuals module i reads x_{i-2}, so the all-reduce of module i-1 runs while module i computes).
 * The model handed to ladder_model_create is ONE RANK'S SLICE: n_q_heads, n_kv_heads and d_ff are the rank's share
 * (w_qkv the rows of its heads, w_o the matching columns, w_gate_up the rows of its hidden units, w_down the
 * matching columns); d_model, the norms, the embedding and the LM head are whole and the same on every rank.  The
 * output and down projections then give a partial sum, and `exchange` is called - from inside ladder_prefill* /
 * ladder_decode_step, on the calling host thread, in module order (attention of layer 0, MLP of layer 0, ...) - to
 * ENQUEUE on `cuda_stream` the in-place sum of partial[0 .. count) (device, fp32, count = rows x d_model) over the
 * ranks; it must not block on the device and every rank must get the same bits (the ranks' residual streams have to
 * stay identical).  Non-zero return: the call fails with LADDER_ERR_CUDA.
 * Schedule: every module stores its (partial) output and the sum is added where a later module's input is formed
 * (the pending-output form of Algorithm 1).  Decode: the exchange runs on the stream of the module that produced
 * the partial, so with two streams a ladder layer's other module computes meanwhile, while with standard residuals
 * the next module's input waits for it (Eq. 1: the paper's baseline); all batch sizes run on the tcgen05 GEMMs, one
 * kernel per GEMM.  Prompt pass: exchanges and adds run on a stream of their own and the GEMM stream waits only
 * where a module reads what an add writes.  A layer whose MLP module reads the same input as its attention module
 * (parallel attention + MLP, Sec. 3.3.1) has ONE exchange: the down projection adds the attention module's stored
 * partial sum before it.  capturable != 0: `exchange` may be called while its stream is being
 * captured into a CUDA graph (NCCL collectives may); 0: decode steps are enqueued without a graph.
 * fn == NULL switches it off.  Pipeline-stage calls (ladder_stage_*) work under it (tensor parallelism inside every
 * stage, paper Sec. 5.1): the pair a stage hands on is the summed stream state, identical on all its ranks.
 * Costs 2 x max_prefill_tokens x d_model x 4 bytes of device memory on first use (LADDER_ERR_OOM if there is none).
 * Measured on one GPU only (a world of one, and against recorded partials of the other ranks): the hardware this
 * was built on has one GPU per job, so no multi-GPU timing is claimed. */
typedef ladder_status_t (*ladder_exchange_fn)(void* ctx, float* partial, int64_t count, void* cuda_stream);
ladder_status_t ladder_model_set_exchange(ladder_model_t* m, ladder_exchange_fn fn, void* ctx, int32_t capturable);

/* The exchange over NCCL: one communicator per rank (= process = GPU, the current CUDA device at creation).
 * Rank 0 draws an id with ladder_comm_unique_id (LADDER_COMM_ID_BYTES host bytes) and hands it to the other ranks by
 * any means (e.g. a torch.distributed broadcast); every rank then calls ladder_comm_create (collective: returns when
 * all `world` ranks have called it).  The NCCL library is looked up when first needed (the copy the process has
 * loaded already, else the system's); LADDER_ERR_UNSUPPORTED if there is none, LADDER_ERR_CUDA if NCCL reports an
 * error.  ladder_comm_all_reduce_sum has the ladder_exchange_fn signature (ctx = the communicator);
 * ladder_model_set_tensor_parallel(m, comm) installs it (capturable), comm == NULL switches tensor parallelism off.
 * The communicator is the caller's: destroy it after the models that use it. */
#define LADDER_COMM_ID_BYTES 128
typedef struct ladder_comm ladder_comm_t;
ladder_status_t ladder_comm_unique_id(void* id);
ladder_status_t ladder_comm_create(int32_t world, int32_t rank, const void* id, ladder_comm_t** out);
ladder_status_t ladder_comm_destroy(ladder_comm_t* comm);
int32_t ladder_comm_world(const ladder_comm_t* comm);
int32_t ladder_comm_rank(const ladder_comm_t* comm);
ladder_status_t ladder_comm_all_reduce_sum(void* comm, float* partial, int64_t count, void* cuda_stream);
ladder_status_t ladder_model_set_tensor_parallel(ladder_model_t* m, ladder_comm_t* comm);

/* The exchange over peer memory, for the decode step (paper Sec. 2 Eq. 1; messages of batch x d_model fp32), in two
 * forms: a stand-alone all-reduce (ladder_peer_all_reduce_sum) and, inside a model, an exchange fused into the GEMM
 * before it and the launch after it (further down).  The stand-alone form is one
 * kernel per exchange in which every rank stores its partial sum into a receive slot in each peer's memory (plain
 * stores through the NVLink peer mapping), raises a counter there, waits - bounded, about 0.3 s, then
 * LADDER_DEV_TIMEOUT in the status word and no sum - for its peers' counters in its own memory and adds the slots in
 * rank order, so every rank gets the same bits.  Two channels (0: attention modules, 1: MLP modules: the two chains
 * of a step, each ordered on its own stream) with two receive slots each.
 * Set-up: every rank calls ladder_peer_create(world <= LADDER_PEER_MAX_WORLD, rank, max_floats >= max_batch x d_model,
 * a multiple of 4) on its GPU (allocates and clears 1 KiB + 32 x world x max_floats bytes), hands the
 * LADDER_PEER_HANDLE_BYTES of ladder_peer_export (a CUDA IPC memory handle) to the others, and calls
 * ladder_peer_connect(peer, r, handle_of_r, NULL) for every other rank r (ranks that are threads of one process pass
 * ladder_peer_local_base of r's object as same_process_base instead, with peer access between the devices enabled
 * by the caller).  All ranks must have connected before the first exchange.  ladder_peer_all_reduce_sum enqueues one
 * exchange on `cuda_stream`: partial[0 .. count) (device, fp32, 16-byte aligned, count a multiple of 4 and at most
 * max_floats) becomes the sum over the ranks; every rank must enqueue the same sequence of (channel, count).
 * device_status: a device int32 that receives LADDER_DEV_TIMEOUT, or NULL.  Capturable into a CUDA graph.
 * Inside a model the exchange is FUSED into the kernels on either side of it, with no kernel of its own, no counter
 * and no fence: the output / down projection's epilogue stores every finished element of the partial sum straight
 * into the receive slot on every rank, together with the sequence number of the exchange in ONE aligned 8-byte store
 * (the transfer runs tile by tile under the GEMM); the launch that normalises the next reader's input polls
 * (bounded) each pair it needs until the number is the expected one and adds the slots in rank order while it
 * forms the residual stream.  This rests on aligned 8-byte stores reaching peer memory whole (as NCCL's
 * low-latency protocol does).
 * The fused exchange is one-shot - (world - 1) x batch x d_model x 8 bytes leave every rank per exchange - so a decode
 * step uses it only while that is at most 8 MiB (batch 18 at world 8 and d_model 8192) and the model's `exchange`
 * (NCCL) above; ladder_model_set_peer_max_bytes moves the limit (negative: never fused).
 * ladder_model_set_tensor_parallel_peer(m, comm, peer): decode steps exchange that way over `peer`, the prompt pass
 * (messages of hundreds of MB, where NCCL's algorithms are the right ones) over `comm`; LADDER_ERR_INVALID_ARG if the
 * peer object is too small for max_batch x d_model, not connected or of another world.  ladder_model_set_peer(m, peer)
 * is the second half alone, for a model whose prompt-pass exchange was set with ladder_model_set_exchange
 * (LADDER_ERR_STATE if none is set); NULL switches back.  Both objects stay the caller's; a peer object serves ONE
 * model (each pipeline stage its own), or ladder_peer_all_reduce_sum calls: its channels number their exchanges.
 * ladder_debug_set_peer_hook: a function called on the host right after each decode-step output GEMM has been
 * enqueued (channel, stream), so that a test can enqueue an absent rank's stores there; steps then run ungraphed.
 * ladder_peer_probe_write / _read: connectivity check by host copies (rank a writes a word into rank b's memory, b
 * reads it after a host-side barrier).  ladder_peer_slot / ladder_peer_counter / ladder_peer_ctas_per_exchange expose
 * where a rank's data lands (a slot holds max_floats values for ladder_peer_all_reduce_sum, max_floats (value, number)
 * pairs for the fused exchange) and how the stand-alone kernel counts arrivals (each exchange adds ctas_per_exchange
 * to the sender's counter), so that a test can play an absent rank.
 * Exercised on one GPU only (a world of one, and worlds of two and four with the other ranks' stores made by the test):
 * the IPC path is covered by the probe between two processes; nothing is claimed about multi-GPU speed. */
#define LADDER_PEER_MAX_WORLD 8
#define LADDER_PEER_HANDLE_BYTES 64
typedef struct ladder_peer ladder_peer_t;
ladder_status_t ladder_peer_create(int32_t world, int32_t rank, int64_t max_floats, ladder_peer_t** out);
ladder_status_t ladder_peer_export(const ladder_peer_t* peer, void* handle);
void* ladder_peer_local_base(const ladder_peer_t* peer);
ladder_status_t ladder_peer_connect(ladder_peer_t* peer, int32_t r, const void* ipc_handle, void* same_process_base);
int32_t ladder_peer_connected(const ladder_peer_t* peer);
int32_t ladder_peer_world(const ladder_peer_t* peer);
int32_t ladder_peer_rank(const ladder_peer_t* peer);
int64_t ladder_peer_max_floats(const ladder_peer_t* peer);
int32_t ladder_peer_ctas_per_exchange(void);
ladder_status_t ladder_peer_destroy(ladder_peer_t* peer);
ladder_status_t ladder_peer_all_reduce_sum(ladder_peer_t* peer, int32_t channel, float* partial, int64_t count,
                                           int32_t* device_status, void* cuda_stream);
ladder_status_t ladder_peer_probe_write(ladder_peer_t* peer, int32_t r, uint32_t value);
ladder_status_t ladder_peer_probe_read(const ladder_peer_t* peer, int32_t from, uint32_t* value);
float* ladder_peer_slot(const ladder_peer_t* peer, int32_t channel, int32_t parity, int32_t from);
uint32_t* ladder_peer_counter(const ladder_peer_t* peer, int32_t channel, int32_t from);
ladder_status_t ladder_model_set_tensor_parallel_peer(ladder_model_t* m, ladder_comm_t* comm, ladder_peer_t* peer);
ladder_status_t ladder_model_set_peer(ladder_model_t* m, ladder_peer_t* peer);
ladder_status_t ladder_model_set_peer_max_bytes(ladder_model_t* m, int64_t bytes);
typedef void (*ladder_peer_hook_fn)(void* ctx, int32_t channel, void* cuda_stream);
ladder_status_t ladder_debug_set_peer_hook(ladder_model_t* m, ladder_peer_hook_fn fn, void* ctx);

/* Prompt pass ("prefill phase", paper Sec. 3.2): the module chain of Eq. 1 / Eq. 2 (in the pending-output form of
 * Algorithm 1 with the all-reduce removed) over all prompt positions at once, causal attention within the prompt.
 * d_tokens int32 [batch, seq_len]; every sequence has the same length.
 * Writes cache rows 0..seq_len-1 of sequences 0..batch-1, sets seq_lens[b] = seq_len, and
 * produces outputs for position seq_len-1 (next_tokens = the first generated token).
 * batch*seq_len <= max_prefill_tokens, seq_len <= max_seq_len, else LADDER_ERR_STATE. */
ladder_status_t ladder_prefill(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                               int32_t batch, int32_t seq_len, const ladder_outputs_t* out, void* cuda_stream);

/* Prompt pass over sequences of DIFFERENT lengths in one call.  d_tokens int32 [batch, seq_len] holds every
 * prompt left-aligned and padded to seq_len with any valid token id; h_lens is a HOST array [batch] of the true
 * lengths, 1 <= h_lens[b] <= seq_len (copied before the call returns).  Sequence b gets cache rows
 * 0..h_lens[b]-1 (nothing is written behind them), seq_lens[b] = h_lens[b], and its outputs are those of its own
 * last position h_lens[b]-1; with all_hidden the rows of padding positions are unspecified.  Padding costs its
 * share of the GEMM work (it is computed and discarded); causal attention keeps it from reaching any valid
 * position.  The host-side length the library tracks becomes the longest one (cf. ladder_set_position), so the
 * sequences can be decoded together right away.  The paper has no counterpart (it benchmarks equal lengths). */
ladder_status_t ladder_prefill_ragged(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                      const int32_t* h_lens, int32_t batch, int32_t seq_len, const ladder_outputs_t* out,
                                      void* cuda_stream);

/* Pipeline stages (paper Sec. 5.1: at a pipeline boundary the stream `residual` and the two module outputs that have
 * not been added yet are forwarded to the next stage).  A stage is a model object created over its own layers (the
 * whole model's weight arrays and rule tables, sliced; pass module_stale explicitly when the slice starts with a
 * ladder layer whose predecessor in the previous stage is not one) with its own KV cache.  The state that crosses the
 * boundary is the pair (x_m, x_{m-1}) of residual-stream values after the stage's last module -- in Algorithm 1's
 * variables residual + attn_out + mlp_out and residual + attn_out: the two sums are all the next layer reads -- as
 * fp32 [rows, d_model] buffers, rows = batch * seq_len in the prompt pass and batch in a decode step.
 *   state_in  NULL: first stage, starts from the token embedding (d_tokens required).  Otherwise d_tokens is unused
 *             (may be NULL), `newest` is required; without `older` a first module that asks for x_{m-1} reads x_m
 *             (as module 1 of a whole model reads x_0).
 *   state_out NULL: last stage, runs the final norm, the LM head and the argmax as ladder_prefill / ladder_decode_step
 *             do.  Otherwise the head is skipped, the state is written (`older` optional) and `out` must not ask for
 *             all_hidden; next_tokens / final_hidden / logits are not produced.
 * Every stage updates its own cache and seq_lens.  Stage calls run one kernel per GEMM (no persistent kernel); moving
 * the state between devices is the caller's business (one peer copy of 2 x rows x d_model floats per boundary). */
typedef struct {
  float* newest; /* x_m:     [rows, d_model] fp32 */
  float* older;  /* x_{m-1}: [rows, d_model] fp32, optional */
} ladder_stream_state_t;
ladder_status_t ladder_stage_prefill(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                     const ladder_stream_state_t* state_in, int32_t batch, int32_t seq_len,
                                     const ladder_stream_state_t* state_out, const ladder_outputs_t* out,
                                     void* cuda_stream);
ladder_status_t ladder_stage_decode_step(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                         const ladder_stream_state_t* state_in, int32_t batch,
                                         const ladder_stream_state_t* state_out, const ladder_outputs_t* out,
                                         void* cuda_stream);

/* Continues a prompt (chunked prompt pass): the seq_len new tokens of every sequence sit at positions
 * L .. L+seq_len-1, where L is the common cached length the library tracks (set by ladder_prefill, a previous
 * ladder_prefill_append, decode steps or ladder_set_position).  They attend to cache rows 0..L-1 and causally
 * to each other; rows L..L+seq_len-1 are written, seq_lens[b] = L+seq_len, outputs are for the last new position
 * (all_hidden: [batch, seq_len, d_model] of the new positions).  A prompt longer than max_prefill_tokens / batch
 * is fed as ladder_prefill of its first chunk followed by appends; the result equals the one-call prompt pass up
 * to summation order.  L+seq_len <= max_seq_len and batch*seq_len <= max_prefill_tokens, else LADDER_ERR_STATE.
 * Same model equations as the prompt pass (Eq. 1 / Eq. 2 of the paper; the paper does not discuss chunking). */
ladder_status_t ladder_prefill_append(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                      int32_t batch, int32_t seq_len, const ladder_outputs_t* out, void* cuda_stream);

/* One autoregressive step ("decode phase", paper Sec. 3.2; the workload of Sec. 3.3.1 is 512 of them after a
 * 1024-token prompt): the same module chain (Eq. 1 / Eq. 2, Algorithm 1) for one new position per sequence.
 * Consumes d_tokens int32 [batch] at position seq_lens[b] (read on
 * the device), appends K/V there, attends over positions 0..seq_lens[b], writes the outputs and
 * adds one to seq_lens[b].  d_tokens may alias out->next_tokens (device-side feedback loop).
 * The library tracks the common length on the host (set by prefill / ladder_set_position) and
 * returns LADDER_ERR_STATE instead of overflowing the cache.  After ladder_device_status has reported
 * LADDER_DEV_TIMEOUT the model refuses further steps with LADDER_ERR_TIMEOUT (the step that timed out produced
 * nothing and the cache position is unknown) until ladder_set_position or a new ladder_prefill re-arms it. */
ladder_status_t ladder_decode_step(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                   int32_t batch, const ladder_outputs_t* out, void* cuda_stream);

/* Same step with HOST token buffers: copies h_tokens [batch] to the device, runs the step,
 * copies the greedy tokens back to h_next_tokens [batch] and SYNCHRONISES the stream.
 * Pinned host memory makes the copies asynchronous up to that final sync. */
ladder_status_t ladder_decode_step_host(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* h_tokens,
                                        int32_t batch, int32_t* h_next_tokens, void* cuda_stream);
/* Prompt pass with HOST token buffers [batch, seq_len]; synchronises like the call above. */
ladder_status_t ladder_prefill_host(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* h_tokens,
                                    int32_t batch, int32_t seq_len, int32_t* h_next_tokens, void* cuda_stream);

/* Tell the library that every sequence of the cache now holds `len` tokens (e.g. after the
 * caller restored a cache snapshot or rewound seq_lens itself).  Host-side only.
 * Sequences of different lengths: positions are per sequence on the device, only this host-side overflow
 * check assumes one length.  Fill sequence b alone with a batch-1 prompt pass on a cache struct whose k and v
 * point n_kv_heads*max_seq_len*head_dim elements further per sequence skipped and whose seq_lens points at
 * entry b, then call this with the LONGEST length and decode all sequences together. */
ladder_status_t ladder_set_position(ladder_model_t* m, int32_t len);

/* Synchronises `cuda_stream`, returns the device status word (LADDER_DEV_* bits) and clears it.  Returns
 * LADDER_ERR_TIMEOUT (with *flags filled in) when the word holds LADDER_DEV_TIMEOUT. */
ladder_status_t ladder_device_status(ladder_model_t* m, int32_t* flags, void* cuda_stream);

/* Number of kernels this model has enqueued so far (graph replays count their kernel nodes). */
int64_t ladder_kernel_launches(const ladder_model_t* m);

ladder_status_t ladder_destroy(ladder_model_t* m); /* NULL is fine */
const char* ladder_status_string(ladder_status_t s);
const char* ladder_last_error(const ladder_model_t* m); /* library-owned string; NULL model = last create error */

/* ------------------------------------------------------------------------------------------
 * Single-kernel entry points: the same kernels the model calls, exposed so each can be tested
 * and profiled at its true shape.  They do not synchronise; ladder_op_smallm_gemm keeps a
 * library-owned split-K scratch that it grows (allocating, and then synchronising once) when a
 * larger shape is first seen, so its calls must not overlap on the device; the others allocate nothing.
 * ------------------------------------------------------------------------------------------ */

/* Weight-streaming small-M GEMM  acc[b,n] = sum_k act[b,k] * W[n,k]  (decode: M = batch <= 64),
 * with the activation staging and the epilogue of one step of the decode path.
 *   act      fp32 [batch, K]
 *   act_mode 0: used as is                                         (steps: output / down projection)
 *            1: the kernel applies RMSNorm with gain `gain` bf16 [K] and eps to it
 *               (steps: fused RMSNorm + QKV / gate-up projection, LM head)
 *   epi_mode 0: out_f32[b,n] = addend[b,n] + acc            (residual add; addend may equal out_f32)
 *            1: out_f32[b,j] = silu(acc[b,2j]) * acc[b,2j+1]       (SwiGLU over interleaved rows)
 *            2: out_f32[b,n] = acc                                   (plain, e.g. logits)
 * W bf16 [N,K] row-major; N % 8 == 0, K % 8 == 0, 1 <= batch <= 64. */
ladder_status_t ladder_op_smallm_gemm(const void* W, int32_t N, int32_t K, const void* act, int32_t act_mode,
                                      const void* gain, float eps, int32_t batch, int32_t epi_mode,
                                      const float* addend, void* out, void* cuda_stream);

/* Split-KV grouped-query decode attention for one layer.
 *   q fp32 [batch, Hq*Dh] (already rotated); k,v binary16 [max_batch][Hkv][max_seq_len][Dh] (one layer);
 *   kv_len int32 [batch] = number of keys to attend (positions 0..kv_len-1);
 *   scratch fp32, at least ladder_decode_attention_scratch_bytes(...) bytes;
 *   o fp32 [batch, Hq*Dh].  softmax(q.k/sqrt(Dh)) v per head, fp32 softmax and accumulation.
 * q, k, v, o and scratch must be 16-byte aligned (the kernel uses 16-byte loads), else LADDER_ERR_INVALID_ARG;
 * max_seq_len <= 65536, else LADDER_ERR_UNSUPPORTED.  The same two checks apply to the variant below. */
size_t ladder_decode_attention_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim, int32_t max_seq_len);
ladder_status_t ladder_op_decode_attention(const float* q, const void* k, const void* v, const int32_t* kv_len,
                                           int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                           int32_t max_seq_len, float* scratch, void* o, void* cuda_stream);

/* The same split-KV decode attention for callers that must not allocate device memory (a server
 * whose own pool owns the whole device, a memory-capped container slice, a host framework that
 * forbids cudaMalloc after start-up).  This entry point has no counterpart in the paper; it exists
 * for deployment.  Its scratch is a fixed 8 MiB array inside the library image, resident on every
 * GPU that loads the library until the process exits, so the call needs
 *     batch * n_q_heads * ceil(max_seq_len / 64) * (head_dim + 2) <= 2 * 1024 * 1024 floats
 * and returns LADDER_ERR_UNSUPPORTED otherwise (e.g. batch 4, 64 heads of 128, up to 2048 keys fits).
 * It calls no cudaMalloc / cudaFree and no allocating library routine.  The FIRST call on each
 * device looks up the array's device address (cudaGetSymbolAddress, with that device current):
 * make that first call outside any stream capture.  All calls share the one array, which keeps
 * the previous call's partials; nothing in it needs clearing (every split rewrites its partial
 * before the merge reads it), but two calls that overlap on the GPU -- different streams, or
 * different host threads -- race on it: serialise them.  Arguments and result as
 * ladder_op_decode_attention, minus the scratch. */
ladder_status_t ladder_op_decode_attention_noalloc(const float* q, const void* k, const void* v, const int32_t* kv_len,
                                                   int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                                   int32_t head_dim, int32_t max_seq_len, void* o, void* cuda_stream);

/* Large-M GEMM of the prefill path: C[m,n] = sum_k (A[m,k] + A_lo[m,k]) * W[n,k], A bf16 [M,K], W bf16 [N,K].
 *   A_lo: optional bf16 [M,K] low part of the activation (activation ~ A + A_lo); NULL = single bf16.
 *   epi_mode 0: out_f32[m,n] = addend[m,n] + acc;  1: SwiGLU -> out_bf16 [M, N/2];
 *            2: out_f32 = acc;  3: out_bf16[m,n] = acc.   K % 8 == 0, N % 8 == 0.
 *   out_lo: optional (modes 1 and 3) bf16 buffer of out's shape receiving value - bf16(value). */
ladder_status_t ladder_op_prefill_gemm(const void* A, const void* A_lo, const void* W, int32_t M, int32_t N, int32_t K,
                                       int32_t epi_mode, const float* addend, void* out, void* out_lo,
                                       void* cuda_stream);

/* The same GEMM with binary16 operands, the prompt pass's default for calls of at least 256 tokens: A binary16
 * [M,K] (ONE value per activation, 11 significant bits), W binary16 [N,K]; half the tensor-core work of the
 * bf16 hi + lo pair.  Epilogue modes as above, with the 16-bit outputs of modes 1 and 3 written as binary16
 * (saturating at +-65504).  A, W and out 16-byte aligned. */
ladder_status_t ladder_op_prefill_gemm_f16(const void* A, const void* W, int32_t M, int32_t N, int32_t K, int32_t epi_mode,
                                           const float* addend, void* out, void* cuda_stream);

/* bf16 -> binary16 conversion of n elements (n % 8 == 0, pointers 16-byte aligned): what the prompt pass does to
 * one layer's weights per call.  Exact for magnitudes >= 2^-14 (binary16 carries three more significant bits);
 * smaller magnitudes are rounded to binary16's subnormal grid, at most 2^-25 away. */
ladder_status_t ladder_op_convert_bf16_f16(const void* src, void* dst, int64_t n, void* cuda_stream);

/* Which implementation the prefill GEMMs use.  PROCESS-WIDE and not thread-safe: a switch for tests and A/B
 * measurements, not for serving code (leave it at 0).
 *   0 = default: tcgen05 kernel (TMA, TMEM accumulators) with binary16 operands -- each layer's bf16 weights are
 *       converted to binary16 in a per-model scratch once per call (1.7 GB at the 70B shape; model creation falls
 *       back to mode 3 when that does not fit) and every activation is ONE binary16 value -- for calls of at
 *       least 256 tokens, bf16 hi + lo pairs (mode 3) for shorter ones;
 *   2 = the tcgen05 kernel with ONE bf16 value per activation: the usual bf16 inference precision, but every stored
 *       activation is rounded at 2^-9, which by itself reaches 1.6e-2 of hidden-state error after 8 layers of the
 *       8B shape;
 *   3 = the tcgen05 kernel with bf16 hi + lo activation pairs (two MMAs per product) at every size;
 *   4 = as 0, but every GEMM with one CTA per output tile (0 runs single-value operands on pairs of CTAs,
 *       tcgen05.mma.cta_group::2 with 256 x 256 tiles, wherever there is at least one such tile per pair of SMs). */
void ladder_set_prefill_gemm_impl(int32_t impl);

/* Decode GEMM: 0 = batch 1..4 on the mma.sync weight-streaming kernel, batch 5..64 on the tcgen05 kernel (weights as
 * the M side of the MMA, TMA tiles, TMEM accumulators, equal K-block ranges per CTA with a deterministic fix-up of
 * shared tiles; default); 2 = the tcgen05 kernel for every batch.  PROCESS-WIDE and not thread-safe: a switch for
 * tests and A/B measurements, not for serving code. */
void ladder_set_decode_wide_impl(int32_t impl);

/* Decode attention for batch > 8 (head_dim 128, at most 8 query heads per kv head): 0 = the split step on TMA +
 * tcgen05 (key / value tiles of 128 cache rows streamed into shared memory, scores and P.V on the tensor core) where
 * batch x kv heads x ceil(max_seq_len / 128) >= 2048 tiles, the register-fragment kernel that serves batch <= 8
 * otherwise (default); 1 = the register-fragment kernel always; 2 = the TMA / tcgen05 kernel for every batch > 8.
 * PROCESS-WIDE and not thread-safe: a switch for tests and A/B measurements. */
void ladder_set_decode_attention_impl(int32_t impl);

/* Causal grouped-query attention of the prefill path for one layer:
 *   q binary16 [batch, seq_len, Hq*Dh] (rotated), q_lo its optional low part; k,v binary16 cache of one layer
 *   as above, rows 0..seq_len-1 valid; o bf16 [batch, seq_len, Hq*Dh] (the output projection's operand type),
 *   o_lo its low part (given iff q_lo is).  Query p attends keys t <= p. */
ladder_status_t ladder_op_prefill_attention(const void* q, const void* q_lo, const void* k, const void* v, int32_t batch,
                                            int32_t seq_len, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                            int32_t max_seq_len, void* o, void* o_lo, void* cuda_stream);

/* The same kernel with the arguments the chunked and ragged prompt passes use (ladder_prefill_append,
 * ladder_prefill_ragged; causal Llama attention of paper Sec. 3.3.1 over a cache that already holds pos0 rows):
 *   pos0            the seq_len queries sit at positions pos0 .. pos0+seq_len-1; cache rows 0 .. pos0+seq_len-1 are read
 *                   (pos0 >= 0, pos0 + seq_len <= max_seq_len, else LADDER_ERR_INVALID_ARG);
 *   lens            optional, DEVICE int32 [batch]: sequence b has lens[b] <= seq_len valid query rows; the rows
 *                   behind them are padding: neither read as keys / values nor written to o;
 *   out_binary16    non-zero: o receives ONE binary16 value per element (o_lo must be NULL; q_lo may be given).
 * All pointers are device pointers, 16-byte aligned (else LADDER_ERR_INVALID_ARG); nothing is allocated. */
ladder_status_t ladder_op_prefill_attention_at(const void* q, const void* q_lo, const void* k, const void* v,
                                               int32_t batch, int32_t seq_len, int32_t n_q_heads, int32_t n_kv_heads,
                                               int32_t head_dim, int32_t max_seq_len, int32_t pos0, const int32_t* lens,
                                               int32_t out_binary16, void* o, void* o_lo, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LADDER_H_ */
