// C ABI of libladder: model object, module scheduler (residual routing, two streams,
// CUDA graph of the decode step) and the single-kernel entry points.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <string>
#include <vector>

#include "../../include/ladder.h"
#include "kernels.h"

using namespace ladder;

namespace {

thread_local std::string g_create_error;

// sizeof(ladder_config_t) before layer_mode / module_stale were appended
constexpr size_t kConfigSizeV1 = offsetof(ladder_config_t, layer_mode);

// Copies the caller's configuration (of either size) and drops its host pointers: the rule tables are parsed
// into the model once.
void copy_config(ladder_config_t* dst, const ladder_config_t* src) {
  memset(dst, 0, sizeof(*dst));
  memcpy(dst, src, src->struct_size < sizeof(*dst) ? src->struct_size : sizeof(*dst));
  dst->struct_size = sizeof(*dst);
  dst->layer_is_ladder = nullptr;
  dst->layer_mode = nullptr;
  dst->module_stale = nullptr;
}

bool g_kernels_ready = false;
cudaError_t kernels_ready() {  // opt-in to large dynamic shared memory, once per process
  if (g_kernels_ready) return cudaSuccess;
  cudaError_t e = smallm_gemm_init();
  if (e == cudaSuccess) e = largem_gemm_tc_init();
  if (e == cudaSuccess) e = prefill_attention_tc_init();
  if (e == cudaSuccess) e = decode_attention_tc_init();
  if (e == cudaSuccess) g_kernels_ready = true;
  return e;
}

struct GraphKey {
  int batch = 0, n_streams = 0, pdl = 0;
  const void *k = nullptr, *v = nullptr, *lens = nullptr, *tok = nullptr;
  const void *o_next = nullptr, *o_hid = nullptr, *o_logits = nullptr;
  const void *s_in0 = nullptr, *s_in1 = nullptr, *s_out0 = nullptr, *s_out1 = nullptr;  // pipeline-stage state buffers
  bool operator==(const GraphKey& o) const {
    return batch == o.batch && n_streams == o.n_streams && pdl == o.pdl && k == o.k && v == o.v && lens == o.lens &&
           tok == o.tok && o_next == o.o_next && o_hid == o.o_hid && o_logits == o.o_logits && s_in0 == o.s_in0 &&
           s_in1 == o.s_in1 && s_out0 == o.s_out0 && s_out1 == o.s_out1;
  }
};

}  // namespace

struct ladder_model {
  ladder_config_t cfg;
  std::vector<uint8_t> is_ladder;  // per layer: a ladder layer (both modules read one module back)
  std::vector<uint8_t> mode;       // per layer: LADDER_LAYER_*
  std::vector<uint8_t> stale;      // per module (index m-1): module m reads x_{m-2} instead of x_{m-1}
  const __nv_bfloat16 *tok_embedding, *final_norm, *lm_head;
  std::vector<const __nv_bfloat16*> attn_norm, w_qkv, w_o, mlp_norm, w_gate_up, w_down;
  int sm_count = 0;
  int max_rows = 0;  // rows of the residual buffers
  // workspace (device)
  float* R[2] = {nullptr, nullptr};
  float* q_f32 = nullptr;           // decode [max_batch, Hq*Dh]
  float* o_dec = nullptr;           // decode [max_batch, Hq*Dh]
  float* h_dec = nullptr;           // decode [max_batch, F]
  // batch 9..64: the SwiGLU output / the attention output as the next GEMM's staged operand (bf16 [2 x 64, F] / [2 x 64, Hq*Dh])
  __nv_bfloat16* wide_hpack = nullptr;
  __nv_bfloat16* wide_opack = nullptr;
  float* pend_a = nullptr;  // batch 5..64, pending-output schedule: the attention module's output, stored not added
  float* pend_m = nullptr;  // ... and the MLP module's
  std::vector<cudaEvent_t> ev_sq, ev_sg;  // [layer]: the staging step of layer l's QKV / gate-up input has run ([L]: the head's)
  std::vector<cudaEvent_t> ev_out;        // [module]: the module's stored output is complete (and summed over the ranks)
  // tensor parallelism (Sec. 2, Eq. 1): sums a module's partial output over the ranks, in place, on the given stream
  ladder_exchange_fn exchange = nullptr;
  void* exchange_ctx = nullptr;
  int exchange_capturable = 0;  // the callback may be called while its stream is being captured into a CUDA graph
  ladder_comm* comm = nullptr;  // set by ladder_model_set_tensor_parallel (not owned)
  ladder_peer* peer = nullptr;  // decode-step exchanges over peer memory instead of `exchange` (not owned)
  int64_t peer_max_bytes = 8ll << 20;  // largest outbound volume per exchange the fused exchange is used for
  ladder_peer_hook_fn peer_hook = nullptr;  // test hook: called after each output GEMM of a decode step is enqueued
  void* peer_hook_ctx = nullptr;
  float* pend_pf[2] = {nullptr, nullptr};  // prompt pass under tensor parallelism: the two modules' stored outputs
  cudaStream_t xstream = nullptr;          // ... exchanged and added to the stream on this one
  std::vector<cudaEvent_t> ev_pf_out, ev_pf_add;  // [module]: stored / added
  // the same activations as bf16 hi/lo MMA operands ([chunk][8][2048]), written by the persistent kernel's
  // epilogues for the phase that reads them next (batch <= 4): twins of R[0], R[1], h_dec, o_dec
  __nv_bfloat16 *xpack[2] = {nullptr, nullptr}, *hpack = nullptr, *opack = nullptr;
  float* attn_scratch = nullptr;
  int attn_splits = 1;
  float* gemm_scratch[2] = {nullptr, nullptr};  // split-K partials + tickets, one per stream role
  int32_t* work_slots = nullptr;    // 2 ints per GEMM launch of a step (claim counters)
  int n_work_slots = 0;
  float* logits_ws = nullptr;       // [max_batch, V]
  float* last_x = nullptr;          // [max_batch, d]
  // prefill activations, each a bf16 hi part followed by a lo part (value ~ hi + lo)
  __nv_bfloat16 *n_pf = nullptr, *o_pf = nullptr, *h_pf = nullptr;
  __half* q_pf = nullptr;  // the rotated query as the attention's binary16 operand pair
  __half* w16 = nullptr;   // one layer's four weight matrices as binary16 (prompt pass; NULL: not enough memory)
  __half* w16b = nullptr;  // a second such buffer: the next layer is converted on the side stream meanwhile (optional)
  cudaEvent_t ev_w16_ready[2] = {nullptr, nullptr}, ev_w16_free[2] = {nullptr, nullptr}, ev_pf_fork = nullptr;
  size_t n_lo = 0, q_lo = 0, h_lo = 0;  // element offsets of the lo parts
  float2* rope = nullptr;
  int32_t* status = nullptr;
  int32_t *tok_tmp = nullptr, *next_tmp = nullptr, *lens_tmp = nullptr;
  int32_t* h_lens_pinned = nullptr;  // host (pinned), max_batch entries: staging of per-sequence prompt lengths
  // scheduling
  cudaStream_t side = nullptr, cap = nullptr;
  std::vector<cudaEvent_t> ev;  // ev[m] = end of module m (m = 0: embedding)
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_lens = nullptr;
  int n_streams = 2, use_graph = 1, use_pdl = 1;
  int sms_a = -1;  // SMs given to the attention stream in ladder layers (0 = automatic, -1 = no split)
  cudaGraphExec_t graph_exec = nullptr;
  GraphKey graph_key;
  int64_t graph_kernels = 0;
  // persistent layer-stack kernel (one cooperative launch per decode step, batch <= 8)
  bool stack_ok = false;   // usable on this device and worthwhile for this model
  int stack_begin = 0;     // first layer run by the persistent kernel (layers below: one kernel per GEMM)
  bool stack_usable = false;  // the kernel fits this device and this depth
  int stack_stall_test = 0;  // test hook: the last phase waits for a count its producer never reaches
  int use_stack = 1;
  bool persistent_explicit = false;  // ladder_model_set_persistent was called with on != 0: no second-guessing
  GraphKey stack_key;      // what the uploaded phase list was built for
  bool stack_built = false;
  StackPhase* d_phases = nullptr;
  StackAttn* d_attn = nullptr;
  int32_t* d_counters = nullptr;
  int n_phases = 0, n_attn = 0, n_counters = 0, cap_counters = 0;
  // state
  // pipeline stage (paper Sec. 5.1), set for the duration of a ladder_stage_* call: the stream state this stage
  // starts from instead of the embedding, and where it leaves the state instead of running the head
  ladder_stream_state_t st_in = {nullptr, nullptr}, st_out = {nullptr, nullptr};
  int host_len = 0;
  bool timed_out = false;  // ladder_device_status saw LADDER_DEV_TIMEOUT: steps are refused until re-armed
  int64_t launches = 0;
  std::string err;
  bool sticky_cuda = false;
};

namespace {

ladder_status_t fail(ladder_model* m, ladder_status_t s, const std::string& msg) {
  if (m) m->err = msg;
  else g_create_error = msg;
  return s;
}

#define CK(m, call)                                                                                   \
  do {                                                                                                \
    cudaError_t e_ = (call);                                                                          \
    if (e_ != cudaSuccess) {                                                                          \
      if (m) (m)->sticky_cuda = true;                                                                 \
      return fail(m, LADDER_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_));            \
    }                                                                                                 \
  } while (0)

template <typename T>
cudaError_t dev_alloc(T** p, size_t count) {
  return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T) + 256);
}

const char* check_shape(const ladder_config_t& c) {
  if (c.d_model <= 0 || c.n_layers <= 0 || c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.d_ff <= 0 || c.vocab_size <= 0)
    return "non-positive dimension";
  if (c.head_dim != 64 && c.head_dim != 128) return "head_dim must be 64 or 128";
  if (c.n_q_heads % c.n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
  if (c.d_model % 8 || c.d_ff % 8 || c.vocab_size % 8) return "d_model, d_ff and vocab_size must be multiples of 8";
  if (c.max_batch < 1 || c.max_batch > 64) return "max_batch must be in [1, 64]";
  if (c.max_seq_len < 1) return "max_seq_len must be positive";
  if (c.max_seq_len > kDecodeAttnMaxKeys) return "max_seq_len above 65536 (decode attention merges at most 1024 splits of 64 keys)";
  if (!(c.rms_eps >= 0.f) || !(c.rope_theta > 0.f)) return "bad rms_eps / rope_theta";
  return nullptr;
}

// Residual routing (Eq. 1 / Eq. 2 of the paper on two ping-pong buffers).  Module m reads x_{m-2} (reads_older)
// or x_{m-1}, adds onto x_{m-1} and writes x_m: over the buffer of x_{m-2}, which is dead from then on, or -- when
// it read x_{m-1} and the next module does not need that value any more -- in place.
struct Router {
  int cur = 0, stale = -1;  // buffer holding x_{m-1}; buffer holding x_{m-2} (or -1)
  int writer[2] = {0, -1};  // module that last wrote each buffer
  struct Route {
    int in, add, dst, in_writer;
  };
  Route next(bool reads_older, bool next_reads_older, int module) {
    Route r;
    if (reads_older && stale >= 0) {
      r = {stale, cur, stale, writer[stale]};
      const int old_cur = cur;
      cur = stale;
      stale = old_cur;
    } else if (next_reads_older) {  // reads x_{m-1}, which module m+1 will read too: keep it
      r = {cur, cur, cur ^ 1, writer[cur]};
      stale = cur;
      cur ^= 1;
    } else {
      r = {cur, cur, cur, writer[cur]};
      stale = -1;
    }
    writer[r.dst] = module;
    return r;
  }
};

// Route of module `module` (1-based) of this model.
Router::Route route(const ladder_model* m, Router& rt, int module) {
  const int n = static_cast<int>(m->stale.size());
  // the last module of a stage that hands its state on keeps x_{m-1}: the next stage's first module may read it
  const bool next_reads_older = module < n ? m->stale[module] != 0 : m->st_out.newest != nullptr;
  return rt.next(m->stale[module - 1] != 0, next_reads_older, module);
}

// Start of a forward pass over `rows` tokens: the embedding gather, or -- in a pipeline stage that receives the
// stream state -- copies of (x_{m-1}, x_{m-2}) into the two residual buffers.
cudaError_t begin_stream(ladder_model* m, Router& rt, const int32_t* d_tokens, int rows, cudaStream_t st) {
  const ladder_config_t& c = m->cfg;
  if (!m->st_in.newest)
    return launch_embed(d_tokens, m->tok_embedding, rows, c.d_model, c.vocab_size, m->R[0], m->status, st, false);
  const size_t bytes = static_cast<size_t>(rows) * c.d_model * sizeof(float);
  cudaError_t e = cudaMemcpyAsync(m->R[0], m->st_in.newest, bytes, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess && m->st_in.older) {
    e = cudaMemcpyAsync(m->R[1], m->st_in.older, bytes, cudaMemcpyDeviceToDevice, st);
    rt.stale = 1;
    rt.writer[1] = 0;
  }
  return e;
}

// End of a stage that hands its state on: (x_m, x_{m-1}) out of the residual buffers (x_{m-1} := x_m when the last
// module worked in place and nothing older exists), and the cache lengths.
cudaError_t end_stage(ladder_model* m, const Router& rt, const ladder_kv_cache_t* cache, int batch, int rows, int advance,
                      int set_len, const int32_t* set_lens, cudaStream_t st) {
  const size_t bytes = static_cast<size_t>(rows) * m->cfg.d_model * sizeof(float);
  cudaError_t e = cudaMemcpyAsync(m->st_out.newest, m->R[rt.cur], bytes, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess && m->st_out.older)
    e = cudaMemcpyAsync(m->st_out.older, m->R[rt.stale >= 0 ? rt.stale : rt.cur], bytes, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess)
    e = launch_argmax_advance(nullptr, batch, m->cfg.vocab_size, nullptr, cache->seq_lens, advance, set_len, st, false,
                              set_lens);
  return e;
}

// Gain of the RMSNorm in front of the MLP of layer l: a parallel layer normalises once, with the attention gain.
const __nv_bfloat16* mlp_gain(const ladder_model* m, int l) {
  return m->mode[l] == LADDER_LAYER_PARALLEL ? m->attn_norm[l] : m->mlp_norm[l];
}

// Fills the per-layer / per-module rule tables from the configuration.  Fields past cfg->struct_size are absent
// (a caller compiled against the earlier, shorter struct).
const char* parse_rules(const ladder_config_t* cfg, ladder_model* m) {
  const int L = cfg->n_layers;
  const bool has_ext = cfg->struct_size >= sizeof(ladder_config_t);
  m->mode.assign(L, LADDER_LAYER_LADDER);
  if (cfg->layer_is_ladder)
    for (int l = 0; l < L; ++l) m->mode[l] = cfg->layer_is_ladder[l] ? LADDER_LAYER_LADDER : LADDER_LAYER_STANDARD;
  if (has_ext && cfg->layer_mode)
    for (int l = 0; l < L; ++l) {
      if (cfg->layer_mode[l] > LADDER_LAYER_UPPER_BOUND) return "layer_mode entry outside 0..3";
      // without communication the upper bound is the standard model
      m->mode[l] = cfg->layer_mode[l] == LADDER_LAYER_UPPER_BOUND ? LADDER_LAYER_STANDARD : cfg->layer_mode[l];
    }
  m->is_ladder.assign(L, 0);
  m->stale.assign(2 * L, 0);
  for (int l = 0; l < L; ++l) {
    const bool after_ladder = l > 0 && m->mode[l - 1] == LADDER_LAYER_LADDER;
    if (m->mode[l] == LADDER_LAYER_LADDER) {
      m->is_ladder[l] = 1;
      m->stale[2 * l] = (after_ladder || l == 0) ? 1 : 0;  // after a non-ladder layer: the complete stream
      m->stale[2 * l + 1] = 1;
    } else if (m->mode[l] == LADDER_LAYER_PARALLEL) {
      m->stale[2 * l + 1] = 1;  // the MLP reads the attention module's input
    }
  }
  if (has_ext && cfg->module_stale)
    for (int i = 0; i < 2 * L; ++i) m->stale[i] = cfg->module_stale[i] ? 1 : 0;
  return nullptr;
}

struct Enqueue {
  ladder_model* m;
  cudaStream_t sA, sB;
  bool two;
  bool pdl_ok[2] = {false, false};  // previous op on the stream was a kernel (programmatic edge possible)
  int64_t kernels = 0;
  int slot = 0;  // next claim-counter slot
  int grid_a = 0, grid_b = 0;  // CTAs per GEMM on stream A / B while the two run side by side (0 = all SMs)
  bool force_wide = false;     // the tcgen05 GEMM at batch <= 4 too
  void gemm(int s, SmallMParams& p, bool side_by_side = false) {
    p.scratch = m->gemm_scratch[two ? s : 0];
    p.force_wide = force_wide;
    p.work = m->work_slots + 2 * (slot++ % m->n_work_slots);
    p.status = m->status;
    const int g = (side_by_side && two && grid_a > 0) ? (s ? grid_b : grid_a) : m->sm_count;
    launched(s, launch_smallm_gemm(p, stream(s), pdl(s), g));
  }
  cudaError_t err = cudaSuccess;

  cudaStream_t stream(int s) const { return s ? sB : sA; }
  bool pdl(int s) const { return m->use_pdl && pdl_ok[two ? s : 0]; }
  void launched(int s, cudaError_t e) {
    if (err == cudaSuccess) err = e;
    pdl_ok[two ? s : 0] = true;
    ++kernels;
  }
  void wait(int s, cudaEvent_t ev_from_other) {
    if (!two) return;
    cudaError_t e = cudaStreamWaitEvent(stream(s), ev_from_other, 0);
    if (err == cudaSuccess) err = e;
    pdl_ok[s] = false;
  }
  void record(int s, cudaEvent_t e) {
    if (!two) return;
    cudaError_t r = cudaEventRecord(e, stream(s));
    if (err == cudaSuccess) err = r;
  }
};

// Batch <= 4, every module reading x_{m-2}, small layers AND an attention module much narrower than the hidden size
// (one tensor-parallel rank's slice: 8 of 64 heads at the 70B shape): the persistent kernel loses to the
// pending-output form on the tcgen05 GEMMs with the two chains side by side on 36 / 112 SMs - measured at the
// TP-rank slice, KV 2048: batch 1 / 2 / 4 4.05 / 4.03 / 4.15 ms per step in the persistent kernel, 3.82 / 3.85 / 3.91 ms
// this way (inside the persistent kernel the output projection waits for the attention of its own layer, which at
// this shape takes longer than the gate/up phase beside it).  Where the attention is as wide as the model (1.2B
// shape) the persistent kernel stays ahead (0.80 against 0.85 ms).
bool prefers_wide_small(const ladder_model* m) {
  const ladder_config_t& c = m->cfg;
  if (m->persistent_explicit || m->n_streams != 2 || m->sms_a != -1 || !m->pend_a || !m->pend_m) return false;
  for (uint8_t f : m->stale)
    if (!f) return false;
  const double layer_bytes = 2.0 * (static_cast<double>((c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim) * c.d_model +
                                    static_cast<double>(c.d_model) * c.n_q_heads * c.head_dim + 3.0 * c.d_ff * c.d_model);
  return layer_bytes < 300e6 && 4 * c.n_q_heads * c.head_dim <= c.d_model;
}

// Whether a decode step of this batch exchanges over peer memory (fused into the GEMMs) rather than through
// `exchange`.  The fused exchange is one-shot: every rank stores its whole partial sum, 8 bytes per element, into every
// other rank's memory, (world - 1) x batch x d_model x 8 bytes per rank and exchange.  That is the fastest way for the
// small messages of a decode step and a waste of link bandwidth for large ones, where a reduce-scatter / all-gather
// moves a quarter of it at world 8: above peer_max_bytes (8 MiB unless set otherwise) the step leaves it to `exchange` (NCCL).
bool peer_fused(const ladder_model* m, int batch) {
  if (!m->peer) return false;
  const int64_t out = static_cast<int64_t>(ladder_peer_world(m->peer) - 1) * batch * m->cfg.d_model * 8;
  return out <= m->peer_max_bytes;
}

// The decode step in the pending-output form of Algorithm 1.  The output and down projections STORE their module's
// output (pend_a / pend_m) instead of adding it to the stream, and the stream moves on in the staging step of a
// later reader: the step that forms module j's input x_{j-1} (Eq. 1) or x_{j-2} (Eq. 2) adds the stored outputs
// that are still missing from the newest stream value, in module order (none, one or two of them), and writes the
// sum to the other residual buffer.  The sums are the same fp32 additions in the same order as with the adds in the
// GEMM epilogues: bit-identical results.
// What it buys: (1) with the adds in the epilogues every output projection of a ladder layer has to wait for the
// previous down projection and vice versa, so the two streams move in lock-step; here the only cross-stream
// edges are between the (tiny) staging launches, and the attention-module chain (stage, QKV, attention, Wo) and the
// MLP chain (stage, gate/up, down) run side by side on their shares of the SMs.  (2) Under tensor parallelism
// (Sec. 2, Eq. 1) the stored output is this rank's partial sum: the exchange callback sums it over the ranks on
// the producing stream, and a ladder layer's other module computes meanwhile - the overlap Algorithm 1 is about;
// with standard residuals the next module's staging step waits for it, as in the paper's baseline.
// Not for parallel attention + MLP layers (one sum per layer) and not for pipeline stages.
cudaError_t enqueue_decode_pending(ladder_model* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens, int batch,
                                   const ladder_outputs_t* out, cudaStream_t sA, cudaStream_t sB, int64_t* n_kernels,
                                   int grid_a, int grid_b) {
  const ladder_config_t& c = m->cfg;
  Enqueue q{m, sA, sB, sA != sB};
  q.grid_a = grid_a;
  q.grid_b = grid_b;
  q.force_wide = batch <= 4;
  const int Hq = c.n_q_heads, Hkv = c.n_kv_heads, Dh = c.head_dim, d = c.d_model, F = c.d_ff, L = c.n_layers;
  const size_t layer_elems = static_cast<size_t>(c.max_batch) * Hkv * c.max_seq_len * Dh;
  PeerView view = {};
  const bool use_peer = peer_fused(m, batch) && peer_view(m->peer, &view);
  Router rt;
  q.launched(0, begin_stream(m, rt, d_tokens, batch, sA));
  int cur = rt.cur;  // R[cur]: the newest stream value formed so far = x_0 + outputs of modules 0 .. added
  int added = -1;
  // A pipeline stage that was handed (x_{-1}, x_{-2}): they are in R[cur] and the other buffer; only this stage's
  // first module can read the older one, before any staging step overwrites it.
  const int older_buf = (m->st_in.newest && m->st_in.older) ? (cur ^ 1) : -1;
  auto pend = [&](int j) { return (j & 1) ? m->pend_m : m->pend_a; };
  // Under an exchange, a layer whose MLP does not read its attention module's output and whose attention output
  // nobody reads on its own (parallel attention + MLP, Sec. 3.3.1) sums the two outputs BEFORE the exchange: the
  // down projection adds the stored attention output in its epilogue, and there is one exchange per layer.
  auto merged = [&](int j) {  // module j's output travels inside module j + 1's
    if (!m->exchange || (j & 1) || j + 1 >= 2 * L || m->stale[j] || !m->stale[j + 1]) return false;  // a parallel-shaped layer
    if (j + 2 < 2 * L) return m->stale[j + 2] == 0;
    return m->st_out.newest == nullptr || m->st_out.older == nullptr;  // the head reads everything; a handed-on x_{2L-1} would not
  };
  auto ev_stage = [&](int j) { return (j & 1) ? m->ev_sg[j >> 1] : m->ev_sq[j >> 1]; };
  // Staging step of module `mod` (2L = the head) on stream s: its input is x_0 + outputs of modules 0 .. upto.
  auto form_input = [&](int mod, int s, int upto, SmallMParams& p) {
    if (upto < added) upto = added;  // module 0 has no x_{-1}: it reads x_0 whatever its flag
    if (mod > 0 && ((mod - 1) & 1) != s) q.wait(s, ev_stage(mod - 1));  // the stream value the previous step formed
    int list[2] = {-1, -1}, n = 0;  // the stored outputs still to add, in module order: none, one or two
    for (int j = added + 1; j <= upto; ++j) {
      if (merged(j)) continue;  // inside the next module's
      if ((j & 1) != s) q.wait(s, m->ev_out[j]);  // a stored output of the other stream (same stream: in order)
      list[n++] = j;
    }
    p.act = (mod == 0 && m->stale[0] && older_buf >= 0) ? m->R[older_buf] : m->R[cur];
    WidePeer pull = {};
    if (use_peer) {  // the stored outputs are the ranks' partial sums in this rank's receive slots
      pull.peer = view;
      pull.pull_channel[0] = n >= 1 ? (list[0] & 1) + 1 : 0;
      pull.pull_channel[1] = n >= 2 ? (list[1] & 1) + 1 : 0;
      p.wide_peer = &pull;
    } else {
      p.act_pending = n >= 1 ? pend(list[0]) : nullptr;
      p.act_pending2 = n >= 2 ? pend(list[1]) : nullptr;
    }
    p.act_sum_out = n >= 1 ? m->R[cur ^ 1] : nullptr;
    p.scratch = m->gemm_scratch[q.two ? s : 0];
    p.status = m->status;
    p.force_wide = q.force_wide;
    q.launched(s, launch_smallm_gemm_stage(p, q.stream(s), q.pdl(s)));
    if (n >= 1) cur ^= 1;
    added = upto;
    q.record(s, ev_stage(mod));
    p.wide_prestaged = 1;
    p.wide_peer = nullptr;
  };
  // The module's output is complete in pend(mod): sum it over the tensor-parallel ranks, tell the other stream.
  auto output_stored = [&](int mod, int s) {
    if (merged(mod)) {  // stays local: the down projection of this layer adds it before the exchange
      q.record(s, m->ev_out[mod]);
      return;
    }
    if (use_peer) {  // the GEMM itself has pushed the partial sum to every rank
      if (m->peer_hook) {
        m->peer_hook(m->peer_hook_ctx, mod & 1, q.stream(s));
        q.pdl_ok[q.two ? s : 0] = false;
      }
    } else if (m->exchange) {
      const int64_t n = static_cast<int64_t>(batch) * d;
      const ladder_status_t r = m->exchange(m->exchange_ctx, pend(mod), n, q.stream(s));
      if (r != LADDER_OK && q.err == cudaSuccess) q.err = cudaErrorUnknown;
      q.pdl_ok[q.two ? s : 0] = false;
    }
    q.record(s, m->ev_out[mod]);
  };
  for (int l = 0; l < L; ++l) {
    const bool side = m->stale[2 * l + 1] != 0;  // the two modules of this layer can run side by side
    {  // ---------------- attention module (stream A)
      const int mod = 2 * l, s = 0;
      SmallMParams p = {};
      p.W = m->w_qkv[l];
      p.N = (Hq + 2 * Hkv) * Dh;
      p.K = d;
      p.act_mode = ACT_F32_NORM;
      p.gain = m->attn_norm[l];
      p.eps = c.rms_eps;
      p.batch = batch;
      form_input(mod, s, mod - 1 - (m->stale[mod] ? 1 : 0), p);
      p.epi_mode = EPI_QKV_ROPE;
      p.qkv.q_out_f32 = m->q_f32;
      p.qkv.k_cache = static_cast<kv_t*>(cache->k) + l * layer_elems;
      p.qkv.v_cache = static_cast<kv_t*>(cache->v) + l * layer_elems;
      p.qkv.seq_lens = cache->seq_lens;
      p.qkv.rope = m->rope;
      p.qkv.n_q_heads = Hq;
      p.qkv.n_kv_heads = Hkv;
      p.qkv.head_dim = Dh;
      p.qkv.max_seq_len = c.max_seq_len;
      q.gemm(s, p, side);

      DecodeAttnParams a = {};
      a.q = m->q_f32;
      a.k = p.qkv.k_cache;
      a.v = p.qkv.v_cache;
      a.kv_len = cache->seq_lens;
      a.kv_len_offset = 1;
      a.batch = batch;
      a.n_q_heads = Hq;
      a.n_kv_heads = Hkv;
      a.head_dim = Dh;
      a.max_seq_len = c.max_seq_len;
      a.n_splits = m->attn_splits;
      a.max_len = c.max_seq_len;
      a.scratch = m->attn_scratch;
      a.o = m->o_dec;
      a.status = m->status;
      a.o_pack = m->wide_opack;
      a.o_pack_bp = wide_padded_batch(batch);
      q.launched(s, launch_decode_attention(a, q.stream(s), q.pdl(s)));
      ++q.kernels;  // the split kernel and its merge kernel

      SmallMParams o = {};
      o.W = m->w_o[l];
      o.N = d;
      o.K = Hq * Dh;
      o.act = m->o_dec;
      o.act_mode = ACT_F32;
      o.batch = batch;
      o.epi_mode = EPI_PLAIN;
      o.out = pend(mod);
      o.act_staged = m->wide_opack;
      WidePeer push = {};
      if (use_peer && !merged(mod)) {
        push.peer = view;
        push.push_channel = (mod & 1) + 1;
        o.wide_peer = &push;
      }
      q.gemm(s, o, side);
      output_stored(mod, s);
    }
    {  // ---------------- MLP module (stream B)
      const int mod = 2 * l + 1, s = q.two ? 1 : 0;
      SmallMParams g = {};
      g.W = m->w_gate_up[l];
      g.N = 2 * F;
      g.K = d;
      g.act_mode = ACT_F32_NORM;
      g.gain = mlp_gain(m, l);
      g.eps = c.rms_eps;
      g.batch = batch;
      form_input(mod, s, mod - 1 - (m->stale[mod] ? 1 : 0), g);
      g.epi_mode = EPI_SWIGLU;
      g.out = m->h_dec;
      g.wide_pack_out = m->wide_hpack;
      q.gemm(s, g, side);

      SmallMParams dn = {};
      dn.W = m->w_down[l];
      dn.N = d;
      dn.K = F;
      dn.act = m->h_dec;
      dn.act_mode = ACT_F32;
      dn.batch = batch;
      dn.epi_mode = EPI_PLAIN;
      dn.out = pend(mod);
      dn.act_staged = m->wide_hpack;
      if (merged(mod - 1)) {  // attention + MLP output of this layer as one sum
        q.wait(s, m->ev_out[mod - 1]);
        dn.epi_mode = EPI_RESID;
        dn.addend = pend(mod - 1);
      }
      WidePeer push = {};
      if (use_peer) {
        push.peer = view;
        push.push_channel = (mod & 1) + 1;
        dn.wide_peer = &push;
      }
      q.gemm(s, dn, side);
      output_stored(mod, s);
    }
  }
  if (m->st_out.newest) {  // a stage that hands its state on: x_{2L-1} (all outputs but the last) and x_{2L}, no head
    const size_t bytes = static_cast<size_t>(batch) * d * sizeof(float);
    auto note = [&](cudaError_t e) {
      if (q.err == cudaSuccess) q.err = e;
    };
    for (int i = 0; i < 2; ++i) {
      if (i == 0 && !m->st_out.older) continue;
      SmallMParams t = {};
      t.K = d;
      t.act_mode = ACT_F32;
      t.batch = batch;
      form_input(2 * L + i, 0, 2 * L - 2 + i, t);  // a staging launch for its sum only
      note(cudaMemcpyAsync(i == 0 ? m->st_out.older : m->st_out.newest, m->R[cur], bytes, cudaMemcpyDeviceToDevice, sA));
      q.pdl_ok[0] = false;
    }
    q.launched(0, launch_argmax_advance(nullptr, batch, c.vocab_size, nullptr, cache->seq_lens, 1, -1, sA, false, nullptr));
    *n_kernels = q.kernels;
    return q.err;
  }
  // ---------------- head on stream A: reads x_{2L} (every output added)
  float* logits = (out && out->logits) ? out->logits : m->logits_ws;
  SmallMParams h = {};
  h.W = m->lm_head;
  h.N = c.vocab_size;
  h.K = d;
  h.act_mode = ACT_F32_NORM;
  h.gain = m->final_norm;
  h.eps = c.rms_eps;
  h.batch = batch;
  form_input(2 * L, 0, 2 * L - 1, h);
  h.epi_mode = EPI_PLAIN;
  h.out = logits;
  q.gemm(0, h);
  if (out && out->final_hidden)
    q.launched(0, launch_rmsnorm_f32(m->R[cur], m->final_norm, c.rms_eps, batch, d, d, out->final_hidden, sA, q.pdl(0)));
  q.launched(0, launch_argmax_advance(logits, batch, c.vocab_size, out ? out->next_tokens : nullptr, cache->seq_lens, 1,
                                      -1, sA, q.pdl(0)));
  *n_kernels = q.kernels;
  return q.err;
}

// One decode step: enqueue every kernel on sA (attention modules, head) and sB (MLP modules).
// l_end < n_layers: only the embedding and layers [0, l_end) (the rest of the step is run by the persistent kernel).
cudaError_t enqueue_decode(ladder_model* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens, int batch,
                           const ladder_outputs_t* out, cudaStream_t sA, cudaStream_t sB, int64_t* n_kernels,
                           int l_end = -1) {
  const ladder_config_t& c = m->cfg;
  Enqueue q{m, sA, sB, sA != sB};
  const int Hq = c.n_q_heads, Hkv = c.n_kv_heads, Dh = c.head_dim, d = c.d_model, F = c.d_ff;
  const size_t layer_elems = static_cast<size_t>(c.max_batch) * Hkv * c.max_seq_len * Dh;
  // Optional: in ladder layers the attention module and the MLP module run side by side, and the SMs
  // can be divided between the two streams (in proportion to the bytes each has to stream, plus a
  // margin for the attention stream) so that ramp, tail and launch gaps of one stream overlap with the
  // other's steady weight stream.  Measured on the 70B shape this loses to letting every GEMM take all
  // SMs (25.1 ms at the best split of 40 SMs vs 24.4 ms): a subset of SMs streams at ~47 GB/s each and
  // the module chain (Wo waits for the previous down projection and vice versa) leaves it idle in
  // between.  Off by default.
  // Batch 5..64 (one tcgen05 kernel per GEMM) with small layers is the exception: there a launch costs more than it
  // streams (7 us of set-up and 4-11 us of shared-tile fix-up against 3-17 us of weights at the TP-rank slice), and
  // two launches side by side overlap those costs: 60 of 148 SMs for the attention stream measured 581 -> 553 us per
  // 8 layers at batch 16 and 921 -> 865 us at batch 64 (at the 70B shape the split loses at every batch).
  const double layer_bytes = 2.0 * (static_cast<double>((Hq + 2 * Hkv) * Dh) * d + static_cast<double>(d) * Hq * Dh + 3.0 * F * d);
  const bool auto_wide = (m->sms_a == -1 || m->sms_a == -3) && batch > 4 && layer_bytes < 300e6;
  const bool auto_small = batch <= 4 && !m->st_in.newest && !m->st_out.newest && (l_end < 0 || l_end == c.n_layers) &&
                          prefers_wide_small(m);
  if (q.two && (m->sms_a >= 0 || auto_wide || auto_small)) {
    // of 148 SMs for the attention stream (swept 20 .. 72 in the pending-output form): 36 for batch <= 4, 56 for batch
    // 5..32, 44 above
    const int share = auto_small ? 36 : (batch <= 32 ? 56 : 44);
    int ga = (auto_small || auto_wide) ? (share * m->sm_count + 74) / 148 : m->sms_a;
    if (ga == 0) {
      const double ba = static_cast<double>((Hq + 2 * Hkv) * Dh) * d + static_cast<double>(d) * Hq * Dh;
      const double bb = 3.0 * F * d;
      ga = static_cast<int>(m->sm_count * ba / (ba + bb) * 1.2 + 0.5);
    }
    if (ga < 4) ga = 4;
    if (ga > m->sm_count / 2) ga = m->sm_count / 2;
    q.grid_a = ga;
    q.grid_b = m->sm_count - ga;
    // every module reads x_{m-2} (all layers ladder), batch 5..64, the whole step here: the pending-output schedule
    bool all_stale = (batch > 4 || m->sms_a >= 0 || auto_small) && m->sms_a != -3 && m->pend_a && m->pend_m && !m->st_in.newest && !m->st_out.newest &&
                     (l_end < 0 || l_end == c.n_layers);
    for (size_t i = 0; i < m->stale.size() && all_stale; ++i) all_stale = m->stale[i] != 0;
    if (all_stale && !m->exchange)
      return enqueue_decode_pending(m, cache, d_tokens, batch, out, sA, sB, n_kernels, q.grid_a, q.grid_b);
  }
  if (m->exchange)  // tensor parallelism: the pending-output form at every batch size (shares of the SMs as above)
    return enqueue_decode_pending(m, cache, d_tokens, batch, out, sA, sB, n_kernels, q.grid_a, q.grid_b);

  Router rt;
  q.launched(0, begin_stream(m, rt, d_tokens, batch, sA));
  q.pdl_ok[0] = m->st_in.newest == nullptr;  // a programmatic edge needs a kernel in front
  q.record(0, m->ev[0]);
  bool b_joined = false;  // has sB been ordered after the embedding yet

  int last_wait[2] = {0, -1};  // latest module each stream has (transitively) waited for
  auto need = [&](int s, int module) {
    // make stream s wait for the end of `module` unless that is already implied
    if (!q.two) return;
    const int owner = module == 0 ? 0 : ((module & 1) ? 0 : 1);
    if (owner == s) return;  // same stream: program order
    if (last_wait[s] >= module) return;
    q.wait(s, m->ev[module]);
    last_wait[s] = module;
    if (s == 1) b_joined = true;
  };

  if (l_end < 0) l_end = c.n_layers;
  for (int l = 0; l < l_end; ++l) {
    const bool lad = m->stale[2 * l + 1] != 0;  // the MLP module does not read the attention module's output (ladder and
                                                // parallel layers): the two modules' GEMMs may run side by side
    // ---------------- attention module (module index 2l+1) on stream A
    {
      const int mod = 2 * l + 1;
      const Router::Route r = route(m, rt, mod);
      need(0, r.in_writer);
      SmallMParams p = {};
      p.W = m->w_qkv[l];
      p.N = (Hq + 2 * Hkv) * Dh;
      p.K = d;
      p.act = m->R[r.in];
      p.act_mode = ACT_F32_NORM;
      p.gain = m->attn_norm[l];
      p.eps = c.rms_eps;
      p.batch = batch;
      p.epi_mode = EPI_QKV_ROPE;
      p.qkv.q_out_f32 = m->q_f32;
      p.qkv.k_cache = static_cast<kv_t*>(cache->k) + l * layer_elems;
      p.qkv.v_cache = static_cast<kv_t*>(cache->v) + l * layer_elems;
      p.qkv.seq_lens = cache->seq_lens;
      p.qkv.rope = m->rope;
      p.qkv.n_q_heads = Hq;
      p.qkv.n_kv_heads = Hkv;
      p.qkv.head_dim = Dh;
      p.qkv.max_seq_len = c.max_seq_len;
      p.status = m->status;
      q.gemm(0, p, lad);

      DecodeAttnParams a = {};
      a.q = m->q_f32;
      a.k = p.qkv.k_cache;
      a.v = p.qkv.v_cache;
      a.kv_len = cache->seq_lens;
      a.kv_len_offset = 1;
      a.batch = batch;
      a.n_q_heads = Hq;
      a.n_kv_heads = Hkv;
      a.head_dim = Dh;
      a.max_seq_len = c.max_seq_len;
      a.n_splits = m->attn_splits;
      a.max_len = c.max_seq_len;
      a.scratch = m->attn_scratch;
      a.o = m->o_dec;
      a.status = m->status;
      const bool handover = batch > 4 && m->wide_opack;  // operands pass from kernel to kernel
      if (handover) {
        a.o_pack = m->wide_opack;
        a.o_pack_bp = wide_padded_batch(batch);
      }
      q.launched(0, launch_decode_attention(a, sA, q.pdl(0)));
      ++q.kernels;  // the split kernel and its merge kernel

      need(0, mod - 1);  // the epilogue reads x_{m-1} and overwrites the buffer of x_{m-2}
      SmallMParams o = {};
      o.W = m->w_o[l];
      o.N = d;
      o.K = Hq * Dh;
      o.act = m->o_dec;
      o.act_mode = ACT_F32;
      o.batch = batch;
      o.epi_mode = EPI_RESID;
      o.addend = m->R[r.add];
      o.out = m->R[r.dst];
      o.status = m->status;
      if (handover) o.act_staged = m->wide_opack;
      q.gemm(0, o, lad);
      q.record(0, m->ev[mod]);
    }
    // ---------------- MLP module (module index 2l+2) on stream B
    {
      const int mod = 2 * l + 2;
      const Router::Route r = route(m, rt, mod);
      need(1, r.in_writer);
      if (q.two && !b_joined) {  // first use of sB in this step: order it after the embedding
        q.wait(1, m->ev[0]);
        b_joined = true;
      }
      SmallMParams p = {};
      p.W = m->w_gate_up[l];
      p.N = 2 * F;
      p.K = d;
      p.act = m->R[r.in];
      p.act_mode = ACT_F32_NORM;
      p.gain = mlp_gain(m, l);
      p.eps = c.rms_eps;
      p.batch = batch;
      p.epi_mode = EPI_SWIGLU;
      p.out = m->h_dec;
      p.status = m->status;
      const bool handover = batch > 4 && m->wide_hpack;
      if (handover) p.wide_pack_out = m->wide_hpack;
      q.gemm(1, p, lad);

      need(1, mod - 1);
      SmallMParams o = {};
      o.W = m->w_down[l];
      o.N = d;
      o.K = F;
      o.act = m->h_dec;
      o.act_mode = ACT_F32;
      o.batch = batch;
      o.epi_mode = EPI_RESID;
      o.addend = m->R[r.add];
      o.out = m->R[r.dst];
      o.status = m->status;
      if (handover) o.act_staged = m->wide_hpack;
      q.gemm(1, o, lad);
      q.record(1, m->ev[mod]);
    }
  }
  if (l_end < c.n_layers) {  // prefix only: stream A joins stream B, the persistent kernel does the rest
    need(0, 2 * l_end);
    *n_kernels = q.kernels;
    return q.err;
  }
  // ---------------- head on stream A (joins stream B)
  need(0, 2 * c.n_layers);
  if (m->st_out.newest) {  // a stage that hands its state on: no final norm, no head
    q.launched(0, end_stage(m, rt, cache, batch, batch, 1, -1, nullptr, sA));
    *n_kernels = q.kernels;
    return q.err;
  }
  const float* xf = m->R[rt.cur];
  float* logits = (out && out->logits) ? out->logits : m->logits_ws;
  SmallMParams h = {};
  h.W = m->lm_head;
  h.N = c.vocab_size;
  h.K = d;
  h.act = xf;
  h.act_mode = ACT_F32_NORM;
  h.gain = m->final_norm;
  h.eps = c.rms_eps;
  h.batch = batch;
  h.epi_mode = EPI_PLAIN;
  h.out = logits;
  h.status = m->status;
  q.gemm(0, h);
  if (out && out->final_hidden)
    q.launched(0, launch_rmsnorm_f32(xf, m->final_norm, c.rms_eps, batch, d, d, out->final_hidden, sA, q.pdl(0)));
  q.launched(0, launch_argmax_advance(logits, batch, c.vocab_size, out ? out->next_tokens : nullptr, cache->seq_lens, 1,
                                      -1, sA, q.pdl(0)));
  *n_kernels = q.kernels;
  return q.err;
}

// pos0: position of the first of the S new tokens of every sequence (0 = a fresh prompt; > 0 = the prompt is
// continued: the new tokens attend to the pos0 cached positions and to each other causally).
// d_lens (device, optional; fresh prompts only): per-sequence prompt lengths <= S; rows behind them are padding.
cudaError_t enqueue_prefill(ladder_model* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens, int batch, int S,
                            const ladder_outputs_t* out, cudaStream_t st, int64_t* n_kernels, int pos0 = 0,
                            const int32_t* d_lens = nullptr) {
  const ladder_config_t& c = m->cfg;
  const int Hq = c.n_q_heads, Hkv = c.n_kv_heads, Dh = c.head_dim, d = c.d_model, F = c.d_ff;
  const int M = batch * S;
  const size_t layer_elems = static_cast<size_t>(c.max_batch) * Hkv * c.max_seq_len * Dh;
  int64_t k = 0;
  cudaError_t err = cudaSuccess;
  auto did = [&](cudaError_t e) {
    if (err == cudaSuccess) err = e;
    ++k;
  };
  Router rt;
  did(begin_stream(m, rt, d_tokens, M, st));
  // Operand precision of the prompt-pass GEMMs.  Default for calls of >= kPrefillF16MinTokens tokens: binary16,
  // ONE value per activation (11 significant bits) against the layer's weights converted to binary16 once per
  // call (exact but for magnitudes below 2^-14) -- half the tensor-core work of a bf16 hi + lo pair.  Otherwise
  // (short chunks, no room for the converted layer, or a mode selected for tests) bf16 hi + lo pairs / single bf16.
  const bool f16 = prefill_gemm_impl() == 0 && m->w16 && M >= kPrefillF16MinTokens;
  const bool split = !f16 && !prefill_single_bf16();
  __nv_bfloat16* const n_lo = split ? m->n_pf + m->n_lo : nullptr;
  __half* const q_lo = m->q_pf + m->q_lo;  // the query always goes to the attention as a binary16 pair
  __nv_bfloat16* const o_lo = split ? m->o_pf + m->q_lo : nullptr;
  __nv_bfloat16* const h_lo = split ? m->h_pf + m->h_lo : nullptr;
  const size_t n_qkv = static_cast<size_t>(Hq + 2 * Hkv) * Dh * d, n_o = static_cast<size_t>(d) * Hq * Dh;
  const size_t n_gu = 2 * static_cast<size_t>(F) * d, n_dn = static_cast<size_t>(d) * F;
  // Two scratch buffers: the conversion of layer l + 1 runs on the side stream while layer l's GEMMs run here
  // (they leave most of the DRAM bandwidth unused).  With one buffer it runs in line.
  const bool overlap = f16 && m->w16b != nullptr;
  auto convert_layer = [&](int l, __half* dst, cudaStream_t cs) {
    did(launch_convert_bf16_f16(m->w_qkv[l], dst, n_qkv, cs));
    did(launch_convert_bf16_f16(m->w_o[l], dst + n_qkv, n_o, cs));
    did(launch_convert_bf16_f16(m->w_gate_up[l], dst + n_qkv + n_o, n_gu, cs));
    did(launch_convert_bf16_f16(m->w_down[l], dst + n_qkv + n_o + n_gu, n_dn, cs));
  };
  auto note = [&](cudaError_t e) {
    if (err == cudaSuccess) err = e;
  };
  if (overlap) {  // the side stream starts after everything already queued here (an earlier call may still use the buffers)
    note(cudaEventRecord(m->ev_pf_fork, st));
    note(cudaStreamWaitEvent(m->side, m->ev_pf_fork, 0));
    convert_layer(0, m->w16, m->side);
    note(cudaEventRecord(m->ev_w16_ready[0], m->side));
  }
  // Tensor parallelism (Sec. 2, Eq. 1; Algorithm 1): the output and down projections store this rank's partial sum,
  // the exchange stream sums it over the ranks and adds it to the stream value, and this stream goes on with the
  // next module; it waits for an add only where a module reads the buffer that add writes (a ladder module's
  // input x_{m-2} is older than the exchange in flight; with standard residuals the very next module waits).
  const bool tp = m->exchange != nullptr;
  int add_writer[2] = {-1, -1};  // module whose add on the exchange stream last wrote R[i]
  // module j's output travels inside module j + 1's (one exchange for a parallel attention + MLP layer: see the
  // decode step's pending-output form)
  auto merged = [&](int j) {
    const int n_mod = 2 * c.n_layers;
    if (!tp || (j & 1) || j + 1 >= n_mod || m->stale[j] || !m->stale[j + 1]) return false;
    if (j + 2 < n_mod) return m->stale[j + 2] == 0;
    return m->st_out.newest == nullptr || m->st_out.older == nullptr;
  };
  auto norm = [&](int buf, const __nv_bfloat16* gain) {
    if (tp && add_writer[buf] >= 0) note(cudaStreamWaitEvent(st, m->ev_pf_add[add_writer[buf]], 0));
    const float* x = m->R[buf];
    if (f16) did(launch_rmsnorm_f16(x, gain, c.rms_eps, M, d, reinterpret_cast<__half*>(m->n_pf), st));
    else did(launch_rmsnorm_bf16(x, gain, c.rms_eps, M, d, m->n_pf, n_lo, st));
  };
  // Last GEMM of module mod (0-based): x_m = x_{m-1} + output, x_{m-1} in R[r.add], x_m to R[r.dst].
  auto finish_module = [&](int mod, const Router::Route& r, LargeMParams& o) {
    if (!tp) {
      o.epi_mode = EPI_RESID;
      o.addend = m->R[r.add];
      o.out = m->R[r.dst];
      did(launch_largem_gemm(o, st));
      return;
    }
    float* const pend = m->pend_pf[mod & 1];
    o.epi_mode = EPI_PLAIN;
    o.out = pend;
    if (merged(mod)) {  // parallel attention + MLP: stays local, the down projection adds it before the one exchange
      did(launch_largem_gemm(o, st));
      return;
    }
    if (mod >= 2 && !merged(mod - 2)) note(cudaStreamWaitEvent(st, m->ev_pf_add[mod - 2], 0));  // the buffer's previous content is added
    const bool both = (mod & 1) && merged(mod - 1);  // this output plus the attention module's: x_{m} = x_{m-2} + sum
    if (both) {
      o.epi_mode = EPI_RESID;
      o.addend = m->pend_pf[0];
    }
    did(launch_largem_gemm(o, st));
    note(cudaEventRecord(m->ev_pf_out[mod], st));
    note(cudaStreamWaitEvent(m->xstream, m->ev_pf_out[mod], 0));
    if (m->exchange(m->exchange_ctx, pend, static_cast<int64_t>(M) * d, m->xstream) != LADDER_OK) note(cudaErrorUnknown);
    did(launch_add_f32(m->R[both ? r.in : r.add], pend, m->R[r.dst], static_cast<size_t>(M) * d, m->xstream));
    note(cudaEventRecord(m->ev_pf_add[mod], m->xstream));
    add_writer[r.dst] = mod;
  };
  for (int l = 0; l < c.n_layers; ++l) {
    __half* const w16_qkv = overlap && (l & 1) ? m->w16b : m->w16;
    __half* const w16_o = f16 ? w16_qkv + n_qkv : nullptr;
    __half* const w16_gu = f16 ? w16_o + n_o : nullptr;
    __half* const w16_dn = f16 ? w16_gu + n_gu : nullptr;
    if (overlap) {
      if (l + 1 < c.n_layers) {  // next layer into the other buffer, once layer l - 1 has finished with it
        if (l >= 1) note(cudaStreamWaitEvent(m->side, m->ev_w16_free[(l + 1) & 1], 0));
        convert_layer(l + 1, (l + 1) & 1 ? m->w16b : m->w16, m->side);
        note(cudaEventRecord(m->ev_w16_ready[(l + 1) & 1], m->side));
      }
      note(cudaStreamWaitEvent(st, m->ev_w16_ready[l & 1], 0));
    } else if (f16) {  // in line: the previous layer's GEMMs are done with the scratch (same stream)
      convert_layer(l, m->w16, st);
    }
    {
      const Router::Route r = route(m, rt, 2 * l + 1);
      norm(r.in, m->attn_norm[l]);
      LargeMParams p = {};
      p.A = m->n_pf;
      p.A_lo = n_lo;
      p.W = f16 ? reinterpret_cast<const __nv_bfloat16*>(w16_qkv) : m->w_qkv[l];
      p.f16 = f16;
      p.M = M;
      p.N = (Hq + 2 * Hkv) * Dh;
      p.K = d;
      p.epi_mode = EPI_QKV_ROPE;
      p.qkv.q_out_f16 = m->q_pf;
      p.qkv.q_out_lo = q_lo;
      p.qkv.k_cache = static_cast<kv_t*>(cache->k) + l * layer_elems;
      p.qkv.v_cache = static_cast<kv_t*>(cache->v) + l * layer_elems;
      p.qkv.rope = m->rope;
      p.qkv.n_q_heads = Hq;
      p.qkv.n_kv_heads = Hkv;
      p.qkv.head_dim = Dh;
      p.qkv.max_seq_len = c.max_seq_len;
      p.qkv.prefill_seq_len = S;
      p.qkv.prefill_pos0 = pos0;
      p.qkv.prefill_lens = d_lens;
      p.status = m->status;
      did(launch_largem_gemm(p, st));
      did(launch_prefill_attention(m->q_pf, q_lo, p.qkv.k_cache, p.qkv.v_cache, batch, S, Hq, Hkv, Dh, c.max_seq_len,
                                   m->o_pf, o_lo, st, pos0, f16, d_lens, m->status));
      LargeMParams o = {};
      o.A = m->o_pf;
      o.A_lo = o_lo;
      o.W = f16 ? reinterpret_cast<const __nv_bfloat16*>(w16_o) : m->w_o[l];
      o.f16 = f16;
      o.M = M;
      o.N = d;
      o.K = Hq * Dh;
      o.status = m->status;
      finish_module(2 * l, r, o);
    }
    {
      const Router::Route r = route(m, rt, 2 * l + 2);
      norm(r.in, mlp_gain(m, l));
      LargeMParams p = {};
      p.A = m->n_pf;
      p.A_lo = n_lo;
      p.W = f16 ? reinterpret_cast<const __nv_bfloat16*>(w16_gu) : m->w_gate_up[l];
      p.f16 = f16;
      p.M = M;
      p.N = 2 * F;
      p.K = d;
      p.epi_mode = EPI_SWIGLU;
      p.out = m->h_pf;
      p.out_lo = h_lo;
      p.status = m->status;
      did(launch_largem_gemm(p, st));
      LargeMParams o = {};
      o.A = m->h_pf;
      o.A_lo = h_lo;
      o.W = f16 ? reinterpret_cast<const __nv_bfloat16*>(w16_dn) : m->w_down[l];
      o.f16 = f16;
      o.M = M;
      o.N = d;
      o.K = F;
      o.status = m->status;
      finish_module(2 * l + 1, r, o);
    }
    if (overlap) note(cudaEventRecord(m->ev_w16_free[l & 1], st));
  }
  if (tp && c.n_layers > 0) note(cudaStreamWaitEvent(st, m->ev_pf_add[2 * c.n_layers - 1], 0));  // every add (in order)
  if (m->st_out.newest) {  // a stage that hands its state on: every position's stream state, no head
    did(end_stage(m, rt, cache, batch, M, 0, pos0 + S, d_lens, st));
    *n_kernels = k;
    return err;
  }
  const float* xf = m->R[rt.cur];
  if (out && out->all_hidden) did(launch_rmsnorm_f32(xf, m->final_norm, c.rms_eps, M, d, d, out->all_hidden, st, false));
  did(launch_gather_rows(xf, batch, d, S, S - 1, m->last_x, st, d_lens));
  float* logits = (out && out->logits) ? out->logits : m->logits_ws;
  SmallMParams h = {};
  h.W = m->lm_head;
  h.N = c.vocab_size;
  h.K = d;
  h.act = m->last_x;
  h.act_mode = ACT_F32_NORM;
  h.gain = m->final_norm;
  h.eps = c.rms_eps;
  h.batch = batch;
  h.epi_mode = EPI_PLAIN;
  h.out = logits;
  h.status = m->status;
  h.scratch = m->gemm_scratch[0];
  h.work = m->work_slots + 2 * (m->n_work_slots - 1);
  did(launch_smallm_gemm(h, st, false, m->sm_count));
  if (out && out->final_hidden)
    did(launch_rmsnorm_f32(m->last_x, m->final_norm, c.rms_eps, batch, d, d, out->final_hidden, st, false));
  did(launch_argmax_advance(logits, batch, c.vocab_size, out ? out->next_tokens : nullptr, cache->seq_lens, 0, pos0 + S,
                            st, false, d_lens));
  *n_kernels = k;
  return err;
}


// --------------------------------------------------------------------------- persistent layer stack
// Builds the phase list of one decode step for the persistent kernel: the GEMMs of every layer in the
// order the residual rule allows (ladder layer: QKV, gate/up, Wo, down -- the MLP's first GEMM does
// not depend on the attention module; standard layer: QKV, Wo, gate/up, down), the attention nodes,
// and for every access to a buffer another phase touches the counters it has to wait for:
// read-after-write on the last writer, write-after-read on every reader since, write-after-write.
struct StackBuilder {
  struct Buf {
    int writer = -1;
    std::vector<int> readers;
  };
  std::map<const void*, Buf> bufs;
  std::vector<int> need;  // need[counter] = value that means "complete" (-1: not usable as a dependency)
  bool overflow = false;

  int counter(int complete_at) {
    need.push_back(complete_at);
    return static_cast<int>(need.size()) - 1;
  }
  static void push(std::vector<int>& v, int c) {
    if (c >= 0 && std::find(v.begin(), v.end(), c) == v.end()) v.push_back(c);
  }
  void raw(const void* b, std::vector<int>& deps) {
    if (b) push(deps, bufs[b].writer);
  }
  void war(const void* b, std::vector<int>& deps) {
    if (!b) return;
    Buf& s = bufs[b];
    for (int r : s.readers) push(deps, r);
    push(deps, s.writer);
  }
  void did_read(const void* b, int me) {
    if (b) push(bufs[b].readers, me);
  }
  void did_write(const void* b, int me) {
    if (!b) return;
    Buf& s = bufs[b];
    s.readers.clear();
    s.writer = me;
  }
  void emit(const std::vector<int>& deps, int self, int* n_out, int* dep_out, int* need_out) {
    int n = 0;
    for (int c : deps) {
      if (c == self) continue;
      if (n == kStackMaxDeps || need[c] < 0) {
        overflow = true;
        return;
      }
      dep_out[n] = c;
      need_out[n] = need[c];
      ++n;
    }
    *n_out = n;
  }
};

// First layer of the ladder stretch at the top of the model (n_layers if the top layer is standard).
int stack_first_layer(const std::vector<uint8_t>& is_ladder) {
  int b = static_cast<int>(is_ladder.size());
  while (b > 0 && is_ladder[b - 1]) --b;
  return b;
}

// First layer the persistent kernel runs by default.  A standard-residual layer makes every phase wait for the
// one before; for layers that stream a lot (measured: 436 MB per layer at the 8B shape, 1.7 GB at the 70B shape)
// separate kernels with their dynamically balanced GEMMs are then 2.5-3 % faster, so only the ladder stretch at
// the top goes into the kernel.  For small layers (214 MB per layer at the tensor-parallel slice: 6 % the other
// way) the launch gaps weigh more than the balance and every layer goes in.
int stack_default_begin(const ladder_config_t& c, const std::vector<uint8_t>& is_ladder) {
  const double layer_bytes = 2.0 * (static_cast<double>((c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim) * c.d_model +
                                    static_cast<double>(c.d_model) * c.n_q_heads * c.head_dim + 3.0 * c.d_ff * c.d_model);
  return layer_bytes < 300e6 ? 0 : stack_first_layer(is_ladder);
}

// Returns false (with a reason) when this step cannot be expressed; the caller then uses the
// multi-kernel schedule.
bool build_stack(ladder_model* m, const ladder_kv_cache_t* cache, int batch, float* logits, std::vector<StackPhase>& phases,
                 std::vector<StackAttn>& attn, int* n_counters, int l_begin) {
  const ladder_config_t& c = m->cfg;
  const int Hq = c.n_q_heads, Hkv = c.n_kv_heads, Dh = c.head_dim, d = c.d_model, F = c.d_ff;
  const size_t layer_elems = static_cast<size_t>(c.max_batch) * Hkv * c.max_seq_len * Dh;
  if (m->attn_splits > 1024) return false;  // merge weights are held in shared memory
  StackBuilder sb;
  phases.clear();
  attn.clear();

  int cur_layer = 0;
  // A phase whose fp32 input was produced inside this launch gets it as a ready MMA operand as well: the
  // producer's epilogue (or the attention merge) writes the bf16 hi/lo copy, with the reader's RMSNorm gain
  // folded in, and the reader's stagers only copy it (with ordinary loads: a bulk copy by the TMA engine read
  // stale bytes now and then, whatever proxy fences were placed on either side).  Only for batch <= 4 (hi
  // and lo share one MMA tile).
  std::map<const void*, __nv_bfloat16*> twin = {
      {m->R[0], m->xpack[0]}, {m->R[1], m->xpack[1]}, {m->h_dec, m->hpack}, {m->o_dec, m->opack}};
  std::map<const void*, std::pair<int, int>> last_writer;  // fp32 buffer -> (0 = phase | 1 = attention node, index)
  auto add_gemm = [&](int kind, SmallMParams p, const void* act_buf, const void* add_buf, const void* out0,
                      const void* out1, const void* out2) {
    StackPhase P = {};
    P.kind = kind;
    P.layer = cur_layer;
    if (batch <= 4) {
      auto wr = last_writer.find(act_buf);
      auto tw = twin.find(act_buf);
      if (wr != last_writer.end() && tw != twin.end() && tw->second) {
        const __nv_bfloat16* want_gain = p.act_mode == ACT_F32_NORM ? p.gain : nullptr;
        if (wr->second.first == 0) {
          SmallMParams& w = phases[wr->second.second].p;
          if (!w.pack_out) {
            w.pack_out = tw->second;
            w.pack_gain = want_gain;
            P.act_packed = tw->second;
          } else if (w.pack_out == tw->second && w.pack_gain == want_gain) {
            P.act_packed = tw->second;  // a second reader with the same gain (parallel layer: QKV and gate/up)
          }
        } else {
          StackAttn& w = attn[wr->second.second];
          if (!w.o_pack) {
            w.o_pack = tw->second;
            P.act_packed = tw->second;
          }
        }
      }
    }
    if (p.epi_mode == EPI_RESID || p.epi_mode == EPI_SWIGLU) last_writer[out0] = {0, static_cast<int>(phases.size())};
    p.batch = batch;
    p.status = m->status;
    P.p = p;
    P.W = p.W;
    P.K = p.K;
    P.act = static_cast<const float*>(p.act);
    P.gain = p.gain;
    P.act_mode = p.act_mode;
    P.n_units = p.N / 8;
    P.nchunk = (p.K + kStackChunkK - 1) / kStackChunkK;
    P.work_idx = sb.counter(-1);
    P.done_idx = sb.counter(P.n_units);
    const Schedule sc = make_schedule(P.n_units, m->sm_count);
    if (sc.n > kStackRounds) sb.overflow = true;
    P.sched_n = sc.n < kStackRounds ? sc.n : kStackRounds;
    for (int r = 0; r < P.sched_n; ++r) {
      P.count[r] = sc.count[r];
      P.size[r] = sc.size[r];
    }
    P.n_static = sc.n_static;
    P.n_claims = sc.n_claims;
    std::vector<int> ad, ed;
    sb.raw(act_buf, ad);
    sb.raw(add_buf, ed);
    sb.war(out0, ed);
    sb.war(out1, ed);
    sb.war(out2, ed);
    sb.emit(ad, P.done_idx, &P.n_act_deps, P.act_dep, P.act_need);
    sb.emit(ed, P.done_idx, &P.n_epi_deps, P.epi_dep, P.epi_need);
    sb.did_read(act_buf, P.done_idx);
    sb.did_read(add_buf, P.done_idx);
    sb.did_write(out0, P.done_idx);
    sb.did_write(out1, P.done_idx);
    sb.did_write(out2, P.done_idx);
    phases.push_back(P);
  };

  Router rt;
  int prev_merge = -1;
  for (int l = 0; l < c.n_layers; ++l) {
    const Router::Route ra = route(m, rt, 2 * l + 1);
    const Router::Route rm = route(m, rt, 2 * l + 2);
    if (l < l_begin) continue;  // run by separate kernels before the launch: only the routing state matters
    cur_layer = l;
    kv_t* kc = static_cast<kv_t*>(cache->k) + l * layer_elems;
    kv_t* vc = static_cast<kv_t*>(cache->v) + l * layer_elems;

    auto qkv = [&]() {
      SmallMParams p = {};
      p.W = m->w_qkv[l];
      p.N = (Hq + 2 * Hkv) * Dh;
      p.K = d;
      p.act = m->R[ra.in];
      p.act_mode = ACT_F32_NORM;
      p.gain = m->attn_norm[l];
      p.eps = c.rms_eps;
      p.epi_mode = EPI_QKV_ROPE;
      p.qkv.q_out_f32 = m->q_f32;
      p.qkv.k_cache = kc;
      p.qkv.v_cache = vc;
      p.qkv.seq_lens = cache->seq_lens;
      p.qkv.rope = m->rope;
      p.qkv.n_q_heads = Hq;
      p.qkv.n_kv_heads = Hkv;
      p.qkv.head_dim = Dh;
      p.qkv.max_seq_len = c.max_seq_len;
      add_gemm(0, p, m->R[ra.in], nullptr, m->q_f32, kc, vc);
      // the attention of this layer, on the attention warps
      StackAttn A = {};
      A.a.q = m->q_f32;
      A.a.k = kc;
      A.a.v = vc;
      A.a.kv_len = cache->seq_lens;
      A.a.kv_len_offset = 1;
      A.a.batch = batch;
      A.a.n_q_heads = Hq;
      A.a.n_kv_heads = Hkv;
      A.a.head_dim = Dh;
      A.a.max_seq_len = c.max_seq_len;
      A.a.n_splits = m->attn_splits;
      A.a.max_len = c.max_seq_len;
      A.a.scratch = m->attn_scratch;
      A.a.o = m->o_dec;
      A.split_done = sb.counter(-1);
      A.merge_done = sb.counter(batch * Hq);
      std::vector<int> sd, md;
      sb.raw(m->q_f32, sd);
      sb.raw(kc, sd);
      sb.raw(vc, sd);
      StackBuilder::push(sd, prev_merge);  // the partials of the previous layer have been merged
      sb.war(m->o_dec, md);
      sb.emit(sd, A.merge_done, &A.n_deps, A.dep, A.need);
      sb.emit(md, A.merge_done, &A.n_mdeps, A.mdep, A.mneed);
      sb.did_read(m->q_f32, A.merge_done);
      sb.did_read(kc, A.merge_done);
      sb.did_read(vc, A.merge_done);
      sb.did_write(m->o_dec, A.merge_done);
      prev_merge = A.merge_done;
      last_writer[m->o_dec] = {1, static_cast<int>(attn.size())};
      attn.push_back(A);
    };
    auto wo = [&]() {
      SmallMParams p = {};
      p.W = m->w_o[l];
      p.N = d;
      p.K = Hq * Dh;
      p.act = m->o_dec;
      p.act_mode = ACT_F32;
      p.epi_mode = EPI_RESID;
      p.addend = m->R[ra.add];
      p.out = m->R[ra.dst];
      add_gemm(2, p, m->o_dec, m->R[ra.add], m->R[ra.dst], nullptr, nullptr);
    };
    auto gate_up = [&]() {
      SmallMParams p = {};
      p.W = m->w_gate_up[l];
      p.N = 2 * F;
      p.K = d;
      p.act = m->R[rm.in];
      p.act_mode = ACT_F32_NORM;
      p.gain = mlp_gain(m, l);
      p.eps = c.rms_eps;
      p.epi_mode = EPI_SWIGLU;
      p.out = m->h_dec;
      add_gemm(1, p, m->R[rm.in], nullptr, m->h_dec, nullptr, nullptr);
    };
    auto down = [&]() {
      SmallMParams p = {};
      p.W = m->w_down[l];
      p.N = d;
      p.K = F;
      p.act = m->h_dec;
      p.act_mode = ACT_F32;
      p.epi_mode = EPI_RESID;
      p.addend = m->R[rm.add];
      p.out = m->R[rm.dst];
      add_gemm(3, p, m->h_dec, m->R[rm.add], m->R[rm.dst], nullptr, nullptr);
    };
    // An MLP module that reads x_{m-2} (ladder layer, parallel layer) reads a value that exists before the
    // attention module of the same layer has produced anything (in the first ladder layer after a standard
    // one and in a parallel layer it is the attention module's own input: still not its output).
    const bool mlp_independent = m->stale[2 * l + 1] != 0 && rm.in != ra.dst;
    qkv();
    if (mlp_independent) {
      gate_up();
      wo();
    } else {
      wo();
      gate_up();
    }
    down();
  }
  {
    SmallMParams h = {};
    h.W = m->lm_head;
    h.N = c.vocab_size;
    h.K = d;
    h.act = m->R[rt.cur];
    h.act_mode = ACT_F32_NORM;
    h.gain = m->final_norm;
    h.eps = c.rms_eps;
    h.epi_mode = EPI_PLAIN;
    h.out = logits;
    cur_layer = c.n_layers;
    add_gemm(4, h, m->R[rt.cur], nullptr, logits, nullptr, nullptr);
  }
  if (m->stack_stall_test && !phases.empty() && phases.back().n_act_deps > 0) phases.back().act_need[0] += 1;
  *n_counters = static_cast<int>(sb.need.size());
  return !sb.overflow && static_cast<int>(phases.size()) <= kStackMaxPhases;
}

// One decode step through the persistent kernel: embedding, zeroed counters, the layer stack, head outputs.
cudaError_t enqueue_decode_stack(ladder_model* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens, int batch,
                                 const ladder_outputs_t* out, cudaStream_t st, int64_t* n_kernels) {
  const ladder_config_t& c = m->cfg;
  const int d = c.d_model;
  float* logits = (out && out->logits) ? out->logits : m->logits_ws;
  int64_t k = 2;
  cudaError_t e;
  if (m->stack_begin > 0) {  // embedding + the standard-residual layers below the ladder stretch, kernel by kernel
    int64_t kp = 0;
    e = enqueue_decode(m, cache, d_tokens, batch, out, st, st, &kp, m->stack_begin);
    k += kp - 1;
  } else {
    e = launch_embed(d_tokens, m->tok_embedding, batch, d, c.vocab_size, m->R[0], m->status, st, false);
  }
  if (e == cudaSuccess) e = cudaMemsetAsync(m->d_counters, 0, static_cast<size_t>(m->n_counters) * sizeof(int32_t), st);
  StackParams sp = {};
  sp.phases = m->d_phases;
  sp.n_phases = m->n_phases;
  sp.attn = m->d_attn;
  sp.n_attn = m->n_attn;
  sp.counters = m->d_counters;
  sp.status = m->status;
  sp.batch = batch;
  if (e == cudaSuccess) e = launch_decode_stack(sp, m->sm_count, st);
  // the final hidden state is the input of the last phase (the LM head)
  Router rt;
  for (int mod = 1; mod <= 2 * c.n_layers; ++mod) route(m, rt, mod);
  if (out && out->final_hidden) {
    if (e == cudaSuccess)
      e = launch_rmsnorm_f32(m->R[rt.cur], m->final_norm, c.rms_eps, batch, d, d, out->final_hidden, st, false);
    ++k;
  }
  if (e == cudaSuccess)
    e = launch_argmax_advance(logits, batch, c.vocab_size, out ? out->next_tokens : nullptr, cache->seq_lens, 1, -1, st,
                              false);
  ++k;
  *n_kernels = k;
  return e;
}

void drop_graph(ladder_model* m) {
  if (m->graph_exec) cudaGraphExecDestroy(m->graph_exec);
  m->graph_exec = nullptr;
  m->graph_key = GraphKey();
}

}  // namespace

// =========================================================================== C ABI
extern "C" {

const char* ladder_status_string(ladder_status_t s) {
  switch (s) {
    case LADDER_OK: return "ok";
    case LADDER_ERR_INVALID_ARG: return "invalid argument";
    case LADDER_ERR_UNSUPPORTED: return "unsupported configuration";
    case LADDER_ERR_OOM: return "out of device memory";
    case LADDER_ERR_CUDA: return "CUDA error";
    case LADDER_ERR_STATE: return "invalid state (cache overflow / batch too large)";
    case LADDER_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

const char* ladder_last_error(const ladder_model_t* m) { return m ? m->err.c_str() : g_create_error.c_str(); }

void ladder_set_prefill_gemm_impl(int32_t impl) { set_prefill_gemm_impl(impl); }

void ladder_set_decode_wide_impl(int32_t impl) { set_decode_wide_impl(impl); }
void ladder_set_decode_attention_impl(int32_t impl) { set_decode_attention_impl(impl); }

size_t ladder_kv_cache_bytes(const ladder_config_t* c) {
  if (!c) return 0;
  return static_cast<size_t>(c->n_layers) * c->max_batch * c->n_kv_heads * c->max_seq_len * c->head_dim * 2;
}

ladder_status_t ladder_model_create(const ladder_config_t* cfg, const ladder_weights_t* w, ladder_model_t** out) {
  if (out) *out = nullptr;
  if (!cfg || !w || !out) return fail(nullptr, LADDER_ERR_INVALID_ARG, "NULL argument");
  if (cfg->struct_size != sizeof(ladder_config_t) && cfg->struct_size != kConfigSizeV1)
    return fail(nullptr, LADDER_ERR_INVALID_ARG, "struct_size mismatch");
  if (const char* why = check_shape(*cfg)) return fail(nullptr, LADDER_ERR_UNSUPPORTED, why);
  if (!w->tok_embedding || !w->final_norm || !w->lm_head || !w->attn_norm || !w->w_qkv || !w->w_o || !w->mlp_norm ||
      !w->w_gate_up || !w->w_down)
    return fail(nullptr, LADDER_ERR_INVALID_ARG, "NULL weight pointer");
  ladder_model* m = new ladder_model();
  copy_config(&m->cfg, cfg);
  const int L = cfg->n_layers;
  if (const char* why = parse_rules(cfg, m)) {
    delete m;
    return fail(nullptr, LADDER_ERR_INVALID_ARG, why);
  }
  m->tok_embedding = static_cast<const __nv_bfloat16*>(w->tok_embedding);
  m->final_norm = static_cast<const __nv_bfloat16*>(w->final_norm);
  m->lm_head = static_cast<const __nv_bfloat16*>(w->lm_head);
  auto grab = [&](const void* const* src, std::vector<const __nv_bfloat16*>& dst) -> bool {
    dst.resize(L);
    for (int l = 0; l < L; ++l) {
      dst[l] = static_cast<const __nv_bfloat16*>(src[l]);
      if (!dst[l] || (reinterpret_cast<uintptr_t>(dst[l]) & 15)) return false;
    }
    return true;
  };
  if (!grab(w->attn_norm, m->attn_norm) || !grab(w->w_qkv, m->w_qkv) || !grab(w->w_o, m->w_o) ||
      !grab(w->mlp_norm, m->mlp_norm) || !grab(w->w_gate_up, m->w_gate_up) || !grab(w->w_down, m->w_down)) {
    delete m;
    return fail(nullptr, LADDER_ERR_INVALID_ARG, "NULL or misaligned (16 B) per-layer weight pointer");
  }
  if ((reinterpret_cast<uintptr_t>(m->tok_embedding) | reinterpret_cast<uintptr_t>(m->final_norm) |
       reinterpret_cast<uintptr_t>(m->lm_head)) & 15) {
    delete m;
    return fail(nullptr, LADDER_ERR_INVALID_ARG, "misaligned (16 B) weight pointer");
  }
  const ladder_config_t& c = m->cfg;
  if (m->cfg.max_prefill_tokens <= 0) m->cfg.max_prefill_tokens = c.max_batch * c.max_seq_len;
  m->max_rows = c.max_prefill_tokens > c.max_batch ? c.max_prefill_tokens : c.max_batch;

  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&m->sm_count, cudaDevAttrMultiProcessorCount, dev);
  int smem_optin = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e == cudaSuccess) e = kernels_ready();
  if (e == cudaSuccess) e = decode_stack_init(m->sm_count, &m->stack_ok);
  if (e != cudaSuccess) {
    delete m;
    return fail(nullptr, LADDER_ERR_CUDA, std::string("device query: ") + cudaGetErrorString(e));
  }
  if (4 * L + 1 > kStackMaxPhases) m->stack_ok = false;
  // The persistent kernel pays off most where the ladder rule decouples consecutive modules: by default it runs
  // the ladder layers at the top of the model (and the LM head) and, for small layers, the standard ones too.
  m->stack_usable = m->stack_ok;
  m->stack_begin = stack_default_begin(c, m->is_ladder);
  if (m->stack_begin == L) m->stack_ok = false;
  if (static_cast<size_t>(smem_optin) < smallm_gemm_smem_bytes(c.max_batch)) {
    delete m;
    return fail(nullptr, LADDER_ERR_UNSUPPORTED, "device has too little shared memory per block (needs sm_100-class)");
  }

  const size_t rows = m->max_rows, d = c.d_model, qd = static_cast<size_t>(c.n_q_heads) * c.head_dim, F = c.d_ff;
  const size_t MB = c.max_batch, MP = c.max_prefill_tokens;
  m->attn_splits = decode_attention_splits(c.max_batch, c.n_kv_heads, c.max_seq_len, m->sm_count);
  const size_t scratch_floats = decode_attention_scratch_floats(c.max_batch, c.n_q_heads, c.head_dim, m->attn_splits);
  bool oom = false;
  auto A = [&](cudaError_t r) {
    if (r != cudaSuccess) oom = true;
  };
  A(dev_alloc(&m->R[0], rows * d));
  A(dev_alloc(&m->R[1], rows * d));
  A(dev_alloc(&m->q_f32, MB * qd));
  A(dev_alloc(&m->o_dec, MB * qd));
  A(dev_alloc(&m->h_dec, MB * F));
  A(dev_alloc(&m->wide_hpack, 2 * 64 * F));
  A(dev_alloc(&m->wide_opack, 2 * 64 * qd));
  A(dev_alloc(&m->pend_a, MB * d));
  A(dev_alloc(&m->pend_m, MB * d));
  const auto pack_elems = [](size_t K) { return ((K + 2047) / 2048) * 8 * 2048; };
  A(dev_alloc(&m->xpack[0], pack_elems(d)));
  A(dev_alloc(&m->xpack[1], pack_elems(d)));
  A(dev_alloc(&m->hpack, pack_elems(F)));
  A(dev_alloc(&m->opack, pack_elems(qd)));
  if (!oom) {  // the stagers copy whole 4 KB rows: what no epilogue ever writes must be finite
    for (auto pk : {std::make_pair(m->xpack[0], pack_elems(d)), std::make_pair(m->xpack[1], pack_elems(d)),
                    std::make_pair(m->hpack, pack_elems(F)), std::make_pair(m->opack, pack_elems(qd))})
      if (cudaMemset(pk.first, 0, pk.second * sizeof(__nv_bfloat16)) != cudaSuccess) oom = true;
  }
  A(dev_alloc(&m->attn_scratch, scratch_floats));
  {
    const int qkv_rows = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
    size_t sa = smallm_gemm_scratch_floats(qkv_rows, c.d_model, c.max_batch);
    sa = std::max(sa, smallm_gemm_scratch_floats(c.d_model, static_cast<int>(qd), c.max_batch));
    sa = std::max(sa, smallm_gemm_scratch_floats(c.vocab_size, c.d_model, c.max_batch));
    size_t sb = std::max(smallm_gemm_scratch_floats(2 * c.d_ff, c.d_model, c.max_batch),
                         smallm_gemm_scratch_floats(c.d_model, c.d_ff, c.max_batch));
    m->n_work_slots = 4 * L + 4;
    A(dev_alloc(&m->gemm_scratch[0], sa + 64));
    A(dev_alloc(&m->gemm_scratch[1], sb + 64));
    A(dev_alloc(&m->work_slots, static_cast<size_t>(2 * m->n_work_slots)));
    if (!oom) {
      if (cudaMemset(m->gemm_scratch[0], 0, (sa + 64) * sizeof(float)) != cudaSuccess) oom = true;
      if (cudaMemset(m->gemm_scratch[1], 0, (sb + 64) * sizeof(float)) != cudaSuccess) oom = true;
      if (cudaMemset(m->work_slots, 0, 2 * m->n_work_slots * sizeof(int32_t)) != cudaSuccess) oom = true;
    }
  }
  m->cap_counters = 2 * (4 * L + 1) + 2 * L;
  A(dev_alloc(&m->d_phases, static_cast<size_t>(4 * L + 1)));
  A(dev_alloc(&m->d_attn, static_cast<size_t>(L)));
  A(dev_alloc(&m->d_counters, static_cast<size_t>(m->cap_counters)));
  A(dev_alloc(&m->logits_ws, MB * c.vocab_size));
  A(dev_alloc(&m->last_x, MB * d));
  m->n_lo = MP * d;
  m->q_lo = MP * qd;
  m->h_lo = MP * F;
  A(dev_alloc(&m->n_pf, 2 * MP * d));
  A(dev_alloc(&m->q_pf, 2 * MP * qd));
  A(dev_alloc(&m->o_pf, 2 * MP * qd));
  A(dev_alloc(&m->h_pf, 2 * MP * F));
  A(dev_alloc(&m->rope, static_cast<size_t>(c.max_seq_len) * (c.head_dim / 2)));
  A(dev_alloc(&m->status, 4));
  A(dev_alloc(&m->tok_tmp, MP > MB ? MP : MB));
  A(dev_alloc(&m->next_tmp, MB));
  A(dev_alloc(&m->lens_tmp, MB));
  A(cudaMallocHost(reinterpret_cast<void**>(&m->h_lens_pinned), MB * sizeof(int32_t)));
  if (oom) {
    cudaGetLastError();
    ladder_destroy(m);
    return fail(nullptr, LADDER_ERR_OOM, "workspace allocation failed");
  }
  // Optional: room for one layer's weights as binary16 (the prompt pass then runs its GEMMs with one binary16 value
  // per activation).  Without it the prompt pass uses bf16 hi + lo pairs: slower, never wrong.
  if (c.max_prefill_tokens >= kPrefillF16MinTokens) {
    const size_t layer_elems = (static_cast<size_t>(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim + qd + 3 * F) * d;
    if (dev_alloc(&m->w16, layer_elems) != cudaSuccess) {
      cudaGetLastError();
      m->w16 = nullptr;
    } else if (dev_alloc(&m->w16b, layer_elems) != cudaSuccess) {
      cudaGetLastError();
      m->w16b = nullptr;
    }
  }
  // rotary table in double precision: angle = p * theta^(-2j/Dh)
  {
    const int half = c.head_dim / 2;
    std::vector<float2> tab(static_cast<size_t>(c.max_seq_len) * half);
    for (int j = 0; j < half; ++j) {
      const double inv = pow(static_cast<double>(c.rope_theta), -2.0 * j / c.head_dim);
      for (int p = 0; p < c.max_seq_len; ++p) {
        const double a = p * inv;
        tab[static_cast<size_t>(p) * half + j] = make_float2(static_cast<float>(cos(a)), static_cast<float>(sin(a)));
      }
    }
    e = cudaMemcpy(m->rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess) e = cudaMemset(m->status, 0, 16);
  if (e == cudaSuccess) e = cudaMemset(m->attn_scratch, 0, scratch_floats * sizeof(float));
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&m->side, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&m->cap, cudaStreamNonBlocking);
  m->ev.resize(2 * L + 1, nullptr);
  for (auto& ev : m->ev)
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
  m->ev_sq.resize(L + 1, nullptr);
  m->ev_sg.resize(L + 1, nullptr);
  m->ev_out.resize(2 * L, nullptr);
  m->ev_pf_out.resize(2 * L, nullptr);
  m->ev_pf_add.resize(2 * L, nullptr);
  for (auto* vec : {&m->ev_sq, &m->ev_sg, &m->ev_out, &m->ev_pf_out, &m->ev_pf_add})
    for (auto& ev : *vec)
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&m->xstream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_join, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_pf_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_lens, cudaEventDisableTiming);
  for (int i = 0; i < 2; ++i) {
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_w16_ready[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m->ev_w16_free[i], cudaEventDisableTiming);
  }
  if (e != cudaSuccess) {
    std::string msg = std::string("set-up: ") + cudaGetErrorString(e);
    ladder_destroy(m);
    return fail(nullptr, LADDER_ERR_CUDA, msg);
  }
  *out = m;
  return LADDER_OK;
}

ladder_status_t ladder_destroy(ladder_model_t* m) {
  if (!m) return LADDER_OK;
  drop_graph(m);
  for (auto ev : m->ev)
    if (ev) cudaEventDestroy(ev);
  for (auto* vec : {&m->ev_sq, &m->ev_sg, &m->ev_out, &m->ev_pf_out, &m->ev_pf_add})
    for (auto ev : *vec)
      if (ev) cudaEventDestroy(ev);
  if (m->xstream) cudaStreamDestroy(m->xstream);
  if (m->pend_pf[0]) cudaFree(m->pend_pf[0]);
  if (m->pend_pf[1]) cudaFree(m->pend_pf[1]);
  if (m->ev_fork) cudaEventDestroy(m->ev_fork);
  if (m->ev_join) cudaEventDestroy(m->ev_join);
  if (m->ev_pf_fork) cudaEventDestroy(m->ev_pf_fork);
  if (m->ev_lens) cudaEventDestroy(m->ev_lens);
  for (int i = 0; i < 2; ++i) {
    if (m->ev_w16_ready[i]) cudaEventDestroy(m->ev_w16_ready[i]);
    if (m->ev_w16_free[i]) cudaEventDestroy(m->ev_w16_free[i]);
  }
  if (m->side) cudaStreamDestroy(m->side);
  if (m->cap) cudaStreamDestroy(m->cap);
  void* bufs[] = {m->w16, m->w16b, m->wide_hpack, m->wide_opack, m->pend_a, m->pend_m, m->xpack[0], m->xpack[1], m->hpack, m->opack, m->d_phases, m->d_attn, m->d_counters, m->gemm_scratch[0], m->gemm_scratch[1], m->work_slots, m->R[0], m->R[1], m->q_f32, m->o_dec, m->h_dec, m->attn_scratch, m->logits_ws, m->last_x,
                  m->n_pf, m->q_pf,  m->o_pf,  m->h_pf,  m->rope,  m->status,       m->tok_tmp,   m->next_tmp};
  for (void* b : bufs)
    if (b) cudaFree(b);
  if (m->lens_tmp) cudaFree(m->lens_tmp);
  if (m->h_lens_pinned) cudaFreeHost(m->h_lens_pinned);
  delete m;
  return LADDER_OK;
}

ladder_status_t ladder_model_set_schedule(ladder_model_t* m, int32_t n_streams, int32_t use_graph, int32_t use_pdl) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (n_streams != 1 && n_streams != 2) return fail(m, LADDER_ERR_INVALID_ARG, "n_streams must be 1 or 2");
  m->n_streams = n_streams;
  m->use_graph = use_graph ? 1 : 0;
  m->use_pdl = use_pdl ? 1 : 0;
  drop_graph(m);
  return LADDER_OK;
}

ladder_status_t ladder_model_set_persistent(ladder_model_t* m, int32_t on) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  m->use_stack = on ? 1 : 0;
  m->persistent_explicit = on != 0;
  // 2: every layer in the persistent kernel, standard-residual ones included; 1: the default choice
  const int L = m->cfg.n_layers;
  m->stack_begin = on == 2 ? 0 : stack_default_begin(m->cfg, m->is_ladder);
  m->stack_ok = m->stack_usable && m->stack_begin < L;
  m->stack_built = false;
  return LADDER_OK;
}

ladder_status_t ladder_debug_stall_last_phase(ladder_model_t* m, int32_t on) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  m->stack_stall_test = on ? 1 : 0;
  m->stack_built = false;  // rebuild the phase list on the next step
  return LADDER_OK;
}

int32_t ladder_model_persistent_active(const ladder_model_t* m) {
  return (m && m->use_stack && m->stack_ok && !prefers_wide_small(m)) ? 1 : 0;
}

ladder_status_t ladder_model_set_exchange(ladder_model_t* m, ladder_exchange_fn fn, void* ctx, int32_t capturable) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (fn && (!m->pend_pf[0] || !m->pend_pf[1])) {
    const size_t n = static_cast<size_t>(m->cfg.max_prefill_tokens) * m->cfg.d_model;
    for (int i = 0; i < 2; ++i)
      if (!m->pend_pf[i] && dev_alloc(&m->pend_pf[i], n) != cudaSuccess) {
        cudaGetLastError();
        return fail(m, LADDER_ERR_OOM, "no room for the prompt pass's stored module outputs");
      }
  }
  m->exchange = fn;
  m->exchange_ctx = fn ? ctx : nullptr;
  m->exchange_capturable = (fn && capturable) ? 1 : 0;
  m->comm = nullptr;
  m->peer = nullptr;
  drop_graph(m);
  return LADDER_OK;
}

ladder_status_t ladder_model_set_tensor_parallel(ladder_model_t* m, ladder_comm_t* comm) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (!comm) return ladder_model_set_exchange(m, nullptr, nullptr, 0);
  const ladder_status_t s = ladder_model_set_exchange(m, ladder_comm_all_reduce_sum, comm, 1);
  if (s == LADDER_OK) m->comm = comm;
  return s;
}

ladder_status_t ladder_model_set_peer(ladder_model_t* m, ladder_peer_t* peer) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (peer) {
    if (!m->exchange) return fail(m, LADDER_ERR_STATE, "set the exchange of the prompt pass first");
    if (!ladder_peer_connected(peer) ||
        ladder_peer_max_floats(peer) < static_cast<int64_t>(m->cfg.max_batch) * m->cfg.d_model)
      return fail(m, LADDER_ERR_INVALID_ARG, "peer object not connected, or smaller than max_batch x d_model");
  }
  m->peer = peer;
  drop_graph(m);
  return LADDER_OK;
}

ladder_status_t ladder_model_set_tensor_parallel_peer(ladder_model_t* m, ladder_comm_t* comm, ladder_peer_t* peer) {
  if (!m || !comm || !peer) return LADDER_ERR_INVALID_ARG;
  if (ladder_peer_world(peer) != ladder_comm_world(comm) || ladder_peer_rank(peer) != ladder_comm_rank(comm))
    return fail(m, LADDER_ERR_INVALID_ARG, "peer object and communicator of different worlds");
  const ladder_status_t s = ladder_model_set_tensor_parallel(m, comm);
  return s == LADDER_OK ? ladder_model_set_peer(m, peer) : s;
}

ladder_status_t ladder_model_set_peer_max_bytes(ladder_model_t* m, int64_t bytes) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  m->peer_max_bytes = bytes;
  drop_graph(m);
  return LADDER_OK;
}

ladder_status_t ladder_debug_set_peer_hook(ladder_model_t* m, ladder_peer_hook_fn fn, void* ctx) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  m->peer_hook = fn;
  m->peer_hook_ctx = fn ? ctx : nullptr;
  drop_graph(m);
  return LADDER_OK;
}

ladder_status_t ladder_model_set_sm_split(ladder_model_t* m, int32_t sms_attention_stream) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (sms_attention_stream < -3 || sms_attention_stream > m->sm_count / 2)
    return fail(m, LADDER_ERR_INVALID_ARG, "sms_attention_stream must be -3 .. 0 or at most half the SMs");
  m->sms_a = sms_attention_stream;
  drop_graph(m);
  return LADDER_OK;
}

ladder_status_t ladder_set_position(ladder_model_t* m, int32_t len) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (len < 0 || len > m->cfg.max_seq_len) return fail(m, LADDER_ERR_INVALID_ARG, "length outside [0, max_seq_len]");
  m->host_len = len;
  m->timed_out = false;
  return LADDER_OK;
}

int64_t ladder_kernel_launches(const ladder_model_t* m) { return m ? m->launches : 0; }

int32_t ladder_stack_plan(const ladder_config_t* cfg, int32_t batch, int32_t sm_count, int32_t* out, int32_t cap) {
  if (!cfg || !out || cap < 4 || batch < 1 || sm_count < 1) return -1;
  if ((cfg->struct_size != sizeof(ladder_config_t) && cfg->struct_size != kConfigSizeV1) || check_shape(*cfg)) return -1;
  // a model object that owns nothing: every buffer is a distinct made-up address, never dereferenced
  ladder_model m;
  copy_config(&m.cfg, cfg);
  const int L = cfg->n_layers;
  if (parse_rules(cfg, &m)) return -1;
  m.sm_count = sm_count;
  m.attn_splits = decode_attention_splits(cfg->max_batch, cfg->n_kv_heads, cfg->max_seq_len, sm_count);
  uintptr_t next = 0x10000000u;
  auto fake = [&]() {
    next += 0x1000000u;
    return next;
  };
  m.R[0] = reinterpret_cast<float*>(fake());
  m.R[1] = reinterpret_cast<float*>(fake());
  m.q_f32 = reinterpret_cast<float*>(fake());
  m.o_dec = reinterpret_cast<float*>(fake());
  m.h_dec = reinterpret_cast<float*>(fake());
  m.attn_scratch = reinterpret_cast<float*>(fake());
  m.xpack[0] = reinterpret_cast<__nv_bfloat16*>(fake());
  m.xpack[1] = reinterpret_cast<__nv_bfloat16*>(fake());
  m.hpack = reinterpret_cast<__nv_bfloat16*>(fake());
  m.opack = reinterpret_cast<__nv_bfloat16*>(fake());
  m.status = reinterpret_cast<int32_t*>(fake());
  m.rope = reinterpret_cast<float2*>(fake());
  m.lm_head = reinterpret_cast<const __nv_bfloat16*>(fake());
  m.final_norm = reinterpret_cast<const __nv_bfloat16*>(fake());
  for (auto* v : {&m.attn_norm, &m.w_qkv, &m.w_o, &m.mlp_norm, &m.w_gate_up, &m.w_down}) {
    v->resize(L);
    for (int l = 0; l < L; ++l) (*v)[l] = reinterpret_cast<const __nv_bfloat16*>(fake());
  }
  ladder_kv_cache_t cache;
  cache.k = reinterpret_cast<void*>(fake() + 0x40000000u);
  cache.v = reinterpret_cast<void*>(fake() + 0x80000000u);
  cache.seq_lens = reinterpret_cast<int32_t*>(fake());
  std::vector<StackPhase> ph;
  std::vector<StackAttn> at;
  int nc = 0;
  const int begin = stack_default_begin(m.cfg, m.is_ladder);
  const bool ok = build_stack(&m, &cache, batch, reinterpret_cast<float*>(fake()), ph, at, &nc, begin);
  m.ev.clear();
  std::vector<int32_t> o = {static_cast<int32_t>(ph.size()), static_cast<int32_t>(at.size()), nc, begin, ok ? 1 : 0};
  for (const StackPhase& P : ph) {
    o.insert(o.end(), {P.kind, P.layer, P.p.N, P.K, P.n_units, P.n_static, P.n_claims, P.work_idx, P.done_idx, P.sched_n});
    for (int r = 0; r < kStackRounds; ++r) o.push_back(P.count[r]);
    for (int r = 0; r < kStackRounds; ++r) o.push_back(P.size[r]);
    o.push_back(P.n_act_deps);
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? P.act_dep[i] : 0);
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? P.act_need[i] : 0);
    o.push_back(P.n_epi_deps);
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? P.epi_dep[i] : 0);
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? P.epi_need[i] : 0);
  }
  int li = 0;
  for (const StackAttn& A : at) {
    o.insert(o.end(), {begin + li++, A.split_done, A.merge_done, A.n_deps});
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? A.dep[i] : 0);
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? A.need[i] : 0);
    o.push_back(A.n_mdeps);
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? A.mdep[i] : 0);
    for (int i = 0; i < 6; ++i) o.push_back(i < kStackMaxDeps ? A.mneed[i] : 0);
  }
  if (static_cast<int>(o.size()) > cap) return -static_cast<int32_t>(o.size());
  memcpy(out, o.data(), o.size() * sizeof(int32_t));
  return static_cast<int32_t>(o.size());
}

ladder_status_t ladder_device_status(ladder_model_t* m, int32_t* flags, void* cuda_stream) {
  if (!m || !flags) return LADDER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CK(m, cudaStreamSynchronize(st));
  CK(m, cudaMemcpy(flags, m->status, sizeof(int32_t), cudaMemcpyDeviceToHost));
  CK(m, cudaMemset(m->status, 0, sizeof(int32_t)));
  if (*flags & LADDER_DEV_TIMEOUT) {
    m->timed_out = true;
    return fail(m, LADDER_ERR_TIMEOUT, "a wait inside the persistent decode kernel gave up: that step produced nothing; "
                                        "call ladder_set_position or ladder_prefill to continue");
  }
  return LADDER_OK;
}

static ladder_status_t check_call(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* tokens, int batch,
                                  bool rearm = false) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (m->sticky_cuda) return fail(m, LADDER_ERR_CUDA, "an earlier CUDA call failed: " + m->err);
  if (rearm) m->timed_out = false;
  if (m->timed_out)
    return fail(m, LADDER_ERR_TIMEOUT, "an earlier step timed out on the device; call ladder_set_position or ladder_prefill");
  if (!cache || !cache->k || !cache->v || !cache->seq_lens || (!tokens && !m->st_in.newest))
    return fail(m, LADDER_ERR_INVALID_ARG, "NULL argument");
  if ((reinterpret_cast<uintptr_t>(cache->k) | reinterpret_cast<uintptr_t>(cache->v)) & 15)
    return fail(m, LADDER_ERR_INVALID_ARG, "cache buffers must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(cache->seq_lens) | reinterpret_cast<uintptr_t>(tokens)) & 3)
    return fail(m, LADDER_ERR_INVALID_ARG, "seq_lens / token buffers must be 4-byte aligned");
  if (batch < 1) return fail(m, LADDER_ERR_INVALID_ARG, "batch must be >= 1");
  if (batch > m->cfg.max_batch) return fail(m, LADDER_ERR_STATE, "batch exceeds max_batch");
  return LADDER_OK;
}

ladder_status_t ladder_prefill(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens, int32_t batch,
                               int32_t seq_len, const ladder_outputs_t* out, void* cuda_stream) {
  ladder_status_t s = check_call(m, cache, d_tokens, batch, /*rearm=*/true);
  if (s != LADDER_OK) return s;
  if (seq_len < 1) return fail(m, LADDER_ERR_INVALID_ARG, "seq_len must be >= 1");
  if (seq_len > m->cfg.max_seq_len) return fail(m, LADDER_ERR_STATE, "seq_len exceeds max_seq_len");
  if (static_cast<int64_t>(batch) * seq_len > m->cfg.max_prefill_tokens)
    return fail(m, LADDER_ERR_STATE, "batch*seq_len exceeds max_prefill_tokens");
  int64_t k = 0;
  CK(m, enqueue_prefill(m, cache, d_tokens, batch, seq_len, out, static_cast<cudaStream_t>(cuda_stream), &k));
  m->launches += k;
  m->host_len = seq_len;
  return LADDER_OK;
}

ladder_status_t ladder_prefill_ragged(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                      const int32_t* h_lens, int32_t batch, int32_t seq_len, const ladder_outputs_t* out,
                                      void* cuda_stream) {
  ladder_status_t s = check_call(m, cache, d_tokens, batch, /*rearm=*/true);
  if (s != LADDER_OK) return s;
  if (!h_lens) return fail(m, LADDER_ERR_INVALID_ARG, "NULL lengths");
  if (seq_len < 1) return fail(m, LADDER_ERR_INVALID_ARG, "seq_len must be >= 1");
  if (seq_len > m->cfg.max_seq_len) return fail(m, LADDER_ERR_STATE, "seq_len exceeds max_seq_len");
  if (static_cast<int64_t>(batch) * seq_len > m->cfg.max_prefill_tokens)
    return fail(m, LADDER_ERR_STATE, "batch*seq_len exceeds max_prefill_tokens");
  int longest = 0;
  for (int b = 0; b < batch; ++b) {
    if (h_lens[b] < 1 || h_lens[b] > seq_len) return fail(m, LADDER_ERR_INVALID_ARG, "a length outside [1, seq_len]");
    longest = std::max(longest, h_lens[b]);
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the lengths go to the device through a small pinned staging buffer of the model, so that the copy is
  // stream-ordered and h_lens may be reused by the caller as soon as this call returns
  CK(m, cudaEventSynchronize(m->ev_lens));  // the previous call's copy out of the staging buffer has run (usually long ago)
  memcpy(m->h_lens_pinned, h_lens, static_cast<size_t>(batch) * sizeof(int32_t));
  CK(m, cudaMemcpyAsync(m->lens_tmp, m->h_lens_pinned, static_cast<size_t>(batch) * sizeof(int32_t),
                        cudaMemcpyHostToDevice, st));
  CK(m, cudaEventRecord(m->ev_lens, st));
  int64_t k = 0;
  CK(m, enqueue_prefill(m, cache, d_tokens, batch, seq_len, out, st, &k, 0, m->lens_tmp));
  m->launches += k;
  m->host_len = longest;
  return LADDER_OK;
}

// ---- pipeline stages (paper Sec. 5.1)
namespace {
struct StageScope {  // sets the stage state for one call and clears it again
  ladder_model* m;
  StageScope(ladder_model* mm, const ladder_stream_state_t* in, const ladder_stream_state_t* out) : m(mm) {
    if (in) m->st_in = *in;
    if (out) m->st_out = *out;
  }
  ~StageScope() {
    m->st_in = {nullptr, nullptr};
    m->st_out = {nullptr, nullptr};
  }
};
const char* check_stage(const ladder_stream_state_t* in, const ladder_stream_state_t* out, const int32_t* tokens) {
  if (in && !in->newest) return "state_in without its newest buffer";
  if (out && !out->newest) return "state_out without its newest buffer";
  if (!in && !tokens) return "a first stage needs tokens";
  const uintptr_t a = (in ? reinterpret_cast<uintptr_t>(in->newest) | reinterpret_cast<uintptr_t>(in->older) : 0) |
                      (out ? reinterpret_cast<uintptr_t>(out->newest) | reinterpret_cast<uintptr_t>(out->older) : 0);
  return (a & 15) ? "stream-state buffers must be 16-byte aligned" : nullptr;
}
}  // namespace

ladder_status_t ladder_stage_prefill(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                     const ladder_stream_state_t* state_in, int32_t batch, int32_t seq_len,
                                     const ladder_stream_state_t* state_out, const ladder_outputs_t* out,
                                     void* cuda_stream) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (const char* why = check_stage(state_in, state_out, d_tokens)) return fail(m, LADDER_ERR_INVALID_ARG, why);
  if (state_out && out && out->all_hidden) return fail(m, LADDER_ERR_INVALID_ARG, "a stage that hands its state on has no head outputs");
  StageScope scope(m, state_in, state_out);
  return ladder_prefill(m, cache, d_tokens, batch, seq_len, out, cuda_stream);
}

ladder_status_t ladder_stage_decode_step(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                         const ladder_stream_state_t* state_in, int32_t batch,
                                         const ladder_stream_state_t* state_out, const ladder_outputs_t* out,
                                         void* cuda_stream) {
  if (!m) return LADDER_ERR_INVALID_ARG;
  if (const char* why = check_stage(state_in, state_out, d_tokens)) return fail(m, LADDER_ERR_INVALID_ARG, why);
  StageScope scope(m, state_in, state_out);
  return ladder_decode_step(m, cache, d_tokens, batch, out, cuda_stream);
}

ladder_status_t ladder_prefill_append(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                      int32_t batch, int32_t seq_len, const ladder_outputs_t* out, void* cuda_stream) {
  ladder_status_t s = check_call(m, cache, d_tokens, batch);
  if (s != LADDER_OK) return s;
  if (seq_len < 1) return fail(m, LADDER_ERR_INVALID_ARG, "seq_len must be >= 1");
  const int pos0 = m->host_len;
  if (static_cast<int64_t>(pos0) + seq_len > m->cfg.max_seq_len)
    return fail(m, LADDER_ERR_STATE, "cached length + seq_len exceeds max_seq_len");
  if (static_cast<int64_t>(batch) * seq_len > m->cfg.max_prefill_tokens)
    return fail(m, LADDER_ERR_STATE, "batch*seq_len exceeds max_prefill_tokens");
  int64_t k = 0;
  CK(m, enqueue_prefill(m, cache, d_tokens, batch, seq_len, out, static_cast<cudaStream_t>(cuda_stream), &k, pos0));
  m->launches += k;
  m->host_len = pos0 + seq_len;
  return LADDER_OK;
}

ladder_status_t ladder_decode_step(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* d_tokens,
                                   int32_t batch, const ladder_outputs_t* out, void* cuda_stream) {
  ladder_status_t s = check_call(m, cache, d_tokens, batch);
  if (s != LADDER_OK) return s;
  if (m->host_len + 1 > m->cfg.max_seq_len) return fail(m, LADDER_ERR_STATE, "KV cache is full");
  if (out && out->all_hidden) return fail(m, LADDER_ERR_INVALID_ARG, "all_hidden is a prefill-only output");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool two = m->n_streams == 2;

  const bool staged = m->st_in.newest || m->st_out.newest;  // a pipeline stage runs kernel by kernel
  if (m->use_stack && m->stack_ok && batch <= 4 && !staged && !m->exchange && !prefers_wide_small(m)) {
    GraphKey key;
    key.batch = batch;
    key.k = cache->k;
    key.v = cache->v;
    key.lens = cache->seq_lens;
    key.o_logits = out ? out->logits : nullptr;
    if (!m->stack_built || !(key == m->stack_key)) {
      std::vector<StackPhase> ph;
      std::vector<StackAttn> at;
      int nc = 0;
      float* logits = (out && out->logits) ? out->logits : m->logits_ws;
      if (!build_stack(m, cache, batch, logits, ph, at, &nc, m->stack_begin) || nc > m->cap_counters ||
          static_cast<int>(ph.size()) > 4 * m->cfg.n_layers + 1 || static_cast<int>(at.size()) > m->cfg.n_layers) {
        m->stack_ok = false;  // not expressible: use the multi-kernel schedule from now on
      } else {
        // the previous step may still be reading the old lists
        CK(m, cudaStreamSynchronize(st));
        CK(m, cudaMemcpy(m->d_phases, ph.data(), ph.size() * sizeof(StackPhase), cudaMemcpyHostToDevice));
        CK(m, cudaMemcpy(m->d_attn, at.data(), at.size() * sizeof(StackAttn), cudaMemcpyHostToDevice));
        m->n_phases = static_cast<int>(ph.size());
        m->n_attn = static_cast<int>(at.size());
        m->n_counters = nc;
        m->stack_key = key;
        m->stack_built = true;
      }
    }
    if (m->stack_ok) {
      int64_t k = 0;
      CK(m, enqueue_decode_stack(m, cache, d_tokens, batch, out, st, &k));
      m->launches += k;
      m->host_len += 1;
      return LADDER_OK;
    }
  }

  // a graph only if everything the step calls back into may be captured (with a peer object the step calls nothing)
  const bool fused = peer_fused(m, batch);
  if (!m->use_graph || (m->exchange && !fused && !m->exchange_capturable) || (fused && m->peer_hook)) {
    int64_t k = 0;
    if (two) {
      // the side stream may only start after everything already queued on the caller's stream
      CK(m, cudaEventRecord(m->ev_fork, st));
      CK(m, cudaStreamWaitEvent(m->side, m->ev_fork, 0));
    }
    CK(m, enqueue_decode(m, cache, d_tokens, batch, out, st, two ? m->side : st, &k));
    m->launches += k;
  } else {
    GraphKey key;
    key.batch = batch;
    key.n_streams = m->n_streams;
    key.pdl = m->use_pdl;
    key.k = cache->k;
    key.v = cache->v;
    key.lens = cache->seq_lens;
    key.tok = d_tokens;
    key.o_next = out ? out->next_tokens : nullptr;
    key.o_hid = out ? out->final_hidden : nullptr;
    key.o_logits = out ? out->logits : nullptr;
    key.s_in0 = m->st_in.newest;
    key.s_in1 = m->st_in.older;
    key.s_out0 = m->st_out.newest;
    key.s_out1 = m->st_out.older;
    if (!m->graph_exec || !(key == m->graph_key)) {
      drop_graph(m);
      for (int attempt = 0; attempt < 2 && !m->graph_exec; ++attempt) {
        cudaGraph_t graph = nullptr;
        int64_t k = 0;
        CK(m, cudaStreamBeginCapture(m->cap, cudaStreamCaptureModeRelaxed));
        cudaError_t e = enqueue_decode(m, cache, d_tokens, batch, out, m->cap, two ? m->side : m->cap, &k);
        cudaError_t e2 = cudaStreamEndCapture(m->cap, &graph);
        if (e == cudaSuccess) e = e2;
        if (e == cudaSuccess) e = cudaGraphInstantiate(&m->graph_exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
        if (e != cudaSuccess) {
          cudaGetLastError();
          m->graph_exec = nullptr;
          if (attempt == 0 && m->use_pdl) {  // retry once without programmatic edges
            m->use_pdl = 0;
            key.pdl = 0;
            continue;
          }
          m->sticky_cuda = true;
          return fail(m, LADDER_ERR_CUDA, std::string("graph capture: ") + cudaGetErrorString(e));
        }
        m->graph_kernels = k;
      }
      m->graph_key = key;
    }
    CK(m, cudaGraphLaunch(m->graph_exec, st));
    m->launches += m->graph_kernels;
  }
  m->host_len += 1;
  return LADDER_OK;
}

ladder_status_t ladder_decode_step_host(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* h_tokens,
                                        int32_t batch, int32_t* h_next_tokens, void* cuda_stream) {
  if (!m || !h_tokens || !h_next_tokens) return LADDER_ERR_INVALID_ARG;
  if (batch < 1 || batch > m->cfg.max_batch) return fail(m, LADDER_ERR_STATE, "batch outside [1, max_batch]");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CK(m, cudaMemcpyAsync(m->tok_tmp, h_tokens, batch * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  ladder_outputs_t out = {};
  out.next_tokens = m->next_tmp;
  ladder_status_t s = ladder_decode_step(m, cache, m->tok_tmp, batch, &out, cuda_stream);
  if (s != LADDER_OK) return s;
  CK(m, cudaMemcpyAsync(h_next_tokens, m->next_tmp, batch * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CK(m, cudaStreamSynchronize(st));
  return LADDER_OK;
}

ladder_status_t ladder_prefill_host(ladder_model_t* m, const ladder_kv_cache_t* cache, const int32_t* h_tokens,
                                    int32_t batch, int32_t seq_len, int32_t* h_next_tokens, void* cuda_stream) {
  if (!m || !h_tokens || !h_next_tokens) return LADDER_ERR_INVALID_ARG;
  if (batch < 1 || batch > m->cfg.max_batch) return fail(m, LADDER_ERR_STATE, "batch outside [1, max_batch]");
  if (seq_len < 1 || static_cast<int64_t>(batch) * seq_len > m->cfg.max_prefill_tokens)
    return fail(m, LADDER_ERR_STATE, "batch*seq_len outside [1, max_prefill_tokens]");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CK(m, cudaMemcpyAsync(m->tok_tmp, h_tokens, static_cast<size_t>(batch) * seq_len * sizeof(int32_t),
                        cudaMemcpyHostToDevice, st));
  ladder_outputs_t out = {};
  out.next_tokens = m->next_tmp;
  ladder_status_t s = ladder_prefill(m, cache, m->tok_tmp, batch, seq_len, &out, cuda_stream);
  if (s != LADDER_OK) return s;
  CK(m, cudaMemcpyAsync(h_next_tokens, m->next_tmp, batch * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CK(m, cudaStreamSynchronize(st));
  return LADDER_OK;
}

// --------------------------------------------------------------------------- single-kernel entry points
static int g_sm_count = 0;
static int sm_count_cached() {
  if (!g_sm_count) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess)
      g_sm_count = n;
  }
  return g_sm_count > 0 ? g_sm_count : 148;
}

// Library-owned scratch of the single-kernel GEMM entry point (grown on demand; one per process, so
// calls of that entry point must not overlap on the device).
static float* g_op_scratch = nullptr;
static size_t g_op_scratch_floats = 0;
static int32_t* g_op_work = nullptr;
static int g_op_serial = 0;
static cudaError_t op_scratch(size_t floats) {
  if (!g_op_work) {
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&g_op_work), 2 * 256 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(g_op_work, 0, 2 * 256 * sizeof(int32_t));
    if (e != cudaSuccess) return e;
  }
  if (floats <= g_op_scratch_floats) return cudaSuccess;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return e;
  if (g_op_scratch) cudaFree(g_op_scratch);
  g_op_scratch = nullptr;
  g_op_scratch_floats = 0;
  e = cudaMalloc(reinterpret_cast<void**>(&g_op_scratch), floats * sizeof(float));
  if (e == cudaSuccess) e = cudaMemset(g_op_scratch, 0, floats * sizeof(float));
  if (e == cudaSuccess) g_op_scratch_floats = floats;
  return e;
}

ladder_status_t ladder_op_smallm_gemm(const void* W, int32_t N, int32_t K, const void* act, int32_t act_mode,
                                      const void* gain, float eps, int32_t batch, int32_t epi_mode, const float* addend,
                                      void* out, void* cuda_stream) {
  if (!W || !act || !out || N < 8 || K < 8 || (N % 8) || (K % 8) || batch < 1 || batch > 64) return LADDER_ERR_INVALID_ARG;
  if (act_mode != ACT_F32 && act_mode != ACT_F32_NORM) return LADDER_ERR_INVALID_ARG;
  if (act_mode == ACT_F32_NORM && !gain) return LADDER_ERR_INVALID_ARG;
  if (epi_mode != EPI_RESID && epi_mode != EPI_SWIGLU && epi_mode != EPI_PLAIN) return LADDER_ERR_INVALID_ARG;
  if (epi_mode == EPI_RESID && !addend) return LADDER_ERR_INVALID_ARG;
  SmallMParams p = {};
  p.W = static_cast<const __nv_bfloat16*>(W);
  p.N = N;
  p.K = K;
  p.act = act;
  p.act_mode = act_mode;
  p.gain = static_cast<const __nv_bfloat16*>(gain);
  p.eps = eps;
  p.batch = batch;
  p.epi_mode = epi_mode;
  p.addend = addend;
  p.out = out;
  if (kernels_ready() != cudaSuccess) return LADDER_ERR_CUDA;
  if (op_scratch(smallm_gemm_scratch_floats(N, K, batch) + 64) != cudaSuccess) return LADDER_ERR_OOM;
  p.scratch = g_op_scratch;
  p.work = g_op_work + 2 * (g_op_serial++ & 255);
  cudaError_t e = launch_smallm_gemm(p, static_cast<cudaStream_t>(cuda_stream), false, sm_count_cached());
  return e == cudaSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

static int op_attn_splits(int batch, int n_kv_heads, int max_seq_len) {
  return decode_attention_splits(batch, n_kv_heads, max_seq_len, sm_count_cached());
}

size_t ladder_decode_attention_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim, int32_t max_seq_len) {
  if (batch < 1 || n_q_heads < 1 || max_seq_len < 1) return 0;
  // sized for the finest split any kv-head count can ask for (n_kv_heads = 1 gives the most splits)
  const int splits = op_attn_splits(batch, 1, max_seq_len);
  return decode_attention_scratch_floats(batch, n_q_heads, head_dim, splits) * sizeof(float);
}

ladder_status_t ladder_op_decode_attention(const float* q, const void* k, const void* v, const int32_t* kv_len,
                                           int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                           int32_t max_seq_len, float* scratch, void* o, void* cuda_stream) {
  if (!q || !k || !v || !kv_len || !scratch || !o) return LADDER_ERR_INVALID_ARG;
  if (batch < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || (head_dim != 64 && head_dim != 128) || max_seq_len < 1)
    return LADDER_ERR_INVALID_ARG;
  if (decode_attention_misaligned(q, k, v, o, scratch, kv_len)) return LADDER_ERR_INVALID_ARG;
  if (max_seq_len > kDecodeAttnMaxKeys) return LADDER_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DecodeAttnParams a = {};
  a.q = q;
  a.k = static_cast<const kv_t*>(k);
  a.v = static_cast<const kv_t*>(v);
  a.kv_len = kv_len;
  a.kv_len_offset = 0;
  a.batch = batch;
  a.n_q_heads = n_q_heads;
  a.n_kv_heads = n_kv_heads;
  a.head_dim = head_dim;
  a.max_seq_len = max_seq_len;
  a.max_len = max_seq_len;
  a.n_splits = op_attn_splits(batch, n_kv_heads, max_seq_len);
  a.scratch = scratch;
  a.o = static_cast<float*>(o);
  return launch_decode_attention(a, st, false) == cudaSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

ladder_status_t ladder_op_prefill_gemm(const void* A, const void* A_lo, const void* W, int32_t M, int32_t N, int32_t K,
                                       int32_t epi_mode, const float* addend, void* out, void* out_lo,
                                       void* cuda_stream) {
  if (!A || !W || !out || M < 1 || N < 8 || K < 8 || (N % 8) || (K % 8)) return LADDER_ERR_INVALID_ARG;
  int mode;
  switch (epi_mode) {
    case 0: mode = EPI_RESID; break;
    case 1: mode = EPI_SWIGLU; break;
    case 2: mode = EPI_PLAIN; break;
    case 3: mode = EPI_BF16; break;
    default: return LADDER_ERR_INVALID_ARG;
  }
  if (mode == EPI_RESID && !addend) return LADDER_ERR_INVALID_ARG;
  LargeMParams p = {};
  p.A = static_cast<const __nv_bfloat16*>(A);
  p.A_lo = static_cast<const __nv_bfloat16*>(A_lo);
  p.out_lo = static_cast<__nv_bfloat16*>(out_lo);
  p.W = static_cast<const __nv_bfloat16*>(W);
  p.M = M;
  p.N = N;
  p.K = K;
  p.epi_mode = mode;
  p.addend = addend;
  p.out = out;
  if (kernels_ready() != cudaSuccess) return LADDER_ERR_CUDA;
  return launch_largem_gemm(p, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

ladder_status_t ladder_op_convert_bf16_f16(const void* src, void* dst, int64_t n, void* cuda_stream) {
  if (!src || !dst || n < 8 || (n % 8)) return LADDER_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) return LADDER_ERR_INVALID_ARG;
  return launch_convert_bf16_f16(static_cast<const __nv_bfloat16*>(src), static_cast<__half*>(dst),
                                 static_cast<size_t>(n), static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
             ? LADDER_OK
             : LADDER_ERR_CUDA;
}

ladder_status_t ladder_op_prefill_gemm_f16(const void* A, const void* W, int32_t M, int32_t N, int32_t K, int32_t epi_mode,
                                           const float* addend, void* out, void* cuda_stream) {
  if (!A || !W || !out || M < 1 || N < 8 || K < 8 || (N % 8) || (K % 8)) return LADDER_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(W) | reinterpret_cast<uintptr_t>(out)) & 15)
    return LADDER_ERR_INVALID_ARG;
  int mode;
  switch (epi_mode) {
    case 0: mode = EPI_RESID; break;
    case 1: mode = EPI_SWIGLU; break;
    case 2: mode = EPI_PLAIN; break;
    case 3: mode = EPI_BF16; break;
    default: return LADDER_ERR_INVALID_ARG;
  }
  if (mode == EPI_RESID && !addend) return LADDER_ERR_INVALID_ARG;
  LargeMParams p = {};
  p.A = static_cast<const __nv_bfloat16*>(A);
  p.W = static_cast<const __nv_bfloat16*>(W);
  p.f16 = 1;
  p.M = M;
  p.N = N;
  p.K = K;
  p.epi_mode = mode;
  p.addend = addend;
  p.out = out;
  if (kernels_ready() != cudaSuccess) return LADDER_ERR_CUDA;
  return launch_largem_gemm(p, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

ladder_status_t ladder_op_prefill_attention(const void* q, const void* q_lo, const void* k, const void* v, int32_t batch,
                                            int32_t seq_len, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                            int32_t max_seq_len, void* o, void* o_lo, void* cuda_stream) {
  if (!q || !k || !v || !o || batch < 1 || seq_len < 1 || seq_len > max_seq_len || n_kv_heads < 1 ||
      n_q_heads % n_kv_heads || (head_dim != 64 && head_dim != 128))
    return LADDER_ERR_INVALID_ARG;
  if (kernels_ready() != cudaSuccess) return LADDER_ERR_CUDA;
  if ((q_lo == nullptr) != (o_lo == nullptr)) return LADDER_ERR_INVALID_ARG;
  cudaError_t e = launch_prefill_attention(
      static_cast<const __half*>(q), static_cast<const __half*>(q_lo), static_cast<const kv_t*>(k),
      static_cast<const kv_t*>(v), batch, seq_len, n_q_heads, n_kv_heads, head_dim, max_seq_len,
      static_cast<__nv_bfloat16*>(o), static_cast<__nv_bfloat16*>(o_lo), static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

ladder_status_t ladder_op_prefill_attention_at(const void* q, const void* q_lo, const void* k, const void* v,
                                               int32_t batch, int32_t seq_len, int32_t n_q_heads, int32_t n_kv_heads,
                                               int32_t head_dim, int32_t max_seq_len, int32_t pos0, const int32_t* lens,
                                               int32_t out_binary16, void* o, void* o_lo, void* cuda_stream) {
  if (!q || !k || !v || !o || batch < 1 || seq_len < 1 || pos0 < 0 || seq_len > max_seq_len - pos0 || n_kv_heads < 1 ||
      n_q_heads < 1 || n_q_heads % n_kv_heads || (head_dim != 64 && head_dim != 128))
    return LADDER_ERR_INVALID_ARG;
  if (out_binary16 ? o_lo != nullptr : (q_lo == nullptr) != (o_lo == nullptr)) return LADDER_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(q_lo) | reinterpret_cast<uintptr_t>(k) |
       reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(o) | reinterpret_cast<uintptr_t>(o_lo)) & 15)
    return LADDER_ERR_INVALID_ARG;
  if (kernels_ready() != cudaSuccess) return LADDER_ERR_CUDA;
  cudaError_t e = launch_prefill_attention(
      static_cast<const __half*>(q), static_cast<const __half*>(q_lo), static_cast<const kv_t*>(k),
      static_cast<const kv_t*>(v), batch, seq_len, n_q_heads, n_kv_heads, head_dim, max_seq_len,
      static_cast<__nv_bfloat16*>(o), static_cast<__nv_bfloat16*>(o_lo), static_cast<cudaStream_t>(cuda_stream), pos0,
      out_binary16 != 0, lens);
  return e == cudaSuccess ? LADDER_OK : LADDER_ERR_CUDA;
}

}  // extern "C"
