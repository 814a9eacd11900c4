// Host-side launch interface of the kernels (internal to libladder; no torch types).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "decode_schedule.h"
#include "peer_layout.cuh"

namespace ladder {

// Element type of the KV cache: IEEE binary16.  Keys and values of a normalised-input projection are O(1), far inside
// its range, and its 11 significant bits (bf16: 8) are what keeps the hidden-state error of deep models in bound.
typedef __half kv_t;

// Tensor parallelism over peer memory (tcgen05 decode GEMM and its staging launch; layout in peer_layout.cuh).
// push_channel = channel + 1 (EPI_PLAIN GEMM): every output element is stored into receive slot
// [channel][turn & 1][this rank] of EVERY rank instead of p.out, and each CTA counts its arrival on every rank when
// it is done.  pull_channel[i] = channel + 1 (staging step): pending i is the rank-order sum of this rank's receive
// slots of that channel, read after the ranks' arrival counters have reached this rank's own (bounded wait); the
// staging launch then moves the channel on.  act_pending / act_pending2 are ignored for a pulled pending.
struct WidePeer {
  PeerView peer;
  int push_channel;
  int pull_channel[2];
};

}  // namespace ladder
struct ladder_peer;
namespace ladder {
// The addresses of a connected peer-exchange object (peer_exchange.cu); false if it is not connected.
bool peer_view(const ladder_peer* p, PeerView* out);

enum ActMode { ACT_F32 = 0, ACT_F32_NORM = 1 };  // activations are fp32 [batch, K]; NORM applies RMSNorm
enum EpiMode { EPI_RESID = 0, EPI_SWIGLU = 1, EPI_PLAIN = 2, EPI_QKV_ROPE = 3, EPI_BF16 = 4 };

// Rotary / KV-append epilogue description shared by the decode and prefill QKV projections.
struct QkvEpilogue {
  float* q_out_f32;            // decode: fp32 [batch, Hq*Dh]
  __half* q_out_f16;           // prefill: binary16 [M, Hq*Dh] (hi part; the attention's MMA operand type)
  __half* q_out_lo;            // prefill: lo part (q ~ hi + lo), may be NULL
  kv_t* k_cache;               // one layer: [max_batch][Hkv][max_seq][Dh]
  kv_t* v_cache;
  const int32_t* seq_lens;     // decode: position of row b = seq_lens[b]; prefill: NULL (position = m % seq_len)
  const float2* rope;          // [max_seq][Dh/2] (cos, sin)
  int n_q_heads, n_kv_heads, head_dim, max_seq_len;
  int prefill_seq_len;         // prefill: rows are [batch, seq_len] flattened
  int prefill_pos0;            // prefill: position of a sequence's first row (> 0 when a prompt is continued)
  const int32_t* prefill_lens; // prefill, optional (device, [batch]): sequence b has only prefill_lens[b] valid rows;
                               // keys / values of the padding rows behind them are not stored
};

struct SmallMParams {
  const __nv_bfloat16* W;  // [N, K]
  int N, K;
  const void* act;         // fp32 [batch, K]
  int act_mode;
  const __nv_bfloat16* gain;  // [K] (ACT_F32_NORM)
  float eps;
  int batch;
  int epi_mode;
  const float* addend;     // EPI_RESID: fp32 [batch, N]
  void* out;               // EPI_RESID / EPI_PLAIN: fp32 [batch, N]; EPI_SWIGLU: fp32 [batch, N/2]
  QkvEpilogue qkv;         // EPI_QKV_ROPE
  int32_t* status;         // device status word (may be NULL)
  // batch 9..64 (tcgen05 kernel): operands handed from kernel to kernel without a staging launch.
  //   wide_pack_out: EPI_SWIGLU also writes its output as the next GEMM's staged operand, bf16 [2 Bp, N / 2]
  //                  (hi parts in rows 0..Bp-1, lo parts in rows Bp..2Bp-1, rows of sequences >= batch zero);
  //   act_staged:    this GEMM's activations are already staged that way ([2 Bp, K]; act_mode ACT_F32 only).
  __nv_bfloat16* wide_pack_out;
  const __nv_bfloat16* act_staged;
  // The pending-output form of Algorithm 1 (tcgen05 kernel): the staging step first forms
  // y = act + act_pending + act_pending2 (module outputs that were stored, not added; in that order) and, if
  // act_sum_out is given, writes y there (the residual stream moves on in the staging step instead of in a GEMM
  // epilogue).  wide_prestaged: the staging for this GEMM has already been launched with
  // launch_smallm_gemm_stage on the same scratch; the GEMM does not repeat it.  force_wide: the tcgen05 kernel
  // at batch <= 4 too (it is the one that knows this form).
  const float* act_pending;
  const float* act_pending2;
  float* act_sum_out;
  int wide_prestaged;
  int force_wide;
  const WidePeer* wide_peer;  // tensor parallelism over peer memory (HOST pointer, read while launching), or NULL
  // Optional second copy of an fp32 output (EPI_RESID: out, EPI_SWIGLU: h) as the next GEMM's MMA operand:
  // y = value (* pack_gain[n]), bf16 hi at [n / 2048][b][n % 2048], lo at [n / 2048][4 + b][n % 2048]; batch <= 4.
  __nv_bfloat16* pack_out;
  const __nv_bfloat16* pack_gain;
  float* scratch;          // smallm_gemm_scratch_floats(N, K, batch) floats, zero at first use (batch 9..64: staged
                           // activations, tickets and shared-tile pieces); kernels that may run concurrently
                           // need distinct scratch
  int32_t* work;           // batch <= 8: 2 ints, zero: claim counter + finished-CTA counter of THIS launch (left zero)
};

cudaError_t launch_smallm_gemm(const SmallMParams& p, cudaStream_t stream, bool pdl, int sm_count);
// tcgen05 kernel only (batch > 4 or force_wide): the staging launch of a GEMM on its own (p.act, p.act_pending,
// p.act_pending2, p.act_sum_out, p.gain, p.act_mode, p.K, p.batch, p.scratch), so that an event can sit between it
// and the GEMM.
cudaError_t launch_smallm_gemm_stage(const SmallMParams& p, cudaStream_t stream, bool pdl);
size_t smallm_gemm_smem_bytes(int batch);
size_t smallm_gemm_scratch_floats(int N, int K, int batch);
void set_decode_wide_impl(int impl);  // 0 = tcgen05 kernel for batch 5..64 (default), 2 = for every batch

// Decode attention (split over the cache) and its combine step.
struct DecodeAttnParams {
  const float* q;               // [batch, Hq*Dh]
  const kv_t* k;                // one layer
  const kv_t* v;
  const int32_t* kv_len;        // [batch]
  int kv_len_offset;            // keys attended = kv_len[b] + kv_len_offset (decode passes seq_lens and 1)
  int batch, n_q_heads, n_kv_heads, head_dim, max_seq_len;
  int n_splits;                 // CTAs per (b, kv head); each covers ceil(max_len / n_splits) keys
  int max_len;                  // host upper bound on keys attended (sizes the split)
  float* scratch;               // [batch][Hq][n_splits][Dh + 2]
  float* o;                     // [batch, Hq*Dh]
  __nv_bfloat16* o_pack;        // optional: o also as a staged GEMM operand, bf16 [2 o_pack_bp, Hq*Dh] (hi rows, lo rows)
  int o_pack_bp;                // padded batch of that operand (16 / 32 / 64); rows batch..bp-1 are written as zero
  int32_t* status;              // optional device status word (the TMA / tcgen05 kernel of batch > 8 reports timeouts)
};
int wide_padded_batch(int batch);  // Bp of the batch 9..64 GEMM kernel
int decode_attention_splits(int batch, int n_kv_heads, int max_len, int sm_count);
// Longest cache the decode attention handles: its merge step holds one weight per 64-key split, at most 1024.
constexpr int kDecodeAttnMaxKeys = 64 * 1024;
// The kernels read q / o / scratch with 16-byte and K / V with 16-byte vector loads: true when any pointer is not
// aligned for them (the caller then gets an argument error instead of a misaligned-address fault on the device).
inline bool decode_attention_misaligned(const void* q, const void* k, const void* v, const void* o, const void* scratch,
                                        const void* kv_len) {
  const uintptr_t a = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
                      reinterpret_cast<uintptr_t>(o) | reinterpret_cast<uintptr_t>(scratch);
  return (a & 15) != 0 || (reinterpret_cast<uintptr_t>(kv_len) & 3) != 0;
}
size_t decode_attention_scratch_floats(int batch, int n_q_heads, int head_dim, int n_splits);
cudaError_t launch_decode_attention(const DecodeAttnParams& p, cudaStream_t stream, bool pdl);
// Batch > 8 at head_dim 128: the split step on TMA + tcgen05 (decode_attention_tc.cu), one partial per 128 keys.
cudaError_t decode_attention_tc_init();
bool decode_attention_tc_usable(const DecodeAttnParams& p);
cudaError_t launch_decode_attention_tc(const DecodeAttnParams& p, int n_tiles, int32_t* status, cudaStream_t stream,
                                       bool pdl);
void set_decode_attention_impl(int impl);  // 0 = default (TMA / tcgen05 kernel for batch > 8 and >= 2048 tiles), 1 = register-fragment
                                           // kernel always, 2 = TMA / tcgen05 kernel wherever its shapes allow (batch > 8)

// Persistent layer-stack kernel of the decode step: every weight-streaming GEMM of the step is a
// "phase" of ONE cooperative launch, attention runs on dedicated warps of the same CTAs, and the
// kernel boundaries become counters in global memory (units finished per phase) that a reader polls
// before it touches data another SM produced.
constexpr int kStackMaxDeps = 5;
constexpr int kStackMaxPhases = 1023;
constexpr int kStackRounds = 10;
constexpr int kStackChunkK = 2048;  // K elements per chunk of the persistent kernel (4 KB of a weight row)
struct alignas(128) StackPhase {
  // ---- first 128 bytes: what the producer and the consumers need (one cache line)
  const __nv_bfloat16* W;
  int K;
  int n_units;   // N / 8
  int nchunk;    // ceil(K / kStackChunkK)
  int work_idx;  // claim counter (dynamic claims only)
  int done_idx;  // units finished (epilogue written and fenced)
  int n_static;  // claims dealt out statically, claim i to CTA i mod grid
  int n_claims;  // all claims
  int sched_n;   // rounds: count[r] claims of size[r] consecutive units
  int count[kStackRounds], size[kStackRounds];
  int kind;      // 0 QKV, 1 gate/up, 2 Wo, 3 down, 4 LM head (description only)
  int layer;
  // ---- second 128 bytes: the stagers' view and the dependencies
  const float* act;             // fp32 [batch, K]
  const __nv_bfloat16* gain;    // RMSNorm gain or NULL
  int act_mode;
  // counters[dep] >= need must hold before the activations are read ...
  int n_act_deps, act_dep[kStackMaxDeps], act_need[kStackMaxDeps];
  // ... and before the first epilogue (addend read, output buffer overwritten)
  int n_epi_deps, epi_dep[kStackMaxDeps], epi_need[kStackMaxDeps];
  int pad1[1];
  // activations already in MMA operand form (bf16 hi rows 0-3, lo rows 4-7, [chunk][8][2048]), written by the
  // phase that produced them; NULL: convert from the fp32 activations
  const __nv_bfloat16* act_packed;
  int pad2[2];
  // ---- the epilogue description (finishers)
  SmallMParams p;
};
static_assert(offsetof(StackPhase, act) == 128, "producer view must be exactly one line");
static_assert(offsetof(StackPhase, p) == 256, "stager view must be exactly one line");
struct StackAttn {
  DecodeAttnParams a;  // n_splits = stride of the scratch layout; the live split count comes from kv_len
  int n_deps, dep[kStackMaxDeps], need[kStackMaxDeps];      // before the split units (q, K, V written; scratch free)
  int n_mdeps, mdep[kStackMaxDeps], mneed[kStackMaxDeps];   // before the merge units (o free to overwrite)
  int split_done, merge_done;                               // counters: units finished
  __nv_bfloat16* o_pack;                                    // optional MMA-operand copy of o (see SmallMParams::pack_out)
};
struct StackParams {
  const StackPhase* phases;
  int n_phases;
  const StackAttn* attn;
  int n_attn;
  int32_t* counters;  // all zero at launch
  int32_t* status;
  int batch;
};
// 0 = usable on this device (registers and shared memory as expected, co-residency of sm_count CTAs)
cudaError_t decode_stack_init(int sm_count, bool* usable);
cudaError_t launch_decode_stack(const StackParams& sp, int sm_count, cudaStream_t stream);

// Prefill kernels.
struct LargeMParams {
  const __nv_bfloat16* A;  // [M, K] (hi part)
  const __nv_bfloat16* A_lo;  // [M, K] lo part with activation ~ A + A_lo, or NULL (single bf16)
  const __nv_bfloat16* W;  // [N, K]
  int M, N, K;
  int epi_mode;
  const float* addend;     // EPI_RESID
  void* out;
  __nv_bfloat16* out_lo;   // EPI_SWIGLU / EPI_BF16: lo part of the bf16 output, or NULL
  QkvEpilogue qkv;
  int32_t* status;         // device status word (may be NULL)
  int f16;                 // A and W hold binary16 instead of bf16 (one value per activation, A_lo unused), and the
                           // 16-bit outputs (EPI_SWIGLU, EPI_BF16) are written as binary16 too; tcgen05 kernel only
};
// The tcgen05 kernel on every SM of the current device.
cudaError_t launch_largem_gemm(const LargeMParams& p, cudaStream_t stream);
cudaError_t launch_largem_gemm_tc(const LargeMParams& p, cudaStream_t stream, int sm_count);
cudaError_t largem_gemm_tc_init();
// 0 = default: tcgen05 with binary16 operands (one value per activation, the layer's weights converted once per
// call) for calls of at least kPrefillF16MinTokens tokens, bf16 hi + lo pairs below;
// 2 = tcgen05 with single-bf16 activations; 3 = tcgen05 with bf16 hi + lo pairs at every size
void set_prefill_gemm_impl(int impl);
int prefill_gemm_impl();
constexpr int kPrefillF16MinTokens = 256;
bool prefill_single_bf16();            // the prompt pass feeds its GEMMs one bf16 value per activation (no lo part)

// q_lo / o_lo: optional lo parts (value ~ hi + lo) of the query input and the attention output.
// out_f16: o receives ONE binary16 value per element instead of a bf16 value (o_lo must be NULL).
// lens (device, optional): sequence b holds lens[b] <= seq_len valid rows (rows stay seq_len apart); the padding
// rows behind them are neither read as keys nor written as outputs.
// pos0: the seq_len queries sit at positions pos0 .. pos0 + seq_len - 1 and attend to cache rows 0 .. their own.
// status (device, optional): receives LADDER_DEV_TIMEOUT if a bounded wait of the kernel runs out.
cudaError_t launch_prefill_attention(const __half* q, const __half* q_lo, const kv_t* k,
                                     const kv_t* v, int batch, int seq_len, int n_q_heads, int n_kv_heads,
                                     int head_dim, int max_seq_len, __nv_bfloat16* o, __nv_bfloat16* o_lo,
                                     cudaStream_t stream, int pos0 = 0, bool out_f16 = false,
                                     const int32_t* lens = nullptr, int32_t* status = nullptr);
cudaError_t prefill_attention_tc_init();

// Small element-wise / gather kernels.
cudaError_t launch_embed(const int32_t* tokens, const __nv_bfloat16* table, int rows, int d, int vocab, float* x,
                         int32_t* status, cudaStream_t stream, bool pdl);
cudaError_t launch_rmsnorm_bf16(const float* x, const __nv_bfloat16* gain, float eps, int rows, int d,
                                __nv_bfloat16* out, __nv_bfloat16* out_lo, cudaStream_t stream);
cudaError_t launch_rmsnorm_f16(const float* x, const __nv_bfloat16* gain, float eps, int rows, int d, __half* out,
                               cudaStream_t stream);
// n elements, n % 8 == 0, both pointers 16-byte aligned
cudaError_t launch_convert_bf16_f16(const __nv_bfloat16* src, __half* dst, size_t n, cudaStream_t stream);
// out = a + b, n fp32 elements (n a multiple of 4, 16-byte aligned pointers; out may be a or b)
cudaError_t launch_add_f32(const float* a, const float* b, float* out, size_t n, cudaStream_t stream);
cudaError_t launch_rmsnorm_f32(const float* x, const __nv_bfloat16* gain, float eps, int rows, int d, int row_stride,
                               float* out, cudaStream_t stream, bool pdl);
// lens (device, optional): row r is taken at offset lens[r] - 1 instead of src_offset_rows
cudaError_t launch_gather_rows(const float* x, int rows, int d, int src_stride_rows, int src_offset_rows, float* out,
                               cudaStream_t stream, const int32_t* lens = nullptr);
// argmax over logits [batch, vocab] (lowest index on ties) -> next_tokens; then seq_lens[b] = set_lens[b] (device,
// optional), else = set_len (if >= 0), else += advance.
cudaError_t launch_argmax_advance(const float* logits, int batch, int vocab, int32_t* next_tokens, int32_t* seq_lens,
                                  int advance, int set_len, cudaStream_t stream, bool pdl,
                                  const int32_t* set_lens = nullptr);

// One-time opt-in to large dynamic shared memory for every kernel (call once per process/device,
// outside any stream capture).
cudaError_t smallm_gemm_init();

}  // namespace ladder
