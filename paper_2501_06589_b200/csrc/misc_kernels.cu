// Small gather / normalisation / argmax kernels around the GEMMs.
#include "common.cuh"
#include "kernels.h"

namespace ladder {
namespace {

template <typename... KArgs, typename... Args>
cudaError_t launch(void (*kern)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, bool pdl, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// x[r, :] = float(table[tok[r], :]); an id outside [0, vocab) is reported and read as id 0.
__global__ void embed_kernel(const int32_t* tokens, const __nv_bfloat16* table, int d, int vocab, float* x,
                             int32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  int t = tokens[r];
  if (t < 0 || t >= vocab) {
    if (threadIdx.x == 0 && status) atomicOr(status, LADDER_DEV_BAD_TOKEN);
    t = 0;
  }
  const uint4* src = reinterpret_cast<const uint4*>(table + static_cast<size_t>(t) * d);
  float4* dst = reinterpret_cast<float4*>(x + static_cast<size_t>(r) * d);
  for (int i = threadIdx.x; i < d / 8; i += blockDim.x) {
    const uint4 u = __ldg(src + i);
    dst[2 * i] = make_float4(bf16_lo(u.x), bf16_hi(u.x), bf16_lo(u.y), bf16_hi(u.y));
    dst[2 * i + 1] = make_float4(bf16_lo(u.z), bf16_hi(u.z), bf16_lo(u.w), bf16_hi(u.w));
  }
}

__device__ __forceinline__ float block_sum(float v, float* sh) {
  v = warp_sum(v);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float t = 0.f;
  const int nw = (blockDim.x + 31) >> 5;
  for (int w = 0; w < nw; ++w) t += sh[w];
  __syncthreads();
  return t;
}

// y = x / sqrt(mean(x^2) + eps) * gain, one CTA per row; OUT = bf16 or fp32.
// bf16 output is written as a hi part and (if out_lo) a lo part with y ~ hi + lo.
template <typename OUT>
__global__ void rmsnorm_kernel(const float* x, const __nv_bfloat16* gain, float eps, int d, int row_stride, OUT* out,
                               OUT* out_lo) {
  __shared__ float sh[32];
  pdl_launch_dependents();
  pdl_wait();
  const float* xr = x + static_cast<size_t>(blockIdx.x) * row_stride;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
    const float4 v = reinterpret_cast<const float4*>(xr)[i];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  const float rstd = rsqrtf(block_sum(ss, sh) / static_cast<float>(d) + eps);
  OUT* o = out + static_cast<size_t>(blockIdx.x) * d;
  for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
    const float4 v = reinterpret_cast<const float4*>(xr)[i];
    const uint2 gq = __ldg(reinterpret_cast<const uint2*>(gain) + i);
    const float y0 = v.x * rstd * bf16_lo(gq.x), y1 = v.y * rstd * bf16_hi(gq.x);
    const float y2 = v.z * rstd * bf16_lo(gq.y), y3 = v.w * rstd * bf16_hi(gq.y);
    if (sizeof(OUT) == 2) {
      const uint2 hi = make_uint2(pack_bf16x2(y0, y1), pack_bf16x2(y2, y3));
      reinterpret_cast<uint2*>(o)[i] = hi;
      if (out_lo)
        reinterpret_cast<uint2*>(out_lo + static_cast<size_t>(blockIdx.x) * d)[i] =
            make_uint2(pack_bf16x2(y0 - bf16_lo(hi.x), y1 - bf16_hi(hi.x)),
                       pack_bf16x2(y2 - bf16_lo(hi.y), y3 - bf16_hi(hi.y)));
    } else {
      reinterpret_cast<float4*>(o)[i] = make_float4(y0, y1, y2, y3);
    }
  }
}

// The same normalisation written as ONE binary16 value per element (the operand of the binary16 prompt-pass GEMMs).
__global__ void rmsnorm_f16_kernel(const float* x, const __nv_bfloat16* gain, float eps, int d, __half* out) {
  __shared__ float sh[32];
  const float* xr = x + static_cast<size_t>(blockIdx.x) * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
    const float4 v = reinterpret_cast<const float4*>(xr)[i];
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  const float rstd = rsqrtf(block_sum(ss, sh) / static_cast<float>(d) + eps);
  __half* o = out + static_cast<size_t>(blockIdx.x) * d;
  for (int i = threadIdx.x; i < d / 4; i += blockDim.x) {
    const float4 v = reinterpret_cast<const float4*>(xr)[i];
    const uint2 gq = __ldg(reinterpret_cast<const uint2*>(gain) + i);
    reinterpret_cast<uint2*>(o)[i] = make_uint2(pack_kv(v.x * rstd * bf16_lo(gq.x), v.y * rstd * bf16_hi(gq.x)),
                                                pack_kv(v.z * rstd * bf16_lo(gq.y), v.w * rstd * bf16_hi(gq.y)));
  }
}

// bf16 -> binary16, eight elements per thread and iteration.  Exact for |w| >= 2^-14 (binary16 has three more
// significant bits than bf16); smaller magnitudes land on binary16's subnormal grid, at most 2^-25 away.
__global__ void convert_bf16_f16_kernel(const uint4* src, uint4* dst, size_t n8) {
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n8;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const uint4 v = __ldcs(src + i);
    uint4 o;
    o.x = pack_f16x2(bf16_lo(v.x), bf16_hi(v.x));
    o.y = pack_f16x2(bf16_lo(v.y), bf16_hi(v.y));
    o.z = pack_f16x2(bf16_lo(v.z), bf16_hi(v.z));
    o.w = pack_f16x2(bf16_lo(v.w), bf16_hi(v.w));
    dst[i] = o;
  }
}

// out = a + b (fp32, four elements per thread and iteration): the residual add of a module output that was stored
// and summed over the tensor-parallel ranks first (prompt pass).
__global__ void add_f32_kernel(const float4* a, const float4* b, float4* out, size_t n4) {
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n4;
       i += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const float4 x = a[i], y = __ldcs(b + i);
    out[i] = make_float4(x.x + y.x, x.y + y.y, x.z + y.z, x.w + y.w);
  }
}

// out[r, :] = x[(r * stride + offset), :]; with `lens` the offset of row r is lens[r] - 1 (its last valid position)
__global__ void gather_rows_kernel(const float* x, int d, int stride, int offset, const int32_t* lens, float* out) {
  if (lens) offset = min(max(lens[blockIdx.x], 1), stride) - 1;
  const float4* src = reinterpret_cast<const float4*>(x + (static_cast<size_t>(blockIdx.x) * stride + offset) * d);
  float4* dst = reinterpret_cast<float4*>(out + static_cast<size_t>(blockIdx.x) * d);
  for (int i = threadIdx.x; i < d / 4; i += blockDim.x) dst[i] = src[i];
}

// Greedy token per row (lowest index among equal maxima), then the length update.
__global__ void argmax_advance_kernel(const float* logits, int vocab, int32_t* next_tokens, int32_t* seq_lens,
                                      int advance, int set_len, const int32_t* set_lens) {
  __shared__ float bv[32];
  __shared__ int bi[32];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  if (next_tokens) {
    const float* row = logits + static_cast<size_t>(b) * vocab;
    float best = -INFINITY;
    int idx = 0x7fffffff;
    auto take = [&](float v, int i) {
      if (v > best || (v == best && i < idx)) {
        best = v;
        idx = i;
      }
    };
    // 16-byte loads, eight in flight per thread: the scan is latency-bound (one block per row)
    const int n4 = (vocab & 3) == 0 && (reinterpret_cast<uintptr_t>(row) & 15) == 0 ? vocab >> 2 : 0;
    const float4* row4 = reinterpret_cast<const float4*>(row);
    for (int i0 = threadIdx.x; i0 < n4; i0 += 8 * blockDim.x) {
      float4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int i = i0 + j * blockDim.x;
        v[j] = i < n4 ? __ldcg(row4 + i) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int i = (i0 + j * blockDim.x) * 4;
        if (i < vocab) {
          take(v[j].x, i);
          take(v[j].y, i + 1);
          take(v[j].z, i + 2);
          take(v[j].w, i + 3);
        }
      }
    }
    for (int i = n4 * 4 + threadIdx.x; i < vocab; i += blockDim.x) take(row[i], i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      if (ov > best || (ov == best && oi < idx)) {
        best = ov;
        idx = oi;
      }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
      bv[warp] = best;
      bi[warp] = idx;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      const int nw = (blockDim.x + 31) >> 5;
      for (int w = 1; w < nw; ++w)
        if (bv[w] > best || (bv[w] == best && bi[w] < idx)) {
          best = bv[w];
          idx = bi[w];
        }
      next_tokens[b] = idx == 0x7fffffff ? 0 : idx;  // all-NaN row: defined result
    }
  }
  if (threadIdx.x == 0 && seq_lens) {
    if (set_lens) seq_lens[b] = set_lens[b];  // per-sequence prompt lengths
    else if (set_len >= 0) seq_lens[b] = set_len;
    else seq_lens[b] += advance;
  }
}

}  // namespace

cudaError_t launch_embed(const int32_t* tokens, const __nv_bfloat16* table, int rows, int d, int vocab, float* x,
                         int32_t* status, cudaStream_t stream, bool pdl) {
  return launch(embed_kernel, dim3(rows), dim3(256), stream, pdl, tokens, table, d, vocab, x, status);
}

cudaError_t launch_rmsnorm_bf16(const float* x, const __nv_bfloat16* gain, float eps, int rows, int d,
                                __nv_bfloat16* out, __nv_bfloat16* out_lo, cudaStream_t stream) {
  return launch(rmsnorm_kernel<__nv_bfloat16>, dim3(rows), dim3(256), stream, false, x, gain, eps, d, d, out, out_lo);
}

cudaError_t launch_rmsnorm_f16(const float* x, const __nv_bfloat16* gain, float eps, int rows, int d, __half* out,
                               cudaStream_t stream) {
  return launch(rmsnorm_f16_kernel, dim3(rows), dim3(256), stream, false, x, gain, eps, d, out);
}

cudaError_t launch_convert_bf16_f16(const __nv_bfloat16* src, __half* dst, size_t n, cudaStream_t stream) {
  if (n % 8 || ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15)) return cudaErrorInvalidValue;
  const size_t n8 = n / 8;
  const size_t blocks = (n8 + 255) / 256;
  return launch(convert_bf16_f16_kernel, dim3(static_cast<unsigned>(blocks < 148 * 16 ? (blocks ? blocks : 1) : 148 * 16)),
                dim3(256), stream, false, reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst), n8);
}

cudaError_t launch_add_f32(const float* a, const float* b, float* out, size_t n, cudaStream_t stream) {
  if (n % 4 || ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(out)) & 15))
    return cudaErrorInvalidValue;
  const size_t n4 = n / 4;
  const size_t blocks = (n4 + 255) / 256;
  return launch(add_f32_kernel, dim3(static_cast<unsigned>(blocks < 148 * 8 ? (blocks ? blocks : 1) : 148 * 8)), dim3(256),
                stream, false, reinterpret_cast<const float4*>(a), reinterpret_cast<const float4*>(b),
                reinterpret_cast<float4*>(out), n4);
}

cudaError_t launch_rmsnorm_f32(const float* x, const __nv_bfloat16* gain, float eps, int rows, int d, int row_stride,
                               float* out, cudaStream_t stream, bool pdl) {
  return launch(rmsnorm_kernel<float>, dim3(rows), dim3(256), stream, pdl, x, gain, eps, d, row_stride, out,
                static_cast<float*>(nullptr));
}

cudaError_t launch_gather_rows(const float* x, int rows, int d, int src_stride_rows, int src_offset_rows, float* out,
                               cudaStream_t stream, const int32_t* lens) {
  return launch(gather_rows_kernel, dim3(rows), dim3(256), stream, false, x, d, src_stride_rows, src_offset_rows, lens,
                out);
}

cudaError_t launch_argmax_advance(const float* logits, int batch, int vocab, int32_t* next_tokens, int32_t* seq_lens,
                                  int advance, int set_len, cudaStream_t stream, bool pdl, const int32_t* set_lens) {
  return launch(argmax_advance_kernel, dim3(batch), dim3(1024), stream, pdl, logits, vocab, next_tokens, seq_lens,
                advance, set_len, set_lens);
}

}  // namespace ladder
