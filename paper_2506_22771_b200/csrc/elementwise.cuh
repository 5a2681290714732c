// Memory-bound passes of the FF-INT8 step: absmax reduction, SUQ quantisation (Sec. IV) with
// nearest / stochastic rounding (Sec. IV-B), goodness finalisation and length normalisation
// (Sec. III; Alg. 1, goodness step), the loss / look-ahead coefficient kernel (Eq. 1-4) and the output
// gradient quantiser (g^Y to INT8, Sec. IV-B).
// All are coalesced 128-bit-load kernels with warp-shuffle reductions; grids are sized in
// multiples of the SM count by the host code.
#pragma once
#include "common.cuh"

namespace ffi8 {

constexpr int EW_THREADS = 256;
constexpr int FF_MAX_LATER = 31;  // layers after the first in one call
constexpr uint32_t SAMPLE_TILE_GROUPS = 4 * EW_THREADS;  // float4 groups of one sample that a block takes at a time

__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) { return __reduce_max_sync(0xffffffffu, v); }

// Block-wide max of a u32; result valid in thread 0.
__device__ __forceinline__ uint32_t block_max_u32(uint32_t v) {
  __shared__ uint32_t sm[32];
  v = warp_max_u32(v);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) sm[w] = v;
  __syncthreads();
  if (w == 0) {
    v = (lane < (int)((blockDim.x + 31) >> 5)) ? sm[lane] : 0u;
    v = warp_max_u32(v);
  }
  return v;
}

// ---------------------------------------------------------------------------------------------
// absmax over `passes` consecutive slices of n_per_pass floats each; out[p] must be zero before.
// |x| compared as bit patterns (monotone for finite floats); Inf/NaN raise ST_NONFINITE.
// grid = (blocks, passes)
// ---------------------------------------------------------------------------------------------
// out2 (nullable): a second place that receives the same maximum - the other set's slot when both sets are to be
// quantised with one joint range.
__device__ __forceinline__ void absmax_body(const float* __restrict__ xp, size_t n_per_pass, uint32_t* __restrict__ out,
                                            uint32_t* __restrict__ status, uint32_t* __restrict__ out2 = nullptr);
__global__ void __launch_bounds__(EW_THREADS) absmax_kernel(const float* __restrict__ x, size_t n_per_pass,
                                                            float* __restrict__ out, uint32_t* __restrict__ status,
                                                            int joint = 0) {
  uint32_t* o = reinterpret_cast<uint32_t*>(out);
  absmax_body(x + (size_t)blockIdx.y * n_per_pass, n_per_pass, o + blockIdx.y, status, joint ? o + (blockIdx.y ^ 1) : nullptr);
}
// The same over a table of tensors in one launch (blockIdx.y = tensor): the weights of every layer and the two
// sets of the network input are all known when a step starts.  A step of small layers is a chain of short
// launches, so fewer launches is what counts there.
constexpr int MT_MAX = FF_MAX_LATER + 1 + 2;
struct AbsmaxJobs {
  const float* x[MT_MAX];
  unsigned long long n[MT_MAX];
  float* out[MT_MAX];
  float* out2[MT_MAX];   // nullable, see absmax_body
};
__global__ void __launch_bounds__(EW_THREADS) absmax_multi_kernel(AbsmaxJobs jobs, uint32_t* __restrict__ status) {
  const int t = blockIdx.y;
  absmax_body(jobs.x[t], (size_t)jobs.n[t], reinterpret_cast<uint32_t*>(jobs.out[t]), status,
              reinterpret_cast<uint32_t*>(jobs.out2[t]));
}
__device__ __forceinline__ void absmax_body(const float* __restrict__ xp, size_t n_per_pass, uint32_t* __restrict__ out,
                                            uint32_t* __restrict__ status, uint32_t* __restrict__ out2) {
  uint32_t m = 0;
  const bool vec = ((n_per_pass & 3) == 0) && ((((uintptr_t)xp) & 15) == 0);
  size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t stride = (size_t)gridDim.x * blockDim.x;
  if (vec) {
    const uint4* x4 = reinterpret_cast<const uint4*>(xp);
    size_t n4 = n_per_pass >> 2;
#pragma unroll 4
    for (size_t i = tid; i < n4; i += stride) {
      uint4 v = __ldg(x4 + i);
      m = max(m, max(max(v.x & 0x7fffffffu, v.y & 0x7fffffffu), max(v.z & 0x7fffffffu, v.w & 0x7fffffffu)));
    }
  } else {
    for (size_t i = tid; i < n_per_pass; i += stride) m = max(m, __float_as_uint(xp[i]) & 0x7fffffffu);
  }
  m = block_max_u32(m);
  if (threadIdx.x == 0) {
    if (m >= 0x7f800000u) atomicOr(status, ST_NONFINITE);
    if (m) {
      atomicMax(out, m);
      if (out2) atomicMax(out2, m);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// q = clip(round(x * 127/a_p)) for `passes` slices, a_p read from device memory (absmax[p]).
// Linear element index (over the whole tensor) keys the stochastic rounding.  When the tensor is one
// shard of a batch split by rows over several devices, ctr_bias.x / .y (passes 0 / 1) is added to the
// local index so that the counter is the element's index in the unsplit tensor.
// grid = (blocks, passes)
// ---------------------------------------------------------------------------------------------
// zero_S / zero_rowmax (nullable, zero_n entries): per-sample accumulators of the forward epilogue that
// the weight quantiser clears on the side, sparing a launch.
// INT8 tensors of dense layers may have rows padded to a wider pitch (a multiple of 128 bytes keeps every TMA box
// row of the contractions aligned): element e of a [rows, cols] tensor then sits at e + (e / cols) * extra with
// extra = pitch - cols.  extra = 0: dense, no division.
struct RowPad {
  uint32_t cols, extra;
};
__device__ __forceinline__ size_t padded(size_t e, RowPad rp) { return rp.extra ? e + (e / rp.cols) * rp.extra : e; }

// q[i] = quantised x[i] for one tensor of n elements; ctr0 = rounding counter of element 0 (an odd one would
// split the element pairs that share one hash differently from the unsplit tensor: scalar path then).
// qp = start of the output TENSOR, e0 = dense index of xp[0] in it (rows before it are skipped with their padding).
template <int MODE, bool PAD = false>
__device__ __forceinline__ void quantize_body(const float* __restrict__ xp, int8_t* __restrict__ qp, size_t n, float inv,
                                              uint32_t ctr0, RoundKey key, size_t e0 = 0, RowPad rp = RowPad{0u, 0u}) {
  if (!PAD) rp = RowPad{0u, 0u};  // compiled without the row arithmetic
  const bool vec = ((n & 3) == 0) && ((e0 & 3) == 0) && ((((uintptr_t)xp) & 15) == 0) && ((((uintptr_t)qp) & 3) == 0) &&
                   !(ctr0 & 1u) && ((rp.cols | rp.extra) & 3u) == 0;
  size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t stride = (size_t)gridDim.x * blockDim.x;
  if (vec) {
    const float4* x4 = reinterpret_cast<const float4*>(xp);
    size_t n4 = n >> 2;
    // four loads in flight per thread, then the arithmetic (the FP32 source is not read again: streaming loads)
    for (size_t i0 = tid; i0 < n4; i0 += 4 * stride) {
      float4 vv[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (i0 + k * stride < n4) vv[k] = __ldcs(x4 + i0 + k * stride);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const size_t i = i0 + k * stride;
        if (i >= n4) break;
        const float4 v = vv[k];
        uint32_t idx = ctr0 + (uint32_t)(i << 2);
        int q0, q1, q2, q3;
        quant_pair<MODE>(v.x, v.y, inv, idx, key, q0, q1);
        quant_pair<MODE>(v.z, v.w, inv, idx + 2, key, q2, q3);
        *reinterpret_cast<uint32_t*>(qp + (PAD ? padded(e0 + (i << 2), rp) : e0 + (i << 2))) = pack4(q0, q1, q2, q3);
      }
    }
  } else {
    for (size_t i = tid; i < n; i += stride)
      qp[PAD ? padded(e0 + i, rp) : e0 + i] = (int8_t)quant_one<MODE>(xp[i], inv, ctr0 + (uint32_t)i, key);
  }
}

template <int MODE>
__global__ void __launch_bounds__(EW_THREADS) quantize_kernel(const float* __restrict__ x, int8_t* __restrict__ q,
                                                              size_t n_per_pass, const float* __restrict__ a,
                                                              KeySpec ks, unsigned long long* __restrict__ zero_S = nullptr,
                                                              int32_t* __restrict__ zero_rowmax = nullptr, int zero_n = 0,
                                                              uint2 ctr_bias = uint2{0u, 0u}, RowPad rp = RowPad{0u, 0u}) {
  const RoundKey key = (MODE == ROUND_NEAREST) ? RoundKey{0u, 0u} : derive_key(ks);
  const uint32_t bias = blockIdx.y ? ctr_bias.y : ctr_bias.x;
  if (zero_S && blockIdx.y == 0)
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < zero_n; i += gridDim.x * blockDim.x) {
      zero_S[i] = 0ull;
      zero_rowmax[i] = 0;
    }
  const size_t base = (size_t)blockIdx.y * n_per_pass;
  if (rp.extra)
    quantize_body<MODE, true>(x + base, q, n_per_pass, inv_of(a[blockIdx.y]), (uint32_t)base + bias, key, base, rp);
  else
    quantize_body<MODE, false>(x + base, q, n_per_pass, inv_of(a[blockIdx.y]), (uint32_t)base + bias, key, base);
}

// One launch for a table of tensors (blockIdx.y = tensor): the weights of every layer and the two sets of
// the network input, each with its own range, rounding mode, key and first counter.  Also clears the
// per-sample accumulators of every layer's forward epilogue.
struct QuantJobs {
  const float* x[MT_MAX];
  int8_t* q[MT_MAX];
  unsigned long long n[MT_MAX];
  const float* a[MT_MAX];          // address of the tensor's range
  unsigned long long s1[MT_MAX];   // step-independent part of the rounding key
  uint32_t ctr0[MT_MAX];           // counter of the tensor's first element
  unsigned long long e0[MT_MAX];   // dense index of x[t][0] inside the output tensor q[t]
  RowPad pad[MT_MAX];              // row padding of the output tensor
  uint8_t stochastic[MT_MAX];
  unsigned long long* zero_S[FF_MAX_LATER + 1];
  int32_t* zero_rowmax[FF_MAX_LATER + 1];
  int n_zero, zero_n;              // layers whose accumulators are cleared, entries each
  const StepState* ss;
};
template <bool PAD>  // PAD: some output tensor has padded rows (compiled apart so that the dense form stays lean)
__global__ void __launch_bounds__(EW_THREADS) quantize_multi_kernel(const QuantJobs jobs) {
  const int t = blockIdx.y;
  if (t < jobs.n_zero)
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < jobs.zero_n; i += gridDim.x * blockDim.x) {
      jobs.zero_S[t][i] = 0ull;
      jobs.zero_rowmax[t][i] = 0;
    }
  const float inv = inv_of(*jobs.a[t]);
  if (jobs.stochastic[t])
    quantize_body<ROUND_STOCHASTIC, PAD>(jobs.x[t], jobs.q[t], (size_t)jobs.n[t], inv, jobs.ctr0[t],
                                         derive_key(KeySpec{jobs.s1[t], jobs.ss}), (size_t)jobs.e0[t], jobs.pad[t]);
  else
    quantize_body<ROUND_NEAREST, PAD>(jobs.x[t], jobs.q[t], (size_t)jobs.n[t], inv, jobs.ctr0[t], RoundKey{0u, 0u},
                                      (size_t)jobs.e0[t], jobs.pad[t]);
}

// ---------------------------------------------------------------------------------------------
// Goodness per sample from the exact integer sum: G = float(double(S) * c*c), c = s_x[p]*s_w.
// Also the per-pass absmax of the normalised output via the per-sample max of relu(acc):
// max_n y*r = (float(rowmax)*c)*r because each rounded multiply by a fixed non-negative factor is
// monotone.  a_next (and a_next2, if non-NULL) receive it by atomicMax; both must be zero before.
// ---------------------------------------------------------------------------------------------
// write_range = 0: only G is written (the layer's output takes a skip path, so its range is found by the kernel
// that forms the sum); 2: both sets' slots receive the maximum over both sets (one joint range).
__global__ void __launch_bounds__(EW_THREADS) finalize_goodness_kernel(
    const unsigned long long* __restrict__ S, const int32_t* __restrict__ rowmax, const float* __restrict__ absmax,
    int B, float tau, float eps, float* __restrict__ G, float* __restrict__ a_next, float* __restrict__ a_next2,
    int write_range = 1, float* __restrict__ Rn = nullptr) {
  // Rn (nullable, [2B]): receives the per-sample factor tau/(sqrt(G)+eps), so that the normalisation pass of short
  // samples reads it instead of forming a square root and a division per group of four elements
  const int p = blockIdx.y;
  const float c = __fmul_rn(scale_of(absmax[p]), scale_of(absmax[2]));
  const double c2 = __dmul_rn((double)c, (double)c);
  uint32_t mx = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < B; i += gridDim.x * blockDim.x) {
    int m = p * B + i;
    float g = __double2float_rn(__dmul_rn(__ull2double_rn(S[m]), c2));
    G[m] = g;
    float r = __fdiv_rn(tau, __fadd_rn(__fsqrt_rn(g), eps));
    if (Rn) Rn[m] = r;
    float xm = __fmul_rn(__fmul_rn(__int2float_rn(rowmax[m]), c), r);
    mx = max(mx, __float_as_uint(xm));
  }
  mx = block_max_u32(mx);
  if (threadIdx.x == 0 && mx && write_range) {
    atomicMax(reinterpret_cast<uint32_t*>(a_next) + p, mx);
    if (a_next2) atomicMax(reinterpret_cast<uint32_t*>(a_next2) + p, mx);
    if (write_range == 2) {
      atomicMax(reinterpret_cast<uint32_t*>(a_next) + (p ^ 1), mx);
      if (a_next2) atomicMax(reinterpret_cast<uint32_t*>(a_next2) + (p ^ 1), mx);
    }
  }
}

// The per-sample passes below stream float4 groups with a grid-stride loop.  The sample a group
// belongs to is tracked incrementally (one division per thread at the start, none per element):
// advancing by `stride` groups adds stride / g4 samples and stride % g4 groups, with one carry.
struct SampleCursor {
  uint32_t sample, offset;      // current sample (within the pass) and float4 group inside it
  uint32_t step_q, step_r, g4;  // stride / g4, stride % g4, groups per sample
  __device__ __forceinline__ SampleCursor(uint32_t first_group, uint32_t stride, uint32_t groups_per_sample) {
    g4 = groups_per_sample;
    sample = first_group / g4;
    offset = first_group - sample * g4;
    step_q = stride / g4;
    step_r = stride - step_q * g4;
  }
  __device__ __forceinline__ void advance() {
    sample += step_q;
    offset += step_r;
    if (offset >= g4) {
      offset -= g4;
      ++sample;
    }
  }
};

// ---------------------------------------------------------------------------------------------
// Length normalisation x = y * tau/(sqrt(G)+eps) per sample, written as FP32 (xnext, nullable)
// and / or quantised straight to the next layer's INT8 input (xq, nullable) with per-pass range
// a[p].  per_sample = R*N elements per sample; per_pass = B*per_sample.   grid = (blocks, 2)
// ---------------------------------------------------------------------------------------------
template <int MODE, bool PAD = false>
__global__ void __launch_bounds__(EW_THREADS) normalize_kernel(const float* __restrict__ Y, const float* __restrict__ G,
                                                               float tau, float eps, size_t per_sample,
                                                               size_t per_pass, float* __restrict__ xnext,
                                                               int8_t* __restrict__ xq, const float* __restrict__ a,
                                                               KeySpec ks, uint2 ctr_bias = uint2{0u, 0u},
                                                               RowPad rp = RowPad{0u, 0u}, const float* __restrict__ Rn = nullptr) {
  // rp: row padding of xq (dense layers only: a row is a sample, so sample index * extra is the shift)
  // Rn (nullable): the per-sample factors tau/(sqrt(G)+eps) as finalize_goodness_kernel left them (the same bits)
  const RoundKey key = (MODE == ROUND_NEAREST) ? RoundKey{0u, 0u} : derive_key(ks);
  const uint32_t bias = blockIdx.y ? ctr_bias.y : ctr_bias.x;
  const size_t base = (size_t)blockIdx.y * per_pass;
  const float inv = xq ? inv_of(a[blockIdx.y]) : 0.0f;
  const bool vec = ((per_sample & 3) == 0) && ((((uintptr_t)Y) & 15) == 0) &&
                   (!xnext || (((uintptr_t)xnext) & 15) == 0) && (!xq || (((uintptr_t)xq) & 3) == 0);
  const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, stride = gridDim.x * blockDim.x;
  if (vec && per_sample >= 4 * SAMPLE_TILE_GROUPS) {
    // long samples: blocks take (sample, tile of the sample) pairs, so the per-sample factor (a square root and a
    // division) is formed once per tile instead of once per four elements
    const uint32_t g4 = (uint32_t)(per_sample >> 2), n_samples = (uint32_t)(per_pass / per_sample);
    const uint32_t tps = (g4 + SAMPLE_TILE_GROUPS - 1) / SAMPLE_TILE_GROUPS;
    const float* Gp = G + (size_t)blockIdx.y * n_samples;
    for (uint32_t tile = blockIdx.x; tile < n_samples * tps; tile += gridDim.x) {
      const uint32_t smp = tile / tps, g0 = (tile - smp * tps) * SAMPLE_TILE_GROUPS;
      const float r = __fdiv_rn(tau, __fadd_rn(__fsqrt_rn(__ldg(Gp + smp)), eps));
      const size_t e0 = base + (size_t)smp * per_sample;
      float4 vv[SAMPLE_TILE_GROUPS / EW_THREADS];  // all loads of the tile first (Y is read again by the dH quantiser: cached loads)
#pragma unroll
      for (uint32_t k = 0; k < SAMPLE_TILE_GROUPS / EW_THREADS; ++k) {
        const uint32_t i = g0 + k * EW_THREADS + threadIdx.x;
        if (i < g4) vv[k] = __ldg(reinterpret_cast<const float4*>(Y + e0 + ((size_t)i << 2)));
      }
#pragma unroll
      for (uint32_t k = 0; k < SAMPLE_TILE_GROUPS / EW_THREADS; ++k) {
        const uint32_t i = g0 + k * EW_THREADS + threadIdx.x;
        if (i >= g4) break;
        const size_t e = e0 + ((size_t)i << 2);
        float4 v = vv[k];
        v.x = __fmul_rn(v.x, r);
        v.y = __fmul_rn(v.y, r);
        v.z = __fmul_rn(v.z, r);
        v.w = __fmul_rn(v.w, r);
        if (xnext) *reinterpret_cast<float4*>(xnext + e) = v;
        if (xq) {
          int q0, q1, q2, q3;
          quant_pair<MODE>(v.x, v.y, inv, (uint32_t)e + bias, key, q0, q1);
          quant_pair<MODE>(v.z, v.w, inv, (uint32_t)e + bias + 2, key, q2, q3);
          *reinterpret_cast<uint32_t*>(xq + e + (PAD ? (size_t)(blockIdx.y * n_samples + smp) * rp.extra : (size_t)0)) =
              pack4(q0, q1, q2, q3);
        }
      }
    }
  } else if (vec) {
    const uint32_t n4 = (uint32_t)(per_pass >> 2);
    const float* Gp = G + (uint32_t)(base / per_sample);
    const uint32_t pass_row0 = (uint32_t)(base / per_sample);
    SampleCursor cur(tid, stride, (uint32_t)(per_sample >> 2));
    for (uint32_t i0 = tid; i0 < n4; i0 += 4 * stride) {  // four loads in flight, then the arithmetic
      float4 vv[4];
#pragma unroll
      for (uint32_t k = 0; k < 4; ++k)
        if (i0 + k * stride < n4) vv[k] = __ldg(reinterpret_cast<const float4*>(Y + base + ((size_t)(i0 + k * stride) << 2)));
#pragma unroll
      for (uint32_t k = 0; k < 4; ++k, cur.advance()) {
        const uint32_t i = i0 + k * stride;
        if (i >= n4) break;
        const size_t e = base + ((size_t)i << 2);
        const float r = Rn ? __ldg(Rn + pass_row0 + cur.sample) : __fdiv_rn(tau, __fadd_rn(__fsqrt_rn(__ldg(Gp + cur.sample)), eps));
        float4 v = vv[k];
        v.x = __fmul_rn(v.x, r);
        v.y = __fmul_rn(v.y, r);
        v.z = __fmul_rn(v.z, r);
        v.w = __fmul_rn(v.w, r);
        if (xnext) *reinterpret_cast<float4*>(xnext + e) = v;
        if (xq) {
          int q0, q1, q2, q3;
          quant_pair<MODE>(v.x, v.y, inv, (uint32_t)e + bias, key, q0, q1);
          quant_pair<MODE>(v.z, v.w, inv, (uint32_t)e + bias + 2, key, q2, q3);
          *reinterpret_cast<uint32_t*>(xq + e + (PAD ? (size_t)(pass_row0 + cur.sample) * rp.extra : (size_t)0)) =
                pack4(q0, q1, q2, q3);
        }
      }
    }
  } else {
    for (size_t i = tid; i < per_pass; i += stride) {
      size_t e = base + i;
      float g = G[(uint32_t)e / (uint32_t)per_sample];
      float r = __fdiv_rn(tau, __fadd_rn(__fsqrt_rn(g), eps));
      float v = __fmul_rn(Y[e], r);
      if (xnext) xnext[e] = v;
      if (xq) xq[PAD ? padded(e, rp) : e] = (int8_t)quant_one<MODE>(v, inv, (uint32_t)e + bias, key);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Output of a residual block: z = y*r + scale*skip per element (r = tau/(sqrt(G)+eps) of the sample; one rounding
// per operation), written as FP32, and the per-set range max|z| (a maximum: exact, order-free) for the next
// layer's quantiser into a_next[p] and, if given, a_next2[p] (both zero before).  The sum has no range short-cut,
// so the next layer's INT8 input is made from xnext by the ordinary quantiser afterwards.  The paper trains
// residual networks (Sec. IV-C, Table II) without saying how the sum is formed under FF; here the skip path only
// changes what the next layer sees - the layer's own goodness stays ||y||^2 (Sec. III).   grid = (blocks, 2)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS) normalize_skip_kernel(const float* __restrict__ Y, const float* __restrict__ G,
                                                                    float tau, float eps, size_t per_sample, size_t per_pass,
                                                                    const float* __restrict__ skip, float scale,
                                                                    float* __restrict__ xnext, float* __restrict__ a_next,
                                                                    float* __restrict__ a_next2, uint32_t* __restrict__ status,
                                                                    int joint = 0) {
  const size_t base = (size_t)blockIdx.y * per_pass;
  const bool vec = ((per_sample & 3) == 0) && ((((uintptr_t)Y) & 15) == 0) && ((((uintptr_t)xnext) & 15) == 0) &&
                   ((((uintptr_t)skip) & 15) == 0);
  const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, stride = gridDim.x * blockDim.x;
  uint32_t mx = 0u;
  if (vec) {
    const uint32_t n4 = (uint32_t)(per_pass >> 2);
    const float* Gp = G + (uint32_t)(base / per_sample);
    SampleCursor cur(tid, stride, (uint32_t)(per_sample >> 2));
    for (uint32_t i = tid; i < n4; i += stride, cur.advance()) {
      const size_t e = base + ((size_t)i << 2);
      const float r = __fdiv_rn(tau, __fadd_rn(__fsqrt_rn(__ldg(Gp + cur.sample)), eps));
      const float4 y = __ldg(reinterpret_cast<const float4*>(Y + e));
      const float4 s = __ldcs(reinterpret_cast<const float4*>(skip + e));
      float4 z;
      z.x = __fadd_rn(__fmul_rn(y.x, r), __fmul_rn(scale, s.x));
      z.y = __fadd_rn(__fmul_rn(y.y, r), __fmul_rn(scale, s.y));
      z.z = __fadd_rn(__fmul_rn(y.z, r), __fmul_rn(scale, s.z));
      z.w = __fadd_rn(__fmul_rn(y.w, r), __fmul_rn(scale, s.w));
      *reinterpret_cast<float4*>(xnext + e) = z;
      mx = max(mx, max(max(__float_as_uint(z.x) & 0x7fffffffu, __float_as_uint(z.y) & 0x7fffffffu),
                       max(__float_as_uint(z.z) & 0x7fffffffu, __float_as_uint(z.w) & 0x7fffffffu)));
    }
  } else {
    for (size_t i = tid; i < per_pass; i += stride) {
      const size_t e = base + i;
      const float r = __fdiv_rn(tau, __fadd_rn(__fsqrt_rn(G[(uint32_t)e / (uint32_t)per_sample]), eps));
      const float z = __fadd_rn(__fmul_rn(Y[e], r), __fmul_rn(scale, skip[e]));
      xnext[e] = z;
      mx = max(mx, __float_as_uint(z) & 0x7fffffffu);
    }
  }
  mx = block_max_u32(mx);
  if (threadIdx.x == 0) {
    if (mx >= 0x7f800000u) atomicOr(status, ST_NONFINITE);   // a skip tensor that held Inf / NaN
    if (mx) {
      atomicMax(reinterpret_cast<uint32_t*>(a_next) + blockIdx.y, mx);
      if (a_next2) atomicMax(reinterpret_cast<uint32_t*>(a_next2) + blockIdx.y, mx);
      if (joint) {
        atomicMax(reinterpret_cast<uint32_t*>(a_next) + (blockIdx.y ^ 1), mx);
        if (a_next2) atomicMax(reinterpret_cast<uint32_t*>(a_next2) + (blockIdx.y ^ 1), mx);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The same with 2x2 max pooling (stride 2) over the positions of a spatial layer before the scaling:
// out[m, i, j, c] = max of Y[m, 2i..2i+1, 2j..2j+1, c] * tau/(sqrt(G[m])+eps)  (the maximum commutes with the
// positive factor and needs no rounding).  Y [2B, Ho, Wo, N] -> xnext / xq [2B, Ho/2, Wo/2, N]; the rounding
// counters are the element indices of the pooled tensor.  One thread per pooled value (V = 1) or per four
// channels (V = 4, N % 4 == 0).   grid = (blocks, 2)
// ---------------------------------------------------------------------------------------------
template <int MODE, int V>
__global__ void __launch_bounds__(EW_THREADS) normalize_pool_kernel(const float* __restrict__ Y, const float* __restrict__ G,
                                                                    float tau, float eps, int B, int Ho, int Wo, int N,
                                                                    float* __restrict__ xnext, int8_t* __restrict__ xq,
                                                                    const float* __restrict__ a, KeySpec ks,
                                                                    uint2 ctr_bias = uint2{0u, 0u}) {
  const RoundKey key = (MODE == ROUND_NEAREST) ? RoundKey{0u, 0u} : derive_key(ks);
  const uint32_t bias = blockIdx.y ? ctr_bias.y : ctr_bias.x;
  const float inv = xq ? inv_of(a[blockIdx.y]) : 0.0f;
  const uint32_t Hp = Ho >> 1, Wp = Wo >> 1, NG = N / V;
  const uint32_t per_pass = (uint32_t)B * Hp * Wp * NG;          // work items of this pass
  const size_t row = (size_t)N, line = (size_t)Wo * N;
  for (uint32_t it = blockIdx.x * blockDim.x + threadIdx.x; it < per_pass; it += gridDim.x * blockDim.x) {
    const uint32_t pos = it / NG, cg = it - pos * NG;
    const uint32_t j = pos % Wp, t = pos / Wp, i = t % Hp, m = t / Hp + blockIdx.y * B;
    const float r = __fdiv_rn(tau, __fadd_rn(__fsqrt_rn(__ldg(G + m)), eps));
    const float* src = Y + (((size_t)m * Ho + 2 * i) * Wo + 2 * j) * N + (size_t)V * cg;
    const size_t e = ((size_t)blockIdx.y * per_pass + it) * V;   // element index in the pooled tensor
    if (V == 4) {
      const float4 p00 = __ldg(reinterpret_cast<const float4*>(src)), p01 = __ldg(reinterpret_cast<const float4*>(src + row));
      const float4 p10 = __ldg(reinterpret_cast<const float4*>(src + line));
      const float4 p11 = __ldg(reinterpret_cast<const float4*>(src + line + row));
      float4 v;
      v.x = __fmul_rn(fmaxf(fmaxf(p00.x, p01.x), fmaxf(p10.x, p11.x)), r);
      v.y = __fmul_rn(fmaxf(fmaxf(p00.y, p01.y), fmaxf(p10.y, p11.y)), r);
      v.z = __fmul_rn(fmaxf(fmaxf(p00.z, p01.z), fmaxf(p10.z, p11.z)), r);
      v.w = __fmul_rn(fmaxf(fmaxf(p00.w, p01.w), fmaxf(p10.w, p11.w)), r);
      if (xnext) *reinterpret_cast<float4*>(xnext + e) = v;
      if (xq) {
        int q0, q1, q2, q3;
        quant_pair<MODE>(v.x, v.y, inv, (uint32_t)e + bias, key, q0, q1);
        quant_pair<MODE>(v.z, v.w, inv, (uint32_t)e + bias + 2, key, q2, q3);
        *reinterpret_cast<uint32_t*>(xq + e) = pack4(q0, q1, q2, q3);
      }
    } else {
      const float v = __fmul_rn(fmaxf(fmaxf(__ldg(src), __ldg(src + row)), fmaxf(__ldg(src + line), __ldg(src + line + row))), r);
      if (xnext) xnext[e] = v;
      if (xq) xq[e] = (int8_t)quant_one<MODE>(v, inv, (uint32_t)e + bias, key);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// e^v for v <= 0 in FP64 by a fixed recipe so that every implementation agrees bit for bit:
// clamp at -700, n = rint(v*log2e), r = (v - n*LN2_HI) - n*LN2_LO, degree-13 Taylor polynomial by
// Horner with separately rounded multiply and add, exact scaling by 2^n.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double exp_nonpos(double v) {
  constexpr double LOG2E = 1.4426950408889634;
  constexpr double LN2_HI = 6.93147180369123816490e-01;
  constexpr double LN2_LO = 1.90821492927058770002e-10;
  constexpr double C[14] = {1.0 / 1.0,         1.0 / 1.0,          1.0 / 2.0,          1.0 / 6.0,         1.0 / 24.0,
                            1.0 / 120.0,       1.0 / 720.0,        1.0 / 5040.0,       1.0 / 40320.0,     1.0 / 362880.0,
                            1.0 / 3628800.0,   1.0 / 39916800.0,   1.0 / 479001600.0,  1.0 / 6227020800.0};
  v = fmax(v, -700.0);
  double n = rint(__dmul_rn(v, LOG2E));
  double r = __dsub_rn(__dsub_rn(v, __dmul_rn(n, LN2_HI)), __dmul_rn(n, LN2_LO));
  double p = C[13];
#pragma unroll
  for (int k = 12; k >= 0; --k) p = __dadd_rn(__dmul_rn(p, r), C[k]);
  return scalbn(p, (int)n);
}
// sigma(x) from e = e^{-|x|}: x >= 0 -> 1/(1+e), else e/(1+e).
__device__ __forceinline__ double sigmoid_spec(double x) {
  double e = exp_nonpos(-fabs(x));
  double d = __dadd_rn(1.0, e);
  return x >= 0.0 ? __ddiv_rn(1.0, d) : __ddiv_rn(e, d);
}

// log(1 + e^z) for the reported loss value only (it feeds no state and is compared at 1e-5): the
// correction term in FP32, which keeps the long FP64 library chains out of the kernel's critical path.
__device__ __forceinline__ double softplus_value(double z) {
  const float az = fabsf((float)z);
  return fmax(z, 0.0) + (double)log1pf(expf(-az));
}

struct LaterLayers {
  const float* G[FF_MAX_LATER];
  float theta[FF_MAX_LATER];
  int n;
};

// ---------------------------------------------------------------------------------------------
// Loss (Eq. 1, Eq. 2), look-ahead loss (Eq. 3) and the per-sample coefficient of Eq. 4 under the
// scalar-coefficient reading: coef_m = (g'_l,m + lambda * sum_{j>l} g'_j,m)/M with g' = dL/dG.
// Also the per-pass absmax of dH = 2*coef*y via the per-sample max of relu(acc).
// Several blocks; each leaves its partial loss sum and maxima in `scratch`, and the block that
// finishes last (ticket counter) combines them in block order, so the loss is reproducible and
// nothing has to be zeroed beforehand.  scratch: LossScratch, ticket zero on entry and on exit.
// ---------------------------------------------------------------------------------------------
constexpr int LOSS_THREADS = 64;      // small blocks: the FP64 work of a few thousand samples spreads over many SMs
constexpr int LOSS_MAX_BLOCKS = 1024;
struct LossScratch {
  unsigned int ticket;
  unsigned int pad[3];
  double lsum[LOSS_MAX_BLOCKS];
  uint32_t amax[2][LOSS_MAX_BLOCKS];
};
__device__ __forceinline__ void loss_coef_body(const float* __restrict__ G, float theta, const float* const* later_G,
                                               const float* later_theta, int later_n, float lambda, int B,
                                               const int32_t* __restrict__ rowmax, float* __restrict__ absmax,
                                               float* __restrict__ coef, float* __restrict__ loss,
                                               LossScratch* __restrict__ scratch, int m_total);
__global__ void __launch_bounds__(LOSS_THREADS) loss_coef_kernel(const float* __restrict__ G, float theta, LaterLayers later,
                                                                 float lambda, int B, const int32_t* __restrict__ rowmax,
                                                                 float* __restrict__ absmax, float* __restrict__ coef,
                                                                 float* __restrict__ loss, LossScratch* __restrict__ scratch,
                                                                 const StepState* __restrict__ ss = nullptr,
                                                                 int m_total = 0) {
  if (ss) lambda = ss->lambda;  // a step run through the library's own launch sequence keeps lambda in device memory
  loss_coef_body(G, theta, later.G, later.theta, later.n, lambda, B, rowmax, absmax, coef, loss, scratch, m_total);
}
// Every layer of a step in one launch (blockIdx.y = layer): the losses depend on the goodness values alone,
// which are all there once the forward has run.  Layer l looks ahead at layers l+1 .. n-1 of the same table;
// each layer has its own scratch.
struct LossJobs {
  const float* G[FF_MAX_LATER + 1];
  float theta[FF_MAX_LATER + 1];
  const int32_t* rowmax[FF_MAX_LATER + 1];
  float* absmax[FF_MAX_LATER + 1];
  float* coef[FF_MAX_LATER + 1];
  float* loss[FF_MAX_LATER + 1];
  int n;
};
__global__ void __launch_bounds__(LOSS_THREADS) loss_coef_multi_kernel(const LossJobs jobs, int B, LossScratch* __restrict__ scratch,
                                                                       const StepState* __restrict__ ss, int m_total,
                                                                       int first = 0) {
  const int l = blockIdx.y + first;  // layers before `first` are frozen: no loss, no gradient
  loss_coef_body(jobs.G[l], jobs.theta[l], jobs.G + l + 1, jobs.theta + l + 1, jobs.n - 1 - l, ss->lambda, B, jobs.rowmax[l],
                 jobs.absmax[l], jobs.coef[l], jobs.loss[l], scratch + l, m_total);
}
__device__ __forceinline__ void loss_coef_body(const float* __restrict__ G, float theta, const float* const* later_G,
                                               const float* later_theta, int later_n, float lambda, int B,
                                               const int32_t* __restrict__ rowmax, float* __restrict__ absmax,
                                               float* __restrict__ coef, float* __restrict__ loss,
                                               LossScratch* __restrict__ scratch, int m_total) {
  __shared__ double red[LOSS_THREADS / 32];
  __shared__ uint32_t redmax[2][LOSS_THREADS / 32];
  __shared__ bool is_last;
  const int M = 2 * B;
  const double lam = (double)lambda;
  // the mean of Eq. 1 / Eq. 2 runs over the whole batch: m_total samples when these 2B are one shard of it
  const double inv_m = __ddiv_rn(1.0, (double)(m_total > 0 ? m_total : M));
  const float s_w = scale_of(absmax[2]);
  const float cpass[2] = {__fmul_rn(scale_of(absmax[0]), s_w), __fmul_rn(scale_of(absmax[1]), s_w)};
  double lsum = 0.0;
  uint32_t amax[2] = {0u, 0u};
  for (int m = blockIdx.x * LOSS_THREADS + threadIdx.x; m < M; m += gridDim.x * LOSS_THREADS) {
    const int p = m >= B;
    const double sign = p ? 1.0 : -1.0;
    double arg = __dmul_rn(sign, __dsub_rn((double)G[m], (double)theta));
    double g0 = __dmul_rn(sign, sigmoid_spec(arg));
    double L0 = softplus_value(arg);
    double gsum = 0.0, Lsum = 0.0;
    for (int j = 0; j < later_n; ++j) {
      double aj = __dmul_rn(sign, __dsub_rn((double)later_G[j][m], (double)later_theta[j]));
      gsum = __dadd_rn(gsum, __dmul_rn(sign, sigmoid_spec(aj)));
      Lsum += softplus_value(aj);
    }
    float cf = __double2float_rn(__dmul_rn(__dadd_rn(g0, __dmul_rn(lam, gsum)), inv_m));
    coef[m] = cf;
    lsum += L0 + lam * Lsum;
    float k2 = __fmul_rn(2.0f, cf);
    float d = fabsf(__fmul_rn(k2, __fmul_rn(__int2float_rn(rowmax[m]), cpass[p])));
    amax[p] = max(amax[p], __float_as_uint(d));
  }
  // block reduction (fixed order)
  for (int o = 16; o > 0; o >>= 1) lsum += __shfl_down_sync(0xffffffffu, lsum, o);
  amax[0] = warp_max_u32(amax[0]);
  amax[1] = warp_max_u32(amax[1]);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) {
    red[w] = lsum;
    redmax[0][w] = amax[0];
    redmax[1][w] = amax[1];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double v = 0.0;
    uint32_t a0 = 0u, a1 = 0u;
    for (int i = 0; i < LOSS_THREADS / 32; ++i) {
      v += red[i];
      a0 = max(a0, redmax[0][i]);
      a1 = max(a1, redmax[1][i]);
    }
    scratch->lsum[blockIdx.x] = v;
    scratch->amax[0][blockIdx.x] = a0;
    scratch->amax[1][blockIdx.x] = a1;
    __threadfence();
    is_last = atomicAdd(&scratch->ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (is_last && threadIdx.x < 32) {
    __threadfence();
    double v = 0.0;
    uint32_t a0 = 0u, a1 = 0u;
    for (int i = lane; i < (int)gridDim.x; i += 32) {
      v += __ldcg(&scratch->lsum[i]);
      a0 = max(a0, __ldcg(&scratch->amax[0][i]));
      a1 = max(a1, __ldcg(&scratch->amax[1][i]));
    }
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    a0 = warp_max_u32(a0);
    a1 = warp_max_u32(a1);
    if (lane == 0) {
      loss[0] = (float)(v * inv_m);
      absmax[3] = __uint_as_float(a0);
      absmax[4] = __uint_as_float(a1);
      scratch->ticket = 0u;  // ready for the next launch on this stream
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Classification by goodness (Sec. III): sample b was presented once per candidate label c (row c*B + b);
// its score for c is the sum over the counted layers of that row's goodness (FP32 additions in layer
// order), its label the candidate with the largest score (lowest label on ties).  One thread per sample.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS) classify_kernel(LaterLayers layers, int B, int n_classes,
                                                              float* __restrict__ scores, int32_t* __restrict__ pred) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  float best = 0.0f;
  int best_c = 0;
  for (int c = 0; c < n_classes; ++c) {
    float total = 0.0f;
    for (int j = 0; j < layers.n; ++j) total = __fadd_rn(total, layers.G[j][(size_t)c * B + b]);
    scores[(size_t)c * B + b] = total;
    if (c == 0 || total > best) {
      best = total;
      best_c = c;
    }
  }
  pred[b] = best_c;
}

// ---------------------------------------------------------------------------------------------
// dHq = clip(round((2*coef_m * y) * 127/a_dh[p])).  grid = (blocks, 2)
// ---------------------------------------------------------------------------------------------
template <int MODE, bool PAD = false>
__device__ __forceinline__ void dh_quantize_body(const float* __restrict__ Y, const float* __restrict__ coef,
                                                 const float* __restrict__ absmax, size_t per_sample, size_t per_pass,
                                                 int8_t* __restrict__ dHq, RoundKey key, int pass, uint32_t bias,
                                                 RowPad rp = RowPad{0u, 0u});
template <int MODE>
__global__ void __launch_bounds__(EW_THREADS) dh_quantize_kernel(const float* __restrict__ Y, const float* __restrict__ coef,
                                                                 const float* __restrict__ absmax, size_t per_sample,
                                                                 size_t per_pass, int8_t* __restrict__ dHq, KeySpec ks,
                                                                 uint2 ctr_bias = uint2{0u, 0u}, RowPad rp = RowPad{0u, 0u}) {
  const RoundKey key = (MODE == ROUND_NEAREST) ? RoundKey{0u, 0u} : derive_key(ks);
  if (rp.extra)
    dh_quantize_body<MODE, true>(Y, coef, absmax, per_sample, per_pass, dHq, key, blockIdx.y, blockIdx.y ? ctr_bias.y : ctr_bias.x, rp);
  else
    dh_quantize_body<MODE, false>(Y, coef, absmax, per_sample, per_pass, dHq, key, blockIdx.y, blockIdx.y ? ctr_bias.y : ctr_bias.x);
}
// Every layer of a step in one launch: blockIdx.y = 2*layer + set.
struct DhJobs {
  const float* Y[FF_MAX_LATER + 1];
  const float* coef[FF_MAX_LATER + 1];
  const float* absmax[FF_MAX_LATER + 1];
  unsigned long long per_sample[FF_MAX_LATER + 1];
  int8_t* dHq[FF_MAX_LATER + 1];
  unsigned long long s1[FF_MAX_LATER + 1];
  uint8_t stochastic[FF_MAX_LATER + 1];
  RowPad pad[FF_MAX_LATER + 1];   // row padding of dHq (dense layers)
  const StepState* ss;
};
template <bool PAD>
__global__ void __launch_bounds__(EW_THREADS) dh_quantize_multi_kernel(const DhJobs jobs, int B, int first = 0) {
  const int l = (blockIdx.y >> 1) + first, pass = blockIdx.y & 1;
  const size_t per_sample = (size_t)jobs.per_sample[l], per_pass = per_sample * B;
  if (jobs.stochastic[l])
    dh_quantize_body<ROUND_STOCHASTIC, PAD>(jobs.Y[l], jobs.coef[l], jobs.absmax[l], per_sample, per_pass, jobs.dHq[l],
                                            derive_key(KeySpec{jobs.s1[l], jobs.ss}), pass, 0u, jobs.pad[l]);
  else
    dh_quantize_body<ROUND_NEAREST, PAD>(jobs.Y[l], jobs.coef[l], jobs.absmax[l], per_sample, per_pass, jobs.dHq[l],
                                         RoundKey{0u, 0u}, pass, 0u, jobs.pad[l]);
}

template <int MODE, bool PAD>
__device__ __forceinline__ void dh_quantize_body(const float* __restrict__ Y, const float* __restrict__ coef,
                                                 const float* __restrict__ absmax, size_t per_sample, size_t per_pass,
                                                 int8_t* __restrict__ dHq, RoundKey key, int pass, uint32_t bias, RowPad rp) {
  const size_t base = (size_t)pass * per_pass;
  const float inv = inv_of(absmax[3 + pass]);
  const bool vec = ((per_sample & 3) == 0) && ((((uintptr_t)Y) & 15) == 0) && ((((uintptr_t)dHq) & 3) == 0);
  const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, stride = gridDim.x * blockDim.x;
  if (vec && per_sample >= 4 * SAMPLE_TILE_GROUPS) {
    // long samples: blocks take (sample, tile of the sample) pairs, so the per-sample factor is read once per
    // tile and no sample bookkeeping rides along with the elements
    const uint32_t g4 = (uint32_t)(per_sample >> 2), n_samples = (uint32_t)(per_pass / per_sample);
    const uint32_t tps = (g4 + SAMPLE_TILE_GROUPS - 1) / SAMPLE_TILE_GROUPS;
    const float* cp = coef + (size_t)pass * n_samples;
    for (uint32_t tile = blockIdx.x; tile < n_samples * tps; tile += gridDim.x) {
      const uint32_t smp = tile / tps, g0 = (tile - smp * tps) * SAMPLE_TILE_GROUPS;
      const float k2 = __fmul_rn(2.0f, __ldg(cp + smp));
      const size_t e0 = base + (size_t)smp * per_sample;
      // all loads of the tile first (Y is not read again in this step: streaming loads), then the arithmetic
      float4 vv[SAMPLE_TILE_GROUPS / EW_THREADS];
#pragma unroll
      for (uint32_t k = 0; k < SAMPLE_TILE_GROUPS / EW_THREADS; ++k) {
        const uint32_t i = g0 + k * EW_THREADS + threadIdx.x;
        if (i < g4) vv[k] = __ldcs(reinterpret_cast<const float4*>(Y + e0 + ((size_t)i << 2)));
      }
#pragma unroll
      for (uint32_t k = 0; k < SAMPLE_TILE_GROUPS / EW_THREADS; ++k) {
        const uint32_t i = g0 + k * EW_THREADS + threadIdx.x;
        if (i >= g4) break;
        const size_t e = e0 + ((size_t)i << 2);
        const float4 v = vv[k];
        int q0, q1, q2, q3;
        quant_pair<MODE>(__fmul_rn(k2, v.x), __fmul_rn(k2, v.y), inv, (uint32_t)e + bias, key, q0, q1);
        quant_pair<MODE>(__fmul_rn(k2, v.z), __fmul_rn(k2, v.w), inv, (uint32_t)e + bias + 2, key, q2, q3);
        *reinterpret_cast<uint32_t*>(dHq + e + (PAD ? (size_t)(pass * n_samples + smp) * rp.extra : (size_t)0)) =
            pack4(q0, q1, q2, q3);
      }
    }
  } else if (vec) {
    const uint32_t n4 = (uint32_t)(per_pass >> 2);
    const float* cp = coef + (uint32_t)(base / per_sample);
    const uint32_t pass_row0 = (uint32_t)(base / per_sample);
    SampleCursor cur(tid, stride, (uint32_t)(per_sample >> 2));
    for (uint32_t i0 = tid; i0 < n4; i0 += 4 * stride) {  // four loads in flight, then the arithmetic
      float4 vv[4];
#pragma unroll
      for (uint32_t k = 0; k < 4; ++k)
        if (i0 + k * stride < n4) vv[k] = __ldcs(reinterpret_cast<const float4*>(Y + base + ((size_t)(i0 + k * stride) << 2)));
#pragma unroll
      for (uint32_t k = 0; k < 4; ++k, cur.advance()) {
        const uint32_t i = i0 + k * stride;
        if (i >= n4) break;
        const size_t e = base + ((size_t)i << 2);
        const float k2 = __fmul_rn(2.0f, __ldg(cp + cur.sample));
        const float4 v = vv[k];
        int q0, q1, q2, q3;
        quant_pair<MODE>(__fmul_rn(k2, v.x), __fmul_rn(k2, v.y), inv, (uint32_t)e + bias, key, q0, q1);
        quant_pair<MODE>(__fmul_rn(k2, v.z), __fmul_rn(k2, v.w), inv, (uint32_t)e + bias + 2, key, q2, q3);
        *reinterpret_cast<uint32_t*>(dHq + e + (PAD ? (size_t)(pass_row0 + cur.sample) * rp.extra : (size_t)0)) =
              pack4(q0, q1, q2, q3);
      }
    }
  } else {
    for (size_t i = tid; i < per_pass; i += stride) {
      size_t e = base + i;
      float k2 = __fmul_rn(2.0f, coef[(uint32_t)e / (uint32_t)per_sample]);
      dHq[PAD ? padded(e, rp) : e] = (int8_t)quant_one<MODE>(__fmul_rn(k2, Y[e]), inv, (uint32_t)e + bias, key);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Positive / negative / candidate batches by label embedding (Sec. III; Alg. 1, sample generation).
// x [B, n] raw samples, labels [sets, B]; out row s*B + b = sample b with labels[s, b] written
// one-hot over the label places (flat positions j*label_stride, j < n_classes: on_value at the label,
// zero elsewhere), then, if tau0 > 0, scaled to length tau0 with
// r = tau0 / (float(sqrt(sum of squares in FP64)) + eps).  The squares of the data entries are summed
// once per sample and shared by all sets.  One block per sample (grid-stride).
// ---------------------------------------------------------------------------------------------
constexpr int EMBED_THREADS = 256;
__global__ void __launch_bounds__(EMBED_THREADS) embed_labels_kernel(const float* __restrict__ x, const int32_t* __restrict__ labels,
                                                                     int B, int n, int sets, int n_classes, int label_stride,
                                                                     float on_value, float tau0, float eps,
                                                                     float* __restrict__ out, uint32_t* __restrict__ status) {
  __shared__ double red[EMBED_THREADS / 32];
  __shared__ double total;
  const int span = (n_classes - 1) * label_stride + 1;      // flat positions below this may be label places
  const int head = min(n, (span + 3) & ~3);                  // handled element by element
  const bool vec = ((n & 3) == 0) && ((((uintptr_t)x) & 15) == 0) && ((((uintptr_t)out) & 15) == 0);
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int b = blockIdx.x; b < B; b += gridDim.x) {
    const float* xr = x + (size_t)b * n;
    double ss = 0.0;
    if (tau0 > 0.0f) {
      for (int k = threadIdx.x; k < head; k += EMBED_THREADS) {
        const bool place = k < span && (k % label_stride) == 0;
        const double v = place ? 0.0 : (double)xr[k];
        ss = fma(v, v, ss);  // the square of a float is exact in double: the fused form rounds once like the sum
      }
      if (vec) {
        for (int k = head + 4 * threadIdx.x; k < n; k += 4 * EMBED_THREADS) {
          const float4 v = __ldg(reinterpret_cast<const float4*>(xr + k));
          ss += (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
        }
      } else {
        for (int k = head + threadIdx.x; k < n; k += EMBED_THREADS) ss += (double)xr[k] * xr[k];
      }
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_down_sync(0xffffffffu, ss, o);
      if (lane == 0) red[wid] = ss;
      __syncthreads();
      if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < EMBED_THREADS / 32; ++i) t += red[i];
        total = t;
      }
      __syncthreads();
    }
    for (int s = 0; s < sets; ++s) {
      int lab = labels[(size_t)s * B + b];
      const bool good = lab >= 0 && lab < n_classes;
      if (!good && threadIdx.x == 0) atomicOr(status, ST_BADLABEL);
      const int hot = good ? lab * label_stride : -1;
      float r = 1.0f;
      if (tau0 > 0.0f) {
        const double sq = total + (good ? (double)on_value * (double)on_value : 0.0);
        r = __fdiv_rn(tau0, __fadd_rn(__double2float_rn(sqrt(sq)), eps));
      }
      float* orow = out + ((size_t)s * B + b) * n;
      for (int k = threadIdx.x; k < head; k += EMBED_THREADS) {
        const bool place = k < span && (k % label_stride) == 0;
        const float v = place ? (k == hot ? on_value : 0.0f) : xr[k];
        orow[k] = tau0 > 0.0f ? __fmul_rn(v, r) : v;
      }
      if (vec) {
        for (int k = head + 4 * threadIdx.x; k < n; k += 4 * EMBED_THREADS) {
          float4 v = __ldg(reinterpret_cast<const float4*>(xr + k));
          if (tau0 > 0.0f) {
            v.x = __fmul_rn(v.x, r);
            v.y = __fmul_rn(v.y, r);
            v.z = __fmul_rn(v.z, r);
            v.w = __fmul_rn(v.w, r);
          }
          __stcs(reinterpret_cast<float4*>(orow + k), v);
        }
      } else {
        for (int k = head + threadIdx.x; k < n; k += EMBED_THREADS) orow[k] = tau0 > 0.0f ? __fmul_rn(xr[k], r) : xr[k];
      }
    }
    __syncthreads();  // `total` is rewritten for the next sample
  }
}

}  // namespace ffi8
