// 3x3 convolution layers with very few input channels (the first layer of an image network: C_in <= 4, so the
// contraction 9*C_in has at most 36 terms) - Sec. IV-B's INT8 MAC for a convolution layer whose contraction is far
// too short for the tensor cores: the layer is bounded by writing its FP32 output, and a tile-based tensor-core
// kernel spends its time on per-tile latencies instead.  Here a block builds the packed INT8 im2col words of 256
// consecutive output positions in shared memory (zero padding by bounds checks; never written to global memory),
// every thread keeps the INT8 weights of its four output channels in registers, and the products are dp4a
// (four INT8 MACs into INT32).  Lanes are laid out so that each store instruction of a warp writes whole rows of
// Y (4*N bytes contiguous per position).  Same integers, same FP32 operations as every other forward route.
#pragma once
#include "common.cuh"

namespace ffi8 {

constexpr int CS_THREADS = 256;   // = output positions per tile

struct ConvSmallGeom {
  int H, W, Ho, Wo, stride;   // input and output extents
  int N;                      // output channels: 16, 32, 64 or 128
  int rows;                   // output positions of both sets
  int rows_per_pass;          // positions of one set
  int rows_per_sample;        // Ho * Wo
  int y_stream;               // Y is larger than L2 can usefully hold: streaming stores
};

inline bool conv_small_ok(int kind_is_conv3x3, int Cin, int N) {
  return kind_is_conv3x3 && Cin >= 1 && Cin <= 4 && (N == 16 || N == 32 || N == 64 || N == 128);
}

template <int CIN, int LP>   // LP = N / 4: lanes that share a position (4 channels each)
__global__ void __launch_bounds__(CS_THREADS) conv3x3_small_fwd_kernel(const int8_t* __restrict__ xq, const int8_t* __restrict__ wq,
                                                                       float* __restrict__ Y, int32_t* __restrict__ acc_dump,
                                                                       unsigned long long* __restrict__ S,
                                                                       int32_t* __restrict__ rowmax,
                                                                       const float* __restrict__ absmax, ConvSmallGeom g) {
  constexpr int K = 9 * CIN, KW = (K + 3) / 4;   // contraction bytes, packed words
  __shared__ uint32_t xi[CS_THREADS * KW];
  __shared__ unsigned long long red_s[CS_THREADS / 32];
  __shared__ int red_m[CS_THREADS / 32];
  const int lane = threadIdx.x & 31, wv = threadIdx.x >> 5;
  constexpr int ppi = 32 / LP;                    // positions a warp takes per iteration
  const int cg = lane % LP, ps = lane / LP;       // channel group, position slot
  // the four channels' weights, packed like the im2col words (k = (r*3+s)*CIN + ci; bytes beyond K are zero)
  uint32_t wr[4][KW];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int8_t* wrow = wq + (size_t)(4 * cg + c) * K;
#pragma unroll
    for (int j = 0; j < KW; ++j) {
      uint32_t v = 0u;
#pragma unroll
      for (int b = 0; b < 4; ++b)
        if (4 * j + b < K) v |= (uint32_t)(uint8_t)wrow[4 * j + b] << (8 * b);
      wr[c][j] = v;
    }
  }
  const float s_w = scale_of(absmax[2]);
  const float c0 = __fmul_rn(scale_of(absmax[0]), s_w), c1 = __fmul_rn(scale_of(absmax[1]), s_w);
  const bool tile_in_sample = (g.rows_per_sample % CS_THREADS) == 0;   // a tile of 256 positions lies in one sample
  const int tiles = (g.rows + CS_THREADS - 1) / CS_THREADS;
  for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    // ---- packed im2col words of the tile's positions: one position per thread ----
    {
      const int p = tile * CS_THREADS + threadIdx.x;
      uint32_t wd[KW];
#pragma unroll
      for (int j = 0; j < KW; ++j) wd[j] = 0u;
      if (p < g.rows) {
        const int wo = p % g.Wo, t = p / g.Wo, ho = t % g.Ho, img = t / g.Ho;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          const int hh = ho * g.stride + r - 1;
#pragma unroll
          for (int s = 0; s < 3; ++s) {
            const int ww = wo * g.stride + s - 1;
            const bool in = hh >= 0 && hh < g.H && ww >= 0 && ww < g.W;
            const int8_t* src = xq + ((size_t)(img * g.H + (in ? hh : 0)) * g.W + (in ? ww : 0)) * CIN;
#pragma unroll
            for (int ci = 0; ci < CIN; ++ci) {
              const int k = (r * 3 + s) * CIN + ci;
              const uint32_t v = in ? (uint32_t)(uint8_t)__ldg(src + ci) : 0u;
              wd[k >> 2] |= v << (8 * (k & 3));
            }
          }
        }
      }
#pragma unroll
      for (int j = 0; j < KW; ++j) xi[threadIdx.x * KW + j] = wd[j];
    }
    __syncthreads();
    // ---- MACs and epilogue: warp wv takes positions 32*wv .. 32*wv+31 of the tile, ppi per iteration ----
    unsigned long long ssum = 0ull;
    int mx = 0;
#pragma unroll 4
    for (int it = 0; it < LP; ++it) {
      const int pl = 32 * wv + it * ppi + ps;
      const int p = tile * CS_THREADS + pl;
      int acc[4] = {0, 0, 0, 0};
#pragma unroll
      for (int j = 0; j < KW; ++j) {
        const int xw = (int)xi[pl * KW + j];
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[c] = __dp4a(xw, (int)wr[c][j], acc[c]);
      }
      unsigned long long ps_sum = 0ull;
      int ps_max = 0;
      if (p < g.rows) {
        const float cs = p < g.rows_per_pass ? c0 : c1;
        float y[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const unsigned rl = (unsigned)max(acc[c], 0);
          y[c] = __fmul_rn(__uint2float_rn(rl), cs);
          ps_sum += (unsigned long long)rl * rl;
          ps_max = max(ps_max, (int)rl);
        }
        float4* dst = reinterpret_cast<float4*>(Y + (size_t)p * g.N + 4 * cg);
        if (g.y_stream)
          __stcs(dst, make_float4(y[0], y[1], y[2], y[3]));
        else
          *dst = make_float4(y[0], y[1], y[2], y[3]);
        if (acc_dump) *reinterpret_cast<int4*>(acc_dump + (size_t)p * g.N + 4 * cg) = make_int4(acc[0], acc[1], acc[2], acc[3]);
      }
      if (tile_in_sample) {
        ssum += ps_sum;
        mx = max(mx, ps_max);
      } else {
        // positions of a warp may belong to different samples: add up over the LP lanes of the position
        for (int o = LP >> 1; o > 0; o >>= 1) {
          ps_sum += __shfl_xor_sync(0xffffffffu, ps_sum, o);
          ps_max = max(ps_max, __shfl_xor_sync(0xffffffffu, ps_max, o));
        }
        if (cg == 0 && p < g.rows && ps_max > 0) {
          atomicAdd(S + p / g.rows_per_sample, ps_sum);
          atomicMax(rowmax + p / g.rows_per_sample, ps_max);
        }
      }
    }
    if (tile_in_sample) {   // one pair of atomics per block and tile
      for (int o = 16; o > 0; o >>= 1) ssum += __shfl_xor_sync(0xffffffffu, ssum, o);
      mx = __reduce_max_sync(0xffffffffu, mx);
      if (lane == 0) {
        red_s[wv] = ssum;
        red_m[wv] = mx;
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        unsigned long long tot = 0ull;
        int m = 0;
        for (int i = 0; i < CS_THREADS / 32; ++i) {
          tot += red_s[i];
          m = max(m, red_m[i]);
        }
        if (m > 0) {
          const int sample = tile * CS_THREADS / g.rows_per_sample;
          atomicAdd(S + sample, tot);
          atomicMax(rowmax + sample, m);
        }
      }
    }
    __syncthreads();   // the next tile rewrites xi (and red_*)
  }
}

}  // namespace ffi8
