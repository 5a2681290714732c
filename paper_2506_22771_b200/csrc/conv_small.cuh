// 3x3 convolution layers with very few input channels (the first layer of an image network: C_in <= 4, so the
// contraction 9*C_in has at most 36 terms) - Sec. IV-B's INT8 MAC for a convolution layer whose contraction is far
// too short for the tcgen05 tiles: the layer is bounded by writing its FP32 output, and a tile-based kernel spends
// its time on per-tile latencies instead.  Here a block builds the packed INT8 im2col words of 256 consecutive
// output positions in shared memory (zero padding by bounds checks; never written to global memory), the layer's
// weights sit beside them in the same packing, and the products are the warp-level INT8 matrix instruction
// (16 positions x 8 channels x 32 contraction bytes; dp4a, used before, issues at a fraction of its rate and left
// the kernel bound by the integer pipe).  Same integers, same FP32 operations as every other forward route.
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

// D (16 x 8, INT32) += A (16 x 32, INT8, row-major) * B (32 x 8, INT8, column-major): the warp-level INT8 matrix
// instruction.  Lane l holds, with g = l / 4 and t = l % 4: A rows g and g + 8, bytes 4t .. 4t+3 and 16+4t .. of the
// 32 (a0: row g low half, a1: row g+8 low, a2: row g high, a3: row g+8 high); B column g, the same bytes of its
// 32 (b0 low, b1 high); D rows g (c0, c1) and g + 8 (c2, c3), columns 2t and 2t + 1.
__device__ __forceinline__ void mma_s8_16x8x32(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int CIN, int N>
__global__ void __launch_bounds__(CS_THREADS) conv3x3_small_fwd_kernel(const int8_t* __restrict__ xq, const int8_t* __restrict__ wq,
                                                                       float* __restrict__ Y, int32_t* __restrict__ acc_dump,
                                                                       unsigned long long* __restrict__ S,
                                                                       int32_t* __restrict__ rowmax,
                                                                       const float* __restrict__ absmax, ConvSmallGeom g) {
  constexpr int K = 9 * CIN, KS = (K + 31) / 32, KW = KS * 8;   // contraction bytes; steps of 32; packed words per row (zero beyond K)
  constexpr int RS = KW + 4;   // row stride in words: = 4 mod 8, so the 8 rows x 4 words of a fragment load fall into 32 banks
  constexpr int NT = N / 8;    // channel tiles of the matrix instruction
  static_assert(127 * 127 * K < (1 << 23), "the INT32 sums must be exact in a float's mantissa");
  __shared__ __align__(16) uint32_t xi[CS_THREADS * RS];   // im2col words of the tile's positions
  __shared__ __align__(16) uint32_t ws[N * RS];            // the layer's weights in the same packing
  __shared__ unsigned long long red_s[CS_THREADS / 32];
  __shared__ int red_m[CS_THREADS / 32];
  const int lane = threadIdx.x & 31, wv = threadIdx.x >> 5;
  const int gq = lane >> 2, tig = lane & 3;
  for (int i = threadIdx.x; i < N * KW; i += CS_THREADS) {
    const int n = i / KW, j = i - n * KW;
    uint32_t v = 0u;
#pragma unroll
    for (int b = 0; b < 4; ++b)
      if (4 * j + b < K) v |= (uint32_t)(uint8_t)wq[(size_t)n * K + 4 * j + b] << (8 * b);
    ws[n * RS + j] = v;
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
      for (int j = 0; j < KW; j += 4)
        *reinterpret_cast<uint4*>(xi + threadIdx.x * RS + j) = make_uint4(wd[j], wd[j + 1], wd[j + 2], wd[j + 3]);
    }
    __syncthreads();   // (also orders the weights' words before their first use)
    // ---- products and epilogue: warp wv takes positions 32*wv .. 32*wv+31 of the tile, 16 per pass ----
    unsigned long long ssum = 0ull;
    int mx = 0;
#pragma unroll 1
    for (int half = 0; half < 2; ++half) {
      const int pl = 32 * wv + 16 * half + gq;    // this lane's rows of the pass: pl and pl + 8
      const uint32_t* xa = xi + pl * RS + tig;
      uint32_t a[KS][4];
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) a[ks][0] = xa[8 * ks], a[ks][1] = xa[8 * RS + 8 * ks], a[ks][2] = xa[8 * ks + 4], a[ks][3] = xa[8 * RS + 8 * ks + 4];
      const int pa = tile * CS_THREADS + pl, pb = pa + 8;
      const bool oka = pa < g.rows, okb = pb < g.rows;
      const float csa = pa < g.rows_per_pass ? c0 : c1, csb = pb < g.rows_per_pass ? c0 : c1;
      float* ya = Y + (size_t)pa * N + 2 * tig;
      float* yb = Y + (size_t)pb * N + 2 * tig;
      unsigned long long sa = 0ull, sb = 0ull;
      int ma = 0, mb = 0;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        int c[4] = {0, 0, 0, 0};
        const uint32_t* wb = ws + (nt * 8 + gq) * RS + tig;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) mma_s8_16x8x32(c, a[ks][0], a[ks][1], a[ks][2], a[ks][3], wb[8 * ks], wb[8 * ks + 4]);
        unsigned rl[4];
        float y[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          rl[q] = (unsigned)max(c[q], 0);
          // exact: rl < 2^23, so placing it in the mantissa of 2^23 and subtracting 2^23 is the integer as a float
          y[q] = __fmul_rn(__fsub_rn(__uint_as_float(rl[q] | 0x4B000000u), 8388608.0f), q < 2 ? csa : csb);
        }
        sa += (unsigned long long)rl[0] * rl[0] + (unsigned long long)rl[1] * rl[1];
        sb += (unsigned long long)rl[2] * rl[2] + (unsigned long long)rl[3] * rl[3];
        ma = max(ma, (int)max(rl[0], rl[1]));
        mb = max(mb, (int)max(rl[2], rl[3]));
        if (oka) {
          if (g.y_stream)
            __stcs(reinterpret_cast<float2*>(ya + nt * 8), make_float2(y[0], y[1]));
          else
            *reinterpret_cast<float2*>(ya + nt * 8) = make_float2(y[0], y[1]);
        }
        if (okb) {
          if (g.y_stream)
            __stcs(reinterpret_cast<float2*>(yb + nt * 8), make_float2(y[2], y[3]));
          else
            *reinterpret_cast<float2*>(yb + nt * 8) = make_float2(y[2], y[3]);
        }
        if (acc_dump) {
          if (oka) *reinterpret_cast<int2*>(acc_dump + (size_t)pa * N + nt * 8 + 2 * tig) = make_int2(c[0], c[1]);
          if (okb) *reinterpret_cast<int2*>(acc_dump + (size_t)pb * N + nt * 8 + 2 * tig) = make_int2(c[2], c[3]);
        }
      }
      if (!oka) sa = 0ull, ma = 0;
      if (!okb) sb = 0ull, mb = 0;
      if (tile_in_sample) {
        ssum += sa + sb;
        mx = max(mx, max(ma, mb));
      } else {
        // positions of a warp may belong to different samples: add up over the four lanes of a position
#pragma unroll
        for (int o = 1; o <= 2; o <<= 1) {
          sa += __shfl_xor_sync(0xffffffffu, sa, o);
          sb += __shfl_xor_sync(0xffffffffu, sb, o);
          ma = max(ma, __shfl_xor_sync(0xffffffffu, ma, o));
          mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
        }
        if (tig == 0 && oka && ma > 0) {
          atomicAdd(S + pa / g.rows_per_sample, sa);
          atomicMax(rowmax + pa / g.rows_per_sample, ma);
        }
        if (tig == 0 && okb && mb > 0) {
          atomicAdd(S + pb / g.rows_per_sample, sb);
          atomicMax(rowmax + pb / g.rows_per_sample, mb);
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

// ---------------------------------------------------------------------------------------------
// Weight gradient of the same layers: sums[set][n][k] = sum over the set's output positions of
// dHq[pos][n] * x_im2col[pos][k]  (k = (r*3+s)*C_in + ci; INT8 x INT8 -> INT32, Sec. IV-B / Alg. 1, update step).
// The contraction runs over positions, so both operands are repacked in shared memory with four CONSECUTIVE
// POSITIONS per word (a 4 x 4 byte transpose of dHq rows, a gather of input bytes) - which is the operand layout
// of the warp-level INT8 matrix instruction (m16n8k32: 16 channels x 8 contraction indices x 32 positions per
// instruction; at 9*C_in <= 36 contraction indices and a few dozen channels the tcgen05 tile sizes do not apply,
// and dp4a issues at a fraction of this rate).  The loads of the next chunk of 256 positions are in flight while
// the current chunk's products run.
// A block works inside one (slab, set) plane: the planes cut each set's positions into parts of at most
// WG_SAFE_LEN positions, so neither a register sum nor a plane's sum can leave INT32; the block's sums go to the
// plane with integer atomics (exact, order-free; the planes are zero before) and the slab update kernel adds the
// planes in 64 bits.  slabs [n_slabs][2][N][9*C_in].
// ---------------------------------------------------------------------------------------------
constexpr int CW_CHUNK = 256;            // positions per chunk (= threads per block)
constexpr int CW_PW = CW_CHUNK / 4;      // position words per chunk

struct ConvSmallWgradGeom {
  int H, W, Ho, Wo, stride;
  int B;                      // images per set
  int rows_per_pass;          // output positions of one set
  int chunks;                 // chunks per set
  int chunks_per_slab;        // <= WG_SAFE_LEN / CW_CHUNK
  int n_slabs;
  int blocks_per_plane;       // gridDim.x = 2 * n_slabs * blocks_per_plane
};

template <int CIN, int N>
__global__ void __launch_bounds__(CS_THREADS, (CIN <= 3 ? 2 : 1)) conv3x3_small_wgrad_kernel(const int8_t* __restrict__ xq, const int8_t* __restrict__ dhq,
                                                                         int32_t* __restrict__ slabs, ConvSmallWgradGeom g) {
  constexpr int K = 9 * CIN, KT = (K + 7) / 8, KT8 = KT * 8;   // contraction indices; tiles of eight; padded count
  constexpr int NG = N / 4;                                    // groups of four channels (one dHq word per position)
  // row strides (words) of dT[pw][n] and xT[pw][k]: = 8 or 24 mod 32, so that the eight channels (indices) x four
  // position words a fragment load touches fall into 32 different banks
  constexpr int NS = N + 8;
  constexpr int XS = (KT8 % 32 == 8 || KT8 % 32 == 24) ? KT8 : KT8 + 8;
  constexpr int MT = N / 16, KGRP = 8 / MT;                    // channel tiles; warps that share a channel tile split the position words
  constexpr int DT_WORDS = CW_PW * NS, XT_WORDS = CW_PW * XS, RED_WORDS = KGRP * N * KT8;
  constexpr int SM_WORDS = (DT_WORDS + XT_WORDS) > RED_WORDS ? (DT_WORDS + XT_WORDS) : RED_WORDS;
  constexpr int DTASKS = (CW_PW * NG + CS_THREADS - 1) / CS_THREADS;   // 4 x 4 transposes per thread and chunk
  constexpr int XTASKS = CW_PW * KT8 / CS_THREADS;                     // gathered words per thread and chunk
  __shared__ __align__(16) uint32_t sm[SM_WORDS];
  __shared__ int4 s_pos[CW_CHUNK];   // per position of the chunk: first input row of its image, input row / column of tap (0, 0)
  uint32_t* dT = sm;
  uint32_t* xT = sm + DT_WORDS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int plane = blockIdx.x / g.blocks_per_plane, bip = blockIdx.x - plane * g.blocks_per_plane;
  const int slab = plane >> 1, set = plane & 1;
  const int c_begin = slab * g.chunks_per_slab, c_end = min(g.chunks, c_begin + g.chunks_per_slab);
  const bool row4 = (g.Wo & 3) == 0;   // the four positions of a word share an output row (and a set's positions are a multiple of four)
  const bool run4 = row4 && g.stride == 1;
  int acc[KT][4];
#pragma unroll
  for (int t = 0; t < KT; ++t)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[t][i] = 0;
  uint32_t dw[DTASKS][4];   // the next chunk's dHq words (rows of four positions) ...
  uint32_t xb[XTASKS][4];   // ... and input bytes
  auto decode_chunk = [&](int ch) {
    const int p = ch * CW_CHUNK + tid;   // position inside the set
    const int wo = p % g.Wo, t = p / g.Wo, ho = t % g.Ho, img = t / g.Ho;
    s_pos[tid] = p < g.rows_per_pass ? make_int4((set * g.B + img) * g.H, ho * g.stride - 1, wo * g.stride - 1, 0)
                                     : make_int4(0, -(1 << 24), 0, 0);   // every tap out of bounds
  };
  auto load_chunk = [&](int ch) {   // needs decode_chunk(ch) and a barrier before
    const int p0 = ch * CW_CHUNK;
#pragma unroll
    for (int q = 0; q < DTASKS; ++q) {
      const int t = tid + q * CS_THREADS, pw = t / NG, cg = t - pw * NG;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int p = p0 + 4 * pw + j;
        dw[q][j] = (t < CW_PW * NG && p < g.rows_per_pass)
                       ? __ldg(reinterpret_cast<const uint32_t*>(dhq + ((size_t)set * g.rows_per_pass + p) * N) + cg)
                       : 0u;
      }
    }
    if (run4) {
      // stride 1 and the four positions of a word in one output row: for filter row r the word's bytes all come
      // from the 6 * C_in consecutive bytes of input pixels wo - 1 .. wo + 4 - one thread per (position word, r)
      if (tid < 3 * CW_PW) {
        const int r = tid / CW_PW, pw = tid - r * CW_PW;
        const int4 ps = s_pos[4 * pw];
        const int hh = ps.y + r;
        const bool row_in = hh >= 0 && hh < g.H;
        const int8_t* src = xq + ((long long)(ps.x + hh) * g.W + ps.z) * CIN;   // dereferenced only where in bounds
#pragma unroll
        for (int i = 0; i < 6 * CIN; ++i) {
          const int ww = ps.z + i / CIN;
          xb[i >> 2][i & 3] = (row_in && ww >= 0 && ww < g.W) ? (uint32_t)(uint8_t)__ldg(src + i) : 0u;
        }
      }
    } else if (row4) {
      // the four positions of a word lie in one output row: one row test and one address per word
      const int dj = g.stride * CIN;
#pragma unroll
      for (int q = 0; q < XTASKS; ++q) {
        const int t = tid + q * CS_THREADS, pw = t / KT8, k = t - pw * KT8;
        const int tap = k / CIN, ci = k - tap * CIN, r = tap / 3, s = tap - 3 * r;
        const int4 ps = s_pos[4 * pw];
        const int hh = ps.y + r, w0 = ps.z + s;
        const bool row_in = k < K && hh >= 0 && hh < g.H;
        const int8_t* src = xq + ((long long)(ps.x + hh) * g.W + w0) * CIN + ci;   // dereferenced only where in bounds
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int ww = w0 + j * g.stride;
          xb[q][j] = (row_in && ww >= 0 && ww < g.W) ? (uint32_t)(uint8_t)__ldg(src + j * dj) : 0u;
        }
      }
    } else {
#pragma unroll
      for (int q = 0; q < XTASKS; ++q) {
        const int t = tid + q * CS_THREADS, pw = t / KT8, k = t - pw * KT8;
        const int tap = k / CIN, ci = k - tap * CIN, r = tap / 3, s = tap - 3 * r;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int4 ps = s_pos[4 * pw + j];
          const int hh = ps.y + r, ww = ps.z + s;
          const bool in = k < K && hh >= 0 && hh < g.H && ww >= 0 && ww < g.W;
          xb[q][j] = in ? (uint32_t)(uint8_t)__ldg(xq + ((size_t)(ps.x + hh) * g.W + ww) * CIN + ci) : 0u;
        }
      }
    }
  };
  const int gq = lane >> 2, tig = lane & 3;          // fragment coordinates of this lane
  const int m0 = (warp % MT) * 16, grp = warp / MT;  // channel tile and position-word group of this warp
  for (int i = tid; i < XT_WORDS; i += CS_THREADS) xT[i] = 0u;   // contraction indices beyond 9 * C_in stay zero
  int ch = c_begin + bip;
  if (ch < c_end) {
    decode_chunk(ch);
    __syncthreads();
    load_chunk(ch);
  }
  for (; ch < c_end; ch += g.blocks_per_plane) {
    __syncthreads();   // the previous chunk's words and positions have been used
    // ---- dT: 4 x 4 byte transposes of the dHq words;  xT: the gathered bytes as words ----
#pragma unroll
    for (int q = 0; q < DTASKS; ++q) {
      const int t = tid + q * CS_THREADS, pw = t / NG, cg = t - pw * NG;
      if (t < CW_PW * NG) {
        const uint32_t t0 = __byte_perm(dw[q][0], dw[q][1], 0x5140), t1 = __byte_perm(dw[q][2], dw[q][3], 0x5140);
        const uint32_t t2 = __byte_perm(dw[q][0], dw[q][1], 0x7362), t3 = __byte_perm(dw[q][2], dw[q][3], 0x7362);
        uint4 o;
        o.x = __byte_perm(t0, t1, 0x5410);
        o.y = __byte_perm(t0, t1, 0x7632);
        o.z = __byte_perm(t2, t3, 0x5410);
        o.w = __byte_perm(t2, t3, 0x7632);
        *reinterpret_cast<uint4*>(dT + pw * NS + 4 * cg) = o;
      }
    }
    if (run4) {
      if (tid < 3 * CW_PW) {
        const int r = tid / CW_PW, pw = tid - r * CW_PW;
#pragma unroll
        for (int sc = 0; sc < 3 * CIN; ++sc) {   // sc = s * C_in + ci: byte j of the word is pixel j + s, channel ci
          const int i0 = sc, i1 = sc + CIN, i2 = sc + 2 * CIN, i3 = sc + 3 * CIN;
          xT[pw * XS + r * 3 * CIN + sc] =
              xb[i0 >> 2][i0 & 3] | (xb[i1 >> 2][i1 & 3] << 8) | (xb[i2 >> 2][i2 & 3] << 16) | (xb[i3 >> 2][i3 & 3] << 24);
        }
      }
    } else {
#pragma unroll
      for (int q = 0; q < XTASKS; ++q) {
        const int t = tid + q * CS_THREADS, pw = t / KT8, k = t - pw * KT8;
        xT[pw * XS + k] = xb[q][0] | (xb[q][1] << 8) | (xb[q][2] << 16) | (xb[q][3] << 24);
      }
    }
    const int next = ch + g.blocks_per_plane;
    if (next < c_end) decode_chunk(next);
    __syncthreads();
    if (next < c_end) load_chunk(next);   // in flight during the products
    // ---- products: A = dT (channels x positions), B = xT (positions x contraction indices) ----
#pragma unroll 2
    for (int ks = grp; ks < CW_PW / 8; ks += KGRP) {
      const uint32_t* da = dT + (ks * 8 + tig) * NS + m0 + gq;
      const uint32_t a0 = da[0], a1 = da[8], a2 = da[4 * NS], a3 = da[4 * NS + 8];
      const uint32_t* xa = xT + (ks * 8 + tig) * XS + gq;
#pragma unroll
      for (int t = 0; t < KT; ++t) mma_s8_16x8x32(acc[t], a0, a1, a2, a3, xa[t * 8], xa[4 * XS + t * 8]);
    }
  }
  // ---- the block's sums: add the position-word groups in shared memory, one atomic per (channel, index) ----
  __syncthreads();
#pragma unroll
  for (int t = 0; t < KT; ++t) {
    uint32_t* r0 = sm + ((grp * N + m0 + gq) * KT8 + t * 8 + 2 * tig);
    r0[0] = (uint32_t)acc[t][0], r0[1] = (uint32_t)acc[t][1];
    r0[8 * KT8] = (uint32_t)acc[t][2], r0[8 * KT8 + 1] = (uint32_t)acc[t][3];
  }
  __syncthreads();
  int32_t* out = slabs + (size_t)plane * N * K;
  for (int e = tid; e < N * K; e += CS_THREADS) {
    const int n = e / K, k = e - n * K;
    int sum = 0;
#pragma unroll
    for (int q = 0; q < KGRP; ++q) sum += (int)sm[(q * N + n) * KT8 + k];
    if (sum) atomicAdd(out + e, sum);
  }
}

}  // namespace ffi8
