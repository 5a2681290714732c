// Depthwise 3x3 convolution layers (one filter per channel, no sum over channels; stride 1 or 2, zero
// padding 1, NHWC): the INT8 MAC with INT32 accumulation of Sec. IV-B for the depthwise layers of the
// paper's mobile models (Table II).  Nine multiply-adds per output value and no reuse across channels:
// this is streaming work bound by HBM (1 B read + 4 B written per output), not a contraction, so it runs
// on the integer pipes (dp4a against operands spread one per byte lane) and not on the tensor cores.
#pragma once
#include <cstdint>

#include "common.cuh"

namespace ffi8 {

constexpr int DW_THREADS = 256;
constexpr int DW_WB = 4;  // horizontally adjacent output positions per thread (they share the loaded input window)

struct DwGeom {
  int H, W, C, Ho, Wo, stride;
  int rows;             // output positions of both sets: 2*B*Ho*Wo
  int rows_per_pass;    // B*Ho*Wo
  int rows_per_sample;  // Ho*Wo
  int imgs_per_pass;    // B
  int wblocks;          // ceil(Wo / DW_WB)
};

// The input words (four channels each) under DW_WB adjacent outputs: 3 rows of (DW_WB-1)*STRIDE + 3 pixels
// starting at (hh0, ww0) = (ho*STRIDE - 1, wo0*STRIDE - 1); zero outside the image (zero padding).
template <int STRIDE>
struct DwWindow {
  static constexpr int NW = (DW_WB - 1) * STRIDE + 3;
  uint32_t w[3][NW];
  __device__ __forceinline__ void load(const int8_t* __restrict__ xq, int img, int hh0, int ww0, int cg, const DwGeom& g) {
    const size_t pix = (size_t)g.C, line = (size_t)g.W * pix;
    if (hh0 >= 0 && hh0 + 3 <= g.H && ww0 >= 0 && ww0 + NW <= g.W) {
      // the whole window lies inside the image: one base address, constant offsets, no tests
      const int8_t* base = xq + (((size_t)img * g.H + hh0) * g.W + ww0) * pix + 4 * (size_t)cg;
#pragma unroll
      for (int r = 0; r < 3; ++r)
#pragma unroll
        for (int i = 0; i < NW; ++i) w[r][i] = __ldg(reinterpret_cast<const uint32_t*>(base + r * line + i * pix));
      return;
    }
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const int hh = hh0 + r;
      const bool row_in = hh >= 0 && hh < g.H;
      const int8_t* rowp = xq + ((size_t)img * g.H + (row_in ? hh : 0)) * line + 4 * (size_t)cg;
#pragma unroll
      for (int i = 0; i < NW; ++i) {
        const int ww = ww0 + i;
        w[r][i] = (row_in && ww >= 0 && ww < g.W) ? __ldg(reinterpret_cast<const uint32_t*>(rowp + (size_t)ww * pix)) : 0u;
      }
    }
  }
};

// Position of a work item (four channels cg of output block wb in output row ho of image img) that is
// advanced by a fixed number of items per loop trip with carries instead of divisions.
struct DwCursor {
  int cg, wb, ho, img;
  int d_cg, d_wb, d_ho, d_img;
  int CG, WBK, Ho;
  __device__ __forceinline__ DwCursor(uint32_t item, uint32_t step, int CG_, int WBK_, int Ho_) : CG(CG_), WBK(WBK_), Ho(Ho_) {
    split(item, cg, wb, ho, img);
    split(step, d_cg, d_wb, d_ho, d_img);
  }
  __device__ __forceinline__ void split(uint32_t v, int& c, int& w, int& h, int& i) const {
    uint32_t q = v / (uint32_t)CG;
    c = (int)(v - q * CG);
    uint32_t q2 = q / (uint32_t)WBK;
    w = (int)(q - q2 * WBK);
    uint32_t q3 = q2 / (uint32_t)Ho;
    h = (int)(q2 - q3 * Ho);
    i = (int)q3;
  }
  __device__ __forceinline__ void advance() {
    cg += d_cg;
    int c = cg >= CG;
    cg -= c ? CG : 0;
    wb += d_wb + c;
    c = wb >= WBK;
    wb -= c ? WBK : 0;
    ho += d_ho + c;
    c = ho >= Ho;
    ho -= c ? Ho : 0;
    img += d_img + c;
  }
};

// Forward, C % 4 == 0: acc[pos, c] = sum_{r,s} xq[window(pos, r, s), c] * wq[c, r*3+s];
// y = max(0, float(acc)*c_pass); per-sample exact sum of relu(acc)^2 and max of relu(acc) by integer atomics
// (S and rowmax zero on entry).  One thread per (image row, block of DW_WB outputs, four channels).  The
// weights of all channels sit in shared memory as words holding one weight in byte lane j and zeros
// elsewhere, so that dp4a(x word, weight word) is the product for channel j alone.
template <int STRIDE>
__global__ void __launch_bounds__(DW_THREADS) dwconv3x3_fwd_kernel(const int8_t* __restrict__ xq, const int8_t* __restrict__ wq,
                                                                  float* __restrict__ Y, int32_t* __restrict__ acc_dump,
                                                                  unsigned long long* __restrict__ S, int32_t* __restrict__ rowmax,
                                                                  const float* __restrict__ absmax, DwGeom g) {
  extern __shared__ uint32_t dw_tab[];  // [C/4][9][4] words
  const uint32_t CG = (uint32_t)g.C >> 2;
  for (uint32_t i = threadIdx.x; i < CG * 36; i += DW_THREADS) {
    const uint32_t cg = i / 36, rem = i - cg * 36, t = rem >> 2, j = rem & 3;
    dw_tab[i] = (uint32_t)(uint8_t)wq[(size_t)(4 * cg + j) * 9 + t] << (8 * j);
  }
  __syncthreads();
  const float s_w = scale_of(absmax[2]);
  const float c0 = __fmul_rn(scale_of(absmax[0]), s_w), c1 = __fmul_rn(scale_of(absmax[1]), s_w);
  const uint32_t total = (uint32_t)(2 * g.imgs_per_pass) * g.Ho * g.wblocks * CG;  // < 2^32: fewer items than outputs
  const int lane = threadIdx.x & 31;
  // a block takes a contiguous range of items, so that a warp stays inside one sample for many trips and its
  // goodness statistics can ride in registers until the sample changes
  const uint32_t per_block = ((total + gridDim.x - 1) / gridDim.x + DW_THREADS - 1) / DW_THREADS * DW_THREADS;
  const uint32_t begin = min(total, blockIdx.x * per_block), end = min(total, begin + per_block);
  DwCursor cur(begin + threadIdx.x, DW_THREADS, (int)CG, g.wblocks, g.Ho);
  int held = -1;  // sample whose statistics the warp is holding (warp-uniform), -1: none
  unsigned long long ssum = 0ull;
  int mx = 0;
  auto flush = [&]() {
    if (held >= 0) {
      for (int o = 16; o > 0; o >>= 1) ssum += __shfl_xor_sync(0xffffffffu, ssum, o);
      mx = __reduce_max_sync(0xffffffffu, mx);
      if (lane == 0 && mx > 0) {
        atomicAdd(S + held, ssum);
        atomicMax(rowmax + held, mx);
      }
    }
    held = -1;
    ssum = 0ull;
    mx = 0;
  };
  for (uint32_t base = begin + (threadIdx.x & ~31u); base < end; base += DW_THREADS, cur.advance()) {
    const bool valid = base + lane < end;
    const int img = valid ? cur.img : -1;
    const int first = __shfl_sync(0xffffffffu, img, 0), last = __shfl_sync(0xffffffffu, img, 31);
    const bool uniform = first == last;  // every lane valid and in the same sample
    if (!uniform || first != held) flush();
    if (uniform) held = first;
    if (!valid) continue;
    const int ho = cur.ho, wo0 = cur.wb * DW_WB, cg = cur.cg;
    int acc[DW_WB][4];
#pragma unroll
    for (int o = 0; o < DW_WB; ++o)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[o][j] = 0;
    DwWindow<STRIDE> win;
    win.load(xq, img, ho * STRIDE - 1, wo0 * STRIDE - 1, cg, g);
#pragma unroll
    for (int r = 0; r < 3; ++r)
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        const uint4 tw = *reinterpret_cast<const uint4*>(dw_tab + (cg * 9 + r * 3 + s) * 4);
#pragma unroll
        for (int o = 0; o < DW_WB; ++o) {
          const int xw = (int)win.w[r][o * STRIDE + s];
          acc[o][0] = __dp4a(xw, (int)tw.x, acc[o][0]);
          acc[o][1] = __dp4a(xw, (int)tw.y, acc[o][1]);
          acc[o][2] = __dp4a(xw, (int)tw.z, acc[o][2]);
          acc[o][3] = __dp4a(xw, (int)tw.w, acc[o][3]);
        }
      }
    const float c = img < g.imgs_per_pass ? c0 : c1;
    unsigned long long ts = 0ull;
    int tm = 0;
    const size_t off0 = (((size_t)img * g.Ho + ho) * g.Wo + wo0) * g.C + 4 * (size_t)cg;
#pragma unroll
    for (int o = 0; o < DW_WB; ++o) {
      if (wo0 + o >= g.Wo) break;
      float y[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int a = max(acc[o][j], 0);
        y[j] = __fmul_rn(__uint2float_rn((unsigned)a), c);
        ts += (unsigned long long)(unsigned)a * (unsigned long long)(unsigned)a;  // up to (9*127*127)^2: needs 64 bits
        tm = max(tm, a);
      }
      const size_t off = off0 + (size_t)o * g.C;
      __stcs(reinterpret_cast<float4*>(Y + off), make_float4(y[0], y[1], y[2], y[3]));
      if (acc_dump) *reinterpret_cast<int4*>(acc_dump + off) = make_int4(acc[o][0], acc[o][1], acc[o][2], acc[o][3]);
    }
    if (uniform) {
      ssum += ts;
      mx = max(mx, tm);
    } else if (tm > 0) {  // a warp that straddles two samples (or the end of the range): every lane for itself
      atomicAdd(S + img, ts);
      atomicMax(rowmax + img, tm);
    }
  }
  flush();
}

// Forward for any channel count: one thread per output value (slow path for C % 4 != 0).
__global__ void __launch_bounds__(DW_THREADS) dwconv3x3_fwd_scalar_kernel(const int8_t* __restrict__ xq, const int8_t* __restrict__ wq,
                                                                         float* __restrict__ Y, int32_t* __restrict__ acc_dump,
                                                                         unsigned long long* __restrict__ S,
                                                                         int32_t* __restrict__ rowmax,
                                                                         const float* __restrict__ absmax, DwGeom g) {
  const float s_w = scale_of(absmax[2]);
  const float c0 = __fmul_rn(scale_of(absmax[0]), s_w), c1 = __fmul_rn(scale_of(absmax[1]), s_w);
  const uint32_t total = (uint32_t)g.rows * g.C;
  for (uint32_t item = blockIdx.x * DW_THREADS + threadIdx.x; item < total; item += gridDim.x * DW_THREADS) {
    const uint32_t row = item / g.C, ch = item - row * g.C;
    const int wo = row % g.Wo, t1 = row / g.Wo, ho = t1 % g.Ho, img = t1 / g.Ho;
    int acc = 0;
    for (int r = 0; r < 3; ++r) {
      const int hh = ho * g.stride + r - 1;
      if (hh < 0 || hh >= g.H) continue;
      for (int s = 0; s < 3; ++s) {
        const int ww = wo * g.stride + s - 1;
        if (ww < 0 || ww >= g.W) continue;
        acc += (int)xq[(((size_t)img * g.H + hh) * g.W + ww) * g.C + ch] * (int)wq[(size_t)ch * 9 + r * 3 + s];
      }
    }
    const int a = max(acc, 0);
    Y[item] = __fmul_rn(__uint2float_rn((unsigned)a), img < g.imgs_per_pass ? c0 : c1);
    if (acc_dump) acc_dump[item] = acc;
    if (a > 0) {
      atomicAdd(S + img, (unsigned long long)a * (unsigned long long)a);
      atomicMax(rowmax + img, a);
    }
  }
}

// Weight gradient, C % 4 == 0: accW[p, c, r*3+s] += sum over the positions of set p of
// dhq[pos, c] * xq[window(pos, r, s), c]  (INT32, integer atomics: exact and order-free; accW zero on entry).
// A block takes a chunk of output-position blocks (blockIdx.x) for 32 channel groups (blockIdx.y) of one set
// (blockIdx.z); its 8 warps stride through the chunk, every lane holding the 36 sums of its four channels, and
// meet in shared memory.  dp4a(x word, dh word with only byte j kept) is the product for channel j alone.
// The sums are kept in planes [plane][2][C][9]: blocks_per_plane consecutive chunks share a plane, chosen by the
// host so that no plane sums over more than WG_SAFE_LEN positions (no INT32 sum can wrap; the update kernel adds
// the planes in 64 bits).
template <int STRIDE>
__global__ void __launch_bounds__(DW_THREADS) dwconv3x3_wgrad_kernel(const int8_t* __restrict__ dhq, const int8_t* __restrict__ xq,
                                                                    int32_t* __restrict__ accW, DwGeom g, int pb_per_block,
                                                                    int blocks_per_plane) {
  accW += (size_t)(blockIdx.x / blocks_per_plane) * 2 * g.C * 9;
  __shared__ int red[32][37];
  const int CG = g.C >> 2;
  const int lane = threadIdx.x & 31, slot = threadIdx.x >> 5;
  const int cg = blockIdx.y * 32 + lane;
  const int p = blockIdx.z;
  for (int i = threadIdx.x; i < 32 * 37; i += DW_THREADS) (&red[0][0])[i] = 0;
  __syncthreads();
  int acc[4][9];
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int t = 0; t < 9; ++t) acc[j][t] = 0;
  const int pb_total = g.imgs_per_pass * g.Ho * g.wblocks;  // position blocks of one set
  const int pb_begin = blockIdx.x * pb_per_block;
  const int pb_end = min(pb_total, pb_begin + pb_per_block);
  if (cg < CG && pb_begin + slot < pb_end) {
    // (cg = 0, step in position blocks: the cursor's channel digit stays put)
    DwCursor cur((uint32_t)(pb_begin + slot), DW_THREADS / 32, 1, g.wblocks, g.Ho);
    for (int pb = pb_begin + slot; pb < pb_end; pb += DW_THREADS / 32, cur.advance()) {
      const int wo0 = cur.wb * DW_WB, ho = cur.ho;
      const int img = p * g.imgs_per_pass + cur.img;
      uint32_t dh[DW_WB];
      uint32_t any = 0u;
      const int8_t* dp = dhq + ((((size_t)img * g.Ho + ho) * g.Wo + wo0) * g.C) + 4 * (size_t)cg;
#pragma unroll
      for (int o = 0; o < DW_WB; ++o) {
        dh[o] = wo0 + o < g.Wo ? __ldg(reinterpret_cast<const uint32_t*>(dp + (size_t)o * g.C)) : 0u;
        any |= dh[o];
      }
      if (any == 0u) continue;
      DwWindow<STRIDE> win;
      win.load(xq, img, ho * STRIDE - 1, wo0 * STRIDE - 1, cg, g);
#pragma unroll
      for (int o = 0; o < DW_WB; ++o) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int dm = (int)(dh[o] & (0xFFu << (8 * j)));
#pragma unroll
          for (int r = 0; r < 3; ++r)
#pragma unroll
            for (int s = 0; s < 3; ++s) acc[j][r * 3 + s] = __dp4a((int)win.w[r][o * STRIDE + s], dm, acc[j][r * 3 + s]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int t = 0; t < 9; ++t)
        if (acc[j][t]) atomicAdd(&red[lane][j * 9 + t], acc[j][t]);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 32 * 36; i += DW_THREADS) {
    const int l = i / 36, k = i - l * 36;  // k = j*9 + t: the nine sums of channel 4*cg + j are contiguous in accW
    const int gcg = blockIdx.y * 32 + l;
    const int v = red[l][k];
    if (gcg < CG && v) atomicAdd(accW + ((size_t)p * g.C + 4 * (size_t)gcg) * 9 + k, v);
  }
}

// Weight gradient for any channel count: a block per (chunk of positions, set), a thread per channel.
__global__ void __launch_bounds__(DW_THREADS) dwconv3x3_wgrad_scalar_kernel(const int8_t* __restrict__ dhq,
                                                                           const int8_t* __restrict__ xq,
                                                                           int32_t* __restrict__ accW, DwGeom g, int rows_per_block,
                                                                           int blocks_per_plane) {
  accW += (size_t)(blockIdx.x / blocks_per_plane) * 2 * g.C * 9;   // planes as in the kernel above
  const int p = blockIdx.z;
  const int row_begin = blockIdx.x * rows_per_block, row_end = min(g.rows_per_pass, row_begin + rows_per_block);
  for (int ch = threadIdx.x; ch < g.C; ch += DW_THREADS) {
    int acc[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    for (int row = row_begin; row < row_end; ++row) {
      const int wo = row % g.Wo, t1 = row / g.Wo, ho = t1 % g.Ho, img = t1 / g.Ho + p * g.imgs_per_pass;
      const int d = dhq[((size_t)p * g.rows_per_pass + row) * g.C + ch];
      if (d == 0) continue;
      for (int r = 0; r < 3; ++r) {
        const int hh = ho * g.stride + r - 1;
        if (hh < 0 || hh >= g.H) continue;
        for (int s = 0; s < 3; ++s) {
          const int ww = wo * g.stride + s - 1;
          if (ww < 0 || ww >= g.W) continue;
          acc[r * 3 + s] += d * (int)xq[(((size_t)img * g.H + hh) * g.W + ww) * g.C + ch];
        }
      }
    }
    for (int t = 0; t < 9; ++t)
      if (acc[t]) atomicAdd(accW + ((size_t)p * g.C + ch) * 9 + t, acc[t]);
  }
}

}  // namespace ffi8
