// Shape-generic INT8 x INT8 -> INT32 contraction on the CUDA cores (dp4a), used for every shape
// the tensor-core kernels do not take (ragged K or N, Cin = 3 convolution, tiny layers) and as
// the second implementation the tensor-core kernels are tested against.
//   forward:          acc[m,n] = sum_k A(m,k) * Wq[n,k]             (Sec. IV-B, INT8 MAC)
//   weight gradient:  accW_p[n,k] = sum_{m in set p} dHq[m,n] * A(m,k)   (Sec. IV-B, g^W)
// A(m,k) is Xq[m,k] for a dense layer and the im2col view of the NHWC input for a 3x3
// convolution (zero outside the image).  Epilogues are fused: dequantise + ReLU + goodness
// statistics for the forward, the SGD update for the weight gradient.
#pragma once
#include "common.cuh"

namespace ffi8 {

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 32, SG_THREADS = 256;
constexpr int SG_PITCH = SG_BK + 4;  // bytes per smem row (36 = 9 words)

// ---- operand views -----------------------------------------------------------------------
// load8(row, col0, out): 8 consecutive columns col0..col0+7 of one row, zero outside the matrix.
struct DenseView {
  const int8_t* p;
  int rows, cols;
  int ld;     // bytes from one row to the next (>= cols)
  bool vec8;  // cols % 8 == 0, ld % 8 == 0 and p 8-byte aligned
  __device__ __forceinline__ void load8(int row, int col0, int8_t* out) const {
    if (row < rows && vec8 && col0 + 8 <= cols) {
      *reinterpret_cast<uint2*>(out) = __ldg(reinterpret_cast<const uint2*>(p + (size_t)row * ld + col0));
      return;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int c = col0 + i;
      out[i] = (row < rows && c < cols) ? p[(size_t)row * ld + c] : (int8_t)0;
    }
  }
};
// im2col view of an NHWC INT8 tensor for a 3x3 / pad 1 convolution of stride 1 or 2:
// row = (b*Ho + i)*Wo + j, col = (r*3 + s)*Cin + ci  ->  x[b, stride*i+r-1, stride*j+s-1, ci].
struct Im2colView {
  const int8_t* p;
  int rows, cols;  // rows = Bn*Ho*Wo, cols = 9*Cin
  int H, W, Cin;   // input geometry
  int Ho, Wo, stride;
  bool vec8;  // Cin % 8 == 0 and p 8-byte aligned
  __device__ __forceinline__ void load8(int row, int col0, int8_t* out) const {
    if (row >= rows) {
#pragma unroll
      for (int i = 0; i < 8; ++i) out[i] = 0;
      return;
    }
    int w = row % Wo, t = row / Wo;
    int h = t % Ho, b = t / Ho;
    w *= stride;
    h *= stride;
    if (vec8 && col0 + 8 <= cols) {
      int tap = col0 / Cin, ci = col0 - tap * Cin;
      int hh = h + tap / 3 - 1, ww = w + tap % 3 - 1;
      uint2 v = make_uint2(0u, 0u);
      if (hh >= 0 && hh < H && ww >= 0 && ww < W)
        v = __ldg(reinterpret_cast<const uint2*>(p + ((size_t)(b * H + hh) * W + ww) * Cin + ci));
      *reinterpret_cast<uint2*>(out) = v;
      return;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int c = col0 + i;
      int8_t v = 0;
      if (c < cols) {
        int tap = c / Cin, ci = c - tap * Cin;
        int hh = h + tap / 3 - 1, ww = w + tap % 3 - 1;
        if (hh >= 0 && hh < H && ww >= 0 && ww < W) v = p[((size_t)(b * H + hh) * W + ww) * Cin + ci];
      }
      out[i] = v;
    }
  }
};

// ---- epilogues ---------------------------------------------------------------------------
// Each thread owns a 4x4 patch: rows i0..i0+3, cols j0..j0+3 of the output, acc[pass][r][c].
struct RawEpilogue {  // plain INT32 store
  int32_t* C;
  int rows, cols;
  __device__ __forceinline__ void operator()(int i0, int j0, const int (&acc)[2][4][4]) const {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (i0 + r < rows && j0 + c < cols) C[(size_t)(i0 + r) * cols + j0 + c] = acc[0][r][c];
  }
};

// Forward epilogue (dequantise, ReLU, goodness statistics; Sec. III, Alg. 1, goodness step).
struct ForwardEpilogue {
  float* Y;
  int32_t* acc_dump;  // nullable
  unsigned long long* S;
  int32_t* rowmax;
  const float* absmax;
  int rows, cols;             // M*R, N
  int rows_per_pass;          // B*R
  int rows_per_sample;        // R
  __device__ __forceinline__ void operator()(int i0, int j0, const int (&acc)[2][4][4]) const {
    const float s_w = scale_of(absmax[2]);
    const float c0 = __fmul_rn(scale_of(absmax[0]), s_w), c1 = __fmul_rn(scale_of(absmax[1]), s_w);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int i = i0 + r;
      unsigned long long s = 0ull;
      int mx = 0;
      if (i < rows) {
        const float c = i < rows_per_pass ? c0 : c1;
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const int j = j0 + cc;
          if (j < cols) {
            const int a = acc[0][r][cc];
            Y[(size_t)i * cols + j] = dequant_relu(a, c);
            if (acc_dump) acc_dump[(size_t)i * cols + j] = a;
            const int rl = max(a, 0);
            s += (unsigned long long)rl * (unsigned long long)rl;
            mx = max(mx, rl);
          }
        }
      }
      // the 16 threads that share this row sit in one half-warp (tx = lane & 15)
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, o);
        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
      if ((threadIdx.x & 15) == 0 && i < rows && mx > 0) {
        const int sample = i / rows_per_sample;
        atomicAdd(S + sample, s);
        atomicMax(rowmax + sample, mx);
      }
    }
  }
};

// Weight-gradient epilogue (dequantise both sets, SGD update; Sec. IV-B, Alg. 1, update step).
struct UpdateEpilogue {
  float* W;
  int32_t* accW_dump;  // nullable, [2, rows, cols]
  const float* absmax;
  float lr;
  int rows, cols;  // N, K
  float* Mom;      // nullable: heavy-ball buffer, m = mu*m + g, W -= lr*m
  float mu;
  __device__ __forceinline__ void operator()(int i0, int j0, const int (&acc)[2][4][4]) const {
    const float cP = __fmul_rn(scale_of(absmax[3]), scale_of(absmax[0]));
    const float cN = __fmul_rn(scale_of(absmax[4]), scale_of(absmax[1]));
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int i = i0 + r, j = j0 + c;
        if (i < rows && j < cols) {
          const size_t o = (size_t)i * cols + j;
          float g = __fadd_rn(__fmul_rn(__int2float_rn(acc[0][r][c]), cP), __fmul_rn(__int2float_rn(acc[1][r][c]), cN));
          if (Mom) Mom[o] = g = __fadd_rn(__fmul_rn(mu, Mom[o]), g);
          W[o] = __fsub_rn(W[o], __fmul_rn(lr, g));
          if (accW_dump) {
            accW_dump[o] = acc[0][r][c];
            accW_dump[(size_t)rows * cols + o] = acc[1][r][c];
          }
        }
      }
  }
};

// Split weight-gradient epilogue: the contraction is divided over gridDim.z; every split stores
// its INT32 partial sums of both sets to its own slab [split][set][rows][cols] (plain stores;
// slab_update_kernel adds the slabs, which is exact in integers, and applies the update).
struct SlabEpilogue {
  int32_t* slabs;
  int rows, cols;  // N, K
  __device__ __forceinline__ void operator()(int i0, int j0, const int (&acc)[2][4][4]) const {
    const size_t plane = (size_t)rows * cols;
    int32_t* base = slabs + (size_t)blockIdx.z * 2 * plane;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int i = i0 + r, j = j0 + c;
        if (i < rows && j < cols) {
          const size_t o = (size_t)i * cols + j;
          base[o] = acc[0][r][c];
          base[plane + o] = acc[1][r][c];
        }
      }
  }
};

// Adds the `splits` INT32 slabs of both sets and applies the dequantised update (Sec. IV-B;
// Alg. 1, update step): W <- W - lr*(float(accP)*cP + float(accN)*cN).  plane = rows*cols elements of W;
// the slabs may have a wider row pitch (cols <= pitch).  A block covers 32 consecutive elements; its
// 8 warps take the splits round-robin (coalesced along the elements) and their integer partial
// sums meet in shared memory.  W == NULL: no update, only the sums are written to accW_dump (dense
// [2][rows][cols]) - the buffer a data-parallel step adds up over the devices before it updates.
// No slab can have wrapped (the host keeps every part of a contraction within WG_SAFE_LEN); the slabs are
// added in 64 bits, and a sum whose magnitude exceeds `limit` (2^31 - 1; a shard of a split batch: its share
// of that) raises ST_RANGE: that weight is then left as it was and its dumped sums saturate.
__device__ __forceinline__ bool wg_in_range(long long aP, long long aN, long long limit, uint32_t* status) {
  const bool ok = aP <= limit && aP >= -limit && aN <= limit && aN >= -limit;
  if (!ok) atomicOr(status, ST_RANGE);
  return ok;
}
__device__ __forceinline__ int wg_saturate(long long a) {
  return a > 2147483647LL ? 2147483647 : (a < -2147483647LL ? -2147483647 : (int)a);
}
__global__ void __launch_bounds__(256) slab_update_kernel(const int32_t* __restrict__ slabs, int splits, size_t plane, int cols,
                                                          int pitch, float* __restrict__ W, const float* __restrict__ absmax,
                                                          UpdateRule rule, int32_t* __restrict__ accW_dump, long long limit,
                                                          uint32_t* __restrict__ status) {
  const UpdateCoefs uc = update_coefs(rule);
  __shared__ long long part[2][8][32];
  const int lane = threadIdx.x & 31, zl = threadIdx.x >> 5;
  const float cP = __fmul_rn(scale_of(absmax[3]), scale_of(absmax[0]));
  const float cN = __fmul_rn(scale_of(absmax[4]), scale_of(absmax[1]));
  const size_t splane = plane / cols * pitch;  // elements of one slab
  for (size_t e0 = (size_t)blockIdx.x * 32; e0 < plane; e0 += (size_t)gridDim.x * 32) {
    const size_t e = e0 + lane;
    long long aP = 0, aN = 0;
    if (e < plane) {
      const size_t se = pitch == cols ? e : e / cols * pitch + e % cols;
      for (int z = zl; z < splits; z += 8) {
        aP += __ldg(slabs + ((size_t)z * 2) * splane + se);
        aN += __ldg(slabs + ((size_t)z * 2 + 1) * splane + se);
      }
    }
    part[0][zl][lane] = aP;
    part[1][zl][lane] = aN;
    __syncthreads();
    if (zl == 0 && e < plane) {
#pragma unroll
      for (int k = 1; k < 8; ++k) {
        aP += part[0][k][lane];
        aN += part[1][k][lane];
      }
      const bool ok = wg_in_range(aP, aN, limit, status);
      if (W && ok) {
        const float g = __fadd_rn(__fmul_rn(__int2float_rn((int)aP), cP), __fmul_rn(__int2float_rn((int)aN), cN));
        float m = rule.Mom ? rule.Mom[e] : 0.0f, v = rule.Var ? rule.Var[e] : 0.0f;
        W[e] = apply_update(rule, uc, W[e], g, m, v);
        if (rule.Mom) rule.Mom[e] = m;
        if (rule.Var) rule.Var[e] = v;
      }
      if (accW_dump) {
        accW_dump[e] = wg_saturate(aP);
        accW_dump[plane + e] = wg_saturate(aN);
      }
    }
    __syncthreads();
  }
}

// The same for one or two slabs of a large output (dense rows, cols % 4 == 0): nothing to share between
// warps, so every thread takes four consecutive elements with 128-bit accesses.
__global__ void __launch_bounds__(256) slab_update_flat_kernel(const int32_t* __restrict__ slabs, int splits, size_t plane,
                                                               float* __restrict__ W, const float* __restrict__ absmax,
                                                               UpdateRule rule, int32_t* __restrict__ accW_dump, long long limit,
                                                               uint32_t* __restrict__ status) {
  const UpdateCoefs uc = update_coefs(rule);
  const float cP = __fmul_rn(scale_of(absmax[3]), scale_of(absmax[0]));
  const float cN = __fmul_rn(scale_of(absmax[4]), scale_of(absmax[1]));
  const size_t n4 = plane >> 2, stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const int4 p0 = __ldcs(reinterpret_cast<const int4*>(slabs) + i);
    const int4 n0 = __ldcs(reinterpret_cast<const int4*>(slabs + plane) + i);
    long long sP[4] = {p0.x, p0.y, p0.z, p0.w}, sN[4] = {n0.x, n0.y, n0.z, n0.w};
    for (int z = 1; z < splits; ++z) {
      const int4 bP = __ldcs(reinterpret_cast<const int4*>(slabs + (size_t)z * 2 * plane) + i);
      const int4 bN = __ldcs(reinterpret_cast<const int4*>(slabs + ((size_t)z * 2 + 1) * plane) + i);
      sP[0] += bP.x, sP[1] += bP.y, sP[2] += bP.z, sP[3] += bP.w;
      sN[0] += bN.x, sN[1] += bN.y, sN[2] += bN.z, sN[3] += bN.w;
    }
    bool ok[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) ok[q] = wg_in_range(sP[q], sN[q], limit, status);
    if (W) {
      float4 w4 = reinterpret_cast<const float4*>(W)[i];
      float4 m4 = rule.Mom ? reinterpret_cast<const float4*>(rule.Mom)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
      float4 v4 = rule.Var ? reinterpret_cast<const float4*>(rule.Var)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
      float* w = reinterpret_cast<float*>(&w4);
      float* m = reinterpret_cast<float*>(&m4);
      float* v = reinterpret_cast<float*>(&v4);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (!ok[q]) continue;
        const float g = __fadd_rn(__fmul_rn(__int2float_rn((int)sP[q]), cP), __fmul_rn(__int2float_rn((int)sN[q]), cN));
        w[q] = apply_update(rule, uc, w[q], g, m[q], v[q]);
      }
      if (rule.Mom) reinterpret_cast<float4*>(rule.Mom)[i] = m4;
      if (rule.Var) reinterpret_cast<float4*>(rule.Var)[i] = v4;
      reinterpret_cast<float4*>(W)[i] = w4;
    }
    if (accW_dump) {
      reinterpret_cast<int4*>(accW_dump)[i] = make_int4(wg_saturate(sP[0]), wg_saturate(sP[1]), wg_saturate(sP[2]), wg_saturate(sP[3]));
      reinterpret_cast<int4*>(accW_dump + plane)[i] =
          make_int4(wg_saturate(sN[0]), wg_saturate(sN[1]), wg_saturate(sN[2]), wg_saturate(sN[3]));
    }
  }
}

// Explicit INT8 im2col for 3x3 / stride 1 / zero-pad 1 convolutions with few input channels (the
// first layer of an image network: 9*Cin <= 128): row = output position, column (r*3+s)*Cin + ci,
// zero beyond 9*Cin up to the padded width KPAD (a multiple of 16).  The padded matrix feeds the
// dense tensor-core kernels.  One thread per output position.
template <int KPAD>
__global__ void __launch_bounds__(256) im2col3x3_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ out, int rows, int H,
                                                        int W, int Cin, int Ho, int Wo, int stride) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const int t = row / Wo;
  const int w = (row - t * Wo) * stride;
  const int h = (t % Ho) * stride, b = t / Ho;
  __align__(16) int8_t v[KPAD];
#pragma unroll
  for (int i = 0; i < KPAD; ++i) v[i] = 0;
  int k = 0;
  for (int r = 0; r < 3; ++r)
    for (int s = 0; s < 3; ++s) {
      const int hh = h + r - 1, ww = w + s - 1;
      const bool in = hh >= 0 && hh < H && ww >= 0 && ww < W;
      const int8_t* src = x + ((size_t)(b * H + hh) * W + ww) * Cin;
      for (int ci = 0; ci < Cin; ++ci, ++k) {
        const int8_t val = in ? src[ci] : (int8_t)0;
#pragma unroll
        for (int i = 0; i < KPAD; ++i)  // static indexing keeps v in registers
          if (i == k) v[i] = val;
      }
    }
  uint4* dst = reinterpret_cast<uint4*>(out + (size_t)row * KPAD);
#pragma unroll
  for (int i = 0; i < KPAD / 16; ++i) dst[i] = reinterpret_cast<const uint4*>(v)[i];
}
// Rows of an INT8 matrix [rows, cols] copied to a zero-padded pitch.
__global__ void __launch_bounds__(256) pad_rows_kernel(const int8_t* __restrict__ in, int8_t* __restrict__ out, int rows, int cols,
                                                       int pitch) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * pitch) return;
  const int r = i / pitch, c = i - r * pitch;
  out[i] = c < cols ? in[(size_t)r * cols + c] : (int8_t)0;
}

// ---- kernel ------------------------------------------------------------------------------
// !TRANS: C[i,j] = sum_c LA(i,c) * LB(j,c)          (operands contraction-contiguous)
//  TRANS: C[i,j] = sum_c LA(c,i) * LB(c,j)          (operands contraction-strided)
// The contraction index runs over NPASS consecutive ranges of `clen` each (one accumulator set
// per range: the positive and the negative set of the weight gradient).  Block z of the grid
// takes the part [z*csplit, (z+1)*csplit) of every range (csplit = clen: no split).
template <class LA, class LB, bool TRANS, int NPASS, class Epi>
__global__ void __launch_bounds__(SG_THREADS) gemm_simt_kernel(LA la, LB lb, int clen, int csplit, Epi epi) {
  __shared__ __align__(16) int8_t As[SG_BM * SG_PITCH];
  __shared__ __align__(16) int8_t Bs[SG_BN * SG_PITCH];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int i_blk = blockIdx.y * SG_BM, j_blk = blockIdx.x * SG_BN;
  int acc[2][4][4];
#pragma unroll
  for (int p = 0; p < 2; ++p)
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[p][r][c] = 0;

#pragma unroll
  for (int pass = 0; pass < NPASS; ++pass) {
    const int cbeg = pass * clen + (int)blockIdx.z * csplit, cend = min(pass * clen + clen, cbeg + csplit);
    for (int c0 = cbeg; c0 < cend; c0 += SG_BK) {
      int8_t va[8], vb[8];
      if (!TRANS) {
        const int row = tid >> 2, kk = (tid & 3) * 8;  // 64 rows x 4 groups of 8 contraction bytes
        la.load8(i_blk + row, c0 + kk, va);
        lb.load8(j_blk + row, c0 + kk, vb);
        // mask the tail of the contraction range (ranges need not be multiples of SG_BK)
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (c0 + kk + i >= cend) {
            va[i] = 0;
            vb[i] = 0;
          }
        *reinterpret_cast<uint32_t*>(&As[row * SG_PITCH + kk]) = *reinterpret_cast<uint32_t*>(&va[0]);
        *reinterpret_cast<uint32_t*>(&As[row * SG_PITCH + kk + 4]) = *reinterpret_cast<uint32_t*>(&va[4]);
        *reinterpret_cast<uint32_t*>(&Bs[row * SG_PITCH + kk]) = *reinterpret_cast<uint32_t*>(&vb[0]);
        *reinterpret_cast<uint32_t*>(&Bs[row * SG_PITCH + kk + 4]) = *reinterpret_cast<uint32_t*>(&vb[4]);
      } else {
        const int cl = tid >> 3, g = (tid & 7) * 8;  // 32 contraction rows x 8 groups of 8 outputs
        const bool ok = c0 + cl < cend;
        if (ok) {
          la.load8(c0 + cl, i_blk + g, va);
          lb.load8(c0 + cl, j_blk + g, vb);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          As[(g + i) * SG_PITCH + cl] = ok ? va[i] : (int8_t)0;
          Bs[(g + i) * SG_PITCH + cl] = ok ? vb[i] : (int8_t)0;
        }
      }
      __syncthreads();
#pragma unroll
      for (int kw = 0; kw < SG_BK / 4; ++kw) {
        int a[4], b[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) a[r] = *reinterpret_cast<const int*>(&As[(ty * 4 + r) * SG_PITCH + kw * 4]);
#pragma unroll
        for (int c = 0; c < 4; ++c) b[c] = *reinterpret_cast<const int*>(&Bs[(tx * 4 + c) * SG_PITCH + kw * 4]);
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[pass][r][c] = __dp4a(a[r], b[c], acc[pass][r][c]);
      }
      __syncthreads();
    }
  }
  epi(i_blk + ty * 4, j_blk + tx * 4, acc);
}

}  // namespace ffi8
