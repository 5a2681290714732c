// INT8 x INT8 -> INT32 contractions of the FF-INT8 step on the 5th-generation tensor cores
// (tcgen05.mma kind::i8, accumulators in tensor memory, operands staged by TMA):
//   forward           acc[m,n]    = sum_k Xq[m,k] * Wq[n,k]                    (Sec. IV-B, INT8 MAC)
//   weight gradient   accW_p[n,k] = sum_{m in set p} dHq[m,n] * Xq[m,k]        (Sec. IV-B, g^W)
// for dense layers and, as implicit GEMMs, for 3x3 / stride 1 / zero-pad 1 convolutions over NHWC
// tensors (Sec. IV-B names both layer types): the im2col matrix is never written; the
// producer fetches, per filter tap, a box of the input shifted by the tap offset with a 4-D TMA
// copy whose out-of-image part is zero-filled (zero is exact in the symmetric quantiser).
//
// One kernel template.  320 threads: warp 0 = TMA producer, warp 1 = MMA issuer (one elected lane
// each), warps 2..9 = epilogue (two warps per TMEM lane quadrant; they share the tile's columns).
// NCTA = 1: output tile 128 x 256 per CTA.  NCTA = 2: the two CTAs of a cluster share a 256 x 256
// tile (tcgen05 cta_group::2): each stages its own 128 rows of A and one half (128 columns) of B;
// the CTA of cluster rank 0 issues the MMAs for both and holds the barriers the pair synchronises
// on.  The pair halves the B-operand traffic per MMA.
// Forward operands are K-major (contraction contiguous), CH = 128 or 64 contraction bytes per
// block (64: convolution with 64 input channels; 64-byte swizzle).  Weight-gradient operands are
// read in their natural row-major layout as MN-major operands (contraction block = 128 rows), so no
// transposed copy of dHq or Xq is ever written; CH is then the width of one B box in bytes.
// The forward double-buffers the accumulator (2 x 256 TMEM columns) so that the epilogue of tile
// i overlaps the MMAs of tile i+1; the weight gradient holds the accumulators of the positive and
// the negative set side by side (2 x 256 columns) and either applies the update
// W <- W - lr*(float(accP)*cP + float(accN)*cN) (Alg. 1, update step) in its epilogue (dense layers) or,
// when the contraction is split over several CTAs because the output has few tiles
// (convolutions), stores INT32 partial sums to slabs that slab_update_kernel adds exactly.
// Every wait is bounded: when one runs out the CTA raises ST_TIMEOUT, drains and returns.
#pragma once
#include <cuda.h>

#include <cstdio>
#include <cstring>
#include <unordered_map>

#include "../../include/ffint8.h"
#include "common.cuh"

namespace ffi8 {

constexpr int TC_BM = 128, TC_BN = 256;  // tile rows per CTA, tile columns
constexpr int TC_THREADS = 320;
constexpr int TC_EPI_WARPS = 8;                           // two per TMEM lane quadrant
constexpr int TC_EPI_COLS = TC_BN / 2;                    // most accumulator columns one epilogue warp takes
constexpr int TC_MAX_STAGES = 8;
constexpr uint32_t TC_PATCH_BYTES = 32 * 32 * 4;          // one 32 x 32 FP32 staging patch (128-byte swizzle)
constexpr int TC_PATCHES = 2;                             // patches per epilogue warp: a store may still be reading one while the next fills
constexpr uint32_t TC_RING_BYTES = 160 * 1024;            // operand ring budget
constexpr int TC_PREFETCH_KB = 8;                         // W tile is prefetched into L2 this many k-blocks before the epilogue
// Tile rows per rasterisation group.  K-major forward: the group's A row panels stay in L2 while the B
// column panels stream past once per group, so a tall group pays.  MN-major weight gradient: the
// contraction is so long that panels are only shared by tiles running at the same time; a group of
// 8 makes a wave of 74 CTA pairs nearly square (8 x 9 panels instead of 16 x 5).
constexpr int TC_GROUP_M_KMAJOR = 16, TC_GROUP_M_MNMAJOR = 8;
constexpr uint32_t TC_TMEM_COLS = 512;
constexpr uint32_t TC_TALL_ROWS = 192;                    // rows of a tall convolution stage: (128 / W + 2) * W for W <= 32
constexpr int TC_MAX_ACC = 4;                             // most accumulator stages (narrow forward tiles)
constexpr unsigned long long TC_WAIT_NS = 2000000000ull;  // 2 s bound on every wait

// Shared-memory geometry of one pipeline stage.
template <bool MN_MAJOR, int NCTA, int CH>
struct TcGeom {
  // K-major: A = 128 rows x CH bytes, B = (256/NCTA) rows x CH bytes.
  // MN-major: A = 128 contraction rows x 128 bytes, B = 128 contraction rows x (256/NCTA) bytes in boxes of CH bytes.
  static constexpr uint32_t A_BYTES = MN_MAJOR ? 128u * 128u : 128u * CH;
  static constexpr uint32_t B_BYTES = MN_MAJOR ? 128u * (TC_BN / NCTA) : (uint32_t)(TC_BN / NCTA) * CH;
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (int)(TC_RING_BYTES / STAGE_BYTES) < TC_MAX_STAGES ? (int)(TC_RING_BYTES / STAGE_BYTES) : TC_MAX_STAGES;
  static constexpr uint32_t SMEM_BYTES = STAGES * STAGE_BYTES + TC_EPI_WARPS * TC_PATCHES * TC_PATCH_BYTES + 1024 /*align*/ + 512 /*barriers*/;
  static constexpr int MMAS = MN_MAJOR ? 4 : CH / 32;            // MMAs (K = 32) per contraction block
  static constexpr int B_BOXES = MN_MAJOR ? (TC_BN / NCTA) / CH : 1;  // TMA boxes of the B operand per stage
  static constexpr uint32_t SWZ = CH == 128 ? 2u : 4u;             // descriptor swizzle code: 128-byte / 64-byte
};

enum { TC_MODE_RAW = 0, TC_MODE_FWD = 1, TC_MODE_UPD = 2, TC_MODE_SLAB = 3 };

struct TcParams {
  int out_rows, out_cols;   // extent of the output matrix
  int tiles_m, tiles_n;
  int group_m;              // tile rows per rasterisation group
  int kblocks;              // contraction blocks per pass
  int npass;                // 1, or 2 for the weight gradient (positive / negative set)
  int splits, kb_per_split; // the contraction blocks of a pass are divided over `splits` work items
  int bn;                   // K-major kernels: tile columns (a multiple of 32, at most TC_BN) - the MMA's N and the rows of
                            // B a stage holds follow it, so a narrow layer wastes neither, and a wide one can pick the
                            // width that fills its last wave of tiles best; MN-major kernels always use TC_BN
  int acc_stages;           // K-major forward: accumulator stages in tensor memory (512 / bn, at most 4)
  int tall_slots;           // tall stages in the ring: TC_TALL_ROWS rows of A each and, when the weights are streamed, the
  int tall_stride;          // three B boxes (vertical taps) that go with them; tall_stride = bytes from slot to slot
  int b_resident;           // K-major, one tile column: the whole B operand (all contraction blocks of this CTA's rows of
                            // B) is loaded once and stays in shared memory; the stages then hold A only.  A convolution's
                            // weights are the same for every tile, and the loads from L2 are what bounds these kernels.
  uint32_t* status;
  // raw
  int32_t* C;
  // forward epilogue
  float* Y;
  int32_t* acc_dump;
  unsigned long long* S;
  int32_t* rowmax;
  const float* absmax;
  int rows_per_pass, rows_per_sample;
  int y_tma;                // Y leaves through TMA stores (needs N % 4 == 0); else plain stores
  int w_tma;                // update epilogue: W comes and goes as 32 x 32 TMA patches (the Y map slot holds W's map)
  int y_stream;             // Y is larger than what L2 can usefully hold for the kernels that follow
  // update epilogue
  float* W;
  int32_t* accW_dump;
  float lr;
  float* mom;               // nullable heavy-ball buffer [out_rows, out_cols]: m = mu*m + g, W -= lr*m
  float mu;
  // split weight gradient
  int conv_tall;            // convolution forward with resident weights, stride 1: one input box of conv_TH + 2 image rows
                            // per horizontal tap offset and channel chunk serves the three vertical taps (the taps are the
                            // same box shifted by whole image rows, i.e. by whole swizzle atoms): a third of the box loads
  int32_t* slabs;
  int splits_per_slab;      // > 1: that many consecutive splits add their partial sums into one slab with integer
                            // atomics (exact, order-free; the slab is cleared before the launch); 1: a slab per split
  // convolution geometry (conv_W = 0: dense layer).  A 128-row block of positions is conv_TH image
  // rows of conv_W pixels; conv_cpt = channel chunks of CH bytes per filter tap; images per set.
  // conv_W / conv_H are the OUTPUT extents; the input box of an output position starts conv_stride
  // input pixels further per output pixel (the tensor map steps through the input with that stride).
  int conv_W, conv_H, conv_TH, conv_cin, conv_cpt, conv_imgs_per_pass, conv_stride;
};

// ---- PTX wrappers --------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Waits that may be released by the other CTA of a pair use cluster-scope acquire.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in the CTA of cluster rank `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// Arrive on a barrier of another CTA of the cluster.  CTA-scope release (the default) on purpose: what the arrive
// hands over is tensor memory, ordered by the tcgen05 fences around it; a cluster-scope release would also wait for
// every global store and atomic the thread has in flight (measured: 1500 - 2800 cycles per tile in the epilogue).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false when the time limit ran out or another role already gave up.
template <bool CLUSTER = false>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          unsigned long long limit_ns = TC_WAIT_NS) {
  auto poll = [&]() { return CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity); };
  if (poll()) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!poll()) {
    if ((++spins & 0xFFu) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit_ns) return false;
    }
  }
  return true;
}
// Self-test of the bounded wait: one thread waits, with the limit given, on a barrier that nothing ever arrives
// on.  The wait must give up, the thread raises ST_TIMEOUT exactly as the contraction kernels' roles do, and the
// kernel returns normally.  No copy, no tensor memory, no other thread is involved.
__global__ void bounded_wait_probe_kernel(uint32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_word;
  if (threadIdx.x == 0) {
    abort_word = 0u;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait<false>(smem_u32(&bar), 0u, &abort_word, limit_ns)) atomicOr(status, ST_TIMEOUT);
  }
}
// Tiled TMA loads into this CTA's shared memory.  NCTA = 2: `bar` is a shared::cluster address and may
// name a barrier of the other CTA of the pair (the cta_group::2 form allows that); no multicast.
template <int NCTA>
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x, int y, uint64_t policy) {
  if (NCTA == 1)
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y), "l"(policy)
        : "memory");
  else
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
template <int NCTA>
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x, int y, int z) {
  if (NCTA == 1)
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y), "r"(z)
                 : "memory");
  else
    asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
template <int NCTA>
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x, int y, int z, int w) {
  if (NCTA == 1)
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w)
                 : "memory");
  else
    asm volatile("cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w)
                 : "memory");
}
__device__ __forceinline__ void l2_prefetch(const void* gptr, uint32_t bytes) {  // 16-byte aligned, multiple of 16
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(gptr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Arrive on `bar` once all MMAs issued so far by this thread have completed.  NCTA = 2: the arrival is
// delivered to the barrier at the same shared-memory offset in both CTAs of the pair.
template <int NCTA>
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  if (NCTA == 1) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
  } else {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(mask)
                 : "memory");
  }
}
template <int NCTA>
__device__ __forceinline__ void tc_mma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  if (NCTA == 1)
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Load 32 consecutive accumulator columns of this thread's TMEM lane and wait for them.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, int (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// (the wait for the load is part of tc_ld32, so the registers are valid when it returns)
// The same load without the wait: the registers are valid after the next tc_wait_ld().
__device__ __forceinline__ void tc_ld32_async(uint32_t taddr, int (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// Waits for this thread's outstanding TMEM loads.  The loaded registers are passed through as read-write
// operands so that the compiler cannot schedule a use of them above the wait.
__device__ __forceinline__ void tc_wait_ld(int (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
                 "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// TMA store of one staged box to global memory (clipped at the tensor's edge), bulk async-group completion.
// `policy`: an L2 eviction policy (l2_policy_evict_first: the stored lines are the first to leave L2, so a
// stream of output written once does not push the operand panels out).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, uint32_t src, int x, int y, uint64_t policy) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;" ::"l"(
                   reinterpret_cast<uint64_t>(tm)),
               "r"(src), "r"(x), "r"(y), "l"(policy)
               : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }

// Shared-memory matrix descriptor for a swizzled operand tile whose rows are CH = 128 (swz = 2) or
// 64 (swz = 4) bytes long; 8 rows form one swizzle atom.  K-major: rows are M/N indices, SBO = 8 rows
// between atoms, LBO unused.  MN-major: rows are contraction indices, SBO = 8 contraction rows,
// LBO = distance between successive CH-element chunks along M/N.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swz) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;  // descriptor version of this architecture
  d |= (uint64_t)swz << 61;
  return d;
}
// The same descriptor in halves, for the MMA issuer's inner loops (one thread issues every MMA of the CTA group, so
// its instruction count per MMA is on the critical path of short contractions): the high word is a constant of the
// kernel, the low word is a constant plus the start address in 16-byte units, so moving the start by `bytes` adds
// bytes / 16 to the low word (every address is below 256 KB: the 14-bit field cannot carry).
__device__ __forceinline__ uint32_t smem_desc_hi(uint32_t sbo_bytes, uint32_t swz) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (swz << 29);
}
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ uint64_t smem_desc_join(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
// Instruction descriptor: INT8 x INT8 -> INT32, dense, M = 128 per CTA of the group, N = 256.
__host__ __device__ constexpr uint32_t make_idesc_i8(bool a_mn_major, bool b_mn_major, int ncta, int n = TC_BN) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)((TC_BM * ncta) >> 4) << 24);
}

// Tile order: groups of TC_GROUP_M tile rows, column by column inside a group, so that the CTAs
// running at one time share a small set of operand row / column panels in L2.
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int group_m, int& tm, int& tn) {
  const int per_group = group_m * tiles_n;
  const int g = tile / per_group, r = tile - g * per_group;
  const int rows = min(group_m, tiles_m - g * group_m);
  tm = g * group_m + r % rows;
  tn = r / rows;
}

// ---- kernel --------------------------------------------------------------------------------
template <int MODE, bool MN_MAJOR, int NCTA, int CH>
__global__ void __launch_bounds__(TC_THREADS, 1)
    tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const __grid_constant__ CUtensorMap tmY, const TcParams p) {
  using G = TcGeom<MN_MAJOR, NCTA, CH>;
  constexpr int STAGES = G::STAGES;
  constexpr uint32_t STAGE_BYTES = G::STAGE_BYTES;
  constexpr bool PAIR = NCTA == 2;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte aligned operand ring, then the epilogue patches, then the barriers (identical offsets in
  // both CTAs of a pair)
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t ring = (raw + 1023u) & ~1023u;
  uint8_t* ring_ptr = smem_raw + (ring - raw);
  uint8_t* patch_all = ring_ptr + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(patch_all + TC_EPI_WARPS * TC_PATCHES * TC_PATCH_BYTES);
  const uint32_t bar_full = smem_u32(bars);                      // [STAGES]  used in the leader CTA
  const uint32_t bar_empty = bar_full + 8 * TC_MAX_STAGES;       // [STAGES]  one set per CTA
  const uint32_t bar_tfull = bar_empty + 8 * TC_MAX_STAGES;      // [TC_MAX_ACC] one set per CTA
  const uint32_t bar_tempty = bar_tfull + 8 * TC_MAX_ACC;        // [TC_MAX_ACC] used in the leader CTA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * TC_MAX_STAGES + 2 * TC_MAX_ACC);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const uint32_t bar_wpatch = bar_full + 8 * (2 * TC_MAX_STAGES + 2 * TC_MAX_ACC + 4);  // [TC_EPI_WARPS][TC_PATCHES] W patches (update epilogue)
  const uint32_t bar_bres = bar_wpatch + 8 * (TC_EPI_WARPS * TC_PATCHES);               // [1] resident B operand landed (leader CTA)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;           // 0 = leader of the pair
  const int group = blockIdx.x / NCTA, n_groups = gridDim.x / NCTA;
  constexpr bool TWO_SETS = MODE == TC_MODE_UPD || MODE == TC_MODE_SLAB;  // accumulators of both sets side by side
  const int BN = MN_MAJOR ? TC_BN : p.bn;                        // tile columns
  const uint32_t ACC_STAGES = (TWO_SETS || MN_MAJOR) ? 1u : (uint32_t)p.acc_stages;
  const int total_items = p.tiles_m * p.tiles_n * p.splits;      // work item = (tile of (128*NCTA) x 256, split)

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int s = 0; s < TC_MAX_ACC; ++s) {
      mbar_init(bar_tfull + 8 * s, 1);
      mbar_init(bar_tempty + 8 * s, TC_EPI_WARPS * NCTA);  // one arrive per epilogue warp of every CTA of the group
    }
    if (MODE == TC_MODE_UPD)
      for (int s = 0; s < TC_EPI_WARPS * TC_PATCHES; ++s) mbar_init(bar_wpatch + 8 * s, 1);
    mbar_init(bar_bres, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {  // one warp of every CTA of the group takes part in the allocation
    if (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TC_TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TC_TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();  // the other CTA's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // barriers of the leader CTA as seen from this CTA
  const uint32_t lead_full = PAIR ? map_to_cta(bar_full, 0) : bar_full;
  const uint32_t lead_tempty = PAIR ? map_to_cta(bar_tempty, 0) : bar_tempty;
  auto raise_abort = [&]() {
    atomicOr(p.status, ST_TIMEOUT);
    *abort_flag = 1;
    if (PAIR) st_cluster_u32(map_to_cta(smem_u32(const_cast<uint32_t*>(abort_flag)), rank ^ 1u), 1u);
  };

  if (warp == 0) {
    // ------------------------------- TMA producer (every CTA loads its own operand parts) ----
    if (lane == 0) {
      uint32_t it = 0;  // running k-block counter (ring position)
      uint32_t tall_s = 0, tall_ph = 0;  // the same for the tall convolution stages, as slot and phase
      bool ok = true;
      const int a_rows0 = (int)rank * TC_BM;            // this CTA's rows inside the group's tile
      const int b_cols0 = (int)rank * (BN / NCTA);      // this CTA's share of the tile's columns
      // L2 policies of the K-major loads.  Dense forward: the group's row panels of A are reused by every
      // tile column of the rasterisation group (keep), a column panel of B only by the tiles in flight
      // (stream).  Convolution: the small weight matrix is reused by every tile (keep).
      const uint64_t pol_keep = l2_policy_evict_last(), pol_stream = l2_policy_evict_first();
      const int hw = p.conv_H * p.conv_W;
      const int blocks_per_img = p.conv_W ? p.conv_H / p.conv_TH : 1;
      const bool b_res = !MN_MAJOR && p.b_resident;
      const uint32_t b_box_bytes = (uint32_t)(BN / NCTA) * CH;               // one contraction block of this CTA's B rows
      const uint32_t bres_base = ring + STAGES * G::A_BYTES;                 // resident B: behind the (A-only) stages
      if (b_res && group < total_items) {
        if (rank == 0) mbar_expect_tx(bar_bres, b_box_bytes * (uint32_t)p.kblocks * NCTA);
        const uint32_t rb = PAIR ? map_to_cta(bar_bres, 0) : bar_bres;
        for (int kb = 0; kb < p.kblocks; ++kb) tma_load_2d<NCTA>(bres_base + kb * b_box_bytes, &tmB, rb, kb * CH, b_cols0, pol_keep);
      }
      for (int item = group; item < total_items && ok; item += n_groups) {
        const int tile = item / p.splits, split = item - tile * p.splits;
        const int kb0 = split * p.kb_per_split, kb1 = min(p.kblocks, kb0 + p.kb_per_split);
        int tm, tn;
        tile_coords(tile, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
        const int row0 = tm * (TC_BM * NCTA) + a_rows0, col0 = tn * BN + b_cols0;
        // forward convolution: image and first image row of this CTA's 128 output positions
        const int f_img = (!MN_MAJOR && p.conv_W) ? row0 / hw : 0;
        const int f_h0 = (!MN_MAJOR && p.conv_W) ? (row0 - f_img * hw) / p.conv_W : 0;
        // bytes the leader's barrier expects per stage from all CTAs of the group
        uint32_t stage_tx = MN_MAJOR ? STAGE_BYTES * NCTA : (G::A_BYTES + (b_res ? 0u : b_box_bytes)) * NCTA;
        // weight-gradient convolution: filter tap and first channel of each of this CTA's B boxes
        int b_ci0[G::B_BOXES], b_r[G::B_BOXES], b_s[G::B_BOXES];
        if (MN_MAJOR && p.conv_W) {
          const int valid_cols = min(TC_BN, p.out_cols - tn * TC_BN);  // a multiple of CH
          stage_tx = G::A_BYTES * NCTA + (uint32_t)valid_cols * 128u;
#pragma unroll
          for (int q = 0; q < G::B_BOXES; ++q) {
            const int c = col0 + q * CH, tap = c / p.conv_cin;
            b_ci0[q] = c - tap * p.conv_cin;
            b_r[q] = tap / 3;
            b_s[q] = tap - b_r[q] * 3;
          }
        }
        if (!MN_MAJOR && p.conv_tall) {
          // tall boxes: stage = (conv_TH + 2) image rows x conv_W pixels x CH channels for tap column s, chunk cc
          const uint32_t tall_rows = (uint32_t)(p.conv_TH + 2) * p.conv_W, slots = (uint32_t)p.tall_slots;
          for (int ts = 0; ts < 3 && ok; ++ts)
            for (int cc = 0; cc < p.conv_cpt; ++cc) {
              const uint32_t s = tall_s, ph = tall_ph;   // ring position, kept by counting
              if (++tall_s == slots) tall_s = 0u, tall_ph ^= 1u;
              if (!mbar_wait<PAIR>(bar_empty + 8 * s, ph ^ 1u, abort_flag)) {
                ok = false;
                break;
              }
              if (rank == 0) mbar_expect_tx(bar_full + 8 * s, (tall_rows * CH + (b_res ? 0u : 3u * b_box_bytes)) * NCTA);
              const uint32_t slot = ring + s * (uint32_t)p.tall_stride;
              tma_load_4d<NCTA>(slot, &tmA, lead_full + 8 * s, cc * CH, ts - 1, f_h0 - 1, f_img);
              if (!b_res)   // the weights of the three vertical taps (tr, ts) for this channel chunk
                for (int tr = 0; tr < 3; ++tr)
                  tma_load_2d<NCTA>(slot + TC_TALL_ROWS * CH + tr * b_box_bytes, &tmB, lead_full + 8 * s,
                                    ((tr * 3 + ts) * p.conv_cpt + cc) * CH, col0, pol_keep);
            }
          continue;
        }
        for (int pass = 0; pass < p.npass && ok; ++pass) {
          // forward convolution: (filter row, filter column, channel chunk) of k-block kb, kept by counting
          int f_r = 0, f_s = 0, f_cc = 0;
          if (!MN_MAJOR && p.conv_W) {
            const int tap = kb0 / p.conv_cpt;
            f_cc = kb0 - tap * p.conv_cpt;
            f_r = tap / 3;
            f_s = tap - f_r * 3;
          }
          // weight-gradient convolution: image and block of image rows of contraction block kb
          int g_img = 0, g_blk = 0;
          if (MN_MAJOR && p.conv_W) {
            g_img = kb0 / blocks_per_img;
            g_blk = kb0 - g_img * blocks_per_img;
            g_img += pass * p.conv_imgs_per_pass;
          }
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            if (!mbar_wait<PAIR>(bar_empty + 8 * s, ph ^ 1u, abort_flag)) {
              ok = false;
              break;
            }
            const uint32_t a_dst = ring + s * (b_res ? G::A_BYTES : STAGE_BYTES), b_dst = a_dst + G::A_BYTES;
            if (MODE == TC_MODE_UPD && pass == p.npass - 1 && kb == max(kb0, kb1 - TC_PREFETCH_KB)) {
              // pull this CTA's W rows of the tile into L2 shortly before the epilogue's read-modify-write
              const int c0w = tn * TC_BN;
              const int ncols = min(TC_BN, p.out_cols - c0w);
              if ((p.out_cols & 3) == 0 && ncols > 0) {
                const int nrows = min(TC_BM, p.out_rows - row0);
                for (int r = 0; r < nrows; ++r)
                  l2_prefetch(p.W + (size_t)(row0 + r) * p.out_cols + c0w, (uint32_t)ncols * 4u);
              }
            }
            if (rank == 0) mbar_expect_tx(bar_full + 8 * s, stage_tx);
            const uint32_t fb = lead_full + 8 * s;
            if (!MN_MAJOR) {
              if (p.conv_W) {
                // k-block = CH channels of one filter tap (r, s): the input box shifted by (r-1, s-1)
                tma_load_4d<NCTA>(a_dst, &tmA, fb, f_cc * CH, f_s - 1, f_h0 * p.conv_stride + f_r - 1, f_img);
                if (++f_cc == p.conv_cpt) {
                  f_cc = 0;
                  if (++f_s == 3) {
                    f_s = 0;
                    ++f_r;
                  }
                }
              } else {
                tma_load_2d<NCTA>(a_dst, &tmA, fb, kb * CH, row0, pol_keep);
              }
              if (!b_res) tma_load_2d<NCTA>(b_dst, &tmB, fb, kb * CH, col0, p.conv_W ? pol_keep : pol_stream);
            } else {
              // boxes of 128 contraction rows x 128 (A) or CH (B) output indices
              tma_load_3d<NCTA>(a_dst, &tmA, fb, row0, kb * 128, pass);
              if (p.conv_W) {
                // contraction block kb of set `pass` = conv_TH rows of one image; B column chunk q of the
                // tile = CH channels of one filter tap, fetched from the shifted input box
                const int h0 = g_blk * p.conv_TH * p.conv_stride;
#pragma unroll
                for (int q = 0; q < G::B_BOXES; ++q)
                  if (col0 + q * CH < p.out_cols)
                    tma_load_4d<NCTA>(b_dst + q * (128 * CH), &tmB, fb, b_ci0[q], b_s[q] - 1, h0 + b_r[q] - 1, g_img);
                if (++g_blk == blocks_per_img) {
                  g_blk = 0;
                  ++g_img;
                }
              } else {
#pragma unroll
                for (int q = 0; q < G::B_BOXES; ++q)
                  tma_load_3d<NCTA>(b_dst + q * (128 * CH), &tmB, fb, col0 + q * CH, kb * 128, pass);
              }
            }
          }
        }
      }
      if (!ok) raise_abort();
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (leader CTA only) ----------------------------
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = make_idesc_i8(MN_MAJOR, MN_MAJOR, NCTA, BN);
      uint32_t it = 0, tile_it = 0, tall_s = 0, tall_ph = 0;
      bool ok = true;
      const bool b_res = !MN_MAJOR && p.b_resident;
      const uint32_t b_box_bytes = (uint32_t)(BN / NCTA) * CH, bres_base = ring + STAGES * G::A_BYTES;
      if (b_res && group < total_items && !mbar_wait<PAIR>(bar_bres, 0u, abort_flag)) ok = false;
      for (int item = group; item < total_items && ok; item += n_groups, ++tile_it) {
        const int split = item % p.splits;
        const int kb0 = split * p.kb_per_split, kb1 = min(p.kblocks, kb0 + p.kb_per_split);
        const uint32_t as = tile_it % ACC_STAGES, aph = (tile_it / ACC_STAGES) & 1u;
        if (!mbar_wait<PAIR>(bar_tempty + 8 * as, aph ^ 1u, abort_flag)) {
          ok = false;
          break;
        }
        tc_fence_after();
        if (!MN_MAJOR && p.conv_tall) {
          const uint32_t d_tmem = tmem_base + as * BN, slots = (uint32_t)p.tall_slots;
          // descriptor low words: start addresses in 16-byte units.  One image row of the box is the step between
          // vertical taps; a weight box follows the previous tap's box of the same (ts, cc) after 3 * cpt boxes (resident)
          // or directly (streamed, inside the stage)
          const uint32_t hi = smem_desc_hi(8 * CH, G::SWZ);
          const uint32_t a_lo0 = smem_desc_lo(ring, 16), a_step = (uint32_t)p.tall_stride >> 4, a_tap = ((uint32_t)p.conv_W * CH) >> 4;
          const uint32_t b_box = b_box_bytes >> 4;
          const uint32_t b_tap = b_res ? 3u * (uint32_t)p.conv_cpt * b_box : b_box;
          const uint32_t b_lo0 = b_res ? smem_desc_lo(bres_base, 16) : a_lo0 + ((TC_TALL_ROWS * CH) >> 4);
          uint32_t acc = 0u, chunk = 0u;   // chunk = ts * cpt + cc
          for (int n = 3 * p.conv_cpt; n > 0; --n, ++chunk) {
            const uint32_t s = tall_s, ph = tall_ph;   // ring position, kept by counting (no division in this loop)
            if (++tall_s == slots) tall_s = 0u, tall_ph ^= 1u;
            if (!mbar_wait<PAIR>(bar_full + 8 * s, ph, abort_flag)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + s * a_step;
            const uint32_t b_lo = b_lo0 + (b_res ? chunk * b_box : s * a_step);
#pragma unroll
            for (int tr = 0; tr < 3; ++tr) {
#pragma unroll
              for (int k = 0; k < G::MMAS; ++k) {
                tc_mma_i8<NCTA>(d_tmem, smem_desc_join(a_lo + tr * a_tap + 2 * k, hi), smem_desc_join(b_lo + tr * b_tap + 2 * k, hi), idesc, acc);
                acc = 1u;
              }
            }
            tc_commit<NCTA>(bar_empty + 8 * s);
          }
          if (ok) tc_commit<NCTA>(bar_tfull + 8 * as);
          continue;
        }
        for (int pass = 0; pass < p.npass && ok; ++pass) {
          const uint32_t d_tmem = tmem_base + (TWO_SETS ? pass * TC_BN : as * BN);
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            if (!mbar_wait<PAIR>(bar_full + 8 * s, ph, abort_flag)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t a_src = ring + s * (b_res ? G::A_BYTES : STAGE_BYTES);
            const uint32_t b_src = b_res ? bres_base + (uint32_t)kb * b_box_bytes : a_src + G::A_BYTES;
#pragma unroll
            for (int k = 0; k < G::MMAS; ++k) {
              uint64_t ad, bd;
              if (!MN_MAJOR) {
                ad = make_smem_desc(a_src + k * 32, 16, 8 * CH, G::SWZ);
                bd = make_smem_desc(b_src + k * 32, 16, 8 * CH, G::SWZ);
              } else {
                ad = make_smem_desc(a_src + k * 4096, 16384, 1024, 2u);
                bd = make_smem_desc(b_src + k * (32 * CH), 128 * CH, 8 * CH, G::SWZ);
              }
              tc_mma_i8<NCTA>(d_tmem, ad, bd, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
            }
            tc_commit<NCTA>(bar_empty + 8 * s);  // frees the smem stage (in every CTA) once these MMAs have read it
          }
        }
        if (ok) tc_commit<NCTA>(bar_tfull + 8 * as);  // accumulator complete (signalled in every CTA)
      }
      if (!ok) raise_abort();
    }
    __syncwarp();
  } else {
    // ------------------------------- epilogue (warps 2..9 of every CTA) -----------------------
    const int quad = warp & 3;                           // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;                    // which of the quadrant's two warps
    uint8_t* patch0 = patch_all + (warp - 2) * TC_PATCHES * TC_PATCH_BYTES;
    uint32_t pflip = 0;  // which of the warp's two patches the next chunk fills (forward epilogue)
    (void)pflip;
    uint32_t wuse = 0, wdone = 0;  // W patches requested / consumed so far (update epilogue): slot = count & 1, parity = count >> 1
    (void)wuse;
    (void)wdone;
    const uint64_t w_policy = l2_policy_evict_normal();
    (void)w_policy;
    // A large Y is written once and read much later: let it leave L2 first.  A small one is read back by
    // the next kernels (normalisation, dH quantiser) while it still sits in L2: keep it.
    const uint64_t y_policy = p.y_stream ? l2_policy_evict_first() : l2_policy_evict_last();
    (void)y_policy;
    uint32_t tile_it = 0;
    bool ok = true;
    float c0 = 0.f, c1 = 0.f, cP = 0.f, cN = 0.f;
    if (MODE == TC_MODE_FWD) {
      const float s_w = scale_of(p.absmax[2]);
      c0 = __fmul_rn(scale_of(p.absmax[0]), s_w);
      c1 = __fmul_rn(scale_of(p.absmax[1]), s_w);
    }
    if (MODE == TC_MODE_UPD) {
      cP = __fmul_rn(scale_of(p.absmax[3]), scale_of(p.absmax[0]));
      cN = __fmul_rn(scale_of(p.absmax[4]), scale_of(p.absmax[1]));
    }
    for (int item = group; item < total_items && ok; item += n_groups, ++tile_it) {
      const int tile = item / p.splits, split = item - tile * p.splits;
      (void)split;
      int tm, tn;
      tile_coords(tile, p.tiles_m, p.tiles_n, p.group_m, tm, tn);
      const uint32_t as = tile_it % ACC_STAGES, aph = (tile_it / ACC_STAGES) & 1u;
      const int wrow0 = tm * (TC_BM * NCTA) + (int)rank * TC_BM + quad * 32;  // first output row of this warp
      const int row = wrow0 + lane;
      const bool row_ok = row < p.out_rows;
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
      const int col0 = tn * BN;
      // the quadrant's two warps share the tile's valid 32-column chunks (a narrow last tile keeps both busy)
      const int chunks = (min(BN, p.out_cols - col0) + 31) >> 5;
      const int cbeg = half ? ((chunks + 1) >> 1) * 32 : 0;
      const int cend = half ? chunks * 32 : ((chunks + 1) >> 1) * 32;
      // Update epilogue with W patches: the 32 x 32 block of W under chunk `cb` comes into one of the warp's two
      // swizzled patches by TMA (the box is clipped / zero-filled at the edges of W) and goes back the same way.
      // A patch is reloaded only after the store that last left from it has read it.
      const bool w_patches = MODE == TC_MODE_UPD && p.w_tma && wrow0 < p.out_rows;
      auto w_patch_load = [&](int cb) {
        if (lane == 0) {
          const uint32_t slot = wuse & 1u;
          bulk_wait_read0();
          mbar_expect_tx(bar_wpatch + 8 * ((warp - 2) * TC_PATCHES + slot), TC_PATCH_BYTES);
          tma_load_2d<1>(smem_u32(patch0 + slot * TC_PATCH_BYTES), &tmY, bar_wpatch + 8 * ((warp - 2) * TC_PATCHES + slot), col0 + cb,
                         wrow0, w_policy);
        }
        ++wuse;
      };
      // Hands the accumulator stage back to the MMA issuer (in the leader CTA).  Called as soon as the warp's last
      // tensor-memory load of the tile has completed - the values are in registers then - and before the warp's
      // global-memory traffic for the tile (stores, integer atomics): the arrive has release semantics, so placed
      // after them it would wait for their round trips to L2, and the next tile's MMAs with it.
      bool released = false;
      auto release_acc = [&]() {
        if (released) return;
        released = true;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (PAIR)
            mbar_arrive_cluster(lead_tempty + 8 * as);
          else
            mbar_arrive(bar_tempty + 8 * as);
        }
      };
      if (w_patches && cbeg < cend) w_patch_load(cbeg);  // nobody else writes this tile of W: fetch while the MMAs still run
      if (!mbar_wait<PAIR>(bar_tfull + 8 * as, aph, abort_flag)) {
        ok = false;
        break;
      }
      tc_fence_after();
      if (MODE == TC_MODE_RAW) {
#pragma unroll 1
        for (int cb = cbeg; cb < cend; cb += 32) {
          int v[32];
          tc_ld32(t_row + as * BN + cb, v);
          if (cb + 32 >= cend) release_acc();
          if (row_ok) {
            int32_t* dst = p.C + (size_t)row * p.out_cols + col0 + cb;
            if (col0 + cb + 32 <= p.out_cols && (p.out_cols & 3) == 0) {
#pragma unroll
              for (int j = 0; j < 32; j += 4) *reinterpret_cast<int4*>(dst + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + cb + j < p.out_cols) dst[j] = v[j];
            }
          }
        }
      } else if (MODE == TC_MODE_FWD) {
        // thread = one accumulator row.  Rows and columns outside the output hold zero accumulators (their
        // operand rows were zero-filled by TMA), so the goodness statistics need no masks.  y is staged in
        // a swizzled 32 x 32 patch and leaves with one TMA store per patch (clipped at the output's edge);
        // the TMEM load of the next 32 columns is in flight while this chunk is processed.
        const float c = row < p.rows_per_pass ? c0 : c1;
        unsigned long long ssum = 0ull;
        int mx = 0;
        int v[2][32];
        if (cbeg < cend) tc_ld32_async(t_row + as * BN + cbeg, v[0]);
#pragma unroll
        for (int i = 0; i < TC_EPI_COLS / 32; ++i) {
          const int cb = cbeg + i * 32;
          if (cb < cend) tc_wait_ld(v[i & 1]);
          if (i + 1 < TC_EPI_COLS / 32 && cb + 32 < cend) tc_ld32_async(t_row + as * BN + cb + 32, v[(i + 1) & 1]);
          if (cb < cend && cb + 32 >= cend) release_acc();  // the tile's last chunk is in registers
          if (cb < cend) {  // uniform across the warp
            const int(&a)[32] = v[i & 1];
            uint8_t* patch = patch0 + pflip * TC_PATCH_BYTES;
            pflip ^= 1u;
            if (p.y_tma) {  // the store issued two chunks ago must have read this patch
              if (lane == 0) bulk_wait_read1();
              __syncwarp();
            }
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              float y[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                // relu on the integer first: float(max(acc,0))*c equals max(0, float(acc)*c) bit for bit (c >= 0)
                const unsigned rl = (unsigned)max(a[j + q], 0);
                y[q] = __fmul_rn(__uint2float_rn(rl), c);
                ssum += (unsigned long long)rl * rl;  // one 32x32+64 multiply-add
                mx = max(mx, (int)rl);
              }
              *reinterpret_cast<float4*>(patch + lane * 128 + (((j >> 2) ^ (lane & 7)) << 4)) = make_float4(y[0], y[1], y[2], y[3]);
            }
            if (p.y_tma) {
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
              if (lane == 0 && wrow0 < p.out_rows) {  // a box that starts inside the output; its overhang is clipped
                tma_store_2d(&tmY, smem_u32(patch), col0 + cb, wrow0, y_policy);
                bulk_commit();
              }
            } else {
              __syncwarp();
              // lanes 0..7 of each quarter-warp cover one staged row: 4 rows x 128 bytes per store instruction
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                const int r = k * 4 + (lane >> 3), cc = lane & 7;
                const int grow = wrow0 + r, gcol = col0 + cb + cc * 4;
                if (grow < p.out_rows) {
                  const float4 yv = *reinterpret_cast<const float4*>(patch + r * 128 + ((cc ^ (r & 7)) << 4));
                  float* dst = p.Y + (size_t)grow * p.out_cols + gcol;
                  const float yy[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
                  for (int q = 0; q < 4; ++q)
                    if (gcol + q < p.out_cols) dst[q] = yy[q];
                }
              }
              __syncwarp();
            }
            if (p.acc_dump && row_ok) {  // parity dump: plain per-row stores
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + cb + j < p.out_cols) p.acc_dump[(size_t)row * p.out_cols + col0 + cb + j] = a[j];
            }
          }
        }
        if ((p.rows_per_sample & 31) == 0) {
          // the warp's 32 rows belong to one sample (convolution: a sample has H*W rows): one atomic per warp
          ssum += __shfl_xor_sync(0xffffffffu, ssum, 16);
          ssum += __shfl_xor_sync(0xffffffffu, ssum, 8);
          ssum += __shfl_xor_sync(0xffffffffu, ssum, 4);
          ssum += __shfl_xor_sync(0xffffffffu, ssum, 2);
          ssum += __shfl_xor_sync(0xffffffffu, ssum, 1);
          mx = __reduce_max_sync(0xffffffffu, mx);
          if (lane == 0 && wrow0 < p.out_rows && mx > 0) {
            const int sample = wrow0 / p.rows_per_sample;
            atomicAdd(p.S + sample, ssum);
            atomicMax(p.rowmax + sample, mx);
          }
        } else if (row_ok && mx > 0) {
          const int sample = row / p.rows_per_sample;
          atomicAdd(p.S + sample, ssum);
          atomicMax(p.rowmax + sample, mx);
        }
      } else if (MODE == TC_MODE_SLAB) {
        // raw INT32 partial sums of both sets to this split's slab [split][set][rows][cols].  A thread
        // holds one accumulator row; the 32 x 32 chunk is turned through a swizzled smem patch so that each
        // store instruction of the warp writes four whole 128-byte row segments.
        uint8_t* patch = patch0;
        for (int pass = 0; pass < 2; ++pass) {
          const bool shared_slab = p.splits_per_slab > 1;
          int32_t* slab = p.slabs + (size_t)((shared_slab ? split / p.splits_per_slab : split) * 2 + pass) * p.out_rows * p.out_cols;
          int v[2][32];
          if (cbeg < cend) tc_ld32_async(t_row + pass * TC_BN + cbeg, v[0]);
#pragma unroll
          for (int i = 0; i < TC_EPI_COLS / 32; ++i) {
            const int cb = cbeg + i * 32;
            if (cb < cend) tc_wait_ld(v[i & 1]);
            if (i + 1 < TC_EPI_COLS / 32 && cb + 32 < cend) tc_ld32_async(t_row + pass * TC_BN + cb + 32, v[(i + 1) & 1]);
            if (pass == 1 && cb < cend && cb + 32 >= cend) release_acc();  // both sets' sums have left tensor memory
            if (cb < cend) {  // uniform across the warp
              const int(&a)[32] = v[i & 1];
              if ((p.out_cols & 3) == 0) {  // groups of four columns are whole or absent, the last chunk included
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                  *reinterpret_cast<int4*>(patch + lane * 128 + (((j >> 2) ^ (lane & 7)) << 4)) =
                      make_int4(a[j], a[j + 1], a[j + 2], a[j + 3]);
                __syncwarp();
                if (shared_slab) {
                  // one staged row per instruction: the warp's 32 lanes add 32 consecutive columns (128 bytes)
                  if (col0 + cb + lane < p.out_cols) {
#pragma unroll 8
                    for (int r = 0; r < 32; ++r) {
                      const int val = *reinterpret_cast<const int*>(patch + r * 128 + ((((lane >> 2) ^ (r & 7))) << 4) + (lane & 3) * 4);
                      if (wrow0 + r < p.out_rows && val != 0) atomicAdd(slab + (size_t)(wrow0 + r) * p.out_cols + col0 + cb + lane, val);
                    }
                  }
                } else {
#pragma unroll
                  for (int q = 0; q < 8; ++q) {
                    const int r = q * 4 + (lane >> 3), cc = lane & 7;
                    if (wrow0 + r < p.out_rows && col0 + cb + cc * 4 < p.out_cols)
                      *reinterpret_cast<int4*>(slab + (size_t)(wrow0 + r) * p.out_cols + col0 + cb + cc * 4) =
                          *reinterpret_cast<const int4*>(patch + r * 128 + ((cc ^ (r & 7)) << 4));
                  }
                }
                __syncwarp();
              } else if (row_ok) {
                int32_t* dst = slab + (size_t)row * p.out_cols + col0 + cb;
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (col0 + cb + j < p.out_cols) {
                    if (shared_slab) {
                      if (a[j] != 0) atomicAdd(dst + j, a[j]);
                    } else {
                      dst[j] = a[j];
                    }
                  }
              }
            }
          }
        }
      } else if (MODE == TC_MODE_UPD && p.w_tma) {
        // thread = one accumulator row: g = float(accP)*cP + float(accN)*cN stays in registers, the thread updates
        // its own row of the W patch in shared memory, one TMA store per patch writes it back
        if (wrow0 < p.out_rows) {
          const size_t plane = (size_t)p.out_rows * p.out_cols;
#pragma unroll 1
          for (int cb = cbeg; cb < cend && ok; cb += 32) {
            if (cb + 32 < cend) w_patch_load(cb + 32);
            int vp[32], vn[32];
            tc_ld32_async(t_row + cb, vp);
            tc_ld32_async(t_row + TC_BN + cb, vn);
            tc_wait_ld(vp);
            tc_wait_ld(vn);
            if (cb + 32 >= cend) release_acc();
            float d[32];
#pragma unroll
            for (int j = 0; j < 32; ++j)
              d[j] = __fmul_rn(p.lr, __fadd_rn(__fmul_rn(__int2float_rn(vp[j]), cP), __fmul_rn(__int2float_rn(vn[j]), cN)));
            const uint32_t slot = wdone & 1u, par = (wdone >> 1) & 1u;
            ++wdone;
            if (!mbar_wait<false>(bar_wpatch + 8 * ((warp - 2) * TC_PATCHES + slot), par, abort_flag)) {
              ok = false;
              break;
            }
            uint8_t* patch = patch0 + slot * TC_PATCH_BYTES;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              float4* q = reinterpret_cast<float4*>(patch + lane * 128 + (((j >> 2) ^ (lane & 7)) << 4));
              float4 w = *q;
              w.x = __fsub_rn(w.x, d[j]);
              w.y = __fsub_rn(w.y, d[j + 1]);
              w.z = __fsub_rn(w.z, d[j + 2]);
              w.w = __fsub_rn(w.w, d[j + 3]);
              *q = w;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmY, smem_u32(patch), col0 + cb, wrow0, w_policy);
              bulk_commit();
            }
            if (p.accW_dump && row_ok) {  // parity dump
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + cb + j < p.out_cols) {
                  p.accW_dump[(size_t)row * p.out_cols + col0 + cb + j] = vp[j];
                  p.accW_dump[plane + (size_t)row * p.out_cols + col0 + cb + j] = vn[j];
                }
            }
          }
        }
      } else {  // TC_MODE_UPD
        // thread = one accumulator row computes g = float(accP)*cP + float(accN)*cN; g is staged
        // through smem so that the read-modify-write of W (and of the momentum buffer) is row-contiguous
        const size_t plane = (size_t)p.out_rows * p.out_cols;
        uint8_t* patch = patch0;
#pragma unroll 1
        for (int cb = cbeg; cb < cend; cb += 32) {
          // out_cols % 4 == 0: a lane's group of four columns is whole or absent, in the ragged last chunk too
          const bool vec = (p.out_cols & 3) == 0;
          const bool full = vec && col0 + cb + (lane & 7) * 4 < p.out_cols;
          // issue the (row-contiguous) W loads first so that they are in flight during the TMEM reads
          float4 wv[8];
          if (full) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int grow = wrow0 + i * 4 + (lane >> 3);
              if (grow < p.out_rows)
                wv[i] = *reinterpret_cast<const float4*>(p.W + (size_t)grow * p.out_cols + col0 + cb + (lane & 7) * 4);
            }
          }
          int vp[32], vn[32];
          tc_ld32_async(t_row + cb, vp);
          tc_ld32_async(t_row + TC_BN + cb, vn);
          tc_wait_ld(vp);
          tc_wait_ld(vn);
          if (cb + 32 >= cend) release_acc();
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            float d[4];
#pragma unroll
            for (int q = 0; q < 4; ++q)
              d[q] = __fadd_rn(__fmul_rn(__int2float_rn(vp[j + q]), cP), __fmul_rn(__int2float_rn(vn[j + q]), cN));
            *reinterpret_cast<float4*>(patch + lane * 128 + (((j >> 2) ^ (lane & 7)) << 4)) = make_float4(d[0], d[1], d[2], d[3]);
          }
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = i * 4 + (lane >> 3), cc = lane & 7;
            const int grow = wrow0 + r, gcol = col0 + cb + cc * 4;
            if (grow < p.out_rows && (full || !vec)) {
              float4 dv = *reinterpret_cast<const float4*>(patch + r * 128 + ((cc ^ (r & 7)) << 4));
              float* dst = p.W + (size_t)grow * p.out_cols + gcol;
              if (p.mom) {  // heavy ball: the step is taken along m = mu*m + g
                float* mp = p.mom + (size_t)grow * p.out_cols + gcol;
                if (full) {
                  const float4 m = *reinterpret_cast<const float4*>(mp);
                  dv.x = __fadd_rn(__fmul_rn(p.mu, m.x), dv.x);
                  dv.y = __fadd_rn(__fmul_rn(p.mu, m.y), dv.y);
                  dv.z = __fadd_rn(__fmul_rn(p.mu, m.z), dv.z);
                  dv.w = __fadd_rn(__fmul_rn(p.mu, m.w), dv.w);
                  *reinterpret_cast<float4*>(mp) = dv;
                } else {
                  float* dd = reinterpret_cast<float*>(&dv);
#pragma unroll
                  for (int q = 0; q < 4; ++q)
                    if (gcol + q < p.out_cols) mp[q] = dd[q] = __fadd_rn(__fmul_rn(p.mu, mp[q]), dd[q]);
                }
              }
              dv.x = __fmul_rn(p.lr, dv.x);
              dv.y = __fmul_rn(p.lr, dv.y);
              dv.z = __fmul_rn(p.lr, dv.z);
              dv.w = __fmul_rn(p.lr, dv.w);
              if (full) {
                float4 w = wv[i];
                w.x = __fsub_rn(w.x, dv.x);
                w.y = __fsub_rn(w.y, dv.y);
                w.z = __fsub_rn(w.z, dv.z);
                w.w = __fsub_rn(w.w, dv.w);
                *reinterpret_cast<float4*>(dst) = w;
              } else {
                const float dd[4] = {dv.x, dv.y, dv.z, dv.w};
#pragma unroll
                for (int q = 0; q < 4; ++q)
                  if (gcol + q < p.out_cols) dst[q] = __fsub_rn(dst[q], dd[q]);
              }
            }
          }
          if (p.accW_dump && row_ok) {  // parity dump
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + cb + j < p.out_cols) {
                p.accW_dump[(size_t)row * p.out_cols + col0 + cb + j] = vp[j];
                p.accW_dump[plane + (size_t)row * p.out_cols + col0 + cb + j] = vn[j];
              }
          }
          __syncwarp();
        }
      }
      release_acc();  // a warp without chunks in this tile, or a path that gave up early
    }
    if ((MODE == TC_MODE_FWD || MODE == TC_MODE_UPD) && lane == 0) bulk_wait_read0();  // the last stores have read their patches
    if (!ok && lane == 0) raise_abort();
  }

  // ---- teardown: everyone meets, outstanding copies are waited for, TMEM is released ---------
  __syncthreads();
  if (*abort_flag && threadIdx.x == 0) {
    // give in-flight TMA copies a bounded time to land before the CTA (and its smem) goes away
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 2000000ull) {
    }
  }
  tc_fence_before();
  __syncthreads();
  // neither CTA of a pair leaves (or frees its tensor memory) while the other may still use it
  if (PAIR) cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    if (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
  }
}

// ---- host side -----------------------------------------------------------------------------
typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
  int sm_count = 148;
  int force_ncta = 0;  // 0: choose by problem size; 1 / 2: always that CTA-group size
  PFN_encodeTiled encode = nullptr;
  std::unordered_map<const void*, int> max_groups;  // CTA groups resident at one time, per kernel instance
  char err[256] = {0};
};

inline ff_status tc_init(TcState& t) {
  if (t.encode) return FF_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
  if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
    snprintf(t.err, sizeof(t.err), "cuTensorMapEncodeTiled not available");
    return FF_ERR_CUDA;
  }
  t.encode = reinterpret_cast<PFN_encodeTiled>(fn);
  return FF_OK;
}

inline ff_status tc_encode(TcState& t, CUtensorMap* tm, const int8_t* base, cuuint32_t rank, const cuuint64_t* dims,
                           const cuuint64_t* strides, const cuuint32_t* box, int swizzle_bytes,
                           const cuuint32_t* element_strides = nullptr) {
  cuuint32_t ones[4] = {1, 1, 1, 1};
  const cuuint32_t* estr = element_strides ? element_strides : ones;
  CUresult r = t.encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, rank, const_cast<int8_t*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(t.err, sizeof(t.err), "cuTensorMapEncodeTiled failed (%d) rank=%u dims=%llu,%llu box=%u,%u", (int)r, rank,
             (unsigned long long)dims[0], (unsigned long long)dims[1], box[0], box[1]);
    return FF_ERR_CUDA;
  }
  return FF_OK;
}

// INT8 row-major matrix [rows, cols] viewed as `passes` stacked matrices of rows_per_pass rows (passes = 0:
// a plain 2-D map); box = box_cols x box_rows (x 1), swizzle = box_cols bytes (128 or 64), zero fill outside.
// pitch: bytes from one row to the next (0: rows are contiguous)
inline ff_status tc_make_map(TcState& t, CUtensorMap* tm, const int8_t* base, uint64_t cols, uint64_t rows_per_pass, uint64_t passes,
                             uint32_t box_cols, uint32_t box_rows, uint64_t pitch = 0) {
  if (!pitch) pitch = cols;
  // A pitched row is mapped over its whole pitch: boxes that reach past `cols` then stay inside the map and
  // take the plain copy path.  Whatever the padding bytes hold only meets zero-filled columns of the other
  // operand (forward) or lands in output rows / columns that the epilogue discards (weight gradient).
  cuuint64_t dims[3] = {pitch, rows_per_pass, passes ? passes : 1};
  cuuint64_t strides[2] = {pitch, pitch * rows_per_pass};
  cuuint32_t box[3] = {box_cols, box_rows, 1};
  return tc_encode(t, tm, base, passes > 0 ? 3 : 2, dims, strides, box, (int)box_cols);
}
// NHWC INT8 tensor [imgs, H, W, C] stepped through with `stride` pixels in both image directions;
// one copy brings ch_box channels of wo x th positions of one image (the box spans stride times as
// many input pixels).
inline ff_status tc_make_map_nhwc(TcState& t, CUtensorMap* tm, const int8_t* base, uint64_t C, uint64_t W, uint64_t H, uint64_t imgs,
                                  uint32_t ch_box, uint32_t wo, uint32_t th, uint32_t stride) {
  cuuint64_t dims[4] = {C, W, H, imgs};
  cuuint64_t strides[3] = {C, C * W, C * W * H};
  cuuint32_t box[4] = {ch_box, wo * stride, th * stride, 1};
  cuuint32_t estr[4] = {1, stride, stride, 1};
  return tc_encode(t, tm, base, 4, dims, strides, box, (int)ch_box, estr);
}
inline int tc_conv_stride(const ff_layer_desc& L) {
  return ((L.kind == FF_CONV3X3 || L.kind == FF_DWCONV3X3) && L.stride == 2) ? 2 : 1;
}
inline int tc_out_h(const ff_layer_desc& L) { return (L.H - 1) / tc_conv_stride(L) + 1; }
inline int tc_out_w(const ff_layer_desc& L) { return (L.Wd - 1) / tc_conv_stride(L) + 1; }

inline int cdiv(long long a, long long b) { return (int)((a + b - 1) / b); }

// CTA-group size for an output of out_rows x out_cols: a pair whenever the output has at least two
// 128-row blocks (the pair halves the B-operand traffic per MMA; measured at least as fast as single
// CTAs from one wave of tiles upwards), single CTAs for outputs of at most 128 rows.
inline int tc_pick_ncta(const TcState& t, long long out_rows, long long out_cols, long long splits = 1) {
  (void)out_cols;
  (void)splits;
  if (t.force_ncta == 1 || t.force_ncta == 2) return t.force_ncta;
  return out_rows > TC_BM ? 2 : 1;
}

// FP32 row-major matrix [rows, cols] for the forward epilogue's TMA stores: boxes of 32 x 32, 128-byte swizzle.
inline ff_status tc_make_store_map(TcState& t, CUtensorMap* tm, float* base, uint64_t cols, uint64_t rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * sizeof(float)};
  cuuint32_t box[2] = {32, 32};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = t.encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(t.err, sizeof(t.err), "cuTensorMapEncodeTiled (store map) failed (%d) cols=%llu rows=%llu", (int)r,
             (unsigned long long)cols, (unsigned long long)rows);
    return FF_ERR_CUDA;
  }
  return FF_OK;
}

// Shared-memory budget of the K-major kernels as the host sees it (mirrors TcGeom<false, NCTA, CH>).
inline int tc_kmajor_stages(int ncta, int ch) {
  const int stage = 128 * ch + (TC_BN / ncta) * ch;
  const int n = (int)(TC_RING_BYTES / stage);
  return n < TC_MAX_STAGES ? n : TC_MAX_STAGES;
}
// The B operand stays resident when the contraction has one tile column, more tiles than CTA groups (some group
// reuses B), and all of B's contraction blocks fit where the stages' B parts were.
inline bool tc_resident_ok(long long out_rows, long long out_cols, int bn, int kblocks, int ncta, int ch, int sm_count) {
  if (cdiv(out_cols, bn) != 1 || cdiv(out_rows, TC_BM * ncta) <= sm_count / ncta) return false;
  return (size_t)kblocks * (bn / ncta) * ch <= (size_t)tc_kmajor_stages(ncta, ch) * (TC_BN / ncta) * ch;
}
inline int tc_tall_slots(int ncta, int ch) { return (int)((size_t)tc_kmajor_stages(ncta, ch) * 128 * ch / ((size_t)TC_TALL_ROWS * ch)); }

template <int MODE, bool MN_MAJOR, int NCTA, int CH>
inline ff_status tc_launch_n(TcState& t, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& y, TcParams p,
                             cudaStream_t st) {
  using G = TcGeom<MN_MAJOR, NCTA, CH>;
  auto kern = tc_gemm_kernel<MODE, MN_MAJOR, NCTA, CH>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)G::SMEM_BYTES);
  if (e != cudaSuccess) {
    snprintf(t.err, sizeof(t.err), "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    return FF_ERR_CUDA;
  }
  if (MN_MAJOR || p.bn <= 0) p.bn = TC_BN;
  p.acc_stages = (int)TC_TMEM_COLS / p.bn < TC_MAX_ACC ? (int)TC_TMEM_COLS / p.bn : TC_MAX_ACC;
  p.tiles_m = cdiv(p.out_rows, TC_BM * NCTA);
  p.tiles_n = cdiv(p.out_cols, p.bn);
  p.b_resident = (!MN_MAJOR && (MODE == TC_MODE_FWD || MODE == TC_MODE_RAW) && p.splits <= 1 &&
                  tc_resident_ok(p.out_rows, p.out_cols, p.bn, p.kblocks, NCTA, CH, t.sm_count)) ? 1 : 0;
  p.tall_stride = (int)TC_TALL_ROWS * CH + (p.b_resident ? 0 : 3 * (p.bn / NCTA) * CH);
  p.tall_slots = p.b_resident ? tc_tall_slots(NCTA, CH) : (int)(G::STAGES * G::STAGE_BYTES / (uint32_t)p.tall_stride);
  if (p.tall_slots > TC_MAX_STAGES) p.tall_slots = TC_MAX_STAGES;
  if (p.conv_tall && p.tall_slots < 2) {   // the caller's tensor map was made for tall boxes
    snprintf(t.err, sizeof(t.err), "tall convolution boxes do not fit the operand ring");
    return FF_ERR_ARG;
  }
  p.group_m = MN_MAJOR ? TC_GROUP_M_MNMAJOR : TC_GROUP_M_KMAJOR;
  if (p.splits < 1) p.splits = 1;
  p.kb_per_split = cdiv(p.kblocks, p.splits);
  p.splits = cdiv(p.kblocks, p.kb_per_split);  // no empty split
  const int items = p.tiles_m * p.tiles_n * p.splits;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(TC_THREADS, 1, 1);
  cfg.dynamicSmemBytes = G::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = NCTA;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int& max_groups = t.max_groups[reinterpret_cast<const void*>(kern)];
  if (max_groups == 0) {
    // a persistent grid must be resident as a whole: ask how many CTA groups fit on the device
    max_groups = t.sm_count / NCTA;
    if (NCTA > 1) {
      cfg.gridDim = dim3(t.sm_count / NCTA * NCTA, 1, 1);
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n > 0 && n < max_groups) max_groups = n;
    }
  }
  const int groups = items < max_groups ? items : max_groups;
  cfg.gridDim = dim3(groups * NCTA, 1, 1);
  e = cudaLaunchKernelEx(&cfg, kern, a, b, y, p);
  if (e != cudaSuccess) {
    snprintf(t.err, sizeof(t.err), "launch: %s", cudaGetErrorString(e));
    return FF_ERR_CUDA;
  }
  return FF_OK;
}

template <int MODE, bool MN_MAJOR, int CH>
inline ff_status tc_launch(TcState& t, int ncta, const CUtensorMap& a, const CUtensorMap& b, const TcParams& p, cudaStream_t st,
                           const CUtensorMap* y = nullptr) {
  CUtensorMap none;
  memset(&none, 0, sizeof(none));
  const CUtensorMap& ym = y ? *y : none;
  if (ncta == 2) return tc_launch_n<MODE, MN_MAJOR, 2, CH>(t, a, b, ym, p, st);
  return tc_launch_n<MODE, MN_MAJOR, 1, CH>(t, a, b, ym, p, st);
}

// Tile width of a K-major contraction with out_rows x out_cols outputs on `groups` CTA groups of `rows_per_tile`
// rows.  An output at most TC_BN wide takes its own width (rounded up to 32): the MMA and the B rows of a stage then
// carry no padding.  A wider one takes, of 256, 224, 192, the width whose tiles fill the waves best - cost =
// waves x (width + 32), the 32 standing for a tile's fixed overhead - and 256 unless a narrower one wins by 5 %:
// narrower tiles re-read the A panel more often.
inline int tc_pick_bn(long long out_rows, long long out_cols, int rows_per_tile, int groups) {
  if (out_cols <= TC_BN) return (int)((out_cols + 31) / 32 * 32);
  const long long tm = cdiv(out_rows, rows_per_tile);
  auto cost = [&](int bn) { return (double)cdiv(tm * cdiv(out_cols, bn), groups) * (bn + 32); };
  const double base = cost(TC_BN);
  int best = TC_BN;
  double best_cost = base;
  for (int bn = TC_BN - 32; bn >= 192; bn -= 32) {
    const double c = cost(bn);
    if (c < 0.95 * base && c < best_cost) {
      best = bn;
      best_cost = c;
    }
  }
  return best;
}

// K-major ("NT") problem: A [M,K], B [N,K]; K % 16 == 0 (TMA row pitch), everything else ragged.
inline bool tc_nt_ok(long long M, long long N, long long K) { return K % 16 == 0 && K >= 16 && M >= 1 && N >= 1; }
// MN-major ("TN") problem: A [Kc,M], B [Kc,N]; M % 16 == 0 and N % 16 == 0.
inline bool tc_tn_ok(long long M, long long N, long long Kc) { return M % 16 == 0 && N % 16 == 0 && Kc >= 1; }

inline bool tc_gemm_supported(int M, int N, int K, int trans) { return trans ? tc_tn_ok(M, N, K) : tc_nt_ok(M, N, K); }
// 3x3 convolution as an implicit GEMM: whole 128-byte (or 64-byte) channel chunks per filter tap, image
// width a power of two up to 128 so that 128 consecutive output positions are whole image rows.
inline bool tc_conv_ok(const ff_layer_desc& L) {
  if (L.kind != FF_CONV3X3 || L.Cin % 64 != 0) return false;
  const int W = tc_out_w(L);   // 128 consecutive OUTPUT positions must be whole output rows
  if (W < 8 || W > 128 || (W & (W - 1)) != 0) return false;
  return tc_out_h(L) % (128 / W) == 0;
}
inline bool tc_forward_supported(const ff_layer_desc& L, int B) {
  if (L.kind == FF_CONV3X3) return tc_conv_ok(L);
  return tc_nt_ok(2LL * B * (L.kind == FF_LINEAR ? 1 : tc_out_h(L) * tc_out_w(L)), L.N, L.K);
}
inline bool tc_update_supported(const ff_layer_desc& L, int B) {
  if (L.kind == FF_CONV3X3) return tc_conv_ok(L) && L.N % 16 == 0;
  return tc_tn_ok(L.N, L.K, (long long)B * (L.kind == FF_LINEAR ? 1 : tc_out_h(L) * tc_out_w(L)));
}

// Fewest splits of a contraction of `kblocks` blocks of 128 such that no split is longer than WG_SAFE_LEN,
// i.e. no INT32 partial sum can wrap whatever the codes (Sec. IV-B: INT32 accumulation).
constexpr int TC_SAFE_KBLOCKS = (int)(WG_SAFE_LEN / 128);   // 1040 blocks = 133120 contraction elements
inline int tc_min_splits(long long kblocks) { return (int)((kblocks + TC_SAFE_KBLOCKS - 1) / TC_SAFE_KBLOCKS); }

// Split count of the convolution weight gradient (its output N x 9*Cin has few tiles, its contraction
// runs over every output position of a set): as many splits as keep every SM (pair) busy with one
// work item, at least 8 contraction blocks each, and at least tc_min_splits.  sm_count <= 0: assume 148.
inline int tc_conv_update_splits(const ff_layer_desc& L, int B, int sm_count, int force_ncta) {
  if (sm_count <= 0) sm_count = 148;
  const int ncta = force_ncta ? force_ncta : (L.N > TC_BM ? 2 : 1);
  const long long tiles = (long long)cdiv(L.N, TC_BM * ncta) * cdiv(L.K, TC_BN);
  const long long kblocks = (long long)B * tc_out_h(L) * tc_out_w(L) / 128;
  long long splits = (sm_count / ncta) / tiles;
  if (splits > kblocks / 8) splits = kblocks / 8;
  if (splits < tc_min_splits(kblocks)) splits = tc_min_splits(kblocks);
  return splits < 1 ? 1 : (int)splits;
}
// Splits that may share one slab: as many consecutive ones as keep the slab's whole contraction within
// TC_SAFE_KBLOCKS blocks, so that a shared INT32 sum cannot wrap either.  Sets p.splits_per_slab, clears the
// slabs a shared accumulation adds into, and returns the number of slabs the launch will leave.
// The arithmetic alone: *per = splits that share a slab, *kb_per_split = contraction blocks of a split; returns the slabs.
inline int tc_shared_slab_plan(int kblocks, int splits_asked, int* per, int* kb_per_split) {
  *kb_per_split = cdiv(kblocks, splits_asked < 1 ? 1 : splits_asked);
  const int splits = cdiv(kblocks, *kb_per_split);
  *per = TC_SAFE_KBLOCKS / *kb_per_split;
  if (*per < 1) *per = 1;
  if (*per > splits) *per = splits;
  return cdiv(splits, *per);
}
inline int tc_plan_shared_slabs(TcParams& p, size_t plane, cudaStream_t st, cudaError_t* err) {
  int per, kb_per_split;
  const int slabs = tc_shared_slab_plan(p.kblocks, p.splits, &per, &kb_per_split);
  p.splits_per_slab = per;
  *err = cudaSuccess;
  if (per > 1) *err = cudaMemsetAsync(p.slabs, 0, (size_t)slabs * 2 * plane * sizeof(int32_t), st);
  return slabs;
}
inline size_t tc_conv_update_slab_bytes(const ff_layer_desc& L, int splits) {
  return (size_t)splits * 2 * L.N * L.K * sizeof(int32_t);
}

inline ff_status tc_gemm(TcState& t, const int8_t* A, const int8_t* Bm, int32_t* C, int M, int N, int K, int trans,
                         uint32_t* status, cudaStream_t st) {
  ff_status s = tc_init(t);
  if (s != FF_OK) return s;
  CUtensorMap ta, tb;
  TcParams p = {};
  p.out_rows = M;
  p.out_cols = N;
  p.npass = 1;
  p.splits = 1;
  p.status = status;
  p.C = C;
  const int ncta = tc_pick_ncta(t, M, N);
  if (!trans) {
    p.kblocks = cdiv(K, 128);
    if ((s = tc_make_map(t, &ta, A, K, M, 0, 128, TC_BM)) != FF_OK) return s;
    p.bn = tc_pick_bn(M, N, TC_BM * ncta, t.sm_count / ncta);
    if ((s = tc_make_map(t, &tb, Bm, K, N, 0, 128, p.bn / ncta)) != FF_OK) return s;
    return tc_launch<TC_MODE_RAW, false, 128>(t, ncta, ta, tb, p, st);
  }
  p.kblocks = cdiv(K, 128);
  if ((s = tc_make_map(t, &ta, A, M, K, 1, 128, 128)) != FF_OK) return s;
  if ((s = tc_make_map(t, &tb, Bm, N, K, 1, 128, 128)) != FF_OK) return s;
  return tc_launch<TC_MODE_RAW, true, 128>(t, ncta, ta, tb, p, st);
}

// A convolution whose 9*Cin contraction fits one 128-byte block is run through an explicit, zero-padded
// INT8 im2col matrix (xi [rows, kpad], weights wi [N, kpad]) and the dense kernels.
inline int tc_im2col_kpad(const ff_layer_desc& L) { return (9 * L.Cin + 15) / 16 * 16; }
inline bool tc_im2col_ok(const ff_layer_desc& L) {
  if (L.kind != FF_CONV3X3 || tc_conv_ok(L)) return false;
  const int kp = tc_im2col_kpad(L);
  return kp == 16 || kp == 32 || kp == 48 || kp == 64 || kp == 96 || kp == 128;
}

// xi / wi / kpad: explicit-im2col operands (nullptr / 0: use the layer's Xq and Wq directly).
inline ff_status tc_forward(TcState& t, const ff_layer_desc& L, const ff_layer_bufs& b, int B, uint32_t* status, cudaStream_t st,
                            const int8_t* xi = nullptr, const int8_t* wi = nullptr, int kpad = 0) {
  ff_status s = tc_init(t);
  if (s != FF_OK) return s;
  const bool conv = L.kind == FF_CONV3X3 && !xi;
  const int R = L.kind != FF_LINEAR ? tc_out_h(L) * tc_out_w(L) : 1;
  const int M = 2 * B * R;
  const int K = xi ? kpad : L.K;
  const int8_t* A = xi ? xi : b.Xq;
  const int8_t* Bw = xi ? wi : b.Wq;
  CUtensorMap ta, tb;
  TcParams p = {};
  p.out_rows = M;
  p.out_cols = L.N;
  p.npass = 1;
  p.splits = 1;
  p.status = status;
  p.Y = b.Y;
  p.acc_dump = b.acc_dump;
  p.S = reinterpret_cast<unsigned long long*>(b.S);
  p.rowmax = b.rowmax;
  p.absmax = b.absmax;
  p.rows_per_pass = B * R;
  p.rows_per_sample = R;
  const int ncta = tc_pick_ncta(t, M, L.N);
  CUtensorMap ty;
  p.y_tma = (L.N % 4 == 0) ? 1 : 0;
  p.y_stream = (size_t)M * L.N * sizeof(float) > ((size_t)80 << 20) ? 1 : 0;

  if (p.y_tma && (s = tc_make_store_map(t, &ty, b.Y, L.N, M)) != FF_OK) return s;
  const CUtensorMap* typ = p.y_tma ? &ty : nullptr;
  if (!conv) {
    p.kblocks = cdiv(K, 128);
    if ((s = tc_make_map(t, &ta, A, K, M, 0, 128, TC_BM, xi ? 0 : (uint64_t)b.ld_xq)) != FF_OK) return s;
    p.bn = tc_pick_bn(M, L.N, TC_BM * ncta, t.sm_count / ncta);
    if ((s = tc_make_map(t, &tb, Bw, K, L.N, 0, 128, p.bn / ncta)) != FF_OK) return s;
    return tc_launch<TC_MODE_FWD, false, 128>(t, ncta, ta, tb, p, st, typ);
  }
  const int ch = L.Cin % 128 == 0 ? 128 : 64;
  p.conv_W = tc_out_w(L);
  p.conv_H = tc_out_h(L);
  p.conv_TH = 128 / p.conv_W;
  p.conv_stride = tc_conv_stride(L);
  p.conv_cin = L.Cin;
  p.conv_cpt = L.Cin / ch;
  p.conv_imgs_per_pass = B;
  p.kblocks = 9 * p.conv_cpt;
  p.bn = tc_pick_bn(M, L.N, TC_BM * ncta, t.sm_count / ncta);
  // stride 1, rows of at most 32 pixels, weights resident: boxes of conv_TH + 2 image rows, one per horizontal tap offset
  {
    const bool res = tc_resident_ok(M, L.N, p.bn, p.kblocks, ncta, ch, t.sm_count);
    const int stride_bytes = (int)TC_TALL_ROWS * ch + (res ? 0 : 3 * (p.bn / ncta) * ch);
    const int slots = res ? tc_tall_slots(ncta, ch)
                          : tc_kmajor_stages(ncta, ch) * (128 * ch + (TC_BN / ncta) * ch) / stride_bytes;
    p.conv_tall = (p.conv_stride == 1 && p.conv_W <= 32 && p.conv_H >= p.conv_TH + 2 && slots >= 2) ? 1 : 0;
  }
  if ((s = tc_make_map_nhwc(t, &ta, b.Xq, L.Cin, L.Wd, L.H, 2 * B, ch, p.conv_W, p.conv_TH + (p.conv_tall ? 2 : 0), p.conv_stride)) != FF_OK)
    return s;
  if ((s = tc_make_map(t, &tb, b.Wq, L.K, L.N, 0, ch, p.bn / ncta)) != FF_OK) return s;
  if (ch == 128) return tc_launch<TC_MODE_FWD, false, 128>(t, ncta, ta, tb, p, st, typ);
  return tc_launch<TC_MODE_FWD, false, 64>(t, ncta, ta, tb, p, st, typ);
}

// Dense weight gradient + update in one kernel.  B = rows of one set (samples x positions per sample).
inline ff_status tc_update(TcState& t, const ff_layer_desc& L, const ff_layer_bufs& b, int B, uint32_t* status, cudaStream_t st) {
  ff_status s = tc_init(t);
  if (s != FF_OK) return s;
  CUtensorMap ta, tb;
  TcParams p = {};
  p.out_rows = L.N;
  p.out_cols = L.K;
  p.kblocks = cdiv(B, 128);
  p.npass = 2;
  p.splits = 1;
  p.status = status;
  p.W = b.W;
  p.accW_dump = b.accW_dump;
  p.absmax = b.absmax;
  p.lr = L.lr;
  p.mom = L.momentum != 0.0f ? b.Mom : nullptr;
  p.mu = L.momentum;
  if ((s = tc_make_map(t, &ta, b.dHq, L.N, B, 2, 128, 128, (uint64_t)b.ld_dhq)) != FF_OK) return s;
  if ((s = tc_make_map(t, &tb, b.Xq, L.K, B, 2, 128, 128, (uint64_t)b.ld_xq)) != FF_OK) return s;
  // plain SGD: W travels through the epilogue as 32 x 32 TMA patches (K % 16 == 0 here, so its rows are 16-byte pitched)
  CUtensorMap tw;
  p.w_tma = (!p.mom && (reinterpret_cast<uintptr_t>(b.W) & 15) == 0) ? 1 : 0;
  if (p.w_tma && (s = tc_make_store_map(t, &tw, b.W, L.K, L.N)) != FF_OK) return s;
  return tc_launch<TC_MODE_UPD, true, 128>(t, tc_pick_ncta(t, L.N, L.K), ta, tb, p, st, p.w_tma ? &tw : nullptr);
}

// Convolution weight gradient: split contraction, INT32 partial sums of both sets to `slabs`
// ([splits][2][N][K]); the caller adds the slabs and applies the update.  *splits_out = slabs written.
inline ff_status tc_conv_update(TcState& t, const ff_layer_desc& L, const ff_layer_bufs& b, int B, int32_t* slabs, int splits,
                                int* splits_out, uint32_t* status, cudaStream_t st) {
  ff_status s = tc_init(t);
  if (s != FF_OK) return s;
  CUtensorMap ta, tb;
  TcParams p = {};
  const int ch = L.Cin % 128 == 0 ? 128 : 64;
  const int pos_per_pass = B * tc_out_h(L) * tc_out_w(L);
  p.out_rows = L.N;
  p.out_cols = L.K;
  p.kblocks = pos_per_pass / 128;
  p.npass = 2;
  p.splits = splits;
  p.status = status;
  p.slabs = slabs;
  p.conv_W = tc_out_w(L);
  p.conv_H = tc_out_h(L);
  p.conv_TH = 128 / p.conv_W;
  p.conv_stride = tc_conv_stride(L);
  p.conv_cin = L.Cin;
  p.conv_cpt = L.Cin / ch;
  p.conv_imgs_per_pass = B;
  cudaError_t merr;
  *splits_out = tc_plan_shared_slabs(p, (size_t)L.N * L.K, st, &merr);
  if (merr != cudaSuccess) {
    snprintf(t.err, sizeof(t.err), "cudaMemsetAsync: %s", cudaGetErrorString(merr));
    return FF_ERR_CUDA;
  }
  const int ncta = t.force_ncta ? t.force_ncta : (L.N > TC_BM ? 2 : 1);
  if ((s = tc_make_map(t, &ta, b.dHq, L.N, pos_per_pass, 2, 128, 128)) != FF_OK) return s;
  if ((s = tc_make_map_nhwc(t, &tb, b.Xq, L.Cin, L.Wd, L.H, 2 * B, ch, p.conv_W, p.conv_TH, p.conv_stride)) != FF_OK) return s;
  if (ch == 128) return tc_launch<TC_MODE_SLAB, true, 128>(t, ncta, ta, tb, p, st);
  return tc_launch<TC_MODE_SLAB, true, 64>(t, ncta, ta, tb, p, st);
}

// Dense split weight gradient into slabs: A = dHq [rows_per_pass x 2, N], B = xi [rows_per_pass x 2, kcols]
// (kcols % 16 == 0); slabs [splits][2][N][kcols].
inline int tc_dense_slab_splits(int N, int kcols, long long rows_per_pass, int sm_count) {
  if (sm_count <= 0) sm_count = 148;
  const long long tiles = (long long)cdiv(N, TC_BM) * cdiv(kcols, TC_BN);
  const long long kblocks = (rows_per_pass + 127) / 128;
  long long splits = sm_count / tiles;
  if (splits > kblocks / 8) splits = kblocks / 8;
  if (splits < tc_min_splits(kblocks)) splits = tc_min_splits(kblocks);
  return splits < 1 ? 1 : (int)splits;
}
inline ff_status tc_dense_update_slab(TcState& t, const int8_t* dHq, int N, const int8_t* xi, int kcols, int rows_per_pass,
                                      int32_t* slabs, int splits, int* splits_out, uint32_t* status, cudaStream_t st,
                                      int ld_dhq = 0, int ld_xi = 0) {
  ff_status s = tc_init(t);
  if (s != FF_OK) return s;
  CUtensorMap ta, tb;
  TcParams p = {};
  p.out_rows = N;
  p.out_cols = kcols;
  p.kblocks = cdiv(rows_per_pass, 128);
  p.npass = 2;
  p.splits = splits;
  p.status = status;
  p.slabs = slabs;
  cudaError_t merr;
  *splits_out = tc_plan_shared_slabs(p, (size_t)N * kcols, st, &merr);
  if (merr != cudaSuccess) {
    snprintf(t.err, sizeof(t.err), "cudaMemsetAsync: %s", cudaGetErrorString(merr));
    return FF_ERR_CUDA;
  }
  if ((s = tc_make_map(t, &ta, dHq, N, rows_per_pass, 2, 128, 128, (uint64_t)ld_dhq)) != FF_OK) return s;
  if ((s = tc_make_map(t, &tb, xi, kcols, rows_per_pass, 2, 128, 128, (uint64_t)ld_xi)) != FF_OK) return s;
  // one split: a large output with tiles for every SM, where CTA pairs pay; several: a small output, single CTAs
  const int ncta = t.force_ncta ? t.force_ncta : (splits == 1 ? tc_pick_ncta(t, N, kcols) : 1);
  return tc_launch<TC_MODE_SLAB, true, 128>(t, ncta, ta, tb, p, st);
}

}  // namespace ffi8
