// Tensor-core convolution for sm_100a: implicit GEMM
//     D[ch][px] = sum_k W[ch][k] * X[px][k]
// with ch = output channel, px = output pixel (n, oh, ow) in NHWC order and k = (kh, kw, cin): the
// contraction of Eq. 3 on tcgen05.mma kind::i8 (s8 weights x u8/s8 activations, INT32 accumulators in
// tensor memory), fused with the integer epilogue: INT32 bias (Appendix D), dyadic multiply-shift
// (Eq. 4), dyadically rescaled residual branch (Section 3.3), ReLU, clamp, pack.
//
// Orientation.  The output channels sit on the M side of the MMA, i.e. on the 128 lanes of tensor
// memory, and the pixels on the N side (columns).  An epilogue thread therefore owns ONE channel:
// its dyadic pair, bias and residual pair live in registers for the whole kernel, no per-element
// constant fetch is needed, and the 32 lanes of a warp hold 32 consecutive channels of the same
// pixel, which is a contiguous 32-byte run of the NHWC output.
//
// One persistent CTA per SM, twelve warps (six in the two-CTAs-per-SM shape):
//   warp 0      TMA producer.  X tile = PT consecutive output pixels x BK bytes of one filter tap,
//               fetched by an im2col-mode tensor map straight from the NHWC activation tensor (the
//               hardware walks pixels across rows and images, applies the stride and zero-fills the
//               padding; zero is the right padding value because activations have zero point 0), or by
//               a plain tiled map when the conv is 1x1 / stride 1.  W tile = 128 output channels x BK
//               bytes of the [cout][kh*kw*cin] weight matrix.  When a residual is fused, its
//               [PT][128] tile of the stored 8-bit tensor is prefetched as well.
//   warps 1-3   MMA issuers (one lane each; a single issuer for layers whose weights stream from L2).
//               BK/32 instructions of shape 128 x PT x 32 per stage; two (PT = 256) or four
//               (PT <= 128) accumulator buffers in tensor memory, so the MMAs of the next tiles run
//               while the epilogue works on the current ones.  3x3 / stride 1 layers with resident
//               weights use the strip form: one padded input patch per cin chunk, read by all nine
//               taps as row offsets (see the issuer loop).
//   warps 4-11  epilogue.  Warp (q, half) reads lanes 32q..32q+31 (tcgen05.ld 32x32b) of one half
//               of the tile's pixel columns, applies the integer epilogue in registers and writes
//               bytes to a private staging box that leaves through its own TMA store; no CTA-wide
//               barrier per tile.  The loop is software-pipelined: the accumulator buffer goes back
//               to the MMA issuer as soon as its last chunk has been read, and the first chunk of
//               the next tile is requested from tensor memory before the current tile's staging
//               writes and store hand-over, whose latency it hides.
// The CTA keeps one channel tile for its whole life (grid = multiple of the channel tiles).
// Every wait on an mbarrier is bounded: after the budget the waiter records a code in the
// handle's status word, raises a CTA-wide abort flag and every role leaves its loop, drains what
// it has in flight (again bounded), and the CTA frees its tensor memory and returns.
#include <cuda.h>
#include <climits>
#include <cstdlib>

#include "hq_internal.cuh"

namespace {

constexpr int kTileC = 128;                   // output channels per tile = MMA M = TMEM lanes
constexpr int kMaxStages = 8;
// Dynamic shared memory of a one-CTA-per-SM launch: 224 KiB for the pipeline's pieces + 1 KiB of alignment slack, inside
// the 226 KiB the kernels ask for (227 KiB per block is the limit, the control block is static).
constexpr int kSmemBudget = 224 * 1024;
constexpr int kSmemAttr = 226 * 1024;
constexpr int kMaxAccBufs = 4;                                 // accumulator buffers: 4 x 128 or 2 x 256 columns
constexpr int kMaxResBufs = 8;                                 // residual / output tiles in shared memory
// Four launch shapes of the same kernel:
//   solo  8 epilogue warps, one CTA per SM, up to 512 tensor-memory columns, up to 224 KiB of shared memory;
//   pair  4 epilogue warps, two CTAs per SM with 256 columns and at most 110 KiB each.  Layers with a short
//         reduction are bound by the latency of the hand-over chain between the MMA issuer and the epilogue
//         (barrier, fences, MMA, commit), not by any throughput; two independent CTAs hide each other's chain.
//   rtm   ("residual through tensor memory") 8 epilogue warps, one issuer and a store warp, one CTA per SM, 128-pixel
//         tiles: fused 8-bit residuals with a short reduction.  The residual tile is transposed and widened by an MMA
//         with the identity matrix, the epilogue works on 16 x 8 fragments and writes with transposing matrix stores.
//   duo   the solo roles in clusters of two CTAs that share every MMA (cta_group::2): long reductions whose weights
//         stream; each CTA fetches its own weight rows and half of the pixel rows.
constexpr int kSoloEpilogueWarps = 8;
constexpr int kPairEpilogueWarps = 4;
constexpr int kSoloIssuerWarps = 3;     // 1 + 3 + 8 warps = 384 threads: 168 registers per thread remain
constexpr int kPairIssuerWarps = 1;
constexpr unsigned long long kWaitBudgetNs = 2000000000ull;   // 2 s per wait
constexpr long long kIm2colMinTensorBytes = 128 * 1024;        // smaller activation tensors are not fetched in im2col mode

struct TcParams {
  int32_t P, C;          // output pixels (n*ho*wo) and output channels
  int32_t howo, wo, stride, pad, kw;
  int32_t cchunks;       // K blocks per filter tap
  int32_t bkb;           // bytes of K per stage (32, 64 or 128) = swizzle span
  int32_t k_blocks;      // kh * kw * cchunks
  int32_t pt;            // pixel tile = MMA N: 64, 128 or 256
  int32_t p_tiles, c_tiles, stages;
  int32_t rev;           // 1: a CTA's t-th pixel tile is tile p_tiles - 1 - t: the layer walks its tensors from the end, so
                         //    that it reads first what the kernel before it wrote last (still in the L2)
  int32_t wres;          // 1: the CTA's whole weight slab [k_blocks][128][bkb] is loaded once and stays in shared memory
  uint32_t wres_off;     // its offset from the 1024-aligned dynamic base
  int32_t fold;          // 1: at most 64 output channels: W rows loaded twice, lane quarters 2-3 share the pixel columns
  int32_t halves;        // 2: two warps share a lane quarter's pixel columns; 1 for the 64-pixel tile (warps 6-9 idle)
  int32_t lg_rbufs;      // log2 of the residual-tile buffer count (<= lg_bufs; 0 when a long reduction leaves no room)
  int32_t rtm;           // 1: the 8-bit residual tile reaches the epilogue through tensor memory: an MMA with the identity
                         //    matrix as its A operand turns the [pixels][128 channels] byte tile into INT32 columns beside
                         //    the accumulator, in the accumulator's own layout (see epilogue_loop_frag)
  int32_t acc_bits;      // |accumulator| < 2^acc_bits for every 8-bit operand pair: ceil(log2(K * 255 * 128 + 1))
  int32_t acc_stride;    // tensor-memory columns between accumulator buffers: pt, or 2 * pt with rtm
  uint32_t ident_off;    // rtm: offset of the 128 x 128 identity matrix (16 KiB, 128-byte swizzle) from the 1024-aligned base
  int32_t duo;           // 1: two CTAs of a cluster (adjacent SMs) share every MMA: 256 channels x 256 pixels per pair
  int32_t ni;            // MMA issuer warps in use: min(issuer warps of the launch shape, k_blocks)
  int32_t lg_bufs;       // log2 of the accumulator / residual buffer count: tile t of a CTA uses buffer t mod 2^lg_bufs
  int32_t x_signed;      // activations signed?
  int32_t x_tiled;       // 1: X is a dense [P][cin] matrix (1x1, stride 1, no padding) fetched by a tiled map
  // Strip mode (3x3, stride 1, pad 1): a tile is `rows` output rows of one image, laid out with a power-of-two
  // pitch of 2^lg_wp positions (columns >= wo are scratch); one padded input patch per cin chunk feeds all nine taps.
  int32_t strip;         // 1: strip mode
  int32_t lg_wp, rows;   // log2 of the position pitch; output rows per tile (pt = rows << lg_wp)
  int32_t tpi;           // tiles per image = ceil(ho / rows)
  int32_t ho;            // output (= input) height
  int32_t npatch;        // patch buffers (2 or 3)
  uint32_t patch_bytes, patch_off;   // bytes of one patch [(rows+3) << lg_wp][bkb]; offset from the 1024-aligned base
  uint32_t tmem_cols;
  // epilogue
  int32_t staged_out;    // 1: bytes leave through per-warp staging boxes and TMA stores
  int32_t staged_res;    // 1: the 8-bit residual tile arrives through a TMA load
  int32_t sat_pack;      // 1: clamp bounds equal the 8-bit output type's range (a saturating convert does the clamp)
  int32_t out_signed;
  uint32_t out_stage_off, res_stage_off;   // offsets from the 1024-aligned dynamic base
  const int32_t* bias; const int32_t* b; const int32_t* c;
  const void* res; int32_t res_bits, res_signed; const int32_t* rb; const int32_t* rc;
  const int4* res_narrow;   // optional per-channel {m, a, s, valid} from residual_narrow_kernel
  int32_t narrow_fresh;     // 1: the pairs are written by the kernel launched just before this one
  int32_t relu, qmin, qmax;
  void* out; int32_t out_bits;
  uint32_t* status;
};

struct SharedCtl {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long tfull[kMaxAccBufs];
  unsigned long long tempty[kMaxAccBufs];
  unsigned long long tstart[kMaxAccBufs];   // the tile's first (overwriting) MMA has been issued
  unsigned long long rfull[kMaxResBufs];
  unsigned long long rempty[kMaxResBufs];
  unsigned long long ofull[kMaxResBufs];    // rtm: every epilogue warp has written its pieces of the output tile
  unsigned long long drain;
  unsigned long long wfull;              // resident weight slab landed
  unsigned long long pfull[3], pempty[3];  // strip mode: input patches
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};

// ---------------------------------------------------------------- PTX wrappers ---------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false when the budget ran out or another role already aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, SharedCtl* ctl, uint32_t* status,
                                          uint32_t code) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 63u) == 0) {
      if (ctl->abort_flag) return false;
      if (global_ns() - t0 > kWaitBudgetNs) {
        ctl->abort_flag = 1;
        atomicCAS(status, 0u, code);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
// The same copy with an L2 eviction priority.  Activations and residual tiles that a layer reads exactly once per
// channel tile are fetched "evict first": they then make room before the output lines the layer is writing, and the
// next layer (which starts at the end this one wrote last, see TcParams::rev) finds more of its input in the L2.
__device__ __forceinline__ unsigned long long policy_evict_first() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                                 unsigned long long pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                int c, int w, int h, int n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c, int w, int h, int n) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n) : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c, int w, int h, int n) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(src), "r"(c), "r"(w), "r"(h), "r"(n) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
template <int EPI_THREADS>
__device__ __forceinline__ uint32_t epi_bar_and(uint32_t v) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"(v), "n"(EPI_THREADS) : "memory");
  return r;
}

// True in exactly one lane of a converged warp; tells the compiler the guarded region is
// single-lane, which lets it keep TMA / MMA operands in uniform registers.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ---- two-CTA forms (cta_group::2).  `in_cta(addr, r)` names the same shared-memory offset in the cluster's CTA r.
__device__ __forceinline__ uint32_t in_cta(uint32_t addr, uint32_t cta_rank) {
  uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta_rank)); return r;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma_i8_2cta(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// arrives on ONE barrier (of either CTA of the pair) when the pair's MMAs issued so far have completed
__device__ __forceinline__ void mma_commit_2cta(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
// loads of a CTA pair: the bytes land in the issuing CTA's shared memory and are counted on the leading CTA's barrier
__device__ __forceinline__ void tma_load_2d_2cta(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(in_cta(bar, 0)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_2cta(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                     int c, int w, int h, int n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(in_cta(bar, 0)), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, int (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 lanes x 32 columns in the layout of an MMA accumulator fragment: thread T (t4 = T / 4, q2 = T % 4) receives, for
// every group g of eight columns, v[4g + 0/1] = lane t4, columns 8g + 2 q2 + 0/1 and v[4g + 2/3] = lane t4 + 8, same columns.
__device__ __forceinline__ void tmem_ld_frag16(uint32_t taddr, int (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr) : "memory");
}
// Four 16 x 8 byte matrices, stored transposed: register g of thread T holds, in byte order, the elements
// (m, n) = (t4, 2 q2), (t4, 2 q2 + 1), (t4 + 8, 2 q2), (t4 + 8, 2 q2 + 1) of matrix g -- the byte-packed form of the
// fragment above -- and matrix g's column n becomes the 16 contiguous bytes at the address thread 8 g + n supplies.
__device__ __forceinline__ void stmatrix_t_x4(uint32_t row_addr, unsigned r0, unsigned r1, unsigned r2, unsigned r3) {
  asm volatile("stmatrix.sync.aligned.m16n8.x4.trans.shared.b8 [%0], {%1, %2, %3, %4};"
               ::"r"(row_addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
// four values -> four bytes (s0 lowest), clamped to the unsigned / signed 8-bit range by two chained saturating packs
template <bool OSIGNED>
__device__ __forceinline__ unsigned sat_pack4(int s0, int s1, int s2, int s3) {
  unsigned w23, w;
  if (OSIGNED) {
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(s3), "r"(s2), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(s1), "r"(s0), "r"(w23));
  } else {
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(s3), "r"(s2), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(s1), "r"(s0), "r"(w23));
  }
  return w;
}
// Saturating conversion to a byte.  The packing form of the convert (second source -> byte 0) is a single
// integer-pipe instruction; the plain cvt.sat.u8.s32 measured at twice its issue cost.
__device__ __forceinline__ int sat_u8(int x) {
  int d; asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %1;" : "=r"(d) : "r"(0), "r"(x)); return d;
}
__device__ __forceinline__ int sat_s8(int x) {
  int d; asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %1;" : "=r"(d) : "r"(0), "r"(x)); return d;
}

// Shared-memory matrix descriptor for a K-major operand tile whose rows are `bkb` bytes wide and
// stored with the matching TMA swizzle (32/64/128 B): 8-row groups are bkb*8 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t bkb) {
  const uint64_t layout = (bkb == 128) ? 2ull : (bkb == 64) ? 4ull : 6ull;
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);            // start address
  d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(((bkb * 8) >> 4) & 0x3FFF) << 32;  // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                            // descriptor version for this architecture
  d |= layout << 61;
  return d;
}

// Per-thread (= per output channel) constants of the epilogue.
struct ChanConst {
  int b, sh;            // main branch multiplier; shift (c, or c - min(c,32) on the fast path)
  int sh1;              // fast path: min(c, 32), the part of the shift taken by the funnel shift
  int cmin31;           // fast path: min(c, 31)
  int pre;              // pre-shift form (SMALL == 2): 32 - min(c, 32), the accumulator is shifted left by it first
  long long r0;         // bias*b + 2^(c-1)
  int rb, rh, rsh;      // residual multiplier; fast path: rh = 2^(rc-9), rsh = rc-8; else rsh = rc
  long long rr0;        // general path: 2^(rc-1)
  int bias;
};

// One output value on the 32-bit fast path (Eq. 4; Section 3.3):
//   main      y  = hi32(acc*b + bias*b + 2^(c-1)) >> (c-32)                         (needs c >= 32)
//   residual  y += (hi32((r << 24) * rb) + 2^(rc-9)) >> (rc-8)                      (needs 9 <= rc)
// The residual form is exact: (r<<24)*rb >> 32 = floor(r*rb / 2^8), the rounding constant 2^(rc-1) is
// a multiple of 2^8, and the dropped low 8 bits of r*rb cannot carry across a multiple of 2^(rc-8).
// (A 64-bit multiply-add followed by a funnel shift measured no faster.)  `r` is the stored 8-bit
// residual, already extended.  SMALL: 1 when some channel of the warp has c < 32 (exact funnel-shift form with a
// saturation guard); 2 when, besides, every such channel's accumulator and bias are known to stay below 2^(c-2)
// (TcParams::acc_bits, checked per channel when the constants are set up): the accumulator is then shifted left by
// 32 - c first and r0 was shifted with it, (acc << pre) * b + (r0 << pre) = (acc * b + r0) << pre exactly and without
// overflow, and the plain form applies again at the cost of one shift.
// RN: every channel of the warp has a narrow residual pair (m, a, s) with (r*m + a) >> s equal to the residual
// term for all 256 values of r (found and checked exhaustively by residual_narrow_kernel); rb / rh / rsh hold
// m / a / s then, and a 32-bit multiply-add replaces the shift, multiply-high and add.
// SPELLED: the product is written as the 32 x 32 -> 64 multiply-add instruction it is.  In the fragment loop, left
// to the compiler, the sign extension of k.b is hoisted out of the loop and the product becomes a full 64 x 64
// multiply (three to four multiply instructions per value); the other loops compile to the short form by themselves.
template <bool RES, bool RSIGNED, int SMALL, bool RN = false, bool SPELLED = false>
__device__ __forceinline__ int requant_fast(int acc, int r, const ChanConst& k) {
  if (SMALL == 2) acc <<= k.pre;
  long long t1;
  if (SPELLED) asm("mad.wide.s32 %0, %1, %2, %3;" : "=l"(t1) : "r"(acc), "r"(k.b), "l"(k.r0));
  else t1 = (long long)acc * (long long)k.b + k.r0;
  int s;
  if (SMALL != 1) {
    s = (int)(t1 >> 32) >> k.sh;                       // c >= 32 (or pre-shifted): |s| < 2^30
  } else {
    // some channel of this warp has c < 32: take bits [c, c+32) of the 64-bit value with a funnel shift
    // and saturate to +-2^30 when the exact value does not fit (it is far outside every clamp range then,
    // and |residual term| < 2^30 keeps the sum inside INT32)
    const int hi = (int)(t1 >> 32);
    const unsigned lo = (unsigned)t1;
    const int s0 = (int)__funnelshift_rc(lo, (unsigned)hi, k.sh1);
    const int above = hi >> k.cmin31;                  // the bits above the window (sign for c >= 32)
    s = (above == (s0 >> 31)) ? (s0 >> k.sh) : (hi < 0 ? INT_MIN : INT_MAX);
    s = max(min(s, 1 << 30), -(1 << 30));
  }
  if (RES && RN) {
    s += (r * k.rb + k.rh) >> k.rsh;
  } else if (RES) {
    const unsigned top = (unsigned)r << 24;
    if (RSIGNED) s += (__mulhi((int)top, k.rb) + k.rh) >> k.rsh;
    else s += (int)((__umulhi(top, (unsigned)k.rb) + (unsigned)k.rh) >> k.rsh);
  }
  return s;
}

// Pixel tile behind position `t` of the tile order (see TcParams::rev).
__device__ __forceinline__ int tile_at(const TcParams& p, int t) { return p.rev ? p.p_tiles - 1 - t : t; }

// The finished staging box of one warp leaves for global memory.  Dense tiles: one [columns][32 B] box at pixel
// `p_tile * pt + col0`.  Strip tiles: one box per 32 positions (a row, half a row or two rows of the pitch-2^lg_wp
// raster); columns at or beyond the image width and rows at or beyond its height fall outside the tensor map
// and are clipped by the copy.
__device__ __forceinline__ void store_warp_box(const TcParams& p, const CUtensorMap* map_out, uint32_t my_stage, int chx,
                                               int p_tile, int col0, int px_per_warp) {
  if (!p.strip) {
    const int p_base = p_tile * p.pt + col0;
    if (p_base < p.P) { tma_store_2d(map_out, my_stage, chx, p_base); tma_store_commit(); }
    return;
  }
  const int img = p_tile / p.tpi, y0 = (p_tile - img * p.tpi) * p.rows;
  bool any = false;
  for (int c = 0; c < (px_per_warp >> 5); ++c) {
    const int j0 = col0 + 32 * c;
    const int y = y0 + (j0 >> p.lg_wp), x = j0 & ((1 << p.lg_wp) - 1);
    if (y < p.ho && x < p.wo) { tma_store_4d(map_out, my_stage + (uint32_t)c * 1024u, chx, x, y, img); any = true; }
  }
  if (any) tma_store_commit();
}

// An epilogue warp hands its part of accumulator buffer `as` back.  The barrier that counts is the one the MMA issuer
// waits on: this CTA's, or the leading CTA's when two CTAs share the MMAs.
__device__ __forceinline__ void release_accumulator(const TcParams& p, SharedCtl& ctl, uint32_t as) {
  const uint32_t bar = smem_u32(&ctl.tempty[as]);
  if (p.duo) mbar_arrive_cluster(in_cta(bar, 0)); else mbar_arrive(bar);
}

// Everything an epilogue warp needs, gathered once so the tile loops can live in their own functions.
struct EpiCtx {
  const TcParams* p; SharedCtl* ctl; const CUtensorMap* map_out;
  uint8_t* smem_raw; uint32_t raw, out_stage, res_stage, res_tile_bytes, tmem_base;
  int warp, lane, q, cq, ew, half, col0, px_per_warp, ch, c_tile, p_tile0, p_step, lo, hi;
  bool ch_live, warp_live;
};

// Lean tile loop for the common case: 8-bit output through the staging box, 32-bit fast arithmetic,
// clamp by saturating convert or by min/max, optional 8-bit residual from the prefetched tile.
// Software-pipelined across chunks and tiles: while one 32-pixel accumulator chunk is processed, the
// next one (of this tile, or the first of the group's next tile) streams from tensor memory into the
// other register set; the accumulator buffer is handed back as soon as its last chunk has been read,
// the residual tile as soon as its last bytes have been used, both before the tile's store is issued.
template <bool RES, bool RSIGNED, bool SAT, bool OSIGNED, int SMALL, bool RN, bool OUT4 = false>
__device__ __forceinline__ void epilogue_loop_fast8(const EpiCtx& e_in, const ChanConst& k_in) {
  // Private copies: the caller's objects live in local memory (their address is passed to the general
  // loop), so every asm statement with a memory clobber would force their fields to be re-read.
  const EpiCtx e = e_in;
  ChanConst k_own = k_in;
  if (SMALL == 2) k_own.r0 <<= k_own.pre;          // the pre-shift form of requant_fast
  const ChanConst k = k_own;
  const TcParams& p = *e.p;
  SharedCtl& ctl = *e.ctl;
  const int lane = e.lane, q = e.q, cq = e.cq, col0 = e.col0, px_per_warp = e.px_per_warp;
  const uint32_t my_stage = e.out_stage + (uint32_t)e.ew * (uint32_t)(px_per_warp * 32);
  uint8_t* const my_stage_ptr = e.smem_raw + (my_stage - e.raw);
  const uint8_t* const res_stage_ptr = e.smem_raw + (e.res_stage - e.raw);
  const int nchunks = px_per_warp >> 5;           // 2 or 4
  const uint32_t bmask = (1u << p.lg_bufs) - 1u, rmask = (1u << p.lg_rbufs) - 1u;
  const int tile_step = e.p_step;
  int p_tile = e.p_tile0;
  if (p_tile >= p.p_tiles) return;
  uint32_t tcount = 0;
  uint32_t as = 0, aph = 0;
  const uint32_t t_warp = e.tmem_base + ((uint32_t)(q * 32) << 16) + col0;

  auto wait_bar = [&](unsigned long long* bar, uint32_t ph) -> bool {
    uint32_t w = 1;
    if (lane == 0) w = mbar_wait(smem_u32(bar), ph, &ctl, p.status, HQ_DEV_TIMEOUT_EPILOGUE) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, w, 0) != 0;
  };
  auto chunk = [&](const int (&v)[32], const uint8_t* res_tile, int c) {
    if (!e.warp_live) return;
    int y[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const int r = !RES ? 0 : RSIGNED ? (int)(signed char)res_tile[(c * 32 + j) * kTileC] : (int)res_tile[(c * 32 + j) * kTileC];
      const int s = requant_fast<RES, RSIGNED, SMALL, RN>(v[j], r, k);
      y[j] = SAT ? (OSIGNED ? sat_s8(s) : sat_u8(s)) : min(max(s, e.lo), e.hi);
    }
    if (!OUT4) {
#pragma unroll
      for (int j = 0; j < 32; ++j) my_stage_ptr[(c * 32 + j) * 32 + lane] = (uint8_t)y[j];
    } else {
      // Unsigned 4-bit output (0 <= y <= 15 after the clamp): a byte holds the channel pair of two neighbouring
      // lanes.  Each lane packs its 32 pixels into four words of eight nibbles, the pair exchanges the words
      // (4 shuffles instead of 32), both interleave them into bytes, and the even lane stores pixels 0-3 of every
      // eight, the odd lane pixels 4-7: rows of 16 bytes per pixel in the staging box.
      const bool odd = lane & 1;
      const unsigned sel = odd ? 0x7362u : 0x5140u;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        unsigned mine = (unsigned)y[8 * w + 7];
#pragma unroll
        for (int i = 6; i >= 0; --i) mine = mine * 16u + (unsigned)y[8 * w + i];
        const unsigned other = __shfl_xor_sync(0xffffffffu, mine, 1);
        const unsigned a = odd ? other : mine, b = odd ? mine : other;        // even channel, odd channel
        const unsigned t = (a & 0x0F0F0F0Fu) | ((b << 4) & 0xF0F0F0F0u);        // pixels 0, 2, 4, 6
        const unsigned u = ((a >> 4) & 0x0F0F0F0Fu) | (b & 0xF0F0F0F0u);        // pixels 1, 3, 5, 7
        const unsigned four = __byte_perm(t, u, sel);                          // pixels 0-3 (even lane) or 4-7 (odd lane)
        const int px = c * 32 + 8 * w + (odd ? 4 : 0);
#pragma unroll
        for (int i = 0; i < 4; ++i) my_stage_ptr[(px + i) * 16 + (lane >> 1)] = (uint8_t)(four >> (8 * i));
      }
    }
  };

  int va[32], vb[32];
  bool ok = wait_bar(&ctl.tfull[as], aph);
  if (!ok) return;
  tc_fence_after();
  tmem_ld32_issue(t_warp + as * p.pt, va);
  bool pending = true;                            // a tensor-memory load into va is in flight
  while (true) {
    const uint32_t rs = tcount & rmask, rph = (tcount >> p.lg_rbufs) & 1u;       // residual buffer and its phase
    if (RES && !wait_bar(&ctl.rfull[rs], rph)) break;
    const uint8_t* const res_tile = res_stage_ptr + rs * e.res_tile_bytes + (uint32_t)col0 * kTileC + cq * 32 + lane;
    const uint32_t t_addr = t_warp + as * p.pt;
    const bool has_next = p_tile + tile_step < p.p_tiles;
    const uint32_t nas = (tcount + 1u) & bmask, naph = ((tcount + 1u) >> p.lg_bufs) & 1u;

    for (int c = 0; c < nchunks; c += 2) {
      // ---- chunk c (registers va), while chunk c+1 streams into vb
      tmem_ld_wait();
      tmem_ld32_issue(t_addr + (c + 1) * 32, vb);
      if (c == 0) {                               // the previous tile's store must have read the staging box
        if (lane == 0) tma_store_wait_read0();
        __syncwarp();
      }
      chunk(va, res_tile, c);
      // ---- chunk c+1 (registers vb), while the next chunk streams into va
      tmem_ld_wait();
      pending = false;
      if (c + 2 < nchunks) {
        tmem_ld32_issue(t_addr + (c + 2) * 32, va);
        pending = true;
      } else {
        // every lane has read its last accumulator columns of this tile: hand the buffer back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) release_accumulator(p, ctl, as);
      }
      chunk(vb, res_tile, c + 1);
    }
    if (RES) {                                    // every lane has used its last residual bytes of this tile
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl.rempty[rs]));
    }
    // Only now wait for the group's next tile: its copies may be queued behind the buffers released above.
    if (has_next) {
      ok = wait_bar(&ctl.tfull[nas], naph);
      if (ok) { tc_fence_after(); tmem_ld32_issue(t_warp + nas * p.pt, va); pending = true; }
    }
    fence_async_smem();                           // make this lane's box writes visible to the TMA engine
    __syncwarp();
    if (lane == 0 && e.warp_live) store_warp_box(p, e.map_out, my_stage, (e.c_tile * kTileC + cq * 32) >> (OUT4 ? 1 : 0), tile_at(p, p_tile), col0, px_per_warp);
    if (!has_next || !ok) break;
    p_tile += tile_step; ++tcount; as = nas; aph = naph;
  }
  if (pending) tmem_ld_wait();
  if (lane == 0) tma_store_wait_all();
}

// Per-channel constants of one output channel (Eq. 4 and the residual rescale of Section 3.3), as the loops below want
// them: `fast` selects the 32-bit forms (see requant_fast), `narrow` the checked narrow residual pair of the channel.
__device__ __forceinline__ ChanConst chan_const_for(const TcParams& p, int ch, bool fast, bool narrow, bool pre = false) {
  ChanConst k{};
  const bool live = ch < p.C;
  k.bias = (live && p.bias) ? p.bias[ch] : 0;
  k.b = live ? p.b[ch] : 0;
  const int cc = live ? p.c[ch] : 32;
  k.sh = cc;
  k.r0 = (long long)k.bias * (long long)k.b + (1LL << (cc - 1));
  if (p.res) {
    const int rcc = live ? p.rc[ch] : 32;
    k.rb = live ? p.rb[ch] : 0;
    k.rsh = rcc;
    k.rr0 = 1LL << (rcc - 1);
  }
  if (fast) {
    k.sh1 = k.sh < 32 ? k.sh : 32;
    k.cmin31 = k.sh < 31 ? k.sh : 31;
    k.sh -= k.sh1;
    k.pre = 32 - k.sh1;
    if (pre) k.r0 <<= k.pre;                                         // the pre-shift form (the caller checked its bounds)
    if (p.res) {
      if (k.rsh >= 40) { k.rb = 0; k.rh = 0; k.rsh = 1; }            // |r*rb| < 2^39: rounds to 0
      else { k.rh = 1 << (k.rsh - 9); k.rsh -= 8; }
    }
  }
  if (narrow) {
    const int4 nr = live ? p.res_narrow[ch] : make_int4(0, 0, 0, 1);
    k.rb = nr.x; k.rh = nr.y; k.rsh = nr.z;
  }
  return k;
}

// Tile loop of the launch shape for fused 8-bit residuals (eight epilogue warps and a store warp, 128-pixel tiles).
//
// Nothing moves byte by byte here.  The residual tile [128 pixels][128 channels] lands in shared memory by TMA in the
// 128-byte-swizzled K-major form of an MMA operand, and the MMA issuer multiplies it by the 128 x 128 identity matrix:
// D2[ch][px] = sum_k I[ch][k] * R[px][k] = R[px][ch], i.e. the tensor core transposes the tile and widens it to INT32
// in tensor-memory columns next to the accumulator.  An epilogue warp owns 16 accumulator lanes (channels) and reads
// accumulator and residual with the same 16x256b loads, which hand thread T the values of channels t4, t4 + 8 for
// pixel pairs -- the fragment of a 16 x 8 matrix.  It applies Eq. 4 and the residual add of Section 3.3 with the
// constants of its two channels in registers, packs four results into a word with two saturating converts, and one
// stmatrix (transposing, b8) writes 32 pixels x 16 channels as 16-byte row pieces into the tile the residual came
// from (the MMA has finished reading it: the accumulator barrier is committed after the identity MMAs).  The loads of
// the next 32 columns (or of the next tile's first) are in flight while a unit is processed.  Warps do not wait for
// each other: each arrives on the tile's `ofull` barrier when its pieces are written, and the store warp alone waits
// there, stores the [128][128] box (128-byte swizzle, as it was loaded) and hands the buffer back.
// GEN: 64-bit arithmetic for every shift 1..62 (a residual shift below 9, or an INT32 residual).  SMALL: some channel
// of the warp has c < 32 (common with 4-bit operands, whose accumulators are small): funnel-shift form of Eq. 4.
template <bool GEN, bool RSIGNED, bool SAT, bool OSIGNED, bool RN, int SMALL = 0>
__device__ __forceinline__ void epilogue_loop_frag(const EpiCtx& e_in) {
  const EpiCtx e = e_in;
  const TcParams& p = *e.p;
  SharedCtl& ctl = *e.ctl;
  const int lane = e.lane, q = e.q, hh = e.half;
  const int t4 = lane >> 2;
  ChanConst k[2];                                   // channels 32 q + 16 hh + 8 r + t4, r = 0, 1
#pragma unroll
  for (int r = 0; r < 2; ++r) k[r] = chan_const_for(p, e.c_tile * kTileC + 32 * q + 16 * hh + 8 * r + t4, !GEN, RN, SMALL == 2);
  const uint32_t bmask = (1u << p.lg_bufs) - 1u, rmask = (1u << p.lg_rbufs) - 1u;
  constexpr int units = 4;                          // 32 pixel columns per unit, 128-pixel tiles
  const uint32_t t_lane = e.tmem_base + ((uint32_t)(q * 32 + 16 * hh) << 16);
  // byte offset of this thread's 16-byte piece in a unit's 32 rows: row `lane`, chunk (2 q + hh) ^ (row % 8)
  const uint32_t row_off = (uint32_t)lane * 128u + ((uint32_t)((2 * q + hh) ^ (lane & 7)) << 4);
  if (e.p_tile0 >= p.p_tiles) return;
  auto wait_bar = [&](unsigned long long* bar, uint32_t ph) -> bool {
    uint32_t w = 1;
    if (lane == 0) w = mbar_wait(smem_u32(bar), ph, &ctl, p.status, HQ_DEV_TIMEOUT_EPILOGUE) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, w, 0) != 0;
  };
  auto one = [&](int acc, int r, const ChanConst& c) -> int {
    if (GEN) {
      const long long y = (((long long)acc * (long long)c.b + c.r0) >> c.sh) + (((long long)r * (long long)c.rb + c.rr0) >> c.rsh);
      return hq_clamp_ll(y, p.relu, p.qmin, p.qmax);
    }
    const int y = requant_fast<true, RSIGNED, SMALL, RN, true>(acc, r, c);
    return SAT ? y : min(max(y, e.lo), e.hi);
  };
  // one unit: 16 values per thread -> four words -> one transposing store of 32 pixel rows x 16 channel bytes
  auto unit = [&](const int (&va)[16], const int (&vr)[16], uint32_t tile, int u) {
    unsigned w[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const int y0 = one(va[4 * g + 0], vr[4 * g + 0], k[0]), y1 = one(va[4 * g + 1], vr[4 * g + 1], k[0]);
      const int y2 = one(va[4 * g + 2], vr[4 * g + 2], k[1]), y3 = one(va[4 * g + 3], vr[4 * g + 3], k[1]);
      w[g] = sat_pack4<OSIGNED>(y0, y1, y2, y3);
    }
    // this thread names the row of pixel 32 u + lane: 16 bytes at channel offset 32 q + 16 hh of the row (row_off)
    if (e.warp_live) stmatrix_t_x4(tile + row_off + (uint32_t)u * 4096u, w[0], w[1], w[2], w[3]);
  };
  auto issue = [&](uint32_t as, int u, int (&va)[16], int (&vr)[16]) {
    const uint32_t t_addr = t_lane + as * p.acc_stride + 32 * u;
    tmem_ld_frag16(t_addr, va);
    tmem_ld_frag16(t_addr + p.pt, vr);
  };

  int a0[16], r0[16], a1[16], r1[16];
  uint32_t tcount = 0, as = 0;
  int p_tile = e.p_tile0;
  if (!wait_bar(&ctl.tfull[0], 0)) return;          // accumulator AND transposed residual are in tensor memory
  tc_fence_after();
  issue(0, 0, a0, r0);
  bool pending = true;
  while (true) {
    const uint32_t rs = tcount & rmask;
    const uint32_t tile = e.res_stage + rs * e.res_tile_bytes;          // [128 pixels][128 bytes], 128-byte swizzle
    const bool has_next = p_tile + e.p_step < p.p_tiles;
    const uint32_t nas = (tcount + 1u) & bmask, naph = ((tcount + 1u) >> p.lg_bufs) & 1u;
    bool ok = true, next_issued = false;
#pragma unroll
    for (int u = 0; u < units; u += 2) {
      // ---- unit u (registers a0 / r0), while unit u + 1 streams into a1 / r1
      tmem_ld_wait();
      issue(as, u + 1, a1, r1);
      unit(a0, r0, tile, u);
      // ---- unit u + 1, while the next unit streams into a0 / r0
      tmem_ld_wait();
      pending = false;
      if (u + 2 < units) {
        issue(as, u + 2, a0, r0);
        pending = true;
      } else {
        // every lane has read its last columns of this tile: hand the accumulator buffer back, and start on the next
        // tile's first unit if that tile is already there (else after this unit's arithmetic)
        tc_fence_before();
        __syncwarp();
        if (lane == 0) release_accumulator(p, ctl, as);
        if (has_next) {
          uint32_t there = 0;
          if (lane == 0) there = mbar_try_wait(smem_u32(&ctl.tfull[nas]), naph) ? 1u : 0u;
          if (__shfl_sync(0xffffffffu, there, 0)) { tc_fence_after(); issue(nas, 0, a0, r0); pending = true; next_issued = true; }
        }
      }
      unit(a1, r1, tile, u + 1);
    }
    fence_async_smem();                             // make this lane's pieces visible to the TMA engine
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&ctl.ofull[rs]));
    if (!has_next) break;
    if (!next_issued) {
      ok = wait_bar(&ctl.tfull[nas], naph);
      if (!ok) break;
      tc_fence_after();
      issue(nas, 0, a0, r0);
      pending = true;
    }
    p_tile += e.p_step; ++tcount; as = nas;
  }
  if (pending) tmem_ld_wait();
}

// General tile loop: every output type, direct stores, 64-bit arithmetic, INT32 residuals.
__device__ __noinline__ void epilogue_loop_general(const EpiCtx& e, const ChanConst& k, uint32_t fast) {
  const TcParams& p = *e.p;
  SharedCtl& ctl = *e.ctl;
  const CUtensorMap& map_out = *e.map_out;
  uint8_t* const smem_raw = e.smem_raw;
  const uint32_t raw = e.raw, out_stage = e.out_stage, res_stage = e.res_stage, res_tile_bytes = e.res_tile_bytes;
  const uint32_t tmem_base = e.tmem_base;
  const int lane = e.lane, q = e.q, cq = e.cq, ew = e.ew, col0 = e.col0, px_per_warp = e.px_per_warp, ch = e.ch;
  const int c_tile = e.c_tile, p_tile0 = e.p_tile0, p_step = e.p_step, lo = e.lo, hi = e.hi;
  const bool ch_live = e.ch_live, warp_live = e.warp_live;
  const bool staged_out = p.staged_out != 0;
    // staging box of this warp: [px_per_warp pixels][32 channels] bytes (16 bytes per pixel at 4 bit)
    const int row_b = (p.out_bits == 4) ? 16 : 32;
    const uint32_t my_stage = out_stage + (uint32_t)ew * (uint32_t)(px_per_warp * 32);   // px_per_warp rows x 32 bytes reserved per warp
    // plain pointers to the same bytes: ordinary loads / stores that the compiler may schedule freely
    uint8_t* const my_stage_ptr = smem_raw + (my_stage - raw);
    const uint8_t* const res_stage_ptr = smem_raw + (res_stage - raw);
    const uint32_t bmask = (1u << p.lg_bufs) - 1u;
    uint32_t tcount = 0;
    for (int p_tile = p_tile0; p_tile < p.p_tiles; p_tile += p_step, ++tcount) {
      const uint32_t as = tcount & bmask, aph = (tcount >> p.lg_bufs) & 1u;
      const uint32_t rs = tcount & ((1u << p.lg_rbufs) - 1u), rph = (tcount >> p.lg_rbufs) & 1u;
      uint32_t w = 1;
      if (lane == 0) {
        if (staged_out) tma_store_wait_read0();   // the previous store has read this warp's staging box
        w = mbar_wait(smem_u32(&ctl.tfull[as]), aph, &ctl, p.status, HQ_DEV_TIMEOUT_EPILOGUE) ? 1u : 0u;
        if (w && p.staged_res)
          w = mbar_wait(smem_u32(&ctl.rfull[rs]), rph, &ctl, p.status, HQ_DEV_TIMEOUT_EPILOGUE) ? 1u : 0u;
      }
      w = __shfl_sync(0xffffffffu, w, 0);
      if (!w) break;
      tc_fence_after();                            // lane 0 observed the barriers; the shuffle ordered the warp
      const int p_base = tile_at(p, p_tile) * p.pt + col0;              // first pixel of this warp's columns
      const uint8_t* const res_tile = res_stage_ptr + rs * res_tile_bytes + (uint32_t)col0 * kTileC + cq * 32 + lane;

      for (int cc0 = 0; cc0 < px_per_warp; cc0 += 32) {
        int v[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + as * p.pt + col0 + cc0, v);
        if (!warp_live) continue;
        const int px0 = p_base + cc0;                                     // global pixel of v[0]

        if (p.out_bits == 32) {
          // raw accumulator + bias: 32 lanes write 32 consecutive INT32 channels of one pixel
          if (ch_live) {
            int* dst = (int*)p.out + (long long)px0 * p.C + ch;
#pragma unroll
            for (int j = 0; j < 32; ++j) if (px0 + j < p.P) dst[(long long)j * p.C] = v[j] + k.bias;
          }
          continue;
        }

        int y[32];
        if (fast) {
          unsigned rb8[32];
          if (p.res) {
            if (p.staged_res) {
#pragma unroll
              for (int j = 0; j < 32; ++j) rb8[j] = res_tile[(cc0 + j) * kTileC];
            } else {
              const unsigned char* rp = (const unsigned char*)p.res + (long long)px0 * p.C + ch;
#pragma unroll
              for (int j = 0; j < 32; ++j) rb8[j] = (ch_live && px0 + j < p.P) ? (unsigned)__ldg(rp + (long long)j * p.C) : 0u;
            }
          }
          const int variant = (p.res ? 2 : 0) | (p.res_signed ? 1 : 0);
          if (variant == 2) {
#pragma unroll
            for (int j = 0; j < 32; ++j) y[j] = requant_fast<true, false, true>(v[j], (int)rb8[j], k);
          } else if (variant == 3) {
#pragma unroll
            for (int j = 0; j < 32; ++j) y[j] = requant_fast<true, true, true>(v[j], (int)(signed char)rb8[j], k);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) y[j] = requant_fast<false, false, true>(v[j], 0, k);
          }
          if (p.sat_pack) {
            if (p.out_signed) {
#pragma unroll
              for (int j = 0; j < 32; ++j) y[j] = sat_s8(y[j]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) y[j] = sat_u8(y[j]);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) y[j] = min(max(y[j], lo), hi);
          }
        } else {
          // general CTA: full 64-bit results (any 1 <= c <= 62, INT32 residual operands)
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            long long s = ((long long)v[j] * (long long)k.b + k.r0) >> k.sh;
            if (p.res) {
              int r = 0;
              if (p.staged_res) {
                const unsigned byte = res_tile[(cc0 + j) * kTileC];
                r = p.res_signed ? (int)(signed char)byte : (int)byte;
              } else if (ch_live && px0 + j < p.P) {
                r = hq_load_elem(p.res, (long long)(px0 + j) * p.C + ch, p.res_bits, p.res_signed);
              }
              s += ((long long)r * (long long)k.rb + k.rr0) >> k.rsh;
            }
            y[j] = hq_clamp_ll(s, p.relu, p.qmin, p.qmax);
          }
        }

        if (p.out_bits == 4) {
          // neighbouring channels share a byte: even lanes collect the odd lane's nibble
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int other = __shfl_xor_sync(0xffffffffu, y[j], 1);
            y[j] = (y[j] & 0xF) | ((other & 0xF) << 4);
          }
          if (staged_out) {
            if (!(lane & 1)) {
#pragma unroll
              for (int j = 0; j < 32; ++j) my_stage_ptr[(cc0 + j) * row_b + (lane >> 1)] = (uint8_t)y[j];
            }
          } else if (ch_live && !(lane & 1)) {
            unsigned char* dst = (unsigned char*)p.out + (((long long)px0 * p.C + ch) >> 1);
#pragma unroll
            for (int j = 0; j < 32; ++j) if (px0 + j < p.P) dst[((long long)j * p.C) >> 1] = (unsigned char)y[j];
          }
        } else if (staged_out) {
#pragma unroll
          for (int j = 0; j < 32; ++j) my_stage_ptr[(cc0 + j) * 32 + lane] = (uint8_t)y[j];
        } else if (ch_live) {
          unsigned char* dst = (unsigned char*)p.out + (long long)px0 * p.C + ch;
#pragma unroll
          for (int j = 0; j < 32; ++j) if (px0 + j < p.P) dst[(long long)j * p.C] = (unsigned char)(y[j] & 0xFF);
        }
      }
      // accumulator columns (and the residual tile) are no longer needed by this warp: hand them back
      tc_fence_before();
      if (staged_out) fence_async_smem();        // make this lane's box writes visible to the TMA engine
      __syncwarp();
      if (lane == 0) {
        release_accumulator(p, ctl, as);
        if (p.staged_res) mbar_arrive(smem_u32(&ctl.rempty[rs]));
        if (staged_out && warp_live)
          store_warp_box(p, &map_out, my_stage, ((c_tile * kTileC + cq * 32) * p.out_bits) >> 3, tile_at(p, p_tile), col0, px_per_warp);
      }
    }

    if (staged_out && lane == 0) tma_store_wait_all();
}

// ---------------------------------------------------------------- the kernel -----------------
// DUO: the instantiation that may be launched as clusters of two CTAs sharing their MMAs; only it contains the
// cta_group::2 instructions (a kernel that contains them cannot be launched without clusters).
// RTM: the instantiation for fused 8-bit residuals that travel through tensor memory; it has one more warp, which
// stores the finished output tiles.
template <int EPI_WARPS, int MIN_CTAS, int MMA_WARPS, bool DUO = false, bool RTM = false>
__global__ void __launch_bounds__(32 * (1 + MMA_WARPS + EPI_WARPS + (RTM ? 1 : 0)), MIN_CTAS)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_res,
               const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ SharedCtl ctl;

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;          // operand stages, 1024-byte aligned
  const uint32_t w_bytes = kTileC * p.bkb;
  // strip mode: the stages carry weights only; duo: each CTA of the pair holds half of the pixel rows
  const uint32_t x_bytes = p.strip ? 0u : (uint32_t)((p.pt >> p.duo) * p.bkb);
  uint32_t rank = 0u;                                      // 0 = the CTA that issues the pair's MMAs
  if constexpr (DUO) rank = cluster_ctarank();
  const uint32_t x_off = p.wres ? 0u : w_bytes;          // offset of the X tile inside a stage
  const uint32_t stage_bytes = x_off + x_bytes;
  const uint32_t out_stage = tiles + p.out_stage_off;
  const uint32_t res_stage = tiles + p.res_stage_off;
  const uint32_t res_tile_bytes = p.pt * kTileC;          // [pt pixels][128 channels] bytes
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Tile schedule: the grid is a multiple of c_tiles, so a CTA keeps one channel tile for its whole
  // life (its weights' rows and per-channel constants never change) and strides over the pixel tiles.
  const int c_tile = blockIdx.x % p.c_tiles;
  const int p_tile0 = blockIdx.x / p.c_tiles;
  const int p_step = gridDim.x / p.c_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&ctl.full[s]), 1); mbar_init(smem_u32(&ctl.empty[s]), 1); }
    for (int s = 0; s < (1 << p.lg_bufs); ++s) {
      mbar_init(smem_u32(&ctl.tfull[s]), p.ni); mbar_init(smem_u32(&ctl.tempty[s]), (4 * p.halves) << p.duo);
      mbar_init(smem_u32(&ctl.tstart[s]), 1);
    }
    for (int s = 0; s < (1 << p.lg_rbufs); ++s) {
      mbar_init(smem_u32(&ctl.rfull[s]), 1);
      mbar_init(smem_u32(&ctl.rempty[s]), RTM ? 1 : 4 * p.halves);
      mbar_init(smem_u32(&ctl.ofull[s]), EPI_WARPS);
    }
    mbar_init(smem_u32(&ctl.drain), p.ni);
    mbar_init(smem_u32(&ctl.wfull), 1);
    for (int s = 0; s < 3; ++s) { mbar_init(smem_u32(&ctl.pfull[s]), 1); mbar_init(smem_u32(&ctl.pempty[s]), p.ni); }
    ctl.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) { if constexpr (DUO) tmem_alloc2(smem_u32(&ctl.tmem_base), p.tmem_cols); else tmem_alloc(smem_u32(&ctl.tmem_base), p.tmem_cols); }
  if (p.rtm) {
    // the identity matrix as a K-major MMA operand, [128 rows][128 bytes] with the 128-byte swizzle: 16-byte chunk
    // c of row r sits at chunk position c ^ (r % 8); row r holds a single 1 at byte r
    uint4* ident = (uint4*)(smem_raw + (tiles - raw) + p.ident_off);
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) {
      const int r = i >> 3, c = (i & 7) ^ (r & 7);
      uint32_t word[4] = {0u, 0u, 0u, 0u};
      if (c == (r >> 4)) word[(r & 15) >> 2] = 1u << (8 * (r & 3));
      ident[i] = make_uint4(word[0], word[1], word[2], word[3]);
    }
    fence_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (DUO) cluster_sync_all();   // both CTAs' barriers exist before either touches the other's
  tc_fence_after();
  const uint32_t tmem_base = ctl.tmem_base;
  // Programmatic dependent launch: this grid may have started while the previous kernel of the stream was
  // still finishing (its CTAs leave the SMs one by one); everything above touched only this CTA's own
  // resources.  The threads that read what the previous kernel wrote -- the producer lane (activations and
  // residual tiles by TMA) and epilogue warps that load a residual directly -- wait for that grid to complete
  // first; the other roles only consume what arrives behind the producer's barriers.  The next kernel's CTAs
  // may start filling SMs as ours leave.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      // No division or modulo in this loop: one thread runs it and every dependent instruction
      // costs its full latency, so stage / phase / filter-tap indices are carried incrementally.
      uint32_t it = 0, tcount = 0, s = 0, ph = 0;
      const uint32_t rmask = (1u << p.lg_rbufs) - 1u;
      bool ok = true;
      // (image, row, column) of the tile's first output pixel, advanced by a fixed step per tile
      const int ho = p.howo / p.wo;
      // (duo: this CTA fetches the half of the tile's pixel rows that starts at half_off)
      const int half_off = p.duo ? (int)rank * (p.pt >> 1) : 0;
      const int px_first = tile_at(p, p_tile0) * p.pt + half_off;
      int img = px_first / p.howo;
      int oh = (px_first - img * p.howo) / p.wo;
      int ow = px_first - img * p.howo - oh * p.wo;
      const int step = p_step * p.pt;
      const int d_img = step / p.howo, d_oh = (step - d_img * p.howo) / p.wo, d_ow = step - d_img * p.howo - d_oh * p.wo;
      if (p.wres) {              // the channel tile's weights for every K block, once
        const uint32_t bar = smem_u32(&ctl.wfull);
        mbar_expect_tx(bar, (uint32_t)p.k_blocks * w_bytes);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          const uint32_t w_dst = tiles + p.wres_off + (uint32_t)kb * w_bytes;
          if (p.fold) {
            tma_load_2d(w_dst, &map_w, bar, kb * p.bkb, 0);
            tma_load_2d(w_dst + 64 * p.bkb, &map_w, bar, kb * p.bkb, 0);
          } else {
            tma_load_2d(w_dst, &map_w, bar, kb * p.bkb, c_tile * kTileC);
          }
        }
      }
      // The resident weights above do not wait for the previous kernel: weights are never written by the launch
      // immediately before this one (the helper kernels that prepare weights are always followed by another launch).
      // Everything below reads activations, which the previous kernel may still be writing.
      asm volatile("griddepcontrol.wait;" ::: "memory");
      const unsigned long long pol_first = policy_evict_first();
      uint32_t pit = 0;                                // strip mode: patches started
      if (p.strip) {
        uint32_t ps = 0, pph = 0;
        for (int p_tile = p_tile0; p_tile < p.p_tiles && ok; p_tile += p_step, ++tcount) {
          const int t_act = tile_at(p, p_tile);
          const int img_s = t_act / p.tpi, y0 = (t_act - img_s * p.tpi) * p.rows;
          for (int chunk = 0; chunk < p.cchunks && ok; ++chunk) {
            // the padded patch of this cin chunk: columns -1 .. 2^lg_wp - 2, rows y0-1 .. y0+rows+1 (zeros outside the image)
            if (!mbar_wait(smem_u32(&ctl.pempty[ps]), pph ^ 1u, &ctl, p.status, HQ_DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
            const uint32_t pbar = smem_u32(&ctl.pfull[ps]);
            mbar_expect_tx(pbar, p.patch_bytes);
            tma_load_4d(tiles + p.patch_off + ps * p.patch_bytes, &map_x, pbar, chunk * p.bkb, -1, y0 - 1, img_s);
            ++pit;
            if (++ps == (uint32_t)p.npatch) { ps = 0; pph ^= 1u; }
            if (p.wres) continue;
            for (int tap = 0; tap < 9; ++tap, ++it) {      // the nine weight blocks that meet this patch
              if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, p.status, HQ_DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
              const uint32_t bar = smem_u32(&ctl.full[s]);
              const uint32_t w_dst = tiles + s * stage_bytes;
              const int kb = tap * p.cchunks + chunk;
              mbar_expect_tx(bar, stage_bytes);
              if (p.fold) {
                tma_load_2d(w_dst, &map_w, bar, kb * p.bkb, 0);
                tma_load_2d(w_dst + 64 * p.bkb, &map_w, bar, kb * p.bkb, 0);
              } else {
                tma_load_2d(w_dst, &map_w, bar, kb * p.bkb, c_tile * kTileC);
              }
              if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; }
            }
          }
        }
      }
      for (int p_tile = p_tile0; p_tile < p.p_tiles && ok && !p.strip; p_tile += p_step, ++tcount) {
        const int p0 = tile_at(p, p_tile) * p.pt;
        const int cw = ow * p.stride - p.pad, chh = oh * p.stride - p.pad, img_now = img;
        if (!p.rev) {
          ow += d_ow; if (ow >= p.wo) { ow -= p.wo; ++oh; }
          oh += d_oh; if (oh >= ho) { oh -= ho; ++img; }
          img += d_img;
        } else {                                     // the same step backwards, with borrows (unused after the last tile)
          ow -= d_ow; if (ow < 0) { ow += p.wo; --oh; }
          oh -= d_oh; if (oh < 0) { oh += ho; --img; }
          img -= d_img;
        }
        int chunk = 0, tap_s = 0, tap_r = 0;
        // The residual tile of this output tile is fetched as soon as its buffer is free, but this thread only
        // blocks for the buffer after the tile's last operand block is on its way: the buffer comes back when the
        // epilogue of an earlier tile ends, and the operand copies must not queue behind that.
        bool res_due = p.staged_res != 0;
        auto residual = [&](bool must) -> bool {
          const uint32_t rbuf = tcount & rmask, rph = (tcount >> p.lg_rbufs) & 1u;
          const uint32_t rb = smem_u32(&ctl.rempty[rbuf]);
          if (!mbar_try_wait(rb, rph ^ 1u)) {
            if (!must) return true;
            if (!mbar_wait(rb, rph ^ 1u, &ctl, p.status, HQ_DEV_TIMEOUT_PRODUCER)) return false;
          }
          const uint32_t bar = smem_u32(&ctl.rfull[rbuf]);
          mbar_expect_tx(bar, res_tile_bytes);
          tma_load_2d_hint(res_stage + rbuf * res_tile_bytes, &map_res, bar, c_tile * kTileC, p0, pol_first);
          res_due = false;
          return true;
        };
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          if (res_due && !residual(false)) { ok = false; break; }
          if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, p.status, HQ_DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
          const uint32_t bar = smem_u32(&ctl.full[s]);
          const uint32_t w_dst = tiles + s * stage_bytes;
          if constexpr (DUO) {
            // Both CTAs of the pair fetch their own weight rows and their half of the pixel rows into their own
            // stage; all four copies are counted on the leading CTA's barrier, which alone expects the bytes.
            if (rank == 0) mbar_expect_tx(bar, 2u * stage_bytes);
            if (p.x_tiled) tma_load_2d_2cta(w_dst + x_off, &map_x, bar, chunk * p.bkb, p0 + half_off);
            else tma_load_im2col_2cta(w_dst + x_off, &map_x, bar, chunk * p.bkb, cw, chh, img_now, (uint16_t)tap_s, (uint16_t)tap_r);
            tma_load_2d_2cta(w_dst, &map_w, bar, kb * p.bkb, c_tile * kTileC);
            if (++chunk == p.cchunks) { chunk = 0; if (++tap_s == p.kw) { tap_s = 0; ++tap_r; } }
            if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; }
            if (res_due && kb + 1 == p.k_blocks && !residual(true)) { ok = false; break; }
            continue;
          }
          mbar_expect_tx(bar, stage_bytes);
          if (p.x_tiled) {
            tma_load_2d_hint(w_dst + x_off, &map_x, bar, chunk * p.bkb, p0, pol_first);
          } else {
            tma_load_im2col(w_dst + x_off, &map_x, bar, chunk * p.bkb, cw, chh, img_now, (uint16_t)tap_s, (uint16_t)tap_r);
          }
          if (p.wres) {
            // weights are resident
          } else if (p.fold) {   // 64-row box, twice: accumulator lanes 64-127 repeat lanes 0-63
            tma_load_2d(w_dst, &map_w, bar, kb * p.bkb, 0);
            tma_load_2d(w_dst + 64 * p.bkb, &map_w, bar, kb * p.bkb, 0);
          } else {
            tma_load_2d(w_dst, &map_w, bar, kb * p.bkb, c_tile * kTileC);
          }
          if (++chunk == p.cchunks) { chunk = 0; if (++tap_s == p.kw) { tap_s = 0; ++tap_r; } }
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; }
          if (res_due && kb + 1 == p.k_blocks && !residual(true)) { ok = false; break; }
        }
      }
      // Drain: every copy this thread started must have landed before the CTA may exit.
      // (the odd CTA of a pair sees no completion of its own copies: they are counted on the leading CTA's barriers,
      // whose MMAs consume them before the pair's closing cluster barrier)
      const uint32_t issued = (p.duo && rank != 0) ? 0u : (it < (uint32_t)p.stages ? it : (uint32_t)p.stages);
      for (uint32_t j = 0; j < (p.npatch > 0 ? (pit < (uint32_t)p.npatch ? pit : (uint32_t)p.npatch) : 0u); ++j) {
        const uint32_t k = pit - 1 - j;
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&ctl.pfull[k % p.npatch]), (k / p.npatch) & 1u)) {
          if (global_ns() - t0 > kWaitBudgetNs) { atomicCAS(p.status, 0u, (uint32_t)HQ_DEV_TIMEOUT_DRAIN); break; }
        }
      }
      for (uint32_t j = 0; j < issued; ++j) {
        const uint32_t k = it - 1 - j;
        const uint32_t ds = k % p.stages, dph = (k / p.stages) & 1u;
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&ctl.full[ds]), dph)) {
          if (global_ns() - t0 > kWaitBudgetNs) { atomicCAS(p.status, 0u, (uint32_t)HQ_DEV_TIMEOUT_DRAIN); break; }
        }
      }
      if (p.wres) {
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(smem_u32(&ctl.wfull), 0)) {
          if (global_ns() - t0 > kWaitBudgetNs) { atomicCAS(p.status, 0u, (uint32_t)HQ_DEV_TIMEOUT_DRAIN); break; }
        }
      }
      if (p.staged_res) {
        const uint32_t tiles_done = tcount < rmask + 1u ? tcount : rmask + 1u;
        for (uint32_t j = 0; j < tiles_done; ++j) {
          const uint32_t k = tcount - 1 - j;
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(smem_u32(&ctl.rfull[k & rmask]), (k >> p.lg_rbufs) & 1u)) {
            if (global_ns() - t0 > kWaitBudgetNs) { atomicCAS(p.status, 0u, (uint32_t)HQ_DEV_TIMEOUT_DRAIN); break; }
          }
        }
      }
    }
  } else if (warp <= MMA_WARPS) {
    // ------------------------------------------------------------ MMA issuers
    // The K blocks of the CTA's tiles, numbered through (g = tile * k_blocks + b), are dealt round-robin to p.ni
    // issuer warps (one lane each).  A single thread cannot keep the tensor pipe busy: every shared-memory
    // operation it executes between two batches of MMAs (the wait for the next operands) holds it for a few hundred
    // cycles while its own MMAs are in flight, and the pipe drains meanwhile; with the waits of one issuer falling
    // into the MMAs of the others the pipe stays fed.  The stage count is a multiple of p.ni, so a stage is always
    // read by the same issuer: its parity waits then follow one another like a single thread's (a thread that
    // looked at a stage's barrier a whole fill early would take the fill before for its own).  Integer accumulation
    // does not care about the order of the blocks; only the tile's first MMA, which overwrites the accumulator,
    // must come first: whoever issues it signals `tstart` and the others wait for that.
    const int iss = warp - 1;
    if (iss < p.ni && rank == 0 && elect_one()) {
      // instruction descriptor: D = S32, A = s8 weights, B = u8/s8 activations, both K-major, N = pt,
      // M = 128 (256 over the two CTAs of a pair)
      const uint32_t idesc = (2u << 4) | (1u << 7) | ((uint32_t)(p.x_signed ? 1 : 0) << 10) |
                             ((uint32_t)(p.pt >> 3) << 17) | ((uint32_t)((kTileC << p.duo) >> 4) << 24);
      // completion of the MMAs issued so far, signalled on a barrier of this CTA -- and of its partner in a pair
      auto commit = [&](uint32_t bar) {
        if constexpr (DUO) { mma_commit_2cta(in_cta(bar, 0)); mma_commit_2cta(in_cta(bar, 1)); }
        else mma_commit(bar);
      };
      const uint32_t ni = (uint32_t)p.ni, nstages = (uint32_t)p.stages;
      const bool ring = !(p.strip && p.wres);                 // do the blocks travel through the stage ring?
      uint32_t tcount = 0, s = 0, ph = 0;
      auto advance = [&](uint32_t d) { s += d; while (s >= nstages) { s -= nstages; ph ^= 1u; } };
      if (ring) advance((uint32_t)iss);
      int b = iss;                                           // my next block of the current tile
      const uint32_t bmask = (1u << p.lg_bufs) - 1u;
      bool ok = true;
      const uint64_t desc_hi = smem_desc(0, p.bkb);           // everything but the start address
      const int ksteps = p.bkb >> 5;
      if (p.wres && !mbar_wait(smem_u32(&ctl.wfull), 0, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) ok = false;
      // One issuer, plain form: the lean loop (the hand-over chain of short reductions is latency bound, every
      // instruction on it counts).
      const bool lean = ni == 1 && !p.strip;
      for (int p_tile = p_tile0; p_tile < p.p_tiles && ok && lean; p_tile += p_step, ++tcount) {
        const uint32_t as = tcount & bmask, aph = (tcount >> p.lg_bufs) & 1u;
        // The operands of the tile's first K block have usually landed long ago; looking at them first
        // keeps that check off the path between the epilogue's hand-back and the first MMA.
        if (!mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
        if (!mbar_wait(smem_u32(&ctl.tempty[as]), aph ^ 1u, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * p.acc_stride;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (kb > 0 && !mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
          const uint32_t w_addr = tiles + s * stage_bytes;
          const uint32_t a_addr = p.wres ? tiles + p.wres_off + (uint32_t)kb * w_bytes : w_addr;
          uint64_t adesc = desc_hi | (uint64_t)((a_addr >> 4) & 0x3FFF);
          uint64_t bdesc = desc_hi | (uint64_t)(((w_addr + x_off) >> 4) & 0x3FFF);
          if constexpr (DUO) {
            for (int k = 0; k < ksteps; ++k, adesc += 2, bdesc += 2)
              mma_i8_2cta(d_tmem, adesc, bdesc, idesc, (kb | k) ? 1u : 0u);
          } else {
            for (int k = 0; k < ksteps; ++k, adesc += 2, bdesc += 2)     // 32 bytes of K per instruction
              mma_i8(d_tmem, adesc, bdesc, idesc, (kb | k) ? 1u : 0u);
          }
          // the accumulator's barrier first on the last K block: the epilogue is the one waiting
          if (kb + 1 == p.k_blocks && !p.rtm) commit(smem_u32(&ctl.tfull[as]));
          commit(smem_u32(&ctl.empty[s]));         // frees the stage when these MMAs have read it
          if (++s == nstages) { s = 0; ph ^= 1u; }
        }
        if (p.rtm && ok) {
          // The residual tile through the tensor core: D2[ch][px] = sum_k I[ch][k] * R[px][k] = R[px][ch], INT32, in the
          // pt columns after the accumulator.  Four MMAs of 32 channels of K each; the accumulator barrier then stands
          // for both results, and for the tile in shared memory being free to be overwritten by the outputs.
          const uint32_t rs = tcount & ((1u << p.lg_rbufs) - 1u), rph = (tcount >> p.lg_rbufs) & 1u;
          if (!mbar_wait(smem_u32(&ctl.rfull[rs]), rph, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
          tc_fence_after();
          const uint64_t hi128 = smem_desc(0, 128);
          uint64_t adesc = hi128 | (uint64_t)(((tiles + p.ident_off) >> 4) & 0x3FFF);
          uint64_t bdesc = hi128 | (uint64_t)(((res_stage + rs * res_tile_bytes) >> 4) & 0x3FFF);
          const uint32_t idesc_r = (2u << 4) | (1u << 7) | ((uint32_t)(p.res_signed ? 1 : 0) << 10) |
                                   ((uint32_t)(p.pt >> 3) << 17) | ((uint32_t)(kTileC >> 4) << 24);
          for (int k = 0; k < 4; ++k, adesc += 2, bdesc += 2) mma_i8(d_tmem + p.pt, adesc, bdesc, idesc_r, k ? 1u : 0u);
          commit(smem_u32(&ctl.tfull[as]));
        }
      }
      for (int p_tile = p_tile0; p_tile < p.p_tiles && ok && !lean; p_tile += p_step, ++tcount) {
        const uint32_t as = tcount & bmask, aph = (tcount >> p.lg_bufs) & 1u;
        const uint32_t d_tmem = tmem_base + as * p.pt;
        bool first = true;
        int cur_chunk = -1;
        uint32_t ps = 0;
        for (; b < p.k_blocks; b += (int)ni) {
          uint32_t a_addr, b_addr;
          if (p.strip) {
            // block b = (cin chunk, filter tap): the chunk's patch, read from (tr << lg_wp) + ts rows further on.
            // The start is then not aligned to the swizzle pattern's eight rows, which needs nothing more: the
            // pattern is a function of the shared-memory address, for the copy that wrote the patch and for the
            // MMA that reads it alike (the descriptor's base-offset field stays 0; a phase there gives wrong sums).
            const int chunk = b / 9, tap = b - 9 * chunk, tr = tap / 3, ts = tap - 3 * tr;
            if (chunk != cur_chunk) {
              if (cur_chunk >= 0) mma_commit(smem_u32(&ctl.pempty[ps]));    // my MMAs on the previous patch
              cur_chunk = chunk;
              const uint32_t pidx = tcount * (uint32_t)p.cchunks + (uint32_t)chunk;
              ps = pidx % (uint32_t)p.npatch;
              if (!mbar_wait(smem_u32(&ctl.pfull[ps]), (pidx / (uint32_t)p.npatch) & 1u, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
            }
            b_addr = tiles + p.patch_off + ps * p.patch_bytes + (uint32_t)(((tr << p.lg_wp) + ts) * p.bkb);
            if (p.wres) {
              a_addr = tiles + p.wres_off + (uint32_t)(tap * p.cchunks + chunk) * w_bytes;
            } else {
              if (!mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
              a_addr = tiles + s * stage_bytes;
            }
          } else {
            if (!mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
            const uint32_t w_addr = tiles + s * stage_bytes;
            a_addr = p.wres ? tiles + p.wres_off + (uint32_t)b * w_bytes : w_addr;
            b_addr = w_addr + x_off;
          }
          if (first) {
            // The operands of this issuer's first block have usually landed long ago; looking at them first keeps
            // that check off the path between the epilogue's hand-back and the first MMA.
            if (!mbar_wait(smem_u32(&ctl.tempty[as]), aph ^ 1u, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
            if (b != 0 && !mbar_wait(smem_u32(&ctl.tstart[as]), aph, &ctl, p.status, HQ_DEV_TIMEOUT_MMA)) { ok = false; break; }
            tc_fence_after();
            first = false;
          }
          uint64_t adesc = desc_hi | (uint64_t)((a_addr >> 4) & 0x3FFF);
          uint64_t bdesc = desc_hi | (uint64_t)((b_addr >> 4) & 0x3FFF);
          for (int k = 0; k < ksteps; ++k, adesc += 2, bdesc += 2)     // 32 bytes of K per instruction
            mma_i8(d_tmem, adesc, bdesc, idesc, (b | k) ? 1u : 0u);
          if (b == 0 && ni > 1) mbar_arrive(smem_u32(&ctl.tstart[as]));   // the overwriting MMA is on its way
          // the accumulator's barrier first on this issuer's last block: the epilogue is the one waiting
          if (b + (int)ni >= p.k_blocks) mma_commit(smem_u32(&ctl.tfull[as]));
          if (ring) {
            mma_commit(smem_u32(&ctl.empty[s]));     // frees the stage when these MMAs have read it
            advance(ni);                             // my next block, in this tile or the next
          }
        }
        if (!ok) break;
        if (p.strip && cur_chunk >= 0) mma_commit(smem_u32(&ctl.pempty[ps]));
        b -= p.k_blocks;                             // the numbering runs on into the next tile
      }
      // Drain: all issued MMAs must have completed before tensor memory is freed.
      if constexpr (DUO) mma_commit_2cta(in_cta(smem_u32(&ctl.drain), 0)); else mma_commit(smem_u32(&ctl.drain));
      const unsigned long long t0 = global_ns();
      while (!mbar_try_wait(smem_u32(&ctl.drain), 0)) {
        if (global_ns() - t0 > kWaitBudgetNs) { atomicCAS(p.status, 0u, (uint32_t)HQ_DEV_TIMEOUT_DRAIN); break; }
      }
    }
  } else if (RTM && warp == 1 + MMA_WARPS + EPI_WARPS) {
    // ------------------------------------------------------------ store warp (rtm): finished tiles leave by TMA
    if (elect_one()) {
      const uint32_t rmask = (1u << p.lg_rbufs) - 1u;
      uint32_t tcount = 0;
      for (int p_tile = p_tile0; p_tile < p.p_tiles; p_tile += p_step, ++tcount) {
        const uint32_t rs = tcount & rmask, rph = (tcount >> p.lg_rbufs) & 1u;
        if (!mbar_wait(smem_u32(&ctl.ofull[rs]), rph, &ctl, p.status, HQ_DEV_TIMEOUT_EPILOGUE)) break;
        tma_store_2d(&map_out, res_stage + rs * res_tile_bytes, c_tile * kTileC, tile_at(p, p_tile) * p.pt);
        tma_store_commit();
        if (rmask < 3u) {
          // only two tile buffers: hand this one back as soon as the store has read it
          tma_store_wait_read0();
          mbar_arrive(smem_u32(&ctl.rempty[rs]));
        } else if (tcount > 0) {
          // the store before this one has read its tile by now: that buffer may be loaded again
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          mbar_arrive(smem_u32(&ctl.rempty[(tcount - 1u) & rmask]));
        }
      }
      tma_store_wait_all();
    }
  } else {
    // ------------------------------------------------------------ epilogue (the last EPI_WARPS warps)
    const int q = warp & 3;                       // the TMEM lane quarter this warp may read: channels 32q..32q+31
    const int ew = warp - (1 + MMA_WARPS);        // 0..7
    const int half = ew >> 2;                     // which half of its lane quarter's pixel columns this warp owns
    // Channel tiles of at most 64 channels are folded: the weight rows are loaded twice, so accumulator
    // lanes 64-127 repeat lanes 0-63, and lane quarters 2-3 take the second half of the pixel columns
    // of channels 0-63 instead of idling on channels that do not exist.
    const int cq = p.fold ? (q & 1) : q;          // which 32 channels of the tile
    const int slices = p.halves << p.fold;        // pixel-column slices per channel quarter
    const int px_per_warp = p.pt / slices;        // 128 or 64 pixel columns
    const int col0 = ((p.fold ? (q >> 1) * p.halves : 0) + half) * px_per_warp;
    const int ch = c_tile * kTileC + cq * 32 + lane;         // this thread's output channel
    const bool ch_live = ch < p.C;
    const bool warp_live = (c_tile * kTileC + cq * 32) < p.C; // warp-uniform
    const int lo = p.relu ? (p.qmin > 0 ? p.qmin : 0) : p.qmin, hi = p.qmax;

    // per-channel constants, once per kernel
    ChanConst k{};
    uint32_t fast = (p.out_bits != 32) ? 1u : 0u;
    k.bias = (ch_live && p.bias) ? p.bias[ch] : 0;
    if (p.out_bits != 32) {
      k.b = ch_live ? p.b[ch] : 0;
      const int cc = ch_live ? p.c[ch] : 32;
      k.sh = cc;
      k.r0 = (long long)k.bias * (long long)k.b + (1LL << (cc - 1));
      if (p.res) {
        const int rcc = ch_live ? p.rc[ch] : 32;
        if (rcc < 9 || p.res_bits != 8) fast = 0;
        k.rb = ch_live ? p.rb[ch] : 0;
        k.rsh = rcc;
        k.rr0 = 1LL << (rcc - 1);
      }
    }
    fast = epi_bar_and<32 * EPI_WARPS>(fast);                    // every live channel of the CTA allows 32-bit intermediates
    const bool warp_small = __any_sync(0xffffffffu, k.sh < 32) != 0;     // some channel of this warp has c < 32
    // ... and for each of them accumulator and bias stay below 2^(c-2): the pre-shift form of requant_fast is exact
    // and its result below 2^30 in magnitude, so that the residual term still adds without overflow
    const int babs = k.bias < 0 ? ~k.bias : k.bias;
    const bool warp_pre = warp_small &&
        __all_sync(0xffffffffu, k.sh >= 32 || (k.sh - 2 >= p.acc_bits && k.sh >= 3 && babs < (1 << (k.sh - 2)))) != 0;
    if (fast) {
      k.sh1 = k.sh < 32 ? k.sh : 32;
      k.cmin31 = k.sh < 31 ? k.sh : 31;
      k.sh -= k.sh1;
      k.pre = 32 - k.sh1;                        // (r0 is shifted by the loops that use the pre-shift form)
      if (p.res) {
        if (k.rsh >= 40) { k.rb = 0; k.rh = 0; k.rsh = 1; }            // |r*rb| < 2^39: rounds to 0
        else { k.rh = 1 << (k.rsh - 9); k.rsh -= 8; }
      }
    }
    // narrow residual pairs, when the caller prepared them and every channel of this warp has one
    bool warp_narrow = false;
    if (fast && (!warp_small || warp_pre) && p.res && p.res_narrow) {
      if (p.narrow_fresh) asm volatile("griddepcontrol.wait;" ::: "memory");
      const int4 nr = ch_live ? p.res_narrow[ch] : make_int4(0, 0, 0, 1);
      warp_narrow = __all_sync(0xffffffffu, nr.w != 0) != 0;
      if (warp_narrow) { k.rb = nr.x; k.rh = nr.y; k.rsh = nr.z; }
    }

    if (p.res && !p.staged_res) asm volatile("griddepcontrol.wait;" ::: "memory");   // direct residual loads below
    EpiCtx e;
    e.p = &p; e.ctl = &ctl; e.map_out = &map_out; e.smem_raw = smem_raw; e.raw = raw; e.out_stage = out_stage;
    e.res_stage = res_stage; e.res_tile_bytes = res_tile_bytes; e.tmem_base = tmem_base;
    e.warp = warp; e.lane = lane; e.q = q; e.cq = cq; e.ew = ew; e.half = half; e.col0 = col0; e.px_per_warp = px_per_warp; e.ch = ch;
    e.c_tile = c_tile; e.p_tile0 = p_tile0; e.p_step = p_step; e.lo = lo; e.hi = hi;
    e.ch_live = ch_live; e.warp_live = warp_live;
    if (p.rtm) {
      if constexpr (RTM) {
        // residual through tensor memory: the fragment loop, in its general form when some channel needs 64-bit steps
        const bool rn = warp_narrow;
        if (!fast) {
          if (p.out_signed) epilogue_loop_frag<true, false, false, true, false>(e); else epilogue_loop_frag<true, false, false, false, false>(e);
        } else if (warp_small) {
          // (narrow residual pairs only with the pre-shift form; the funnel-shift form keeps the plain multiply-high term)
#define HQ_FRAG_SMALL(RS, S, OS) do { if (warp_pre && rn) epilogue_loop_frag<false, false, S, OS, true, 2>(e); \
                                      else if (warp_pre) epilogue_loop_frag<false, RS, S, OS, false, 2>(e); \
                                      else epilogue_loop_frag<false, RS, S, OS, false, 1>(e); } while (0)
          if (p.sat_pack) {
            if (p.out_signed) { if (p.res_signed) HQ_FRAG_SMALL(true, true, true); else HQ_FRAG_SMALL(false, true, true); }
            else { if (p.res_signed) HQ_FRAG_SMALL(true, true, false); else HQ_FRAG_SMALL(false, true, false); }
          } else {
            if (p.out_signed) { if (p.res_signed) HQ_FRAG_SMALL(true, false, true); else HQ_FRAG_SMALL(false, false, true); }
            else { if (p.res_signed) HQ_FRAG_SMALL(true, false, false); else HQ_FRAG_SMALL(false, false, false); }
          }
#undef HQ_FRAG_SMALL
        } else if (p.sat_pack) {
          if (p.out_signed) { if (rn) epilogue_loop_frag<false, false, true, true, true>(e); else if (p.res_signed) epilogue_loop_frag<false, true, true, true, false>(e); else epilogue_loop_frag<false, false, true, true, false>(e); }
          else { if (rn) epilogue_loop_frag<false, false, true, false, true>(e); else if (p.res_signed) epilogue_loop_frag<false, true, true, false, false>(e); else epilogue_loop_frag<false, false, true, false, false>(e); }
        } else {
          if (p.out_signed) { if (rn) epilogue_loop_frag<false, false, false, true, true>(e); else if (p.res_signed) epilogue_loop_frag<false, true, false, true, false>(e); else epilogue_loop_frag<false, false, false, true, false>(e); }
          else { if (rn) epilogue_loop_frag<false, false, false, false, true>(e); else if (p.res_signed) epilogue_loop_frag<false, true, false, false, false>(e); else epilogue_loop_frag<false, false, false, false, false>(e); }
        }
      }
    } else if (half >= p.halves) {
      // the 64-pixel tile has one 64-column slice per lane quarter: this warp only took part in the vote above
    } else if (fast && p.staged_out && p.out_bits == 4 && !p.res && !p.strip && lo >= 0 && hi <= 15) {
      // unsigned 4-bit outputs without a residual (the convs inside a 4-bit block)
      if (warp_pre) epilogue_loop_fast8<false, false, false, false, 2, false, true>(e, k);
      else if (warp_small) epilogue_loop_fast8<false, false, false, false, 1, false, true>(e, k);
      else epilogue_loop_fast8<false, false, false, false, 0, false, true>(e, k);
    } else if (fast && p.staged_out && p.out_bits == 8 && (!p.res || p.staged_res)) {
      const int variant = (p.res ? 4 : 0) | ((p.res && p.res_signed) ? 2 : 0) | (p.sat_pack ? 1 : 0);
      switch (variant) {
#define HQ_FAST8(R, RS, S, OS) do { if (RTM) { \
                                    } else if (warp_pre && R && warp_narrow) epilogue_loop_fast8<R, RS, S, OS, 2, R>(e, k); \
                                    else if (warp_pre) epilogue_loop_fast8<R, RS, S, OS, 2, false>(e, k); \
                                    else if (warp_small) epilogue_loop_fast8<R, RS, S, OS, 1, false>(e, k); \
                                    else if (R && warp_narrow) epilogue_loop_fast8<R, RS, S, OS, 0, R>(e, k); \
                                    else epilogue_loop_fast8<R, RS, S, OS, 0, false>(e, k); } while (0)
        case 0: HQ_FAST8(false, false, false, false); break;
        case 1: if (p.out_signed) HQ_FAST8(false, false, true, true); else HQ_FAST8(false, false, true, false); break;
        case 4: HQ_FAST8(true, false, false, false); break;
        case 5: if (p.out_signed) HQ_FAST8(true, false, true, true); else HQ_FAST8(true, false, true, false); break;
        case 6: HQ_FAST8(true, true, false, false); break;
        default: if (p.out_signed) HQ_FAST8(true, true, true, true); else HQ_FAST8(true, true, true, false); break;
#undef HQ_FAST8
      }
    } else {
      epilogue_loop_general(e, k, fast);
    }
  }


  tc_fence_before();
  __syncthreads();
  // A pair leaves together: the leading CTA has seen its MMAs complete (they read the partner's shared memory and
  // signal its barriers), the partner has sent its last remote arrival.
  if constexpr (DUO) cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if constexpr (DUO) tmem_dealloc2(tmem_base, p.tmem_cols); else tmem_dealloc(tmem_base, p.tmem_cols);
  }
}

// ---------------------------------------------------------------- narrow residual pairs ------
// The residual term dn(r, rb, rc) = (r*rb + 2^(rc-1)) >> rc (Section 3.3, Appendix G) has only 256 possible
// inputs per channel.  For most (rb, rc) a 23-bit multiplier m ~ rb / 2^8 with s = rc - 8 and a = 2^(s-1)
// gives (r*m + a) >> s == dn(r, rb, rc) for every one of them, and r*m + a fits 32 bits.  One warp per
// channel tries the two neighbouring multipliers and checks all 256 inputs; channels without such a pair
// are marked invalid and keep the wide form.  Run once per layer when a network is built, and ahead of a
// single large element-wise call.
struct NarrowJob { const int32_t* rb; const int32_t* rc; int is_signed; int4* out; };

__global__ void __launch_bounds__(128) residual_narrow_kernel(NarrowJob j0, NarrowJob j1, int n) {
  // one warp per channel: lane l checks the inputs l, l + 32, ... for both candidate multipliers; warps past the
  // first n channels serve the second job (the other operand of an element-wise call), if there is one
  int ch = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const bool second = ch >= n;
  if (second) ch -= n;
  const NarrowJob& j = second ? j1 : j0;
  if (ch >= n || !j.out) return;
  const long long b = j.rb[ch];
  const int c = j.rc[ch];
  int4 res = make_int4(0, 0, 0, 0);
  const int r_lo = j.is_signed ? -128 : 0;
  if (c >= 41 && c <= 62) {
    res = make_int4(0, 0, 0, 1);                       // |r*rb| < 2^39 <= 2^(rc-2): the term is 0 for every r
  } else if (c >= 9 && c <= 38) {
    const int s = c - 8, a = 1 << (s - 1);
    const long long m0 = b >> 8, m1 = m0 + 1;
    bool same0 = m0 <= (1 << 23), same1 = m1 <= (1 << 23);
    for (int k = 0; k < 8; ++k) {
      const int r = r_lo + lane + 32 * k;
      const long long exact = ((long long)r * b + (1LL << (c - 1))) >> c;
      same0 = same0 && exact == (long long)((r * (int)m0 + a) >> s);
      same1 = same1 && exact == (long long)((r * (int)m1 + a) >> s);
    }
    same0 = __all_sync(0xffffffffu, same0);
    same1 = __all_sync(0xffffffffu, same1);
    if (same0) res = make_int4((int)m0, a, s, 1);
    else if (same1) res = make_int4((int)m1, a, s, 1);
  }
  if (lane == 0) j.out[ch] = res;
}

// ---------------------------------------------------------------- host side ------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;

bool load_driver_entry_points() {
  if (g_encode_tiled && g_encode_im2col) return true;
  cudaDriverEntryPointQueryResult qr;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess ||
      qr != cudaDriverEntryPointSuccess || !fn)
    return false;
  g_encode_tiled = (EncodeTiledFn)fn;
  fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &qr) != cudaSuccess ||
      qr != cudaDriverEntryPointSuccess || !fn)
    return false;
  g_encode_im2col = (EncodeIm2colFn)fn;
  return true;
}

CUtensorMapSwizzle swizzle_for(int row_bytes) {
  return row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
       : row_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
}

// 2-D byte map over a dense [rows][row_bytes] tensor with a box of `ib` bytes x `box_rows` rows.
bool encode_rows_map(CUtensorMap* map, const void* base, long long rows, long long row_bytes, int ib, int box_rows,
                     CUtensorMapSwizzle swz) {
  const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)ib, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Pixel tile: the largest of 256 / 128 / 64 that still gives every SM work, at most `cap`.
int pick_pt(long long pixels, int c_tiles, int sm_count, int cap) {
  const int cands[3] = {256, 128, 64};
  for (int i = 0; i < 3; ++i) {
    const int pt = cands[i];
    if (pt > cap) continue;
    const long long tiles = (pixels + pt - 1) / pt * c_tiles;
    if (tiles >= 2LL * sm_count || pt == 64) return pt;
  }
  return 64;
}

}  // namespace

// One-time set-up that must not happen inside a stream capture: driver entry points for the
// tensor-map encoders and the kernel's dynamic shared-memory limit.
bool hq_conv_tc_init() {
  if (!load_driver_entry_points()) return false;
  return cudaFuncSetAttribute(conv_tc_kernel<kSoloEpilogueWarps, 1, kSoloIssuerWarps>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmemAttr) == cudaSuccess &&
         cudaFuncSetAttribute(conv_tc_kernel<kPairEpilogueWarps, 2, kPairIssuerWarps>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              112 * 1024) == cudaSuccess &&
         cudaFuncSetAttribute(conv_tc_kernel<8, 1, 1, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemAttr) == cudaSuccess &&
         cudaFuncSetAttribute(conv_tc_kernel<kSoloEpilogueWarps, 1, 1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmemAttr) == cudaSuccess;
}

bool hq_conv_tc_supported(const ConvArgs& a) {
  if (a.in_bits != 8) return false;
  if (a.cin % 32 != 0) return false;
  if (a.kh > 255 || a.kw > 255 || a.pad > 127 || a.stride > 8) return false;
  if ((long long)a.n * a.ho * a.wo >= (1ll << 31) - 256) return false;
  if ((long long)a.kh * a.kw * a.cin >= (1ll << 24)) return false;
  if (a.out_bits == 4 && (a.cout & 1)) return false;
  if (a.res && !(a.res_bits == 8 || a.res_bits == 32)) return false;
  // the corners of an im2col-mode tensor map are 8-bit signed offsets: wider filters are declined here, before any
  // map is encoded (more channel tiles than the GPU has SMs are declined by the launcher, which knows the count)
  const int pad_after = a.pad + a.pad_after_delta;
  if (pad_after - (a.kw - 1) < -128 || pad_after - (a.kh - 1) < -128 || pad_after > 127) return false;
  return true;
}

// im2col-mode tensor maps over activation tensors smaller than 128 KiB returned wrong tiles on the driver this
// library was brought up on (the map encoder marks such tensors in a field of the opaque descriptor).  Instead of
// editing the descriptor, layers that would need such a map are not run by the direct kernel at all: they take the
// patch-matrix form (lowering.cu), whose 1x1 convolution uses a plain tiled map.  Only small-batch, late-stage
// layers are affected (every im2col layer of the benchmark configurations is far larger).
bool hq_conv_tc_small_im2col(const ConvArgs& a) {
  const bool tiled = !a.pitch_w && a.kh == 1 && a.kw == 1 && a.stride == 1 && a.pad == 0;
  if (tiled) return false;
  const long long span = a.pitch_n ? (long long)a.n * a.pitch_n : (long long)a.n * a.h * a.w * a.cin;
  return span < kIm2colMinTensorBytes;
}

hq_status hq_launch_conv_tc(hq_handle* h, const ConvArgs& a, cudaStream_t stream) {
  if (!hq_conv_tc_supported(a)) return HQ_ERR_UNSUPPORTED;
  if (!load_driver_entry_points()) return HQ_ERR_CUDA;
  const long long P = (long long)a.n * a.ho * a.wo;
  if (P == 0) return HQ_OK;

  TcParams p{};
  p.rev = h->tile_order ? 1 : 0;
  p.P = (int32_t)P; p.C = a.cout; p.howo = a.ho * a.wo; p.wo = a.wo;
  p.stride = a.stride; p.pad = a.pad; p.kw = a.kw;
  p.bkb = (a.cin % 128 == 0) ? 128 : (a.cin % 64 == 0) ? 64 : 32;
  p.cchunks = a.cin / p.bkb;
  p.k_blocks = a.kh * a.kw * p.cchunks;
  p.c_tiles = (a.cout + kTileC - 1) / kTileC;
  if (p.c_tiles > h->sm_count) return HQ_ERR_UNSUPPORTED;
  // outputs and 8-bit residuals whose rows are 16-byte multiples travel through TMA
  const long long out_row_bytes = (long long)a.cout * a.out_bits / 8;
  p.staged_out = (a.out_bits != 32 && out_row_bytes % 16 == 0) ? 1 : 0;
  p.staged_res = (p.staged_out && a.res && a.res_bits == 8 && a.cout % 16 == 0) ? 1 : 0;
  // Launch shape: pair (two CTAs per SM) for short reductions when the tile pipeline fits half an SM.
  const long long k_total = (long long)a.kh * a.kw * a.cin;
  // (measured: with the weight slab resident the one-CTA shape catches up for K >= 128; the pair shape still
  // wins on the fused-residual expansions with the shortest reduction, and loses where a tile carries little
  // epilogue work, e.g. 64 output channels.  Where the layer is large enough for 256-pixel tiles and its residual
  // travels by TMA, the rtm shape below is faster still: 64 -> 256 at 56x56, batch 256: 129 -> 122 us.)
  const bool wide_fits = p.staged_res && a.out_bits == 8 && a.cout > 64 && pick_pt(P, p.c_tiles, h->sm_count, 256) == 256;
  bool pair = k_total <= 64 && a.res != nullptr && a.res_bits == 8 && a.cout >= 128 && !wide_fits;
  int stages = 0, stage_bytes = 0, res_tile_bytes = 0, out_tile_bytes = 0, wres_bytes = 0;
  if (pair) {
    // 128-pixel tiles, two accumulator buffers (256 columns), K blocks of at most 64 bytes
    if (p.bkb > 64) { p.bkb = 64; p.cchunks = a.cin / p.bkb; p.k_blocks = a.kh * a.kw * p.cchunks; }
    p.pt = pick_pt(P, p.c_tiles, 2 * h->sm_count, 128);
    wres_bytes = p.k_blocks * kTileC * p.bkb;
    p.wres = wres_bytes <= 16 * 1024 ? 1 : 0;              // short reductions: the weight slab stays resident
    if (!p.wres) wres_bytes = 0;
    stage_bytes = ((p.wres ? 0 : kTileC) + p.pt) * p.bkb;
    p.fold = (a.cout <= 64 && p.pt >= 128) ? 1 : 0;
    p.halves = 1;
    p.lg_bufs = 1;
    p.lg_rbufs = 1;
    out_tile_bytes = p.staged_out ? kPairEpilogueWarps * p.pt * 32 : 0;
    res_tile_bytes = p.staged_res ? p.pt * kTileC : 0;
    stages = (110 * 1024 - out_tile_bytes - 2 * res_tile_bytes - wres_bytes) / stage_bytes;
    if (stages < 3 || p.pt < 128) pair = false;
  }
  if (!pair) {
    p.bkb = (a.cin % 128 == 0) ? 128 : (a.cin % 64 == 0) ? 64 : 32;
    p.cchunks = a.cin / p.bkb;
    p.k_blocks = a.kh * a.kw * p.cchunks;
    const int smem_budget = kSmemBudget;                // dynamic bytes after the 1024-byte alignment slack
    // staging: 8 warps x pt/2 pixel rows x 32 bytes (reserved at the 8-bit size), residual 2 or 4 x [pt][128]
    bool chosen = false;
    for (int cap = 256; cap >= 64 && !chosen; cap >>= 1) {   // largest pixel tile that leaves room for >= 3 stages
      p.pt = pick_pt(P, p.c_tiles, h->sm_count, cap);
      // A weight slab of at most 72 KiB stays resident (the stages then hold activations only): a third less
      // traffic into shared memory per K block.  Where the slab would cost the larger pixel tile its stages, the
      // tile wins and the weights travel with the stages.
      for (int keep_w = 1; keep_w >= 0 && !chosen; --keep_w) {
        wres_bytes = p.k_blocks * kTileC * p.bkb;
        p.wres = (keep_w && wres_bytes <= 72 * 1024) ? 1 : 0;
        if (!p.wres) { if (keep_w) continue; wres_bytes = 0; }
        stage_bytes = ((p.wres ? 0 : kTileC) + p.pt) * p.bkb;
        p.fold = (a.cout <= 64 && p.pt >= 128) ? 1 : 0;
        p.halves = p.pt >= (p.fold ? 256 : 128) ? 2 : 1;
        out_tile_bytes = p.staged_out ? 4 * p.pt * 32 : 0;
        p.lg_bufs = p.pt <= 128 ? 2 : 1;
        res_tile_bytes = p.staged_res ? p.pt * kTileC : 0;
        // residual tiles: as many buffers as accumulators, fewer when a long reduction needs the room for stages
        // (its epilogue has slack: a single residual buffer only delays the next tile's prefetch)
        // The rtm shape (below) works in place in the residual tiles and needs no staging box; with the
        // weights resident two stages are enough for its short reductions (the epilogue bounds the tile).
        const bool wide_here = p.pt == 256 && !p.fold && p.staged_out && a.out_bits == 8 && p.staged_res && k_total < 1024;
        if (wide_here) out_tile_bytes = 0;
        const int min_stages = (wide_here && p.wres) ? 2 : 3;
        for (p.lg_rbufs = p.lg_bufs; ; --p.lg_rbufs) {
          stages = (smem_budget - out_tile_bytes - (res_tile_bytes << p.lg_rbufs) - wres_bytes) / stage_bytes;
          if (stages >= min_stages || p.lg_rbufs == 0 || !res_tile_bytes || k_total < 1024) break;
        }
        if (stages >= min_stages || (p.pt == 64 && keep_w == 0)) chosen = true;
      }
    }
  }
  p.p_tiles = (int32_t)((P + p.pt - 1) / p.pt);
  // Strip mode for 3x3 / stride 1 / pad 1: one padded input patch per cin chunk serves all nine taps (a tap is a
  // row offset into the patch), so the activations enter shared memory once instead of nine times.  The tile is
  // 256 positions of a raster whose pitch is the next power of two above the padded width; worth it while at
  // least three quarters of a pitch are real columns.
  size_t patch_total = 0;
  {
    int lg_wp = 0;
    if (a.w >= 11 && a.w <= 14) lg_wp = 4; else if (a.w >= 23 && a.w <= 30) lg_wp = 5; else if (a.w >= 47 && a.w <= 62) lg_wp = 6;
    const bool shape_ok = !pair && lg_wp && a.kh == 3 && a.kw == 3 && a.stride == 1 && a.pad == 1 && !a.pitch_w && !a.res &&
                          p.staged_out && a.out_bits == 8 && a.cin % 64 == 0 && a.n < 65536;
    if (shape_ok) {
      const int bkb = a.cin % 128 == 0 ? 128 : 64;
      const int cchunks = a.cin / bkb, rows = 256 >> lg_wp, tpi = (a.h + rows - 1) / rows;
      const long long tiles_all = (long long)a.n * tpi * p.c_tiles;
      const size_t patch = (size_t)(rows + 3) * (1u << lg_wp) * bkb, wb = (size_t)kTileC * bkb;
      const size_t slab = (size_t)9 * cchunks * wb;
      const bool keep_w = slab <= 72 * 1024;
      const size_t room = (size_t)kSmemBudget - 32 * 1024 - (keep_w ? slab : 0);
      int npatch = 0, wstages = 0;
      if (keep_w) { npatch = (int)(room / patch); if (npatch > 3) npatch = 3; }
      else if (room >= 2 * patch + 3 * wb) { npatch = 2; wstages = (int)((room - 2 * patch) / wb); }
      // measured: with the weights streaming through the stage ring the strip form is no faster than the plain
      // one (both are bound by what the SM can take in per cycle), so it is used where the weights stay resident
      if (((tiles_all >= 2LL * h->sm_count && keep_w) || h->conv_path == 3) && npatch >= 2) {
        p.strip = 1; p.lg_wp = lg_wp; p.rows = rows; p.tpi = tpi; p.ho = a.h; p.npatch = npatch;
        p.patch_bytes = (uint32_t)patch;
        p.bkb = bkb; p.cchunks = cchunks; p.k_blocks = 9 * cchunks;
        p.pt = 256; p.lg_bufs = 1; p.lg_rbufs = 1; p.halves = 2;
        p.fold = a.cout <= 64 ? 1 : 0;
        p.wres = keep_w ? 1 : 0;
        wres_bytes = keep_w ? (int)slab : 0;
        stage_bytes = keep_w ? 0 : (int)wb;
        stages = keep_w ? 0 : (wstages > kMaxStages ? kMaxStages : wstages);
        out_tile_bytes = 4 * 256 * 32;
        res_tile_bytes = 0;
        p.p_tiles = a.n * tpi;
        patch_total = (size_t)npatch * patch;
      }
    }
  }
  // The direct kernel fetches activations through an im2col-mode map unless the layer is 1x1 / stride 1 / unpadded
  // (tiled map) or takes the strip form (tiled map over padded patches).  That mode is not used on tensors below
  // 128 KiB (hq_conv_tc_small_im2col); such a layer is declined here and runs in its lowered form.
  if (!p.strip && hq_conv_tc_small_im2col(a)) return HQ_ERR_UNSUPPORTED;
  p.x_signed = a.in_signed;
  bool wide = false;
  {
    // issuer warps in use: at most one per K block; where the blocks travel through the stage ring, the stage count
    // becomes a multiple of it (every stage then belongs to one issuer)
    // Measured: several issuers pay off where the operands are mostly in shared memory already (strip form,
    // resident weights); where every block waits for 48 KiB from L2 the tile is bound by that stream and the extra
    // issuers only cost a few percent.
    // Third launch shape, *rtm*, for the fused 8-bit residual with a short reduction on layers large enough for
    // 256-pixel tiles (here called `wide` for the condition it shares with the tile choice above): the residual tile
    // goes through the tensor core into tensor memory, see epilogue_loop_frag.  Measured against the shape it replaced
    // (sixteen warps, one channel per thread, one byte load and one byte store per value, in place in the residual tile):
    // 1x1 64 -> 256 at 56x56, batch 256, 125 -> 122 us; 128 -> 512 at 28x28 72 -> 70 us; no byte-wise shared-memory
    // traffic is left, the epilogue is bound by the integer instructions of Eq. 4 and the residual term themselves.
    wide = !pair && !p.strip && p.pt == 256 && !p.fold && p.staged_out && a.out_bits == 8 && p.staged_res && k_total < 1024;
    if (wide) {
      // 128-pixel tiles, two buffers of (accumulator + transposed residual) = 512 tensor-memory columns; the two
      // residual tiles double as the output boxes; the identity matrix takes 16 KiB
      p.rtm = 1; p.halves = 2;
      p.pt = 128; p.lg_bufs = 1; p.lg_rbufs = 1;
      p.p_tiles = (int32_t)((P + p.pt - 1) / p.pt);
      out_tile_bytes = 0;
      res_tile_bytes = p.pt * kTileC;
      wres_bytes = p.k_blocks * kTileC * p.bkb;
      p.wres = wres_bytes <= 72 * 1024 ? 1 : 0;
      if (!p.wres) wres_bytes = 0;
      stage_bytes = ((p.wres ? 0 : kTileC) + p.pt) * p.bkb;
      // four residual / output tiles when they leave room for three operand stages: a tile is held from its load to
      // the end of its store, and the loads of the next tiles must be in flight meanwhile to cover the memory latency
      for (p.lg_rbufs = 2; ; --p.lg_rbufs) {
        stages = (kSmemBudget - (res_tile_bytes << p.lg_rbufs) - wres_bytes - 16 * 1024) / stage_bytes;
        if (stages >= 3 || p.lg_rbufs == 1) break;
      }
    }
    // Fourth shape, *duo*: clusters of two CTAs on adjacent SMs share every MMA (cta_group::2, M = 256): each CTA
    // fetches its own 128 weight rows and HALF of the tile's pixel rows, 32 KiB per K block and SM instead of
    // 48 KiB for the same MMA time.  For the long reductions whose weights stream, which the operand fetch bounds.
    p.duo = (!pair && !wide && !p.strip && !p.wres && !p.fold && p.pt >= 128 && p.bkb == 128 && a.cout % 256 == 0 &&
             k_total >= 2048 && (long long)p.p_tiles * p.c_tiles >= 2LL * h->sm_count) ? 1 : 0;
    if (p.duo) {
      stage_bytes = (kTileC + p.pt / 2) * p.bkb;
      stages = (kSmemBudget - out_tile_bytes - (res_tile_bytes << p.lg_rbufs)) / stage_bytes;
    }
    const int issuers = pair ? kPairIssuerWarps : wide ? 1 : (p.strip || p.wres) ? kSoloIssuerWarps : 1;
    p.ni = p.k_blocks < issuers ? p.k_blocks : issuers;
    if (!(p.strip && p.wres)) {
      while (p.ni > 1 && stages < p.ni) --p.ni;
      if (stages > kMaxStages) stages = kMaxStages;
      // every stage counts more than the third issuer: the bytes in flight set the tile rate of the layers that wait
      // on memory latency (first layer: three 32 KiB stages 163 us, four with two issuers 143 us)
      while (p.ni > 1 && stages % p.ni) --p.ni;
      stages -= stages % p.ni;
    }
  }
  p.acc_stride = p.rtm ? 2 * p.pt : p.pt;
  { const long long bound = k_total * 255 * 128; int bits = 0; while ((1LL << bits) <= bound) ++bits; p.acc_bits = bits; }
  p.tmem_cols = (uint32_t)(p.acc_stride << p.lg_bufs);  // 512 columns, or 256 for the smallest tile
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2 && !p.strip) return HQ_ERR_UNSUPPORTED;
  p.stages = stages;
  p.out_stage_off = (uint32_t)(stages * stage_bytes);             // all pieces are multiples of 1024 bytes
  p.res_stage_off = p.out_stage_off + (uint32_t)out_tile_bytes;
  p.wres_off = p.res_stage_off + ((uint32_t)res_tile_bytes << p.lg_rbufs);
  p.patch_off = p.wres_off + (uint32_t)wres_bytes;
  p.ident_off = p.patch_off + (uint32_t)patch_total;
  p.bias = a.bias; p.b = a.b; p.c = a.c;
  p.res = a.res; p.res_bits = a.res_bits; p.res_signed = a.res_signed; p.rb = a.rb; p.rc = a.rc;
  p.res_narrow = (a.res && a.res_bits == 8) ? (const int4*)a.res_narrow : nullptr;
  p.narrow_fresh = a.res_narrow_fresh;
  p.relu = a.relu; p.qmin = a.qmin; p.qmax = a.qmax;
  p.out = a.out; p.out_bits = a.out_bits; p.out_signed = a.out_signed;
  {
    const int lo = a.relu ? (a.qmin > 0 ? a.qmin : 0) : a.qmin;
    p.sat_pack = (a.out_bits == 8 && ((!a.out_signed && lo == 0 && a.qmax == 255) ||
                                      (a.out_signed && lo == -128 && a.qmax == 127))) ? 1 : 0;
  }
  p.status = h->dev_status;

  const CUtensorMapSwizzle swz = swizzle_for(p.bkb);
  alignas(64) CUtensorMap map_x, map_w, map_out, map_res;
  p.x_tiled = (!a.pitch_w && a.kh == 1 && a.kw == 1 && a.stride == 1 && a.pad == 0) ? 1 : 0;
  if (p.strip) {
    // activations (C, W, H, N), box = one patch: bkb channels x pitch columns x (rows + 3) rows of one image
    const cuuint64_t dims[4] = {(cuuint64_t)a.cin, (cuuint64_t)a.w, (cuuint64_t)a.h, (cuuint64_t)a.n};
    const cuuint64_t strides[3] = {(cuuint64_t)a.cin, (cuuint64_t)a.cin * a.w, (cuuint64_t)a.cin * a.w * a.h};
    const cuuint32_t box[4] = {(cuuint32_t)p.bkb, 1u << p.lg_wp, (cuuint32_t)(p.rows + 3), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (g_encode_tiled(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(a.in), dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return HQ_ERR_CUDA;
    p.x_tiled = 0;
  } else if (p.x_tiled) {
    if (!encode_rows_map(&map_x, a.in, P, a.cin, p.bkb, p.pt >> p.duo, swz)) return HQ_ERR_CUDA;
  } else {
    // activations: (C, W, H, N) with byte strides; base pixels range over
    // [-pad, W + pad - (kw-1)) so that the hardware's pixel walk equals the output raster
    const cuuint64_t dims[4] = {(cuuint64_t)a.cin, (cuuint64_t)a.w, (cuuint64_t)a.h, (cuuint64_t)a.n};
    const cuuint64_t strides[3] = {(cuuint64_t)(a.pitch_w ? a.pitch_w : a.cin),
                                   (cuuint64_t)(a.pitch_h ? a.pitch_h : (long long)a.cin * a.w),
                                   (cuuint64_t)(a.pitch_n ? a.pitch_n : (long long)a.cin * a.w * a.h)};
    const int lower[2] = {-a.pad, -a.pad};
    const int pad_after = a.pad + a.pad_after_delta;
    const int upper[2] = {pad_after - (a.kw - 1), pad_after - (a.kh - 1)};
    const cuuint32_t estr[4] = {1, (cuuint32_t)a.stride, (cuuint32_t)a.stride, 1};
    const CUresult r = g_encode_im2col(&map_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(a.in), dims, strides,
                                       lower, upper, (cuuint32_t)p.bkb, (cuuint32_t)(p.pt >> p.duo), estr,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return HQ_ERR_CUDA;
  }
  if (!encode_rows_map(&map_w, a.wgt, a.cout, (long long)a.kh * a.kw * a.cin, p.bkb, p.fold ? 64 : kTileC, swz)) return HQ_ERR_CUDA;
  map_out = map_w; map_res = map_w;                    // valid placeholders when a path is not staged
  // (with rtm the residual tile is an MMA operand and, later, the output box: 128-byte swizzle both ways)
  const CUtensorMapSwizzle box_swz = p.rtm ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE;
  if (p.strip) {
    // output (C, W, H, N), box = 32 positions of the raster: 32 channels x min(pitch, 32) columns x the rows that makes
    const cuuint32_t bw = p.lg_wp >= 5 ? 32u : (1u << p.lg_wp);
    const cuuint64_t dims[4] = {(cuuint64_t)a.cout, (cuuint64_t)a.wo, (cuuint64_t)a.ho, (cuuint64_t)a.n};
    const cuuint64_t strides[3] = {(cuuint64_t)a.cout, (cuuint64_t)a.cout * a.wo, (cuuint64_t)a.cout * a.wo * a.ho};
    const cuuint32_t box[4] = {32, bw, 32u / bw, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (g_encode_tiled(&map_out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, a.out, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return HQ_ERR_CUDA;
  } else
  if (p.staged_out && !encode_rows_map(&map_out, a.out, P, out_row_bytes, p.rtm ? kTileC : a.out_bits == 4 ? 16 : 32, p.rtm ? p.pt : p.pt / (p.halves << p.fold),
                                       box_swz)) return HQ_ERR_CUDA;
  if (p.staged_res && !encode_rows_map(&map_res, a.res, P, a.cout, kTileC, p.pt, box_swz))
    return HQ_ERR_CUDA;

  const size_t dyn_smem = (size_t)stages * stage_bytes + out_tile_bytes + ((size_t)res_tile_bytes << p.lg_rbufs) + wres_bytes + patch_total +
                          (p.rtm ? 16 * 1024 : 0) + 1024;
  const long long total_tiles = (long long)p.p_tiles * p.c_tiles;
  // a multiple of c_tiles, so that every CTA keeps one channel tile
  const int slots = pair ? 2 * h->sm_count : h->sm_count;
  const int grid = (int)(total_tiles <= slots ? total_tiles : (slots / p.c_tiles) * p.c_tiles);
  // Launched with programmatic stream serialization: the grid may begin (barrier set-up, tensor-memory
  // allocation) while the previous kernel drains; the kernel waits for it before reading any input.
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;          // duo: consecutive CTAs (channel tiles 2j, 2j+1) pair up
  attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid); cfg.stream = stream; cfg.attrs = attr; cfg.numAttrs = p.duo ? 2 : 1;
  cudaError_t err;
  if (p.duo) {
    cfg.blockDim = dim3(32 * (2 + kSoloEpilogueWarps)); cfg.dynamicSmemBytes = dyn_smem < 120 * 1024 ? 120 * 1024 : dyn_smem;
    err = cudaLaunchKernelEx(&cfg, conv_tc_kernel<kSoloEpilogueWarps, 1, 1, true>, map_x, map_w, map_out, map_res, p);
  } else if (wide) {
    cfg.blockDim = dim3(32 * 11); cfg.dynamicSmemBytes = dyn_smem < 120 * 1024 ? 120 * 1024 : dyn_smem;
    err = cudaLaunchKernelEx(&cfg, conv_tc_kernel<8, 1, 1, false, true>, map_x, map_w, map_out, map_res, p);
  } else if (pair) {
    cfg.blockDim = dim3(32 * (1 + kPairIssuerWarps + kPairEpilogueWarps)); cfg.dynamicSmemBytes = dyn_smem;
    err = cudaLaunchKernelEx(&cfg, conv_tc_kernel<kPairEpilogueWarps, 2, kPairIssuerWarps>, map_x, map_w, map_out, map_res, p);
  } else {
    // one CTA per SM (it may allocate all 512 tensor-memory columns): never request less than 120 KiB
    cfg.blockDim = dim3(32 * (1 + kSoloIssuerWarps + kSoloEpilogueWarps)); cfg.dynamicSmemBytes = dyn_smem < 120 * 1024 ? 120 * 1024 : dyn_smem;
    err = cudaLaunchKernelEx(&cfg, conv_tc_kernel<kSoloEpilogueWarps, 1, kSoloIssuerWarps>, map_x, map_w, map_out, map_res, p);
  }
  return err == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

cudaError_t hq_launch_residual_narrow(const int32_t* rb, const int32_t* rc, int res_signed, int channels, void* out,
                                      cudaStream_t s) {
  return hq_launch_residual_narrow2(rb, rc, res_signed, out, nullptr, nullptr, 0, nullptr, channels, s);
}

cudaError_t hq_launch_residual_narrow2(const int32_t* b0, const int32_t* c0, int signed0, void* out0,
                                       const int32_t* b1, const int32_t* c1, int signed1, void* out1, int channels,
                                       cudaStream_t s) {
  if (channels <= 0) return cudaSuccess;
  const NarrowJob j0{b0, c0, signed0, (int4*)out0}, j1{b1, c1, signed1, (int4*)out1};
  const int warps = out1 ? 2 * channels : channels;
  residual_narrow_kernel<<<(warps + 3) / 4, 128, 0, s>>>(j0, j1, channels);
  return cudaGetLastError();
}

namespace {
// The wait of the kernels above in miniature: poll an mbarrier, give up after the budget, say so in the status word.
__global__ void expire_wait_kernel(uint32_t* status, unsigned long long budget_ns) {
  __shared__ unsigned long long bar;
  mbar_init(smem_u32(&bar), 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  const unsigned long long t0 = global_ns();
  while (!mbar_try_wait(smem_u32(&bar), 0)) {
    if (global_ns() - t0 > budget_ns) { atomicCAS(status, 0u, (uint32_t)HQ_DEV_TIMEOUT_EPILOGUE); break; }
  }
}
}  // namespace

cudaError_t hq_launch_expire_wait(uint32_t* status, int budget_ms, cudaStream_t s) {
  expire_wait_kernel<<<1, 1, 0, s>>>(status, (unsigned long long)budget_ms * 1000000ull);
  return cudaGetLastError();
}
