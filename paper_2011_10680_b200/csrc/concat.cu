// Inception-style concatenation with a dyadic rescale per branch (Appendix E, "Concatenation Layer"):
//   q_a[n, h, w, off_i + k] = clamp(dn(q_i[n, h, w, k], b_i[k], c_i[k])),   dn(q, b, c) = (q*b + 2^(c-1)) >> c,
// i.e. every branch (the convolution branches as stored 8- or 4-bit tensors or INT32 accumulators, the pooling
// branch as an INT32 tensor) is brought to the output scale by its own DN pairs and lands beside the others along
// the channel axis.  Memory bound: every operand is read once, the output written once, in ONE launch for all
// branches whose channel count is a multiple of 4 (ragged ones take a second launch in a sixteen-channel form).
// The blocks of the launch are dealt to the branches in proportion to their bytes, so a warp works on one branch
// only.  A thread owns four channels of a branch for the whole kernel -- 16 bytes per pixel of an INT32 branch, one
// word of an 8-bit branch, two bytes of a 4-bit one -- reads its dyadic pairs once, walks the pixels through running
// pointers and keeps several pixels in flight; neighbouring lanes read neighbouring pieces of the dense branch
// tensor and write neighbouring words of the output row.  The pixel loop is compiled per operand signedness, form
// of the arithmetic and output type and chosen once per thread.  Integer arithmetic only.
#include "hq_internal.cuh"

namespace {

struct ConcatBranch {
  const void* in; const int32_t* b; const int32_t* c;
  int32_t bits, is_signed, ch, ch_off;
  int32_t row_ch;     // channels per pixel of the tensor this entry reads (> ch for a piece of a very wide branch)
  int32_t width;      // channels a thread owns: 16, or 4 for an INT32 branch read in 16-byte pieces
  int32_t upp;        // threads (units) per pixel of this branch = ceil(ch / width)
  int32_t block0, nblocks;   // this branch's blocks of the launch
  int32_t vec;        // 1: rows and dyadic arrays allow 16-byte reads (ch % 16 == 0 resp. ch % 4 == 0, aligned arrays)
  int32_t piece16;    // 1: an 8-bit branch whose rows, offset and output rows are whole 16-byte pieces (see concat_uniform8)
};

struct ConcatArgs {
  ConcatBranch br[HQ_CONCAT_MAX_BRANCHES];
  int32_t n_br, out_ch, out_bits, relu, qmin, qmax;
  long long pixels;
  void* out;
  const int4* narrow;   // per OUTPUT channel {m, a, s, valid} from concat_narrow_kernel (8-/4-bit branches), or NULL
  int32_t sat;          // 1: relu and the clamp bounds equal a saturating conversion to the 8-bit output type
  int32_t rev;          // 1: pixels are walked from the last to the first (the handle's tile order): same results
};

// Narrow multiply-add pairs for the 8- and 4-bit branches.  A stored 8-bit value r has 256 possible values, so
// dn(r, b, c) can often be written (r*m + a) >> s in 32-bit arithmetic (on unsigned words for unsigned operands), m ~ b / 2^8: one warp per output channel
// tries the two neighbouring multipliers against the 64-bit definition for every r and records the one that agrees
// everywhere (valid = 1), else valid = 0 and the channel keeps the wide form.  c >= 41 makes the term 0 for every r.
__global__ void __launch_bounds__(128) concat_narrow_kernel(const __grid_constant__ ConcatArgs a, int4* out) {
  const int oc = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (oc >= a.out_ch) return;
  int i = 0;
#pragma unroll
  for (int j = 1; j < HQ_CONCAT_MAX_BRANCHES; ++j)
    if (j < a.n_br && oc >= a.br[j].ch_off) i = j;
  int4 res = make_int4(0, 0, 0, 0);
  if (a.br[i].bits != 32) {
    const int k = oc - a.br[i].ch_off;
    const long long b = a.br[i].b[k];
    const int c = a.br[i].c[k];
    const int r_lo = a.br[i].is_signed ? -128 : 0;
    if (c >= 41) {
      res = make_int4(0, 0, 0, 1);                     // |r*b| < 2^39 <= 2^(c-2)
    } else if (c >= 9 && c <= 38) {
      const int s = c - 8, add = 1 << (s - 1);
      const long long m0 = b >> 8, m1 = m0 + 1;
      bool ok0 = m0 <= (1 << 23), ok1 = m1 <= (1 << 23);
      // signed operands: |r*m| <= 2^30 and a <= 2^29 fit INT32; unsigned ones (r*m + a < 2^32) take the same
      // multiply-add on unsigned words with a logical shift, which the pixel loops mirror
      const bool uns = r_lo == 0;
      for (int t = 0; t < 8; ++t) {
        const int r = r_lo + lane + 32 * t;
        const long long exact = hq_dn(r, (int)b, c);
        const unsigned t0 = (unsigned)r * (unsigned)m0 + (unsigned)add, t1 = (unsigned)r * (unsigned)m1 + (unsigned)add;
        ok0 = ok0 && exact == (uns ? (long long)(t0 >> s) : (long long)((int)t0 >> s));
        ok1 = ok1 && exact == (uns ? (long long)(t1 >> s) : (long long)((int)t1 >> s));
      }
      ok0 = __all_sync(0xffffffffu, ok0);
      ok1 = __all_sync(0xffffffffu, ok1);
      if (ok0) res = make_int4((int)m0, add, s, 1);
      else if (ok1) res = make_int4((int)m1, add, s, 1);
    }
  }
  if (lane == 0) out[oc] = res;
}

// Four values clamped to the unsigned / signed 8-bit range and packed, first value in the low byte.
__device__ __forceinline__ unsigned pack4_sat(int v0, int v1, int v2, int v3, bool is_signed) {
  unsigned hi2, w;
  if (is_signed) {
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi2) : "r"(v3), "r"(v2), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v1), "r"(v0), "r"(hi2));
  } else {
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(hi2) : "r"(v3), "r"(v2), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v1), "r"(v0), "r"(hi2));
  }
  return w;
}

// One value by the 64-bit definition.
__device__ __forceinline__ int concat_dn64(int q, int b, int c, int lo, int hi) {
  long long y = hq_dn(q, b, c);
  if (y < (long long)lo) y = lo;
  if (y > (long long)hi) y = hi;
  return (int)y;
}

constexpr int kPix = 4;      // pixels (16-byte reads) a thread keeps in flight

// Store `n` (<= 16) clamped values of one thread: 8-bit bytes or 4-bit nibbles (low nibble first), widest aligned form.
template <int N>
__device__ __forceinline__ void concat_store(const ConcatArgs& a, int (&o)[N], int n, long long o0, int lo, int hi) {
  if (a.out_bits == 8) {
    unsigned char* op = (unsigned char*)a.out + o0;
    const bool whole = n == N && (o0 & (N - 1)) == 0;
    if (whole) {
      unsigned w[N / 4];
      if (a.sat) {
#pragma unroll
        for (int v = 0; v < N / 4; ++v) w[v] = pack4_sat(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3], lo < 0);
      } else {
#pragma unroll
        for (int j = 0; j < N; ++j) o[j] = min(max(o[j], lo), hi);
#pragma unroll
        for (int v = 0; v < N / 4; ++v)
          w[v] = (unsigned)(o[4 * v] & 0xFF) | ((unsigned)(o[4 * v + 1] & 0xFF) << 8) |
                 ((unsigned)(o[4 * v + 2] & 0xFF) << 16) | ((unsigned)(o[4 * v + 3] & 0xFF) << 24);
      }
      if (N == 16) *(uint4*)op = make_uint4(w[0], w[N / 4 > 1 ? 1 : 0], w[N / 4 > 2 ? 2 : 0], w[N / 4 > 3 ? 3 : 0]);
      else *(unsigned*)op = w[0];
    } else {
#pragma unroll
      for (int j = 0; j < N; ++j) if (j < n) op[j] = (unsigned char)min(max(o[j], lo), hi);
    }
  } else {
    // 4-bit output: channel counts and offsets are even, so a byte's two nibbles belong to this thread
    unsigned char* op = (unsigned char*)a.out + (o0 >> 1);
#pragma unroll
    for (int j = 0; j < N; ++j) o[j] = min(max(o[j], lo), hi) & 0xF;
    const bool whole = n == N && (o0 & (N - 1)) == 0;
    if (whole) {
      unsigned w[N / 8 > 0 ? N / 8 : 1] = {};
#pragma unroll
      for (int j = 0; j < N; ++j) w[j >> 3] |= (unsigned)o[j] << (4 * (j & 7));
      if (N == 16) *(uint2*)op = make_uint2(w[0], w[N / 8 > 1 ? 1 : 0]);
      else *(unsigned short*)op = (unsigned short)w[0];
    } else {
#pragma unroll
      for (int j = 0; j < N; j += 2)
        if (j < n) op[j >> 1] = (unsigned char)(o[j] | (o[j + 1] << 4));
    }
  }
}

// One branch's share of the blocks.  N = channels per thread (16: 8-/4-bit branches and ragged INT32 ones; 4: INT32
// branches read in 16-byte pieces).  Thread t of the block's first upp * ppb threads owns unit t % upp of pixel
// t / upp of every block step, i.e. consecutive lanes walk consecutive 16-byte pieces of the dense branch tensor.
template <int N>
__device__ __forceinline__ void concat_branch(const ConcatArgs& a, const int i) {
  const void* const in = a.br[i].in;
  const int bits = a.br[i].bits, is_signed = a.br[i].is_signed, ch = a.br[i].ch, vec = a.br[i].vec;
  const int upp = a.br[i].upp, ppb = 256 / upp;
  const int tid = threadIdx.x;
  if (tid >= upp * ppb) return;
  const int u = tid % upp, y = tid / upp;
  const int k0 = u * N;
  const int nk = min(N, ch - k0);
  const int off = a.br[i].ch_off + k0;
  const int lo = a.relu ? max(a.qmin, 0) : a.qmin, hi = a.qmax;
  // Per-channel constants, three forms of y = dn(q, b, c):
  //   narrow (8-/4-bit operands with a checked pair)   (q*m + a) >> s
  //   fast   (every c of the thread >= 33)             (mulhi(q, b) + 2^(c-33)) >> (c-32): the rounding constant is
  //          then a multiple of 2^32 and adds to the high word of q*b without a carry; |q*b| < 2^62 keeps it in INT32
  //   else   the 64-bit definition
  int bb[N], hh[N], ss[N];
  bool fast = true;
#pragma unroll
  for (int j = 0; j < N; ++j) {
    const int b = j < nk ? __ldg(a.br[i].b + k0 + j) : 0;
    const int c = j < nk ? __ldg(a.br[i].c + k0 + j) : 33;
    bb[j] = b; ss[j] = c; hh[j] = 0;
    fast = fast && c >= 33;
  }
  bool narrow = a.narrow != nullptr && bits != 32 && nk == N;
  if (narrow) {
#pragma unroll
    for (int j = 0; j < N; ++j) narrow = narrow && __ldg(&a.narrow[off + j].w) != 0;
    if (narrow) {
#pragma unroll
      for (int j = 0; j < N; ++j) { const int4 t = __ldg(a.narrow + off + j); bb[j] = t.x; hh[j] = t.y; ss[j] = t.z; }
    }
  }
  if (fast && !narrow) {
#pragma unroll
    for (int j = 0; j < N; ++j) { hh[j] = 1 << (ss[j] - 33); ss[j] -= 32; }
  }
  const long long step = (long long)a.br[i].nblocks * ppb;
  const long long first = (long long)(blockIdx.x - a.br[i].block0) * ppb + y;
  for (long long px0 = first; px0 < a.pixels; px0 += step * kPix) {
    uint4 raw[kPix];
    if (vec) {
#pragma unroll
      for (int p = 0; p < kPix; ++p) {
        const long long px = px0 + p * step;
        if (px < a.pixels) {
          const long long e0 = (a.rev ? a.pixels - 1 - px : px) * (long long)ch + k0;
          if (bits == 4) { const uint2 t = *(const uint2*)((const unsigned char*)in + (e0 >> 1)); raw[p].x = t.x; raw[p].y = t.y; }
          else raw[p] = *(const uint4*)((const unsigned char*)in + e0 * (bits >> 3));
        }
      }
    }
#pragma unroll 1
    for (int p = 0; p < kPix; ++p) {                 // one copy of the arithmetic: the instruction stream stays small
      const long long pxl = px0 + p * step;
      if (pxl >= a.pixels) break;
      const long long px = a.rev ? a.pixels - 1 - pxl : pxl;
      int q[N];
      if (vec) {
        uint4 r = raw[0];
        if (p == 1) r = raw[1];
        if (p == 2) r = raw[2];
        if (p == 3) r = raw[3];
        const unsigned w[4] = {r.x, r.y, r.z, r.w};
        if (N == 4) {
#pragma unroll
          for (int j = 0; j < N; ++j) q[j] = (int)w[j & 3];
        } else if (bits == 8) {
#pragma unroll
          for (int j = 0; j < N; ++j) {
            const unsigned sh = w[(j >> 2) & 3] >> (8 * (j & 3));
            q[j] = is_signed ? (int)(signed char)sh : (int)(sh & 0xFFu);
          }
        } else {
#pragma unroll
          for (int j = 0; j < N; ++j) {
            const unsigned sh = w[(j >> 3) & 1] >> (4 * (j & 7));
            q[j] = is_signed ? ((int)(sh << 28) >> 28) : (int)(sh & 0xFu);
          }
        }
      } else {
        const long long e0 = px * (long long)ch + k0;
#pragma unroll
        for (int j = 0; j < N; ++j) q[j] = j < nk ? hq_load_elem(in, e0 + j, bits, is_signed) : 0;
      }
      int o[N];
      if (narrow) {
#pragma unroll
        for (int j = 0; j < N; ++j) {
          const unsigned t = (unsigned)q[j] * (unsigned)bb[j] + (unsigned)hh[j];
          o[j] = is_signed ? (int)t >> ss[j] : (int)(t >> ss[j]);
        }
      } else if (fast) {
#pragma unroll
        for (int j = 0; j < N; ++j) o[j] = (__mulhi(q[j], bb[j]) + hh[j]) >> ss[j];
      } else {
#pragma unroll
        for (int j = 0; j < N; ++j) o[j] = concat_dn64(q[j], bb[j], ss[j], lo, hi);
      }
      concat_store<N>(a, o, nk, px * (long long)a.out_ch + off, lo, hi);
    }
  }
}

// An 8-bit branch whose channels all share ONE dyadic pair -- the case Appendix E writes down, DN(S_i / S_a) with
// per-tensor activation scales -- needs no per-channel constants: a thread owns one 16-byte piece (sixteen channels)
// of the pixel row, walks the pixels through running pointers with four pieces in flight, three constants in
// registers, one 16-byte store per piece.  (m, a, s) is the checked narrow pair of the shared (b, c).
template <bool SIGNED, int OUT>
__device__ __forceinline__ void concat_uniform8(const ConcatArgs& a, const int i, const unsigned m, const unsigned add,
                                                const int s, const int lo, const int hi) {
  const ConcatBranch& B = a.br[i];
  const int P = B.ch >> 4;                                        // pieces per pixel (at most 64)
  const int ppb = 256 / P;                                        // pixels per block step
  const int tid = threadIdx.x;
  if (tid >= P * ppb) return;
  const int u = tid % P, y = tid / P;
  const long long step = (long long)B.nblocks * ppb;
  long long px = (long long)((int)blockIdx.x - B.block0) * ppb + y;
  // (px counts positions of the walk; position t is pixel t, or pixel pixels - 1 - t when walking backwards)
  const long long px_at = a.rev ? a.pixels - 1 - px : px, dir = a.rev ? -1 : 1;
  const long long istep = dir * step * B.row_ch, ostep = dir * step * a.out_ch;
  const unsigned char* ip = (const unsigned char*)B.in + px_at * B.row_ch + u * 16;
  unsigned char* op = (unsigned char*)a.out + px_at * a.out_ch + B.ch_off + u * 16;
  auto one = [&](const uint4 r, unsigned char* dst) {
    const unsigned w[4] = {r.x, r.y, r.z, r.w};
    unsigned o[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      int yv[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        // byte j zero- or sign-extended by one byte permute
        const unsigned sx = 8u | (unsigned)j;
        const unsigned q = hq_prmt(w[v], 0u, SIGNED ? (sx << 12) | (sx << 8) | (sx << 4) | (unsigned)j : 0x4440u | (unsigned)j);
        const unsigned t = q * m + add;
        yv[j] = SIGNED ? (int)t >> s : (int)(t >> s);
      }
      if (OUT == 0) o[v] = pack4_sat(yv[0], yv[1], yv[2], yv[3], lo < 0);
      else {
#pragma unroll
        for (int j = 0; j < 4; ++j) yv[j] = min(max(yv[j], lo), hi) & 0xFF;
        o[v] = (unsigned)yv[0] | ((unsigned)yv[1] << 8) | ((unsigned)yv[2] << 16) | ((unsigned)yv[3] << 24);
      }
    }
    *(uint4*)dst = make_uint4(o[0], o[1], o[2], o[3]);
  };
  constexpr int KP = 4;                                           // eight in flight measured the same
  while (px + (KP - 1) * step < a.pixels) {                      // whole groups: all reads first
    uint4 r[KP];
    const unsigned char* q = ip;
#pragma unroll
    for (int k = 0; k < KP; ++k) { r[k] = __ldg((const uint4*)q); q += istep; }
    unsigned char* d = op;
#pragma unroll
    for (int k = 0; k < KP; ++k) { one(r[k], d); d += ostep; }
    px += KP * step; ip = q; op = d;
  }
  for (; px < a.pixels; px += step, ip += istep, op += ostep) one(__ldg((const uint4*)ip), op);
}

struct W4State {
  const unsigned char* ip; unsigned char* op;
  long long px, step, in_row, out_row, pixels, dir;
  int lo, hi; bool word_out;
};

// Pixel loop of the four-channel form.  SIGNED: operand signedness; MODE: 2 narrow pair, 1 high-word form, 0 the
// 64-bit definition; OUT: 0 8-bit output by saturating packs, 1 8-bit output with explicit bounds, 2 4-bit output.
template <int BITS, bool SIGNED, int MODE, int OUT>
__device__ __forceinline__ void concat_w4_loop(W4State t, const int (&bb)[4], const int (&hh)[4], const int (&ss)[4]) {
  constexpr int KP = BITS == 32 ? 4 : 8;
  const long long istep = t.dir * t.step * t.in_row, ostep = t.dir * t.step * t.out_row;
  auto one = [&](const uint4 r, unsigned char* o_ptr) {
    int q[4];
    if (BITS == 32) { q[0] = (int)r.x; q[1] = (int)r.y; q[2] = (int)r.z; q[3] = (int)r.w; }
    else if (BITS == 8) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const unsigned sx = 8u | (unsigned)j;          // one byte permute, zero- or sign-extending
        q[j] = (int)hq_prmt(r.x, 0u, SIGNED ? (sx << 12) | (sx << 8) | (sx << 4) | (unsigned)j : 0x4440u | (unsigned)j);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const unsigned sh = r.x >> (4 * j);
        q[j] = SIGNED ? ((int)(sh << 28) >> 28) : (int)(sh & 0xFu);
      }
    }
    int o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      o[j] = MODE == 2 ? (SIGNED ? (int)((unsigned)q[j] * (unsigned)bb[j] + (unsigned)hh[j]) >> ss[j]
                                 : (int)(((unsigned)q[j] * (unsigned)bb[j] + (unsigned)hh[j]) >> ss[j]))
           : MODE == 1 ? (__mulhi(q[j], bb[j]) + hh[j]) >> ss[j]
                       : concat_dn64(q[j], bb[j], ss[j], t.lo, t.hi);
    if (OUT != 2) {
      unsigned w;
      if (OUT == 0) w = pack4_sat(o[0], o[1], o[2], o[3], t.lo < 0);
      else {
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = min(max(o[j], t.lo), t.hi) & 0xFF;
        w = (unsigned)o[0] | ((unsigned)o[1] << 8) | ((unsigned)o[2] << 16) | ((unsigned)o[3] << 24);
      }
      if (t.word_out) *(unsigned*)o_ptr = w;
      else { o_ptr[0] = (unsigned char)w; o_ptr[1] = (unsigned char)(w >> 8); o_ptr[2] = (unsigned char)(w >> 16); o_ptr[3] = (unsigned char)(w >> 24); }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) o[j] = min(max(o[j], t.lo), t.hi) & 0xF;
      const unsigned w = (unsigned)o[0] | ((unsigned)o[1] << 4) | ((unsigned)o[2] << 8) | ((unsigned)o[3] << 12);
      if (t.word_out) *(unsigned short*)o_ptr = (unsigned short)w;
      else { o_ptr[0] = (unsigned char)w; o_ptr[1] = (unsigned char)(w >> 8); }
    }
  };
  auto fetch = [&](const unsigned char* p) -> uint4 {
    uint4 r = make_uint4(0u, 0u, 0u, 0u);
    if (BITS == 32) r = *(const uint4*)p;
    else if (BITS == 8) r.x = *(const unsigned*)p;
    else r.x = *(const unsigned short*)p;
    return r;
  };
  // whole groups of KP pixels: all reads first, then the arithmetic and the stores
  while (t.px + (KP - 1) * t.step < t.pixels) {
    uint4 raw[KP];
    const unsigned char* q = t.ip;
#pragma unroll
    for (int p = 0; p < KP; ++p) { raw[p] = fetch(q); q += istep; }
    unsigned char* d = t.op;
#pragma unroll
    for (int p = 0; p < KP; ++p) { one(raw[p], d); d += ostep; }
    t.px += KP * t.step; t.ip = q; t.op = d;
  }
  for (; t.px < t.pixels; t.px += t.step, t.ip += istep, t.op += ostep) one(fetch(t.ip), t.op);
}

// Four channels per thread: the form for every branch whose channel count is a multiple of 4 (up to 1024 channels).
// A thread reads 16 bytes (INT32), one word (8 bit) or two bytes (4 bit) per pixel through a running pointer, keeps
// KP pixels in flight and twelve constants in registers, so many warps fit an SM; consecutive lanes read consecutive
// pieces of the dense branch tensor and write consecutive words of the output row.
template <int BITS>
__device__ __forceinline__ void concat_w4(const ConcatArgs& a, const int i) {
  const int is_signed = a.br[i].is_signed;
  const int upp = a.br[i].upp, ppb = 256 / upp;
  const int tid = threadIdx.x;
  const int lo = a.relu ? max(a.qmin, 0) : a.qmin, hi = a.qmax;
  if (BITS == 8 && a.br[i].piece16 && a.narrow != nullptr) {
    // Do all channels of the branch share one pair with a checked narrow form?  The block's threads look at four
    // channels each (together all of them) and vote; the branch and the flag are the same for the whole block.
    const int kc = (tid % upp) * 4;
    const int b0 = __ldg(a.br[i].b), c0 = __ldg(a.br[i].c);
    bool same = true;
#pragma unroll
    for (int j = 0; j < 4; ++j) same = same && __ldg(a.br[i].b + kc + j) == b0 && __ldg(a.br[i].c + kc + j) == c0;
    const int4 n0 = __ldg(a.narrow + a.br[i].ch_off);
    if (__syncthreads_and(same && n0.w != 0)) {
      if (is_signed) { if (a.sat) concat_uniform8<true, 0>(a, i, n0.x, n0.y, n0.z, lo, hi); else concat_uniform8<true, 1>(a, i, n0.x, n0.y, n0.z, lo, hi); }
      else { if (a.sat) concat_uniform8<false, 0>(a, i, n0.x, n0.y, n0.z, lo, hi); else concat_uniform8<false, 1>(a, i, n0.x, n0.y, n0.z, lo, hi); }
      return;
    }
  }
  if (tid >= upp * ppb) return;
  const int u = tid % upp, y = tid / upp;
  const int k0 = u * 4, off = a.br[i].ch_off + k0;
  int bb[4], hh[4], ss[4];
  bool fast = true;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    bb[j] = __ldg(a.br[i].b + k0 + j); ss[j] = __ldg(a.br[i].c + k0 + j); hh[j] = 0;
    fast = fast && ss[j] >= 33;
  }
  bool narrow = a.narrow != nullptr && BITS != 32;
  if (narrow) {
#pragma unroll
    for (int j = 0; j < 4; ++j) narrow = narrow && __ldg(&a.narrow[off + j].w) != 0;
    if (narrow) {
#pragma unroll
      for (int j = 0; j < 4; ++j) { const int4 t = __ldg(a.narrow + off + j); bb[j] = t.x; hh[j] = t.y; ss[j] = t.z; }
    }
  }
  if (fast && !narrow) {
#pragma unroll
    for (int j = 0; j < 4; ++j) { hh[j] = 1 << (ss[j] - 33); ss[j] -= 32; }
  }
  const int mode = narrow ? 2 : fast ? 1 : 0;
  W4State t;
  t.step = (long long)a.br[i].nblocks * ppb;
  t.px = (long long)(blockIdx.x - a.br[i].block0) * ppb + y;
  t.in_row = (long long)a.br[i].row_ch * BITS / 8; t.out_row = (long long)a.out_ch * a.out_bits / 8;
  const long long px_at = a.rev ? a.pixels - 1 - t.px : t.px;      // t.px counts positions of the walk
  t.ip = (const unsigned char*)a.br[i].in + px_at * t.in_row + (long long)k0 * BITS / 8;
  t.op = (unsigned char*)a.out + px_at * t.out_row + (long long)off * a.out_bits / 8;
  t.dir = a.rev ? -1 : 1;
  t.lo = lo; t.hi = hi; t.pixels = a.pixels;
  t.word_out = (off & 3) == 0 && (a.out_ch & 3) == 0;      // the thread's outputs are one aligned word / halfword
  // one straight-line loop per signedness, form of the arithmetic and output type, chosen once
  const int outk = a.out_bits == 4 ? 2 : a.sat ? 0 : 1;
#define HQ_W4_OUT(S, M) \
  do { if (outk == 0) concat_w4_loop<BITS, S, M, 0>(t, bb, hh, ss); \
       else if (outk == 1) concat_w4_loop<BITS, S, M, 1>(t, bb, hh, ss); \
       else concat_w4_loop<BITS, S, M, 2>(t, bb, hh, ss); } while (0)
#define HQ_W4_MODE(S) \
  do { if (mode == 2) HQ_W4_OUT(S, 2); else if (mode == 1) HQ_W4_OUT(S, 1); else HQ_W4_OUT(S, 0); } while (0)
  if (BITS == 32 || is_signed) HQ_W4_MODE(true); else HQ_W4_MODE(false);
#undef HQ_W4_MODE
#undef HQ_W4_OUT
}

// The branch a block works for: the last branch of the wanted width whose first block is not beyond this one.
__device__ __forceinline__ int concat_my_branch(const ConcatArgs& a, int width) {
  int i = -1;
#pragma unroll
  for (int j = 0; j < HQ_CONCAT_MAX_BRANCHES; ++j)
    if (j < a.n_br && a.br[j].width == width && (i < 0 || (int)blockIdx.x >= a.br[j].block0)) i = j;
  return i;
}

// Branches in the four-channel form (few registers, many warps per SM) ...
__global__ void __launch_bounds__(256, 4) concat_requant_kernel(const __grid_constant__ ConcatArgs a) {
  const int i = concat_my_branch(a, 4);
  if (a.br[i].bits == 32) concat_w4<32>(a, i);
  else if (a.br[i].bits == 8) concat_w4<8>(a, i);
  else concat_w4<4>(a, i);
}

// ... and the others (ragged or very wide branches) in the sixteen-channel form, in a launch of their own.
__global__ void __launch_bounds__(256, 2) concat_requant_wide_kernel(const __grid_constant__ ConcatArgs a) {
  concat_branch<16>(a, concat_my_branch(a, 16));
}

inline bool al16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace

extern "C" hq_status hq_concat_requant(hq_handle* h, int32_t n_branches, const hq_tensor* branches,
                                       const hq_dyadic* rescale, int32_t relu, int32_t qmin, int32_t qmax,
                                       hq_tensor* out, void* stream) {
  if (!h || !branches || !rescale || !out || !out->data) return HQ_ERR_INVALID_ARG;
  if (n_branches < 1 || n_branches > HQ_CONCAT_MAX_BRANCHES) return HQ_ERR_INVALID_ARG;
  if (out->bits != 8 && out->bits != 4) return HQ_ERR_INVALID_ARG;
  if (out->n < 0 || out->h < 1 || out->w < 1 || out->c < 1) return HQ_ERR_INVALID_ARG;
  if (!al16(out->data)) return HQ_ERR_ALIGNMENT;
  {
    const long long lo = out->is_signed ? -(1LL << (out->bits - 1)) : 0;
    const long long hi = out->is_signed ? (1LL << (out->bits - 1)) - 1 : (1LL << out->bits) - 1;
    if (qmin > qmax || qmin < lo || qmax > hi) return HQ_ERR_INVALID_ARG;
  }
  ConcatArgs a{};
  int off = 0, nb = 0;
  long long weight[HQ_CONCAT_MAX_BRANCHES], weight_sum = 0;
  // A branch of more than 1024 channels (a multiple of 4) is entered as several pieces of at most 1024, each read
  // with the whole tensor's row pitch, while entries are left; otherwise it takes the sixteen-channel form.
  int spare = HQ_CONCAT_MAX_BRANCHES - n_branches;
  for (int i = 0; i < n_branches; ++i) {
    const hq_tensor& t = branches[i];
    if (!t.data || !rescale[i].b || !rescale[i].c) return HQ_ERR_INVALID_ARG;
    if (t.bits != 4 && t.bits != 8 && t.bits != 32) return HQ_ERR_INVALID_ARG;
    if (t.n != out->n || t.h != out->h || t.w != out->w || t.c < 1) return HQ_ERR_INVALID_ARG;
    if (t.bits == 4 && (t.c & 1)) return HQ_ERR_INVALID_ARG;
    if (out->bits == 4 && (t.c & 1)) return HQ_ERR_UNSUPPORTED;   // a byte of the output would span two branches
    if (!al16(t.data)) return HQ_ERR_ALIGNMENT;
    const bool four = t.c % 4 == 0 && out->c % 2 == 0;
    int pieces = 1;
    if (four && t.c > 1024) {
      pieces = (t.c + 1023) / 1024;
      if (pieces - 1 > spare) pieces = 1; else spare -= pieces - 1;
    }
    for (int pc = 0, k0 = 0; pc < pieces; ++pc) {
      const int chp = pieces == 1 ? t.c : (t.c - k0 < 1024 ? t.c - k0 : 1024);
      ConcatBranch& B = a.br[nb];
      B.in = (const unsigned char*)t.data + (long long)k0 * t.bits / 8; B.b = rescale[i].b + k0; B.c = rescale[i].c + k0;
      B.bits = t.bits; B.is_signed = t.bits == 32 ? 1 : t.is_signed; B.ch = chp; B.ch_off = off; B.row_ch = t.c;
      if (four && chp <= 4 * 256) { B.width = 4; B.vec = 1; }
      else { B.width = 16; B.vec = (t.bits != 32 && t.c % 16 == 0) ? 1 : 0; }
      B.piece16 = (B.width == 4 && t.bits == 8 && out->bits == 8 && chp % 16 == 0 && t.c % 16 == 0 && off % 16 == 0 &&
                   out->c % 16 == 0) ? 1 : 0;
      B.upp = (chp + B.width - 1) / B.width;
      if (B.upp > 256) return HQ_ERR_UNSUPPORTED;                 // more than 4096 channels in one branch
      weight[nb] = (long long)chp * (t.bits + out->bits);
      weight_sum += weight[nb];
      off += chp; k0 += chp; ++nb;
    }
  }
  if (off != out->c) return HQ_ERR_INVALID_ARG;
  a.n_br = nb; a.out_ch = out->c; a.out_bits = out->bits;
  a.relu = relu; a.qmin = qmin; a.qmax = qmax;
  a.rev = h->tile_order ? 1 : 0;
  a.pixels = (long long)out->n * out->h * out->w;
  a.out = out->data;
  if (a.pixels == 0) return HQ_OK;
  // blocks of the one launch, dealt to the branches in proportion to the bytes they move
  const long long cap = (long long)h->sm_count * 8;
  long long blocks4 = 0, blocks16 = 0;
  for (int i = 0; i < nb; ++i) {
    ConcatBranch& B = a.br[i];
    const long long per_block = (long long)(256 / B.upp) * (B.width == 4 && B.bits != 32 ? 8 : kPix);
    const long long need = (a.pixels + per_block - 1) / per_block;
    long long share = (cap * weight[i] + weight_sum - 1) / weight_sum;
    if (share > need) share = need;
    if (share < 1) share = 1;
    long long& blocks = B.width == 4 ? blocks4 : blocks16;          // each form numbers its own launch's blocks
    B.block0 = (int32_t)blocks; B.nblocks = (int32_t)share;
    blocks += share;
  }
  {
    const int lo = relu ? (qmin > 0 ? qmin : 0) : qmin;
    a.sat = (out->bits == 8 && ((!out->is_signed && lo == 0 && qmax == 255) ||
                                (out->is_signed && lo == -128 && qmax == 127))) ? 1 : 0;
  }
  // A large call first works out the narrow pairs of its 8- and 4-bit branches in the handle's buffer (one small
  // launch on the same stream, repaid by the cheaper arithmetic).
  a.narrow = nullptr;
  bool any_narrow = false;
  for (int i = 0; i < n_branches; ++i) any_narrow = any_narrow || branches[i].bits != 32;
  if (any_narrow && h->narrow_pairs && out->c <= 2 * kNarrowChannels && a.pixels * out->c >= (1ll << 22)) {
    int4* tab = (int4*)h->narrow_pairs;
    concat_narrow_kernel<<<(out->c + 3) / 4, 128, 0, (cudaStream_t)stream>>>(a, tab);
    if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
    a.narrow = tab;
  }
  if (blocks4) concat_requant_kernel<<<(unsigned)blocks4, 256, 0, (cudaStream_t)stream>>>(a);
  if (blocks16) concat_requant_wide_kernel<<<(unsigned)blocks16, 256, 0, (cudaStream_t)stream>>>(a);
  return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
