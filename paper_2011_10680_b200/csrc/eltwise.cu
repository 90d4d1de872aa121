// Memory-bound kernels of the integer-only pipeline: residual add / requantization on stored
// tensors (Section 3.3), global average pooling on wide integers (Appendix E) and the stem's max
// pooling.  Each streams its operands once with 16-byte accesses; the arithmetic is the dyadic
// multiply-shift of Eq. 4 in 64-bit integers.  No floating point anywhere.
#include <climits>

#include "hq_internal.cuh"

namespace {

// ---- 16-element group load/store for 4-, 8- and 32-bit dense tensors -----------------------
template <int BITS>
__device__ __forceinline__ void load16(const void* base, long long elem, int is_signed, int (&v)[16]) {
  if constexpr (BITS == 32) {
    const int4* p = (const int4*)((const int*)base + elem);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int4 t = __ldg(p + i);
      v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
    }
  } else if constexpr (BITS == 8) {
    const uint4 t = __ldg((const uint4*)((const unsigned char*)base + elem));
    const unsigned w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const unsigned byte = (w[i >> 2] >> (8 * (i & 3))) & 0xFFu;
      v[i] = is_signed ? (int)(signed char)byte : (int)byte;
    }
  } else {
    const uint2 t = __ldg((const uint2*)((const unsigned char*)base + (elem >> 1)));
    const unsigned w[2] = {t.x, t.y};
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      int nib = (int)((w[i >> 3] >> (4 * (i & 7))) & 0xFu);
      if (is_signed && (nib & 8)) nib -= 16;
      v[i] = nib;
    }
  }
}

template <int BITS>
__device__ __forceinline__ void store16(void* base, long long elem, const int (&v)[16]) {
  if constexpr (BITS == 8) {
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      w[i] = (unsigned)(v[4 * i] & 0xFF) | ((unsigned)(v[4 * i + 1] & 0xFF) << 8) |
             ((unsigned)(v[4 * i + 2] & 0xFF) << 16) | ((unsigned)(v[4 * i + 3] & 0xFF) << 24);
    *(uint4*)((unsigned char*)base + elem) = make_uint4(w[0], w[1], w[2], w[3]);
  } else {
    unsigned w[2] = {0u, 0u};
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i >> 3] |= (unsigned)(v[i] & 0xF) << (4 * (i & 7));
    *(uint2*)((unsigned char*)base + (elem >> 1)) = make_uint2(w[0], w[1]);
  }
}

// Each thread owns one group of 16 channels for the whole launch (its dyadic pairs stay in
// registers) and walks the pixels with a grid stride.
template <int MB, int RB, int OB>
__global__ void __launch_bounds__(256) residual_add_vec_kernel(EltArgs a, int groups, int pix_per_block) {
  const int g = threadIdx.x % groups;
  const int pl = threadIdx.x / groups;
  if (pl >= pix_per_block) return;
  const int ch0 = g * 16;
  int mb[16], mc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) { mb[i] = __ldg(a.mb + ch0 + i); mc[i] = __ldg(a.mc + ch0 + i); }
  int rb[16], rc[16];
  if constexpr (RB != 0) {
#pragma unroll
    for (int i = 0; i < 16; ++i) { rb[i] = __ldg(a.rb + ch0 + i); rc[i] = __ldg(a.rc + ch0 + i); }
  }
  const long long step = (long long)gridDim.x * pix_per_block;
  for (long long p = (long long)blockIdx.x * pix_per_block + pl; p < a.pixels; p += step) {
    const long long e = p * a.ch + ch0;
    int m[16], o[16];
    load16<MB>(a.main_t, e, a.main_signed, m);
    if constexpr (RB != 0) {
      int r[16];
      load16<RB>(a.res, e, a.res_signed, r);
#pragma unroll
      for (int i = 0; i < 16; ++i)
        o[i] = hq_clamp_ll(hq_dn(m[i], mb[i], mc[i]) + hq_dn(r[i], rb[i], rc[i]), a.relu, a.qmin, a.qmax);
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) o[i] = hq_clamp_ll(hq_dn(m[i], mb[i], mc[i]), a.relu, a.qmin, a.qmax);
    }
    store16<OB>(a.out, e, o);
  }
}

// ---- 8-bit operands: 32-bit fast path ----------------------------------------------------------
// A thread owns four consecutive channels (one 32-bit word per pixel) for the whole launch, so its dyadic
// pairs stay in registers and a warp reads / writes 128 contiguous bytes per pixel.  For an 8-bit value q
// and 9 <= c:  (q*b + 2^(c-1)) >> c  ==  (hi32((q << 24) * b) + 2^(c-9)) >> (c-8)   exactly, because
// (q<<24)*b >> 32 = floor(q*b / 2^8), 2^(c-1) is a multiple of 2^8 and the dropped low 8 bits cannot carry
// across a multiple of 2^(c-8); for c >= 40 the term rounds to 0.  Channels with c < 9 take the 64-bit form.
struct Dy8 { int b, h, sh, c; };     // multiplier, 2^(c-9), c-8, original c

__device__ __forceinline__ Dy8 make_dy8(int b, int c) {
  Dy8 d; d.c = c;
  if (c >= 40) { d.b = 0; d.h = 0; d.sh = 1; }
  else if (c >= 9) { d.b = b; d.h = 1 << (c - 9); d.sh = c - 8; }
  else { d.b = b; d.h = 0; d.sh = 0; }                       // c < 9: the thread switches to the 64-bit form
  return d;
}
template <bool SIGNED>
__device__ __forceinline__ int dn8(unsigned top, const Dy8& d) {      // `top` = the byte in bits 31:24; needs d.c >= 9; |result| < 2^30
  if (SIGNED) return (__mulhi((int)top, d.b) + d.h) >> d.sh;
  return (int)((__umulhi(top, (unsigned)d.b) + (unsigned)d.h) >> d.sh);
}

// One pixel's word of four channels.  SLOW: one of the thread's channels has a shift below 9 (64-bit form).
// SATP: 1 / 2 when the clamp bounds equal the range of u8 / s8 (a saturating pack does clamp and packing);
// 3 for a 4-bit output clamped to [0, 15]; 4 the same without a residual and with shifts reduced by four;
// 5 for a byte-wide output clamped to [0, 15].
// 8-bit value i of a word, zero- or sign-extended (one byte permute either way; the signed form needs the full
// selector of hq_prmt: bit 3 of a nibble replicates the selected byte's sign bit).
template <bool SIGNED>
__device__ __forceinline__ int byte_of(unsigned w, int i) {
  const unsigned sx = 8u | (unsigned)i;
  return SIGNED ? (int)hq_prmt(w, 0u, (sx << 12) | (sx << 8) | (sx << 4) | (unsigned)i)
                : (int)__byte_perm(w, 0u, 0x4440u | (unsigned)i);
}

template <bool RES, bool MSIGNED, bool RSIGNED, bool OUT4, bool SLOW, int SATP, bool NARROW = false>
__device__ __forceinline__ void requant8_word(const EltArgs& a, const Dy8 (&m)[4], const Dy8 (&r)[4], int wx, unsigned mw,
                                              unsigned rw, void* dst, int lo, int hi) {
  int s[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (NARROW) {
      // Dy8 holds a narrow pair (b = m, h = a, sh = s): (q*m + a) >> s equals dn(q, b, c) for every 8-bit q
      s[i] = (byte_of<MSIGNED>(mw, i) * m[i].b + m[i].h) >> m[i].sh;
      if (RES) s[i] += (byte_of<RSIGNED>(rw, i) * r[i].b + r[i].h) >> r[i].sh;
    } else if (!SLOW) {
      s[i] = dn8<MSIGNED>(__byte_perm(mw, 0u, 0x0444u | ((unsigned)i << 12)), m[i]);
      if (RES) s[i] += dn8<RSIGNED>(__byte_perm(rw, 0u, 0x0444u | ((unsigned)i << 12)), r[i]);
    } else {
      const unsigned mbyte = (mw >> (8 * i)) & 0xFFu, rbyte = (rw >> (8 * i)) & 0xFFu;
      long long t = hq_dn(MSIGNED ? (int)(signed char)mbyte : (int)mbyte, __ldg(a.mb + 4 * wx + i), m[i].c);
      if (RES) t += hq_dn(RSIGNED ? (int)(signed char)rbyte : (int)rbyte, __ldg(a.rb + 4 * wx + i), r[i].c);
      s[i] = (int)(t < (long long)lo ? (long long)lo : (t > (long long)hi ? (long long)hi : t));
    }
  }
  if constexpr (!OUT4 && SATP == 5) {
    // byte-wide output clamped to [0, 15] (a 4-bit tensor kept one value per byte inside a network): upper bound by a
    // minimum, lower bound and packing by the saturating packs
    unsigned w23, w;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(min(s[3], 15)), "r"(min(s[2], 15)), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(min(s[1], 15)), "r"(min(s[0], 15)), "r"(w23));
    *(unsigned*)dst = w;
  } else if constexpr (!OUT4 && SATP != 0) {
    // two saturating packs; the second carries the first one's halfword in its upper half: bytes s0 s1 s2 s3
    unsigned w23, w;
    if (SATP == 1) {
      asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(s[3]), "r"(s[2]), "r"(0));
      asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(s[1]), "r"(s[0]), "r"(w23));
    } else {
      asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(s[3]), "r"(s[2]), "r"(0));
      asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(s[1]), "r"(s[0]), "r"(w23));
    }
    *(unsigned*)dst = w;
  } else if constexpr (OUT4 && SATP == 4) {
    // No residual, clamp to [0, 15], and the shifts were reduced by four: s = floor(16 v).  The saturating pack
    // clamps 16 v to [0, 255], whose high nibble is min(max(floor(v), 0), 15); the four high nibbles then move
    // next to each other.
    unsigned w23, w;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(s[3]), "r"(s[2]), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(s[1]), "r"(s[0]), "r"(w23));
    const unsigned p0 = __byte_perm(w, 0u, 0x4420), p1 = __byte_perm(w, 0u, 0x4431);    // bytes 0, 2 and bytes 1, 3
    *(unsigned short*)dst = (unsigned short)(((p0 >> 4) & 0x0F0Fu) | (p1 & 0xF0F0u));
  } else if constexpr (OUT4 && SATP == 3) {
    // clamp to [0, 15]: upper bound by a minimum, lower bound by the saturating pack; then the four bytes'
    // low nibbles move next to each other
    unsigned w23, w;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(min(s[3], 15)), "r"(min(s[2], 15)), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(min(s[1], 15)), "r"(min(s[0], 15)), "r"(w23));
    const unsigned t = w | (w >> 4);                       // byte 0 = s0 | s1 << 4, byte 2 = s2 | s3 << 4
    *(unsigned short*)dst = (unsigned short)__byte_perm(t, 0u, 0x4420);
  } else {
    int y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) y[i] = SLOW ? s[i] : min(max(s[i], lo), hi);
    if (OUT4) {
      // 0 <= y <= 15 after the clamp of an unsigned 4-bit output; signed nibbles keep their low four bits
      const unsigned w = (unsigned)(y[0] & 0xF) + ((unsigned)(y[1] & 0xF) << 4) + ((unsigned)(y[2] & 0xF) << 8) + ((unsigned)(y[3] & 0xF) << 12);
      *(unsigned short*)dst = (unsigned short)w;
    } else {
      *(unsigned*)dst = (unsigned)(y[0] & 0xFF) | ((unsigned)(y[1] & 0xFF) << 8) | ((unsigned)(y[2] & 0xFF) << 16) |
                        ((unsigned)(y[3] & 0xFF) << 24);
    }
  }
}

// Destination of word `idx` of the output (four channels: a 32-bit word at 8 bit, a 16-bit word at 4 bit).
template <bool OUT4>
__device__ __forceinline__ void* out_word(const EltArgs& a, long long idx) {
  return OUT4 ? (void*)((unsigned short*)a.out + idx) : (void*)((unsigned*)a.out + idx);
}

template <bool RES, bool MSIGNED, bool RSIGNED, bool OUT4, bool SLOW, int SATP, bool NARROW = false>
__device__ __forceinline__ void requant8_pixels(const EltArgs& a, const Dy8 (&m)[4], const Dy8 (&r)[4], int wx, int words,
                                                int lo, int hi) {
  const unsigned* mp = (const unsigned*)a.main_t;
  const unsigned* rp = (const unsigned*)a.res;
  constexpr int U = RES ? 4 : 8;            // pixels (independent 4-byte loads) in flight per thread
  // A block walks runs of U * blockDim.y consecutive pixels: contiguous bytes per trip, friendly to DRAM pages.
  const long long run = (long long)U * blockDim.y, trip = run * gridDim.y;
  for (long long p0 = (long long)blockIdx.y * run + threadIdx.y; p0 < a.pixels; p0 += trip) {
    if (p0 + (long long)(U - 1) * blockDim.y < a.pixels) {
      unsigned mw[U], rw[U];
#pragma unroll
      for (int u = 0; u < U; ++u) mw[u] = __ldg(mp + (p0 + (long long)u * blockDim.y) * words + wx);
#pragma unroll
      for (int u = 0; u < U; ++u) rw[u] = RES ? __ldg(rp + (p0 + (long long)u * blockDim.y) * words + wx) : 0u;
#pragma unroll
      for (int u = 0; u < U; ++u)
        requant8_word<RES, MSIGNED, RSIGNED, OUT4, SLOW, SATP, NARROW>(a, m, r, wx, mw[u], rw[u],
                                                                       out_word<OUT4>(a, (p0 + (long long)u * blockDim.y) * words + wx), lo, hi);
    } else {
      for (long long p = p0; p < a.pixels; p += blockDim.y)
        requant8_word<RES, MSIGNED, RSIGNED, OUT4, SLOW, SATP, NARROW>(a, m, r, wx, __ldg(mp + p * words + wx),
                                                                       RES ? __ldg(rp + p * words + wx) : 0u, out_word<OUT4>(a, p * words + wx), lo, hi);
    }
  }
}

// 4-bit output clamped to [0, 15] without a residual: when every channel of the thread shifts by at least four,
// the shifts drop by four and the word is packed from the high nibbles (requant8_word, SATP == 4).
__device__ __forceinline__ bool reduce_shifts_by_four(Dy8 (&d)[4], bool usable) {
  bool ok = usable;
#pragma unroll
  for (int i = 0; i < 4; ++i) ok = ok && d[i].sh >= 4;
  return ok;
}

// Flat form for channel counts whose words divide the block (words a power of two, at most 256): the tensor is
// one array of 32-bit words, a block of 256 threads takes 256 consecutive words per step, so a thread keeps its
// four channels (word index mod words is fixed) and every address is a per-trip base plus a constant.
template <bool RES, bool MSIGNED, bool RSIGNED, bool OUT4, bool SLOW, int SATP, bool NARROW = false>
__device__ __forceinline__ void requant8_flat(const EltArgs& a, const Dy8 (&m)[4], const Dy8 (&r)[4], int wx, long long total,
                                              int lo, int hi) {
  constexpr int T = 256, U = RES ? 4 : 8;           // words in flight per thread
  const unsigned* mp = (const unsigned*)a.main_t + threadIdx.x;
  const unsigned* rp = RES ? (const unsigned*)a.res + threadIdx.x : nullptr;
  const long long trip = (long long)gridDim.x * (U * T);
  for (long long base = (long long)blockIdx.x * (U * T); base < total; base += trip) {
    const unsigned* mq = mp + base;
    const unsigned* rq = RES ? rp + base : nullptr;
    void* dst0 = out_word<OUT4>(a, base + threadIdx.x);
    auto dst = [&](int u) { return OUT4 ? (void*)((unsigned short*)dst0 + u * T) : (void*)((unsigned*)dst0 + u * T); };
    if (base + U * T <= total) {
      unsigned mw[U], rw[U];
#pragma unroll
      for (int u = 0; u < U; ++u) mw[u] = __ldg(mq + u * T);
#pragma unroll
      for (int u = 0; u < U; ++u) rw[u] = RES ? __ldg(rq + u * T) : 0u;
#pragma unroll
      for (int u = 0; u < U; ++u)
        requant8_word<RES, MSIGNED, RSIGNED, OUT4, SLOW, SATP, NARROW>(a, m, r, wx, mw[u], rw[u], dst(u), lo, hi);
    } else {
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (base + u * T + threadIdx.x < total)
          requant8_word<RES, MSIGNED, RSIGNED, OUT4, SLOW, SATP, NARROW>(a, m, r, wx, __ldg(mq + u * T),
                                                                         RES ? __ldg(rq + u * T) : 0u, dst(u), lo, hi);
    }
  }
}

template <bool RES, bool MSIGNED, bool RSIGNED, bool OUT4, int SATP, bool FLAT>
__global__ void __launch_bounds__(256) requant8_kernel(EltArgs a, int words, int lo, int hi) {
  // word (4 channels) of the pixel
  const int wx = FLAT ? (int)(threadIdx.x & (unsigned)(words - 1)) : (int)(blockIdx.x * blockDim.x + threadIdx.x);
  if (wx >= words) return;
  const long long total = a.pixels * words;
  Dy8 m[4], r[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = make_dy8(__ldg(a.mb + 4 * wx + i), __ldg(a.mc + 4 * wx + i));
    if (RES) r[i] = make_dy8(__ldg(a.rb + 4 * wx + i), __ldg(a.rc + 4 * wx + i));
    else r[i] = m[i];
  }
  bool slow = false;                       // a shift below 9 on one of this thread's channels: 64-bit form for the thread
#pragma unroll
  for (int i = 0; i < 4; ++i) slow = slow || m[i].c < 9 || (RES && r[i].c < 9);
  // narrow pairs prepared by the caller: usable when every channel of this thread has one
  if (a.m_narrow && (!RES || a.r_narrow)) {
    Dy8 nm[4], nr[4];
    bool ok = true;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int4 pm = __ldg((const int4*)a.m_narrow + 4 * wx + i);
      nm[i].b = pm.x; nm[i].h = pm.y; nm[i].sh = pm.z; nm[i].c = 0; ok = ok && pm.w != 0;
      nr[i] = nm[i];
      if (RES) {
        const int4 pr = __ldg((const int4*)a.r_narrow + 4 * wx + i);
        nr[i].b = pr.x; nr[i].h = pr.y; nr[i].sh = pr.z; ok = ok && pr.w != 0;
      }
    }
    if (ok) {
      if constexpr (FLAT && OUT4 && SATP == 3 && !RES) {
        if (reduce_shifts_by_four(nm, true)) {
#pragma unroll
          for (int i = 0; i < 4; ++i) nm[i].sh -= 4;
          requant8_flat<RES, MSIGNED, RSIGNED, OUT4, false, 4, true>(a, nm, nr, wx, total, lo, hi);
          return;
        }
      }
      if (FLAT) requant8_flat<RES, MSIGNED, RSIGNED, OUT4, false, SATP, true>(a, nm, nr, wx, total, lo, hi);
      else requant8_pixels<RES, MSIGNED, RSIGNED, OUT4, false, SATP, true>(a, nm, nr, wx, words, lo, hi);
      return;
    }
  }
  // two separate loops, so that the common one carries none of the 64-bit form's instructions
  if (FLAT) {
    if constexpr (OUT4 && SATP == 3 && !RES) {
      if (!slow && reduce_shifts_by_four(m, true)) {
#pragma unroll
        for (int i = 0; i < 4; ++i) m[i].sh -= 4;
        requant8_flat<RES, MSIGNED, RSIGNED, OUT4, false, 4>(a, m, r, wx, total, lo, hi);
        return;
      }
    }
    if (slow) requant8_flat<RES, MSIGNED, RSIGNED, OUT4, true, 0>(a, m, r, wx, total, lo, hi);
    else requant8_flat<RES, MSIGNED, RSIGNED, OUT4, false, SATP>(a, m, r, wx, total, lo, hi);
  } else {
    if (slow) requant8_pixels<RES, MSIGNED, RSIGNED, OUT4, true, 0>(a, m, r, wx, words, lo, hi);
    else requant8_pixels<RES, MSIGNED, RSIGNED, OUT4, false, SATP>(a, m, r, wx, words, lo, hi);
  }
}

// ---- the flat form behind a bulk-copy pipeline -------------------------------------------------
// For large tensors.  A persistent block walks chunks of U * 256 consecutive words.  One thread keeps
// kEltStages - 1 chunks ahead with bulk asynchronous copies (global -> shared, completion counted on an
// mbarrier), so the bytes in flight per SM depend neither on registers nor on occupancy; all threads read their
// words from shared memory, requantize and store straight to global memory.  Every wait is bounded: after the
// budget the block records HQ_DEV_TIMEOUT_ELTWISE, waits (bounded) for its copies in flight and returns.
constexpr int kEltStages = 4;
constexpr unsigned long long kEltWaitNs = 2000000000ull;

struct EltPipe {
  unsigned long long full[kEltStages];
  unsigned long long empty[kEltStages];
  volatile unsigned abort_flag;
};

__device__ __forceinline__ unsigned esmem(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ebar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void ebar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void ebar_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool ebar_try_wait(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void ebulk_load(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ unsigned long long elt_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool ebar_wait(unsigned bar, unsigned parity, EltPipe* pipe, uint32_t* status) {
  if (ebar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = elt_ns();
  unsigned spins = 0;
  while (!ebar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0) {
      if (pipe->abort_flag) return false;
      if (elt_ns() - t0 > kEltWaitNs) {
        pipe->abort_flag = 1u;
        if (status) atomicCAS(status, 0u, (uint32_t)HQ_DEV_TIMEOUT_ELTWISE);
        return false;
      }
    }
  }
  return true;
}

template <bool RES, bool MSIGNED, bool RSIGNED, bool OUT4, bool SLOW, int SATP, bool NARROW>
__device__ __forceinline__ void requant8_chunks(const EltArgs& a, const Dy8 (&m)[4], const Dy8 (&r)[4], int wx, long long total,
                                                int lo, int hi, EltPipe* pipe, unsigned char* stage) {
  constexpr int T = 256, U = RES ? 4 : 8;
  constexpr unsigned chunk_bytes = U * T * 4, stage_bytes = RES ? 2u * chunk_bytes : chunk_bytes;
  const int tid = threadIdx.x, lane = tid & 31;
  const long long n_chunks = total / (U * T);
  const unsigned char* mg = (const unsigned char*)a.main_t;
  const unsigned char* rg = (const unsigned char*)a.res;
  auto issue = [&](long long chunk, unsigned slot) {
    const unsigned bar = esmem(&pipe->full[slot]);
    ebar_expect_tx(bar, stage_bytes);
    ebulk_load(esmem(stage + slot * stage_bytes), mg + chunk * chunk_bytes, chunk_bytes, bar);
    if (RES) ebulk_load(esmem(stage + slot * stage_bytes + chunk_bytes), rg + chunk * chunk_bytes, chunk_bytes, bar);
  };
  unsigned issued = 0;                                   // thread 0: chunks handed to the copy engine so far
  if (tid == 0) {
    for (int k = 0; k < kEltStages - 1; ++k) {
      const long long chunk = blockIdx.x + (long long)k * gridDim.x;
      if (chunk < n_chunks) { issue(chunk, (unsigned)k); ++issued; }
    }
  }
  unsigned it = 0;
  bool ok = true;
  for (long long chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x, ++it) {
    const unsigned s = it % kEltStages, ph = (it / kEltStages) & 1u;
    if (tid == 0) {
      const long long nxt = chunk + (long long)(kEltStages - 1) * gridDim.x;
      if (nxt < n_chunks) {
        const unsigned it2 = it + kEltStages - 1, s2 = it2 % kEltStages, use = it2 / kEltStages;
        // the slot's previous use must have been read by every warp (a fresh barrier passes at once)
        ok = ebar_wait(esmem(&pipe->empty[s2]), (use & 1u) ^ 1u, pipe, a.status);
        if (ok) { issue(nxt, s2); ++issued; }
      }
    }
    unsigned w = 1u;
    if (lane == 0) w = (ok && ebar_wait(esmem(&pipe->full[s]), ph, pipe, a.status)) ? 1u : 0u;
    w = __shfl_sync(0xffffffffu, w, 0);
    if (!w) { ok = false; break; }
    const unsigned* ms = (const unsigned*)(stage + s * stage_bytes) + tid;
    const unsigned* rs = (const unsigned*)(stage + s * stage_bytes + chunk_bytes) + tid;
    void* dst0 = out_word<OUT4>(a, chunk * (U * T) + tid);
    unsigned mw[U], rw[U];
#pragma unroll
    for (int u = 0; u < U; ++u) { mw[u] = ms[u * T]; rw[u] = RES ? rs[u * T] : 0u; }
    __syncwarp();
    if (lane == 0) ebar_arrive(esmem(&pipe->empty[s]));     // the words are in registers: the slot may be refilled
#pragma unroll
    for (int u = 0; u < U; ++u)
      requant8_word<RES, MSIGNED, RSIGNED, OUT4, SLOW, SATP, NARROW>(
          a, m, r, wx, mw[u], rw[u], OUT4 ? (void*)((unsigned short*)dst0 + u * T) : (void*)((unsigned*)dst0 + u * T), lo, hi);
  }
  if (ok) {
    // words after the last full chunk: plain loads, spread over the blocks
    const unsigned* mp = (const unsigned*)a.main_t;
    const unsigned* rp = (const unsigned*)a.res;
    for (long long i = n_chunks * (U * T) + (long long)blockIdx.x * T + tid; i < total; i += (long long)gridDim.x * T)
      requant8_word<RES, MSIGNED, RSIGNED, OUT4, SLOW, SATP, NARROW>(a, m, r, wx, __ldg(mp + i), RES ? __ldg(rp + i) : 0u,
                                                                     out_word<OUT4>(a, i), lo, hi);
  } else if (tid == 0) {
    // gave up: the copies already started must land before the block's shared memory is released
    for (unsigned q = it; q < issued; ++q) {
      const unsigned long long t0 = elt_ns();
      while (!ebar_try_wait(esmem(&pipe->full[q % kEltStages]), (q / kEltStages) & 1u)) {
        if (elt_ns() - t0 > kEltWaitNs) break;
      }
    }
  }
}

template <bool RES, bool MSIGNED, bool RSIGNED, bool OUT4, int SATP>
__global__ void __launch_bounds__(256, RES ? 3 : 5) requant8_staged_kernel(EltArgs a, int words, int lo, int hi) {
  extern __shared__ __align__(128) unsigned char stage[];
  __shared__ EltPipe pipe;
  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int k = 0; k < kEltStages; ++k) { ebar_init(esmem(&pipe.full[k]), 1u); ebar_init(esmem(&pipe.empty[k]), 256 / 32); }
    pipe.abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int wx = tid & (words - 1);           // word (4 channels) of the pixel; words is a power of two <= 256
  const long long total = a.pixels * words;
  Dy8 m[4], r[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = make_dy8(__ldg(a.mb + 4 * wx + i), __ldg(a.mc + 4 * wx + i));
    if (RES) r[i] = make_dy8(__ldg(a.rb + 4 * wx + i), __ldg(a.rc + 4 * wx + i));
    else r[i] = m[i];
  }
  bool slow = false;
#pragma unroll
  for (int i = 0; i < 4; ++i) slow = slow || m[i].c < 9 || (RES && r[i].c < 9);
  // the form is chosen per warp, so that a warp's lanes stay together through the pipeline's hand-shakes
  slow = __any_sync(0xffffffffu, slow);
  bool narrow = false;
  Dy8 nm[4], nr[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { nm[i] = m[i]; nr[i] = r[i]; }
  if (a.m_narrow && (!RES || a.r_narrow)) {
    narrow = true;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int4 pm = __ldg((const int4*)a.m_narrow + 4 * wx + i);
      nm[i].b = pm.x; nm[i].h = pm.y; nm[i].sh = pm.z; nm[i].c = 0; narrow = narrow && pm.w != 0;
      nr[i] = nm[i];
      if (RES) {
        const int4 pr = __ldg((const int4*)a.r_narrow + 4 * wx + i);
        nr[i].b = pr.x; nr[i].h = pr.y; nr[i].sh = pr.z; narrow = narrow && pr.w != 0;
      }
    }
  }
  narrow = __all_sync(0xffffffffu, narrow);
  if constexpr (OUT4 && SATP == 3 && !RES) {
    // high-nibble packing, chosen per warp like the other forms
    const bool nib = __all_sync(0xffffffffu, narrow ? reduce_shifts_by_four(nm, true) : reduce_shifts_by_four(m, !slow));
    if (nib) {
#pragma unroll
      for (int i = 0; i < 4; ++i) { nm[i].sh -= 4; m[i].sh -= 4; }
      if (narrow) requant8_chunks<RES, MSIGNED, RSIGNED, OUT4, false, 4, true>(a, nm, nr, wx, total, lo, hi, &pipe, stage);
      else requant8_chunks<RES, MSIGNED, RSIGNED, OUT4, false, 4, false>(a, m, r, wx, total, lo, hi, &pipe, stage);
      return;
    }
  }
  if (narrow) requant8_chunks<RES, MSIGNED, RSIGNED, OUT4, false, SATP, true>(a, nm, nr, wx, total, lo, hi, &pipe, stage);
  else if (slow) requant8_chunks<RES, MSIGNED, RSIGNED, OUT4, true, 0, false>(a, m, r, wx, total, lo, hi, &pipe, stage);
  else requant8_chunks<RES, MSIGNED, RSIGNED, OUT4, false, SATP, false>(a, m, r, wx, total, lo, hi, &pipe, stage);
}

template <bool RES, bool MSIGNED, bool RSIGNED, bool OUT4, int SATP>
cudaError_t launch_requant8_form(const EltArgs& a, dim3 grid, dim3 block, int words, int lo, int hi, int sm_count, cudaStream_t s) {
  if (words <= 256 && (words & (words - 1)) == 0) {
    const long long total = a.pixels * words, per_block = 256 * (RES ? 4 : 8);
    const long long blocks = (total + per_block - 1) / per_block, cap = (long long)sm_count * 16;
    if (total / per_block >= 8ll * sm_count) {      // large: the bulk-copy pipeline, three or five persistent blocks per SM
      const size_t smem = (size_t)kEltStages * per_block * 4 * (RES ? 2 : 1);
      requant8_staged_kernel<RES, MSIGNED, RSIGNED, OUT4, SATP><<<sm_count * (RES ? 3 : 5), 256, smem, s>>>(a, words, lo, hi);
      return cudaGetLastError();
    }
    requant8_kernel<RES, MSIGNED, RSIGNED, OUT4, SATP, true><<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, s>>>(a, words, lo, hi);
  } else {
    requant8_kernel<RES, MSIGNED, RSIGNED, OUT4, SATP, false><<<grid, block, 0, s>>>(a, words, lo, hi);
  }
  return cudaGetLastError();
}

template <bool RES, bool MSIGNED, bool RSIGNED>
cudaError_t launch_requant8(const EltArgs& a, dim3 grid, dim3 block, int words, int lo, int hi, int sm_count, cudaStream_t s) {
  if (a.out_bits == 4 && lo == 0 && hi == 15) return launch_requant8_form<RES, MSIGNED, RSIGNED, true, 3>(a, grid, block, words, lo, hi, sm_count, s);
  if (a.out_bits == 4) return launch_requant8_form<RES, MSIGNED, RSIGNED, true, 0>(a, grid, block, words, lo, hi, sm_count, s);
  if (lo == 0 && hi == 15) return launch_requant8_form<RES, MSIGNED, RSIGNED, false, 5>(a, grid, block, words, lo, hi, sm_count, s);
  if (lo == 0 && hi == 255) return launch_requant8_form<RES, MSIGNED, RSIGNED, false, 1>(a, grid, block, words, lo, hi, sm_count, s);
  if (lo == -128 && hi == 127) return launch_requant8_form<RES, MSIGNED, RSIGNED, false, 2>(a, grid, block, words, lo, hi, sm_count, s);
  return launch_requant8_form<RES, MSIGNED, RSIGNED, false, 0>(a, grid, block, words, lo, hi, sm_count, s);
}

// ---- INT32 main operand, 8-bit output: flat form ------------------------------------------------
// A thread owns four consecutive channels: one 16-byte load of accumulators per pixel (and one word of the 8-bit
// residual), one word stored; quads-per-pixel a power of two up to 256, so the flat index keeps a thread on its
// channels.  For 32 <= c the value is hi32(q*b + 2^(c-1)) >> (c-32) exactly (the low 32 bits cannot matter once
// at least 32 bits are shifted out); a thread with a smaller shift on one of its channels takes the 64-bit form.
struct Dy32 { int b; long long r0; int sh; };
template <bool RES, bool RSIGNED, int SATP>
__global__ void __launch_bounds__(256) requant32_flat_kernel(EltArgs a, int quads, int lo, int hi) {
  constexpr int T = 256, U = 4;
  const int wx = threadIdx.x & (quads - 1);
  const long long total = a.pixels * quads;
  Dy32 m[4];
  Dy8 r[4];
  bool slow = false;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = __ldg(a.mc + 4 * wx + i);
    m[i].b = __ldg(a.mb + 4 * wx + i); m[i].r0 = 1LL << (c - 1); m[i].sh = c - 32;
    slow = slow || c < 32;
    if (RES) { r[i] = make_dy8(__ldg(a.rb + 4 * wx + i), __ldg(a.rc + 4 * wx + i)); slow = slow || r[i].c < 9; }
    else r[i] = make_dy8(0, 40);
  }
  const int4* mp = (const int4*)a.main_t + threadIdx.x;
  const unsigned* rp = RES ? (const unsigned*)a.res + threadIdx.x : nullptr;
  unsigned* op = (unsigned*)a.out + threadIdx.x;
  auto one = [&](const int4& q, unsigned rw, unsigned* dst) {
    const int acc[4] = {q.x, q.y, q.z, q.w};
    int sv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (!slow) {
        sv[i] = (int)(((long long)acc[i] * (long long)m[i].b + m[i].r0) >> 32) >> m[i].sh;
        if (RES) sv[i] += dn8<RSIGNED>(__byte_perm(rw, 0u, 0x0444u | ((unsigned)i << 12)), r[i]);
      } else {
        const unsigned rbyte = (rw >> (8 * i)) & 0xFFu;
        long long t = hq_dn(acc[i], m[i].b, m[i].sh + 32);
        if (RES) t += hq_dn(RSIGNED ? (int)(signed char)rbyte : (int)rbyte, __ldg(a.rb + 4 * wx + i), r[i].c);
        sv[i] = (int)(t < (long long)lo ? (long long)lo : (t > (long long)hi ? (long long)hi : t));
      }
    }
    if (SATP != 0) {
      unsigned w23, w;
      if (SATP == 1) {
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(sv[3]), "r"(sv[2]), "r"(0));
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(sv[1]), "r"(sv[0]), "r"(w23));
      } else {
        asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w23) : "r"(sv[3]), "r"(sv[2]), "r"(0));
        asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(sv[1]), "r"(sv[0]), "r"(w23));
      }
      *dst = w;
    } else {
      unsigned w = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) w |= (unsigned)(min(max(sv[i], lo), hi) & 0xFF) << (8 * i);
      *dst = w;
    }
  };
  const long long trip = (long long)gridDim.x * (U * T);
  for (long long base = (long long)blockIdx.x * (U * T); base < total; base += trip) {
    if (base + U * T <= total) {
      int4 q[U];
      unsigned rw[U];
#pragma unroll
      for (int u = 0; u < U; ++u) q[u] = __ldg(mp + base + u * T);
#pragma unroll
      for (int u = 0; u < U; ++u) rw[u] = RES ? __ldg(rp + base + u * T) : 0u;
#pragma unroll
      for (int u = 0; u < U; ++u) one(q[u], rw[u], op + base + u * T);
    } else {
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (base + u * T + threadIdx.x < total) one(__ldg(mp + base + u * T), RES ? __ldg(rp + base + u * T) : 0u, op + base + u * T);
    }
  }
}

template <bool RES, bool RSIGNED>
cudaError_t launch_requant32(const EltArgs& a, int quads, int lo, int hi, int sm_count, cudaStream_t s) {
  const long long total = a.pixels * quads, per_block = 256 * 4;
  const long long blocks = (total + per_block - 1) / per_block, cap = (long long)sm_count * 16;
  const unsigned grid = (unsigned)(blocks < cap ? blocks : cap);
  if (lo == 0 && hi == 255) requant32_flat_kernel<RES, RSIGNED, 1><<<grid, 256, 0, s>>>(a, quads, lo, hi);
  else if (lo == -128 && hi == 127) requant32_flat_kernel<RES, RSIGNED, 2><<<grid, 256, 0, s>>>(a, quads, lo, hi);
  else requant32_flat_kernel<RES, RSIGNED, 0><<<grid, 256, 0, s>>>(a, quads, lo, hi);
  return cudaGetLastError();
}

// INT32 output (the wide residual stream of Fig. 2: the add of Section 3.3 with its result kept in INT32):
// one thread per element, 64-bit dyadic arithmetic, consecutive threads on consecutive channels.
__global__ void __launch_bounds__(256) residual_add_out32_kernel(EltArgs a) {
  const long long total = a.pixels * a.ch;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const int ch = (int)(e % a.ch);
    long long y = hq_dn(hq_load_elem(a.main_t, e, a.main_bits, a.main_signed), __ldg(a.mb + ch), __ldg(a.mc + ch));
    if (a.res) y += hq_dn(hq_load_elem(a.res, e, a.res_bits, a.res_signed), __ldg(a.rb + ch), __ldg(a.rc + ch));
    ((int*)a.out)[e] = hq_clamp_ll(y, a.relu, a.qmin, a.qmax);
  }
}

// The same for channel counts that are a multiple of four, operands of 8 or 32 bits: a thread owns four channels
// (their pairs stay in registers: the launch makes the thread count a multiple of the quads per pixel), reads
// 16 bytes of an INT32 operand (4 of an 8-bit one) and writes 16 bytes per step, two steps in flight.
template <int MB, int RB>   // operand bits: 8 or 32; RB = 0: no second operand
__global__ void __launch_bounds__(256) residual_add_out32_vec_kernel(EltArgs a) {
  const long long quads = a.pixels * (a.ch >> 2);
  const long long stride = (long long)gridDim.x * blockDim.x;
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= quads) return;
  const int ch = (int)(i % (a.ch >> 2)) << 2;
  int mb[4], mc[4], rb[4], rc[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    mb[j] = a.mb[ch + j]; mc[j] = a.mc[ch + j];
    rb[j] = RB ? a.rb[ch + j] : 0; rc[j] = RB ? a.rc[ch + j] : 1;
  }
  auto load = [&](const void* base, int bits, int is_signed, long long q, int (&v)[4]) {
    if (bits == 32) {
      const int4 t = __ldg((const int4*)base + q);
      v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
      const unsigned t = __ldg((const unsigned*)base + q);
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = is_signed ? (int)(signed char)(t >> (8 * j)) : (int)((t >> (8 * j)) & 0xFFu);
    }
  };
  auto one = [&](long long q) {
    int m[4], r[4] = {0, 0, 0, 0};
    load(a.main_t, MB, a.main_signed, q, m);
    if (RB) load(a.res, RB, a.res_signed, q, r);
    int y[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      long long s = hq_dn(m[j], mb[j], mc[j]);
      if (RB) s += hq_dn(r[j], rb[j], rc[j]);
      y[j] = hq_clamp_ll(s, a.relu, a.qmin, a.qmax);
    }
    ((int4*)a.out)[q] = make_int4(y[0], y[1], y[2], y[3]);
  };
  for (; i + stride < quads; i += 2 * stride) { one(i); one(i + stride); }
  if (i < quads) one(i);
}

// Any channel count: one thread per output byte (one element at 8 bit, two at 4 bit).
__global__ void residual_add_scalar_kernel(EltArgs a) {
  const int per = (a.out_bits == 4) ? 2 : 1;
  const long long total = a.pixels * a.ch / per;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    int q[2] = {0, 0};
    for (int j = 0; j < per; ++j) {
      const long long e = i * per + j;
      const int ch = (int)(e % a.ch);
      long long y = hq_dn(hq_load_elem(a.main_t, e, a.main_bits, a.main_signed), a.mb[ch], a.mc[ch]);
      if (a.res) y += hq_dn(hq_load_elem(a.res, e, a.res_bits, a.res_signed), a.rb[ch], a.rc[ch]);
      q[j] = hq_clamp_ll(y, a.relu, a.qmin, a.qmax);
    }
    if (a.out_bits == 4) ((unsigned char*)a.out)[i] = (unsigned char)((q[0] & 0xF) | ((q[1] & 0xF) << 4));
    else ((unsigned char*)a.out)[i] = (unsigned char)(q[0] & 0xFF);
  }
}

template <int MB, int RB>
cudaError_t launch_vec_out(const EltArgs& a, int groups, int ppb, int grid, cudaStream_t s) {
  if (a.out_bits == 8) residual_add_vec_kernel<MB, RB, 8><<<grid, 256, 0, s>>>(a, groups, ppb);
  else residual_add_vec_kernel<MB, RB, 4><<<grid, 256, 0, s>>>(a, groups, ppb);
  return cudaGetLastError();
}

template <int MB>
cudaError_t launch_vec_res(const EltArgs& a, int groups, int ppb, int grid, cudaStream_t s) {
  if (!a.res) return launch_vec_out<MB, 0>(a, groups, ppb, grid, s);
  switch (a.res_bits) {
    case 4: return launch_vec_out<MB, 4>(a, groups, ppb, grid, s);
    case 8: return launch_vec_out<MB, 8>(a, groups, ppb, grid, s);
    default: return launch_vec_out<MB, 32>(a, groups, ppb, grid, s);
  }
}

// ---- global average pooling -----------------------------------------------------------------
// One thread per (image, 4 channels): 8-bit input read as 32-bit words, coalesced across threads.
__global__ void avgpool_vec4_kernel(const unsigned* __restrict__ in, int n, int hw, int ch, int is_signed,
                                    const int32_t* __restrict__ b, const int32_t* __restrict__ c,
                                    int qmin, int qmax, unsigned* __restrict__ out) {
  const int cg = ch >> 2;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * cg) return;
  const int img = i / cg, g = i - img * cg;
  const unsigned* p = in + (long long)img * hw * cg + g;
  int s0 = 0, s1 = 0, s2 = 0, s3 = 0;
  for (int k = 0; k < hw; ++k) {
    const unsigned v = __ldg(p + (long long)k * cg);
    if (is_signed) {
      s0 += (int)(signed char)(v & 0xFF); s1 += (int)(signed char)((v >> 8) & 0xFF);
      s2 += (int)(signed char)((v >> 16) & 0xFF); s3 += (int)(signed char)(v >> 24);
    } else {
      s0 += (int)(v & 0xFF); s1 += (int)((v >> 8) & 0xFF); s2 += (int)((v >> 16) & 0xFF); s3 += (int)(v >> 24);
    }
  }
  const int sums[4] = {s0, s1, s2, s3};
  unsigned w = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int q = hq_clamp_ll(hq_dn(sums[j], b[4 * g + j], c[4 * g + j]), 0, qmin, qmax);
    w |= (unsigned)(q & 0xFF) << (8 * j);
  }
  out[i] = w;
}

// Same result with more loads in flight: block (64 words, 4 pixel slices) per (image, 64 words); bytes are summed
// as 16-bit lanes of two registers (h*w*255 <= 65535, i.e. up to 257 pixels; signed bytes are offset by 128 and
// corrected at the end), the four slices meet in shared memory.
__global__ void __launch_bounds__(256) avgpool_vec4_sliced_kernel(const unsigned* __restrict__ in, int hw, int ch, int is_signed,
                                                                  const int32_t* __restrict__ b, const int32_t* __restrict__ c,
                                                                  int qmin, int qmax, unsigned* __restrict__ out) {
  __shared__ unsigned part[2][4][64];
  const int cg = ch >> 2;
  const int g = blockIdx.x * 64 + threadIdx.x, img = blockIdx.y;
  unsigned lo = 0, hi = 0;
  if (g < cg) {
    const unsigned* p = in + (long long)img * hw * cg + g;
    const unsigned flip = is_signed ? 0x80808080u : 0u;
    for (int k = threadIdx.y; k < hw; k += 4) {
      const unsigned v = __ldg(p + (long long)k * cg) ^ flip;
      lo += v & 0x00FF00FFu;
      hi += (v >> 8) & 0x00FF00FFu;
    }
  }
  part[0][threadIdx.y][threadIdx.x] = lo;
  part[1][threadIdx.y][threadIdx.x] = hi;
  __syncthreads();
  if (threadIdx.y != 0 || g >= cg) return;
  lo = part[0][0][threadIdx.x] + part[0][1][threadIdx.x] + part[0][2][threadIdx.x] + part[0][3][threadIdx.x];
  hi = part[1][0][threadIdx.x] + part[1][1][threadIdx.x] + part[1][2][threadIdx.x] + part[1][3][threadIdx.x];
  const int off = is_signed ? 128 * hw : 0;
  const int sums[4] = {(int)(lo & 0xFFFFu) - off, (int)(hi & 0xFFFFu) - off, (int)(lo >> 16) - off, (int)(hi >> 16) - off};
  unsigned w = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int q = hq_clamp_ll(hq_dn(sums[j], b[4 * g + j], c[4 * g + j]), 0, qmin, qmax);
    w |= (unsigned)(q & 0xFF) << (8 * j);
  }
  out[(long long)img * cg + g] = w;
}

// 16 channels per thread (one 16-byte load per pixel), SLICES pixel slices per block (two for a 7x7 map, so that
// a thread sums a dozen or more pixels and the block's closing steps weigh little), eight loads of a thread in
// flight at a time; 512 channels per block.  Bytes are summed as 16-bit lanes inside a slice (255 * pixels <= 65535, i.e. up
// to 257 pixels per slice: maps of up to 2056 pixels with eight slices; signed bytes are offset by 128 and corrected at the end).  The slices meet in shared memory and every
// thread then finishes its share of the block's channels, two at a time.
template <int SLICES, bool SIGNED>
__global__ void __launch_bounds__(32 * SLICES) avgpool_vec16_kernel(const uint4* __restrict__ in, int hw, int ch,
                                                                    const int32_t* __restrict__ b, const int32_t* __restrict__ c,
                                                                    int qmin, int qmax, unsigned short* __restrict__ out) {
  __shared__ unsigned part[SLICES][8][32];            // [slice][even / odd byte sums of the four words][channel group]
  const int cg = ch >> 4;
  const int g = blockIdx.x * 32 + threadIdx.x, img = blockIdx.y;
  unsigned acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (g < cg) {
    const uint4* p = in + (long long)img * hw * cg + g;
    constexpr unsigned flip = SIGNED ? 0x80808080u : 0u;
    const int stride = SLICES * cg;
    for (int k0 = threadIdx.y; k0 < hw; k0 += 8 * SLICES) {
      const uint4* q = p + (long long)k0 * cg;
      uint4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        v[u] = k0 + u * SLICES < hw ? __ldg(q + u * stride) : make_uint4(flip, flip, flip, flip);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const unsigned w[4] = {v[u].x ^ flip, v[u].y ^ flip, v[u].z ^ flip, v[u].w ^ flip};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[2 * j] += __byte_perm(w[j], 0u, 0x4240);          // bytes 0 and 2, one per halfword
          acc[2 * j + 1] += __byte_perm(w[j], 0u, 0x4341);      // bytes 1 and 3
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) part[threadIdx.y][j][threadIdx.x] = acc[j];
  __syncthreads();
  // pair index t covers channels 2t and 2t+1 of the block's 512: group t / 8, word (t % 8) / 2, bytes 2 * (t % 2) + {0, 1}
  const int off = SIGNED ? 128 * hw : 0;
  for (int t = threadIdx.y * 32 + threadIdx.x; t < 256; t += 32 * SLICES) {
    const int gl = t >> 3, word = (t & 7) >> 1, half = t & 1;
    const int ch0 = (blockIdx.x * 32 + gl) * 16 + word * 4 + half * 2;
    if (ch0 >= ch) continue;
    // byte 2*half of the word sits in halfword `half` of the even sums, byte 2*half+1 in halfword `half` of the odd sums;
    // a slice's halfword holds at most 257 pixels, the slices are added at full width
    unsigned even = 0, odd = 0;
#pragma unroll
    for (int sl = 0; sl < SLICES; ++sl) {
      even += (part[sl][2 * word][gl] >> (16 * half)) & 0xFFFFu;
      odd += (part[sl][2 * word + 1][gl] >> (16 * half)) & 0xFFFFu;
    }
    const int s0 = (int)even - off, s1 = (int)odd - off;
    const int q0 = hq_clamp_ll(hq_dn(s0, __ldg(b + ch0), __ldg(c + ch0)), 0, qmin, qmax);
    const int q1 = hq_clamp_ll(hq_dn(s1, __ldg(b + ch0 + 1), __ldg(c + ch0 + 1)), 0, qmin, qmax);
    out[((long long)img * ch + ch0) >> 1] = (unsigned short)((q0 & 0xFF) | ((q1 & 0xFF) << 8));
  }
}

template <int SLICES>
void launch_avgpool_vec16(const void* in, int n, int hw, int ch, int in_signed, const int32_t* b, const int32_t* c,
                          int qmin, int qmax, void* out, cudaStream_t s) {
  const dim3 grid((ch / 16 + 31) / 32, n), block(32, SLICES);
  if (in_signed) avgpool_vec16_kernel<SLICES, true><<<grid, block, 0, s>>>((const uint4*)in, hw, ch, b, c, qmin, qmax, (unsigned short*)out);
  else avgpool_vec16_kernel<SLICES, false><<<grid, block, 0, s>>>((const uint4*)in, hw, ch, b, c, qmin, qmax, (unsigned short*)out);
}

__global__ void avgpool_scalar_kernel(const void* in, int n, int hw, int ch, int in_bits, int in_signed,
                                      const int32_t* b, const int32_t* c, int qmin, int qmax,
                                      void* out, int out_bits) {
  const int per = (out_bits == 4) ? 2 : 1;
  const int total = n * ch / per;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  int q[2] = {0, 0};
  for (int j = 0; j < per; ++j) {
    const int e = i * per + j;
    const int img = e / ch, k = e - img * ch;
    long long sum = 0;
    for (int px = 0; px < hw; ++px)
      sum += hq_load_elem(in, ((long long)img * hw + px) * ch + k, in_bits, in_signed);
    q[j] = hq_clamp_ll(hq_dn((int)sum, b[k], c[k]), 0, qmin, qmax);
  }
  if (out_bits == 4) ((unsigned char*)out)[i] = (unsigned char)((q[0] & 0xF) | ((q[1] & 0xF) << 4));
  else ((unsigned char*)out)[i] = (unsigned char)(q[0] & 0xFF);
}

// ---- max pooling ----------------------------------------------------------------------------
// Byte-wise maxima run on the 16-bit pair instructions (a three-input max of two halfword pairs issues like
// a plain integer instruction; the byte-wise intrinsics expand to long sequences): every loaded word is split
// into its even and its odd bytes, widened to halfwords, and the pairs are merged again for the store.
template <bool SIGNED>
struct BytePairMax {
  unsigned e, o;             // running maxima of bytes 0 / 2 and of bytes 1 / 3, one per halfword
  __device__ __forceinline__ static unsigned even(unsigned w) { return hq_prmt(w, 0u, SIGNED ? 0xA280u : 0x4240u); }
  __device__ __forceinline__ static unsigned odd(unsigned w) { return hq_prmt(w, 0u, SIGNED ? 0xB391u : 0x4341u); }
  __device__ __forceinline__ void init(unsigned w) { e = even(w); o = odd(w); }
  __device__ __forceinline__ void add(unsigned w) {
    if (SIGNED) { e = __vmaxs2(e, even(w)); o = __vmaxs2(o, odd(w)); }
    else        { e = __vmaxu2(e, even(w)); o = __vmaxu2(o, odd(w)); }
  }
  __device__ __forceinline__ void add2(unsigned w0, unsigned w1) {
    if (SIGNED) { e = __vimax3_s16x2(e, even(w0), even(w1)); o = __vimax3_s16x2(o, odd(w0), odd(w1)); }
    else        { e = __vimax3_u16x2(e, even(w0), even(w1)); o = __vimax3_u16x2(o, odd(w0), odd(w1)); }
  }
  __device__ __forceinline__ unsigned merged() const { return __byte_perm(e, o, 0x6240); }
};

// One block per (image, output row): no 64-bit index arithmetic per output (a division-heavy flat index is
// instruction-bound); a thread handles 16 channels of one output pixel at a time.  K3: the 3x3 window, fully
// unrolled; rows and columns that fall into the padding are replaced by their nearest valid neighbour, which
// lies inside the same window (pad < k) and leaves the maximum unchanged.
template <bool SIGNED, bool K3>
__global__ void __launch_bounds__(256) maxpool_vec16_kernel(const uint4* __restrict__ in, int h, int w, int cg,
                                                            int k, int stride, int pad, uint4* __restrict__ out, int ho, int wo) {
  const int img = blockIdx.x / ho, oh = blockIdx.x - img * ho;
  const uint4* in_img = in + (long long)img * h * w * cg;
  uint4* out_row = out + ((long long)img * ho + oh) * wo * cg;
  const int row_items = wo * cg;
  if (K3) {
    const int ih1 = oh * stride - pad + 1;                       // centre row of the window
    const int r0 = min(max(ih1 - 1, 0), h - 1), r1 = min(max(ih1, 0), h - 1), r2 = min(max(ih1 + 1, 0), h - 1);
    const uint4* row0 = in_img + (long long)r0 * w * cg;
    const uint4* row1 = in_img + (long long)r1 * w * cg;
    const uint4* row2 = in_img + (long long)r2 * w * cg;
    for (int idx = threadIdx.x; idx < row_items; idx += blockDim.x) {
      const int ow = idx / cg, g = idx - ow * cg;
      const int iw1 = ow * stride - pad + 1;
      const int c0 = min(max(iw1 - 1, 0), w - 1) * cg + g, c1 = min(max(iw1, 0), w - 1) * cg + g,
                c2 = min(max(iw1 + 1, 0), w - 1) * cg + g;
      const uint4 v0 = __ldg(row0 + c0), v1 = __ldg(row0 + c1), v2 = __ldg(row0 + c2);
      const uint4 v3 = __ldg(row1 + c0), v4 = __ldg(row1 + c1), v5 = __ldg(row1 + c2);
      const uint4 v6 = __ldg(row2 + c0), v7 = __ldg(row2 + c1), v8 = __ldg(row2 + c2);
      uint4 m;
#define HQ_MAX9(F) { BytePairMax<SIGNED> a; a.init(v0.F); a.add2(v1.F, v2.F); a.add2(v3.F, v4.F); \
                     a.add2(v5.F, v6.F); a.add2(v7.F, v8.F); m.F = a.merged(); }
      HQ_MAX9(x) HQ_MAX9(y) HQ_MAX9(z) HQ_MAX9(w)
#undef HQ_MAX9
      out_row[idx] = m;
    }
  } else {
    const int r_lo = max(0, pad - oh * stride), r_hi = min(k, h + pad - oh * stride);   // valid filter rows
    for (int idx = threadIdx.x; idx < row_items; idx += blockDim.x) {
      const int ow = idx / cg, g = idx - ow * cg;
      const int s_lo = max(0, pad - ow * stride), s_hi = min(k, w + pad - ow * stride);
      const unsigned init = SIGNED ? 0x80808080u : 0u;
      BytePairMax<SIGNED> mx, my, mz, mw;
      mx.init(init); my.init(init); mz.init(init); mw.init(init);
      for (int r = r_lo; r < r_hi; ++r) {
        const uint4* row = in_img + ((long long)(oh * stride + r - pad) * w + (ow * stride - pad)) * cg + g;
        for (int s = s_lo; s < s_hi; ++s) {
          const uint4 v = __ldg(row + s * cg);
          mx.add(v.x); my.add(v.y); mz.add(v.z); mw.add(v.w);
        }
      }
      out_row[idx] = make_uint4(mx.merged(), my.merged(), mz.merged(), mw.merged());
    }
  }
}

__global__ void maxpool_scalar_kernel(const void* in, int n, int h, int w, int ch, int bits, int is_signed,
                                      int k, int stride, int pad, void* out, int ho, int wo) {
  const long long total = (long long)n * ho * wo * ch;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int cc = (int)(i % ch);
    long long t = i / ch;
    const int ow = (int)(t % wo); t /= wo;
    const int oh = (int)(t % ho);
    const int img = (int)(t / ho);
    int best = bits == 32 ? INT_MIN : is_signed ? -128 : 0;
    for (int r = 0; r < k; ++r) {
      const int ih = oh * stride + r - pad;
      if (ih < 0 || ih >= h) continue;
      for (int s = 0; s < k; ++s) {
        const int iw = ow * stride + s - pad;
        if (iw < 0 || iw >= w) continue;
        const int v = hq_load_elem(in, (((long long)img * h + ih) * w + iw) * ch + cc, bits, is_signed);
        best = v > best ? v : best;
      }
    }
    if (bits == 32) ((int*)out)[i] = best;
    else ((unsigned char*)out)[i] = (unsigned char)(best & 0xFF);
  }
}

}  // namespace

cudaError_t hq_launch_residual_add(const EltArgs& a, int sm_count, cudaStream_t s) {
  if (a.pixels == 0) return cudaSuccess;
  if (a.out_bits == 32) {
    const int quads = a.ch >> 2;
    const bool vec = a.ch % 4 == 0 && (a.main_bits == 8 || a.main_bits == 32) && (!a.res || a.res_bits == 8 || a.res_bits == 32);
    if (vec) {
      // thread count a multiple of the quads per pixel, so that a thread keeps its four channels
      long long blocks = (a.pixels * quads + 255) / 256;
      const long long cap = (long long)sm_count * 16;
      if (blocks > cap) blocks = cap;
      int unit = quads, t = 256;                       // blocks must be a multiple of quads / gcd(quads, 256)
      while (t) { const int r = unit % t; unit = t; t = r; }      // unit = gcd(quads, 256)
      const long long mult = quads / unit;
      blocks = blocks / mult * mult;
      if (blocks >= mult) {
        const int g = (int)blocks;
        const int rbits = a.res ? a.res_bits : 0;
        if (a.main_bits == 32 && rbits == 32) residual_add_out32_vec_kernel<32, 32><<<g, 256, 0, s>>>(a);
        else if (a.main_bits == 32 && rbits == 8) residual_add_out32_vec_kernel<32, 8><<<g, 256, 0, s>>>(a);
        else if (a.main_bits == 32) residual_add_out32_vec_kernel<32, 0><<<g, 256, 0, s>>>(a);
        else if (rbits == 32) residual_add_out32_vec_kernel<8, 32><<<g, 256, 0, s>>>(a);
        else if (rbits == 8) residual_add_out32_vec_kernel<8, 8><<<g, 256, 0, s>>>(a);
        else residual_add_out32_vec_kernel<8, 0><<<g, 256, 0, s>>>(a);
        return cudaGetLastError();
      }
    }
    const long long blocks = (a.pixels * a.ch + 255) / 256, cap = (long long)sm_count * 32;
    residual_add_out32_kernel<<<(int)(blocks < cap ? blocks : cap), 256, 0, s>>>(a);
    return cudaGetLastError();
  }
  // 8-bit operands with a channel count the word mapping covers: 32-bit fast kernel
  const int words = a.ch / 4;
  if (a.main_bits == 8 && (!a.res || a.res_bits == 8) && a.ch % 4 == 0) {
    // more than 256 words per pixel: the fewest blocks along the words, each a whole number of warps wide
    const int xblocks = (words + 255) / 256;
    const int bx = words <= 256 ? words : ((words + xblocks - 1) / xblocks + 31) / 32 * 32;
    int by = 256 / bx; if (by < 1) by = 1;
    dim3 block(bx, by), grid((words + bx - 1) / bx, 1);
    long long gy = (a.pixels + by - 1) / by;
    const long long cap = (long long)sm_count * 16 / grid.x + 1;
    grid.y = (unsigned)(gy < cap ? gy : cap);
    const int lo = a.relu ? (a.qmin > 0 ? a.qmin : 0) : a.qmin, hi = a.qmax;
    const int v = (a.res ? 4 : 0) | (a.main_signed ? 2 : 0) | ((a.res && a.res_signed) ? 1 : 0);
    switch (v) {
      case 0: return launch_requant8<false, false, false>(a, grid, block, words, lo, hi, sm_count, s);
      case 2: return launch_requant8<false, true, false>(a, grid, block, words, lo, hi, sm_count, s);
      case 4: return launch_requant8<true, false, false>(a, grid, block, words, lo, hi, sm_count, s);
      case 5: return launch_requant8<true, false, true>(a, grid, block, words, lo, hi, sm_count, s);
      case 6: return launch_requant8<true, true, false>(a, grid, block, words, lo, hi, sm_count, s);
      default: return launch_requant8<true, true, true>(a, grid, block, words, lo, hi, sm_count, s);
    }
  }
  // INT32 main operand, 8-bit output (and residual, if any): flat kernel when the quads of a pixel divide the block
  if (a.main_bits == 32 && a.out_bits == 8 && (!a.res || a.res_bits == 8) && a.ch % 4 == 0 && words <= 256 &&
      (words & (words - 1)) == 0) {
    const int lo = a.relu ? (a.qmin > 0 ? a.qmin : 0) : a.qmin, hi = a.qmax;
    if (!a.res) return launch_requant32<false, false>(a, words, lo, hi, sm_count, s);
    if (a.res_signed) return launch_requant32<true, true>(a, words, lo, hi, sm_count, s);
    return launch_requant32<true, false>(a, words, lo, hi, sm_count, s);
  }
  const int groups = a.ch / 16;
  if (a.ch % 16 == 0 && groups <= 256) {
    const int ppb = 256 / groups;
    long long blocks = (a.pixels + ppb - 1) / ppb;
    const long long cap = (long long)sm_count * 8;
    const int grid = (int)(blocks < cap ? blocks : cap);
    switch (a.main_bits) {
      case 4: return launch_vec_res<4>(a, groups, ppb, grid, s);
      case 8: return launch_vec_res<8>(a, groups, ppb, grid, s);
      default: return launch_vec_res<32>(a, groups, ppb, grid, s);
    }
  }
  const long long total = a.pixels * a.ch / (a.out_bits == 4 ? 2 : 1);
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)sm_count * 16;
  residual_add_scalar_kernel<<<(int)(blocks < cap ? blocks : cap), 256, 0, s>>>(a);
  return cudaGetLastError();
}

cudaError_t hq_launch_avgpool(const void* in, int n, int h, int w, int ch, int in_bits, int in_signed,
                              const int32_t* b, const int32_t* c, int qmin, int qmax,
                              void* out, int out_bits, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  if (in_bits == 8 && out_bits == 8 && ch % 16 == 0 && h * w <= 8 * 257 && n <= 65535) {
    const int hw = h * w;
    if (hw >= 128) launch_avgpool_vec16<8>(in, n, hw, ch, in_signed, b, c, qmin, qmax, out, s);
    else if (hw >= 64) launch_avgpool_vec16<4>(in, n, hw, ch, in_signed, b, c, qmin, qmax, out, s);
    else launch_avgpool_vec16<2>(in, n, hw, ch, in_signed, b, c, qmin, qmax, out, s);
  } else if (in_bits == 8 && out_bits == 8 && ch % 4 == 0 && h * w <= 257 && n <= 65535) {
    const dim3 grid((ch / 4 + 63) / 64, n), block(64, 4);
    avgpool_vec4_sliced_kernel<<<grid, block, 0, s>>>((const unsigned*)in, h * w, ch, in_signed, b, c, qmin, qmax, (unsigned*)out);
  } else if (in_bits == 8 && out_bits == 8 && ch % 4 == 0) {
    const int total = n * (ch / 4);
    avgpool_vec4_kernel<<<(total + 127) / 128, 128, 0, s>>>((const unsigned*)in, n, h * w, ch, in_signed,
                                                             b, c, qmin, qmax, (unsigned*)out);
  } else {
    const int total = n * ch / (out_bits == 4 ? 2 : 1);
    avgpool_scalar_kernel<<<(total + 127) / 128, 128, 0, s>>>(in, n, h * w, ch, in_bits, in_signed, b, c,
                                                               qmin, qmax, out, out_bits);
  }
  return cudaGetLastError();
}

cudaError_t hq_launch_maxpool(const void* in, int n, int h, int w, int ch, int bits, int is_signed,
                              int k, int stride, int pad, void* out, int ho, int wo, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  if (bits == 8 && ch % 16 == 0 && (long long)n * ho < (1ll << 31) && (long long)wo * (ch / 16) < (1ll << 31)) {
    const uint4* src = (const uint4*)in;
    uint4* dst = (uint4*)out;
    const int cg = ch / 16;
    // the unrolled 3x3 form: with pad <= 1 at most one row / column of a window lies outside the image, next to
    // a valid one of the same window
    const bool k3 = k == 3 && pad <= 1;
    if (is_signed && k3) maxpool_vec16_kernel<true, true><<<n * ho, 256, 0, s>>>(src, h, w, cg, k, stride, pad, dst, ho, wo);
    else if (is_signed)  maxpool_vec16_kernel<true, false><<<n * ho, 256, 0, s>>>(src, h, w, cg, k, stride, pad, dst, ho, wo);
    else if (k3)         maxpool_vec16_kernel<false, true><<<n * ho, 256, 0, s>>>(src, h, w, cg, k, stride, pad, dst, ho, wo);
    else                 maxpool_vec16_kernel<false, false><<<n * ho, 256, 0, s>>>(src, h, w, cg, k, stride, pad, dst, ho, wo);
  } else {
    const long long total = (long long)n * ho * wo * ch;
    long long blocks = (total + 255) / 256;
    if (blocks > (1 << 20)) blocks = 1 << 20;
    maxpool_scalar_kernel<<<(int)blocks, 256, 0, s>>>(in, n, h, w, ch, bits, is_signed, k, stride, pad, out, ho, wo);
  }
  return cudaGetLastError();
}
