// Inception-style concatenation with a dyadic rescale per branch (Appendix E, "Concatenation Layer"):
//   q_a[n, h, w, off_i + k] = clamp(dn(q_i[n, h, w, k], b_i[k], c_i[k])),   dn(q, b, c) = (q*b + 2^(c-1)) >> c,
// i.e. every branch (the convolution branches as stored 8- or 4-bit tensors or INT32 accumulators, the pooling
// branch as an INT32 tensor) is brought to the output scale by its own DN pairs and lands beside the others along
// the channel axis.  Memory bound: every operand is read once, the output written once, in ONE launch for all
// branches.  A thread owns 16 consecutive channels of one branch at one pixel: a 16-byte (8-bit input), 64-byte
// (INT32 input) or 8-byte (4-bit input) read, sixteen exact requantizations, one 16-byte (or 8-byte, 4-bit
// output) write; neighbouring threads take neighbouring channel groups of the same output pixel, so the writes of
// a warp cover contiguous bytes of the concatenated row.  Integer arithmetic only.
#include "hq_internal.cuh"

namespace {

struct ConcatBranch {
  const void* in; const int32_t* b; const int32_t* c;
  int32_t bits, is_signed, ch, ch_off;
  int32_t unit0;      // index of this branch's first 16-channel group among a pixel's groups
  int32_t vec;        // 1: rows and dyadic arrays allow 16-byte accesses (ch % 16 == 0, aligned arrays)
};

struct ConcatArgs {
  ConcatBranch br[HQ_CONCAT_MAX_BRANCHES];
  int32_t n_br, units_per_px, out_ch, out_bits, relu, qmin, qmax;
  long long pixels;
  void* out;
};

// One value: the 64-bit definition, or for c >= 33 its high-word form (the rounding constant 2^(c-1) is then a
// multiple of 2^32, so it adds to the high word of q*b without a carry from the low word).
__device__ __forceinline__ int concat_dn(int q, int b, int c, int relu, int qmin, int qmax) {
  if (c >= 33) {
    int y = (__mulhi(q, b) + (1 << (c - 33))) >> (c - 32);      // |q*b| < 2^62: the sum stays inside INT32
    if (relu) y = max(y, 0);
    return min(max(y, qmin), qmax);
  }
  return hq_clamp_ll(hq_dn(q, b, c), relu, qmin, qmax);
}

__global__ void __launch_bounds__(256) concat_requant_kernel(const __grid_constant__ ConcatArgs a) {
  const long long total = a.pixels * (long long)a.units_per_px;
  for (long long t = (long long)blockIdx.x * 256 + threadIdx.x; t < total; t += (long long)gridDim.x * 256) {
    const long long px = t / a.units_per_px;
    const int u = (int)(t - px * a.units_per_px);
    int i = 0;
#pragma unroll
    for (int j = 1; j < HQ_CONCAT_MAX_BRANCHES; ++j)
      if (j < a.n_br && u >= a.br[j].unit0) i = j;
    const ConcatBranch& B = a.br[i];
    const int k0 = (u - B.unit0) * 16;
    const int nk = min(16, B.ch - k0);
    const long long e0 = px * (long long)B.ch + k0;              // first input element of this thread
    int q[16], bb[16], cc[16];
    if (B.vec) {
      const int4* bp = (const int4*)(B.b + k0);
      const int4* cp = (const int4*)(B.c + k0);
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const int4 x = __ldg(bp + v), y = __ldg(cp + v);
        bb[4 * v] = x.x; bb[4 * v + 1] = x.y; bb[4 * v + 2] = x.z; bb[4 * v + 3] = x.w;
        cc[4 * v] = y.x; cc[4 * v + 1] = y.y; cc[4 * v + 2] = y.z; cc[4 * v + 3] = y.w;
      }
      if (B.bits == 8) {
        const uint4 x = *(const uint4*)((const unsigned char*)B.in + e0);
        const unsigned w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const unsigned byte = (w[j >> 2] >> (8 * (j & 3))) & 0xFFu;
          q[j] = B.is_signed ? (int)(signed char)byte : (int)byte;
        }
      } else if (B.bits == 32) {
        const int4* ip = (const int4*)((const int*)B.in + e0);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const int4 x = ip[v];
          q[4 * v] = x.x; q[4 * v + 1] = x.y; q[4 * v + 2] = x.z; q[4 * v + 3] = x.w;
        }
      } else {
        const uint2 x = *(const uint2*)((const unsigned char*)B.in + (e0 >> 1));
        const unsigned w[2] = {x.x, x.y};
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          int v = (int)((w[j >> 3] >> (4 * (j & 7))) & 0xFu);
          if (B.is_signed && (v & 8)) v -= 16;
          q[j] = v;
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (j < nk) { q[j] = hq_load_elem(B.in, e0 + j, B.bits, B.is_signed); bb[j] = B.b[k0 + j]; cc[j] = B.c[k0 + j]; }
        else { q[j] = 0; bb[j] = 0; cc[j] = 33; }
      }
    }
    int o[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) o[j] = concat_dn(q[j], bb[j], cc[j], a.relu, a.qmin, a.qmax);
    const long long o0 = px * (long long)a.out_ch + B.ch_off + k0;   // first output element
    if (a.out_bits == 8) {
      unsigned char* op = (unsigned char*)a.out + o0;
      if (nk == 16 && (o0 & 15) == 0) {
        unsigned w[4];
#pragma unroll
        for (int v = 0; v < 4; ++v)
          w[v] = (unsigned)(o[4 * v] & 0xFF) | ((unsigned)(o[4 * v + 1] & 0xFF) << 8) |
                 ((unsigned)(o[4 * v + 2] & 0xFF) << 16) | ((unsigned)(o[4 * v + 3] & 0xFF) << 24);
        *(uint4*)op = make_uint4(w[0], w[1], w[2], w[3]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) if (j < nk) op[j] = (unsigned char)o[j];
      }
    } else {
      // 4-bit output: channel counts and offsets are even, so a byte's two nibbles belong to this thread
      unsigned char* op = (unsigned char*)a.out + (o0 >> 1);
      if (nk == 16 && ((o0 >> 1) & 7) == 0) {
        unsigned w[2] = {0u, 0u};
#pragma unroll
        for (int j = 0; j < 16; ++j) w[j >> 3] |= (unsigned)(o[j] & 0xF) << (4 * (j & 7));
        *(uint2*)op = make_uint2(w[0], w[1]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; j += 2)
          if (j < nk) op[j >> 1] = (unsigned char)((o[j] & 0xF) | ((o[j + 1] & 0xF) << 4));
      }
    }
  }
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
  int off = 0, units = 0;
  for (int i = 0; i < n_branches; ++i) {
    const hq_tensor& t = branches[i];
    if (!t.data || !rescale[i].b || !rescale[i].c) return HQ_ERR_INVALID_ARG;
    if (t.bits != 4 && t.bits != 8 && t.bits != 32) return HQ_ERR_INVALID_ARG;
    if (t.n != out->n || t.h != out->h || t.w != out->w || t.c < 1) return HQ_ERR_INVALID_ARG;
    if (t.bits == 4 && (t.c & 1)) return HQ_ERR_INVALID_ARG;
    if (out->bits == 4 && (t.c & 1)) return HQ_ERR_UNSUPPORTED;   // a byte of the output would span two branches
    if (!al16(t.data)) return HQ_ERR_ALIGNMENT;
    ConcatBranch& B = a.br[i];
    B.in = t.data; B.b = rescale[i].b; B.c = rescale[i].c;
    B.bits = t.bits; B.is_signed = t.bits == 32 ? 1 : t.is_signed; B.ch = t.c; B.ch_off = off; B.unit0 = units;
    B.vec = (t.c % 16 == 0 && al16(B.b) && al16(B.c)) ? 1 : 0;
    off += t.c;
    units += (t.c + 15) / 16;
  }
  if (off != out->c) return HQ_ERR_INVALID_ARG;
  a.n_br = n_branches; a.units_per_px = units; a.out_ch = out->c; a.out_bits = out->bits;
  a.relu = relu; a.qmin = qmin; a.qmax = qmax;
  a.pixels = (long long)out->n * out->h * out->w;
  a.out = out->data;
  const long long total = a.pixels * units;
  if (total == 0) return HQ_OK;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)h->sm_count * 16;                // grid-stride beyond eight blocks per SM twice over
  if (blocks > cap) blocks = cap;
  concat_requant_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(a);
  return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
