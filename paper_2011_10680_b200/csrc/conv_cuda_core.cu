// CUDA-core convolution path: used for shapes the tensor-core kernel does not cover (channel
// counts that are not a multiple of 32 bytes, tiny problems) and when the caller forces it.
// One thread per (output pixel, output channel); the contraction of Eq. 3 runs on dp4a (four
// 8-bit products per instruction, INT32 accumulate) when the channel count allows 32-bit reads,
// else element by element.  The epilogue is the same integer sequence as everywhere: bias,
// dyadic multiply-shift (Eq. 4), residual branch (Section 3.3), ReLU, clamp, pack.
#include "hq_internal.cuh"

namespace {

__device__ __forceinline__ int dp4a_us(unsigned a, unsigned b, int c) {   // u8 x s8
  int d;
  asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ int dp4a_ss(unsigned a, unsigned b, int c) {   // s8 x s8
  int d;
  asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// sign-extend the four 4-bit fields that sit in the low nibble of each byte
__device__ __forceinline__ unsigned sext_nibbles(unsigned t) { return t | ((t & 0x08080808u) * 0x1Eu); }

template <int BITS>
__global__ void __launch_bounds__(256) conv_cuda_core_kernel(ConvArgs a) {
  const long long total = (long long)a.n * a.ho * a.wo * a.cout;
  const int epw = (BITS == 8) ? 4 : 8;                    // elements per 32-bit word
  const bool word_path = (a.cin % epw) == 0;
  const int out_per = (a.out_bits == 4) ? 2 : 1;          // one thread writes one output byte / word
  const long long nthreads = total / out_per;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nthreads;
       i += (long long)gridDim.x * blockDim.x) {
    int q[2] = {0, 0};
    for (int j = 0; j < out_per; ++j) {
      const long long o = i * out_per + j;
      const int oc = (int)(o % a.cout);
      long long t = o / a.cout;
      const int ow = (int)(t % a.wo); t /= a.wo;
      const int oh = (int)(t % a.ho);
      const int img = (int)(t / a.ho);
      int acc = 0;
      for (int r = 0; r < a.kh; ++r) {
        const int ih = oh * a.stride + r - a.pad;
        if (ih < 0 || ih >= a.h) continue;
        for (int s = 0; s < a.kw; ++s) {
          const int iw = ow * a.stride + s - a.pad;
          if (iw < 0 || iw >= a.w) continue;
          const long long xe = (((long long)img * a.h + ih) * a.w + iw) * a.cin;
          const long long we = (((long long)oc * a.kh + r) * a.kw + s) * a.cin;
          if (word_path) {
            const unsigned* xp = (const unsigned*)((const unsigned char*)a.in + xe * BITS / 8);
            const unsigned* wp = (const unsigned*)((const unsigned char*)a.wgt + we * BITS / 8);
            const int words = a.cin / epw;
            for (int k = 0; k < words; ++k) {
              const unsigned xv = __ldg(xp + k), wv = __ldg(wp + k);
              if (BITS == 8) {
                acc = a.in_signed ? dp4a_ss(xv, wv, acc) : dp4a_us(xv, wv, acc);
              } else {
                unsigned xl = xv & 0x0F0F0F0Fu, xh = (xv >> 4) & 0x0F0F0F0Fu;
                const unsigned wl = sext_nibbles(wv & 0x0F0F0F0Fu), wh = sext_nibbles((wv >> 4) & 0x0F0F0F0Fu);
                if (a.in_signed) {
                  xl = sext_nibbles(xl); xh = sext_nibbles(xh);
                  acc = dp4a_ss(xl, wl, acc); acc = dp4a_ss(xh, wh, acc);
                } else {
                  acc = dp4a_us(xl, wl, acc); acc = dp4a_us(xh, wh, acc);
                }
              }
            }
          } else {
            for (int k = 0; k < a.cin; ++k)
              acc += hq_load_elem(a.in, xe + k, BITS, a.in_signed) * hq_load_elem(a.wgt, we + k, BITS, 1);
          }
        }
      }
      const int tsum = acc + (a.bias ? a.bias[oc] : 0);
      if (a.out_bits == 32) { ((int*)a.out)[o] = tsum; continue; }
      long long y = hq_dn(tsum, a.b[oc], a.c[oc]);
      if (a.res) y += hq_dn(hq_load_elem(a.res, o, a.res_bits, a.res_signed), a.rb[oc], a.rc[oc]);
      q[j] = hq_clamp_ll(y, a.relu, a.qmin, a.qmax);
    }
    if (a.out_bits == 8) ((unsigned char*)a.out)[i] = (unsigned char)(q[0] & 0xFF);
    else if (a.out_bits == 4) ((unsigned char*)a.out)[i] = (unsigned char)((q[0] & 0xF) | ((q[1] & 0xF) << 4));
  }
}

}  // namespace

cudaError_t hq_launch_conv_cuda_core(const ConvArgs& a, cudaStream_t s) {
  const long long total = (long long)a.n * a.ho * a.wo * a.cout / (a.out_bits == 4 ? 2 : 1);
  if (total == 0) return cudaSuccess;
  long long blocks = (total + 255) / 256;
  if (blocks > (1 << 22)) blocks = 1 << 22;
  if (a.in_bits == 8) conv_cuda_core_kernel<8><<<(int)blocks, 256, 0, s>>>(a);
  else conv_cuda_core_kernel<4><<<(int)blocks, 256, 0, s>>>(a);
  return cudaGetLastError();
}
