// Internal declarations shared by the translation units of libhq.so (CUDA side only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hq.h"

// Device-side status word values (written by a kernel that gave up a bounded wait).
enum : uint32_t {
  HQ_DEV_OK = 0,
  HQ_DEV_TIMEOUT_PRODUCER = 1,   // TMA producer waited too long for a free stage
  HQ_DEV_TIMEOUT_MMA = 2,        // MMA issuer waited too long for operands or a free accumulator
  HQ_DEV_TIMEOUT_EPILOGUE = 3,   // epilogue waited too long for a finished accumulator
  HQ_DEV_TIMEOUT_DRAIN = 4,      // teardown waited too long for work in flight
  HQ_DEV_TIMEOUT_ELTWISE = 5     // a streaming kernel waited too long for a staged chunk or a free stage
};

struct hq_handle {
  int32_t device;
  int32_t conv_path;          // 0 auto, 1 CUDA cores only, 2 tensor cores or fail
  int32_t sm_count;
  uint32_t* dev_status;       // one word in device memory, sticky until hq_sync
  void* workspace;            // scratch owned by the handle (grown on demand, never inside a capture)
  size_t workspace_bytes;
  void* narrow_pairs;         // 2 x kNarrowChannels x 16 bytes: narrow pairs of a single element-wise call's two operands
  int32_t tile_order;         // tensor-core convolutions walk their pixel tiles 0: first to last, 1: last to first
};
constexpr int kNarrowChannels = 4096;

// ------------------------------------------------------------------------------------------
// Dyadic arithmetic (Eq. 4): dn(q, b, c) = (q*b + 2^(c-1)) >> c, 64-bit product, arithmetic shift.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ long long hq_dn(int q, int b, int c) {
  return ((long long)q * (long long)b + (1LL << (c - 1))) >> c;
}

// Byte permute with the full PTX selector: bit 3 of a selector nibble replicates the selected byte's sign bit over the
// target byte.  (The __byte_perm intrinsic keeps three bits per nibble and cannot sign-extend.)
__device__ __forceinline__ unsigned hq_prmt(unsigned a, unsigned b, unsigned sel) {
  unsigned d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// Element access for dense tensors with 4, 8 or 32 bits per element (even element = low nibble).
__device__ __forceinline__ int hq_load_elem(const void* base, long long idx, int bits, int is_signed) {
  if (bits == 32) return ((const int*)base)[idx];
  if (bits == 8) return is_signed ? (int)((const signed char*)base)[idx] : (int)((const unsigned char*)base)[idx];
  const unsigned byte = ((const unsigned char*)base)[idx >> 1];
  int v = (idx & 1) ? (int)(byte >> 4) : (int)(byte & 0xF);
  if (is_signed && (v & 8)) v -= 16;
  return v;
}

__device__ __forceinline__ int hq_clamp_ll(long long y, int relu, int qmin, int qmax) {
  if (relu && y < 0) y = 0;
  if (y < (long long)qmin) y = qmin;
  if (y > (long long)qmax) y = qmax;
  return (int)y;
}

// Launchers implemented in the other translation units.  All return a cudaError_t from the launch.
struct ConvArgs {
  const void* in; int32_t n, h, w, cin, in_bits, in_signed;
  const void* wgt; int32_t cout, kh, kw, stride, pad;
  const int32_t* bias; const int32_t* b; const int32_t* c;
  const void* res; int32_t res_bits, res_signed; const int32_t* rb; const int32_t* rc;
  int32_t relu, qmin, qmax;
  void* out; int32_t ho, wo, out_bits, out_signed;
  // internal (zero for calls that come straight from the ABI):
  const void* res_narrow;    // per-channel narrow residual pairs prepared by hq_launch_residual_narrow, or NULL
  int32_t res_narrow_fresh;  // nonzero: the pairs come from the launch just before on the same stream (the kernel waits for it)
  const void* wgt_widened;   // weights as the lowered form wants them, prepared once by a network, or NULL: 4-bit weights widened
                             // to one byte per value; for the first-layer form the virtual-channel weights and constants
  int32_t pad_after_delta;   // padding after the last row/column minus `pad`
  // byte pitches of the activation tensor along W, H and N when it is not dense (0: dense NHWC).  A W pitch
  // below cin bytes makes neighbouring "pixels" overlap: a pixel is then a window of adjacent stored pixels.
  long long pitch_w, pitch_h, pitch_n;
};

struct EltArgs {
  const void* main_t; int32_t main_bits, main_signed; const int32_t* mb; const int32_t* mc;
  const void* res; int32_t res_bits, res_signed; const int32_t* rb; const int32_t* rc;
  long long pixels; int32_t ch; int32_t relu, qmin, qmax;
  void* out; int32_t out_bits;
  // optional narrow pairs {m, a, s, valid} per channel for 8-bit operands (see hq_launch_residual_narrow), or NULL
  const void* m_narrow; const void* r_narrow;
  uint32_t* status;          // the handle's device status word (bounded waits report here), or NULL
};

cudaError_t hq_launch_conv_cuda_core(const ConvArgs& a, cudaStream_t s);
bool hq_conv_tc_init();
bool hq_conv_tc_supported(const ConvArgs& a);
// True for a layer the direct kernel declines although its shape is supported: it would fetch a tensor below
// 128 KiB through an im2col-mode map.  Such a layer runs in its lowered (patch-matrix) form.
bool hq_conv_tc_small_im2col(const ConvArgs& a);
// Tensor-core path; returns HQ_OK, HQ_ERR_UNSUPPORTED (nothing was launched) or HQ_ERR_CUDA.
hq_status hq_launch_conv_tc(hq_handle* h, const ConvArgs& a, cudaStream_t s);
// Fills `out` (channels x 16 bytes) with the narrow residual pairs of an 8-bit residual branch.
cudaError_t hq_launch_residual_narrow(const int32_t* rb, const int32_t* rc, int res_signed, int channels, void* out,
                                      cudaStream_t s);
// The same for the two operands of an element-wise call in one launch (`out1` NULL: first operand only).
cudaError_t hq_launch_residual_narrow2(const int32_t* b0, const int32_t* c0, int signed0, void* out0,
                                       const int32_t* b1, const int32_t* c1, int signed1, void* out1, int channels,
                                       cudaStream_t s);
// Lowered path for thin first layers: patch matrix + padded weights in scratch, then the tensor-core kernel.
bool hq_conv_lowering_applies(const ConvArgs& a);
size_t hq_conv_lowering_bytes(const ConvArgs& a);
hq_status hq_launch_conv_lowered(hq_handle* h, const ConvArgs& a, void* scratch, cudaStream_t s);
// 7x7 / stride 2 / 3-channel first layer as a 4x4 stride-1 conv over a space-to-depth copy of the image.
bool hq_conv_s2d_applies(const ConvArgs& a);
size_t hq_conv_s2d_bytes(const ConvArgs& a);
hq_status hq_launch_conv_s2d(hq_handle* h, const ConvArgs& a, void* scratch, cudaStream_t s);
size_t hq_conv_s2d_prepared_bytes(const ConvArgs& a);
cudaError_t hq_prepare_conv_s2d(const ConvArgs& a, void* buf, cudaStream_t s);
// 4-bit operands: widen to bytes in scratch, then the tensor-core kernel.
bool hq_conv_widen4_applies(const ConvArgs& a);
size_t hq_conv_widen4_bytes(const ConvArgs& a);
hq_status hq_launch_conv_widen4(hq_handle* h, const ConvArgs& a, void* scratch, cudaStream_t s);
// Widen packed 4-bit weights (cout*kh*kw*cin values, a multiple of 16) to bytes, once, for ConvArgs::wgt_widened.
cudaError_t hq_launch_widen_weights(const void* wgt, long long values, void* out, int sm_count, cudaStream_t s);
// Bytes holding 4-bit values (one per byte) -> packed 4-bit tensor; `values` a multiple of 8.
cudaError_t hq_launch_expire_wait(uint32_t* status, int budget_ms, cudaStream_t s);
cudaError_t hq_launch_pack4(const void* in, long long values, void* out, int sm_count, cudaStream_t s);
// Grow the handle's scratch buffer (not allowed while `s` is capturing).
hq_status hq_reserve_workspace(hq_handle* h, size_t bytes, cudaStream_t s);
cudaError_t hq_launch_residual_add(const EltArgs& a, int sm_count, cudaStream_t s);
cudaError_t hq_launch_avgpool(const void* in, int n, int h, int w, int ch, int in_bits, int in_signed,
                              const int32_t* b, const int32_t* c, int qmin, int qmax,
                              void* out, int out_bits, cudaStream_t s);
cudaError_t hq_launch_maxpool(const void* in, int n, int h, int w, int ch, int bits, int is_signed,
                              int k, int stride, int pad, void* out, int ho, int wo, cudaStream_t s);
