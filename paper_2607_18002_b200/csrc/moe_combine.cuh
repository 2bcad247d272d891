// Router-weighted combine (post-processing): y[t,:] = sum_j w[t,j] * D[flat_to_sorted[t*k+j],:]
// with the k slots added in order in fp32 (Section 2.1 of the paper: the module "combines
// their outputs").  One device routine serves the stand-alone kernel and the combine tiles
// of the persistent kernel.
#pragma once
#include "moe_dev.cuh"

namespace moe {

// Tokens [t0, t1) by `nthr` cooperating threads (thread index tid); 8 bf16 per 16-byte access.
// One item = one 16-byte column slice of one token: the token's k rows of D are fetched
// together (k <= 8: all at once, else eight at a time), so a thread keeps eight 16-byte loads
// in flight, and the routed rows / router weights of the thread's NEXT item are loaded before
// the current item's rows are consumed: the two dependent loads of an item (row index, then
// row) never sit in one latency chain.  The rows are still ADDED in slot order j = 0..k-1.
__device__ inline void combine_tokens(const OpDev* op, int t0, int t1, int k, int H, int tid,
                                      int nthr) {
  const int vec_per_row = H / 8;
  const uint4* D = reinterpret_cast<const uint4*>(op->D);
  uint4* y = reinterpret_cast<uint4*>(op->y);
  const int* f2s = op->flat_to_sorted;
  const float* w = op->topk_w;
  const int total = (t1 - t0) * vec_per_row;
  if (k <= 8) {
    int pj[8];
    float wj[8];
    int t_have = -1;
    auto load_meta = [&](int t) {             // rows and weights of token t
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        pj[i] = 0;
        wj[i] = 0.f;
        if (i < k) {
          pj[i] = f2s[(size_t)t * k + i];
          wj[i] = w[(size_t)t * k + i];
        }
      }
      t_have = t;
    };
    if (tid < total) load_meta(t0 + tid / vec_per_row);
    for (int idx = tid; idx < total; idx += nthr) {
      const int t = t0 + idx / vec_per_row, v = idx % vec_per_row;
      uint4 d[8];
      float wc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        wc[i] = wj[i];
        d[i] = make_uint4(0u, 0u, 0u, 0u);
        if (i < k) d[i] = D[(size_t)pj[i] * vec_per_row + v];
      }
      const int nidx = idx + nthr;
      if (nidx < total) {
        const int nt = t0 + nidx / vec_per_row;
        if (nt != t_have) load_meta(nt);       // issued while the eight row loads above are in flight
      }
      float acc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (i < k) {
          const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&d[i]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float2 f = __bfloat1622float2(h[c]);
            acc[2 * c] = fmaf(wc[i], f.x, acc[2 * c]);
            acc[2 * c + 1] = fmaf(wc[i], f.y, acc[2 * c + 1]);
          }
        }
      }
      uint4 o;
      __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
      y[(size_t)t * vec_per_row + v] = o;
    }
    return;
  }
  for (int idx = tid; idx < total; idx += nthr) {
    const int t = t0 + idx / vec_per_row, v = idx % vec_per_row;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    for (int j0 = 0; j0 < k; j0 += 8) {
      float wj[8];
      uint4 d[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int j = j0 + i;
        wj[i] = 0.f;
        d[i] = make_uint4(0u, 0u, 0u, 0u);
        if (j < k) {
          const int p = f2s[(size_t)t * k + j];
          wj[i] = w[(size_t)t * k + j];
          d[i] = D[(size_t)p * vec_per_row + v];
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (j0 + i < k) {
          const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&d[i]);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float2 f = __bfloat1622float2(h[c]);
            acc[2 * c] = fmaf(wj[i], f.x, acc[2 * c]);
            acc[2 * c + 1] = fmaf(wj[i], f.y, acc[2 * c + 1]);
          }
        }
      }
    }
    uint4 o;
    __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
    y[(size_t)t * vec_per_row + v] = o;
  }
}

}  // namespace moe
