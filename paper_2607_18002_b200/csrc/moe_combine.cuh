// Router-weighted combine (post-processing): y[t,:] = sum_j w[t,j] * D[row(t,j),:], row = flat_to_sorted[t*k+j]
// with the k slots added in order in fp32 (the last step of the MoE module of Section 2.1 of the
// paper).  One device routine serves the stand-alone kernel and the combine tiles of the
// persistent kernel.  A permutation entry outside [0, T*k) -- left by a plan that rejected an
// expert id -- is reported as MOE_EBOUNDS and its slot contributes nothing; no address is formed
// from it.
#pragma once
#include "moe_dev.cuh"

namespace moe {

// Tokens [t0, t1) by `nthr` cooperating threads (thread index tid); 8 bf16 per 16-byte access.
// k <= 8: a group of L adjacent threads (L = 16, 32, ... as many as the thread count allows)
// owns one token, loads its k routed rows and router weights once, and walks the token's row in
// steps of L 16-byte slices.  Slots 0..3 and 4..7 are two buffers: as soon as one has been added
// in, its loads for the next slice are issued, so loads are in flight all the time and the
// dependent pair (row index, then row) is paid once per token.  The rows are ADDED in slot
// order j = 0..k-1.
__device__ __forceinline__ void combine_add4(float (&acc)[8], const uint4 (&d)[4], const float* wj, int n) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (i < n) {
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

__device__ __forceinline__ int f2s_entry(const OpDev* op, int i) { return op->comb_index[i]; }

__device__ __noinline__ inline void combine_tokens(const OpDev* op, int t0, int t1, int k, int H, int tid,
                                                   int nthr) {
  const unsigned n_rows = (unsigned)op->space_rows;    // rows of the packed space D lives in
  // every permutation entry of these tokens is checked once, ahead of the loops that use them
  for (int i = t0 * k + tid; i < t1 * k; i += nthr)
    if ((unsigned)f2s_entry(op, i) >= n_rows) report(op->status, MOE_EBOUNDS, i / k, i % k, f2s_entry(op, i), 2);
  const int vec_per_row = H / 8;
  const uint4* D = reinterpret_cast<const uint4*>(op->D);
  uint4* y = reinterpret_cast<uint4*>(op->y);
  const int* f2s = op->comb_index;
  const float* w = op->topk_w;
  const int total = (t1 - t0) * vec_per_row;
  if (k <= 8 && nthr >= 16 && vec_per_row % 16 == 0) {
    int L = 16;
    while (2 * L * (t1 - t0) <= nthr && vec_per_row % (2 * L) == 0) L *= 2;
    const int tpp = nthr / L;                 // tokens per pass
    const int sub = tid % L, trow = tid / L;
    if (trow >= tpp) return;
    const int nslice = vec_per_row / L;
    for (int t = t0 + trow; t < t1; t += tpp) {
      // row offsets in 16-byte units (moe_create rejects shapes whose D buffer exceeds 2^32 units)
      unsigned off[8];
      float wj[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        off[i] = 0u;
        wj[i] = 0.f;
        if (i < k) {
          const unsigned p = (unsigned)f2s[(size_t)t * k + i];
          const bool ok = p < n_rows;                      // reported by the check above; adds nothing
          off[i] = ok ? p * (unsigned)vec_per_row : 0u;
          wj[i] = ok ? w[(size_t)t * k + i] : 0.f;
        }
      }
      const uint4* src = D + sub;
      uint4* dst = y + (size_t)t * vec_per_row + sub;
      const int na = k < 4 ? k : 4, nb = k - na;          // slots in the two buffers
      uint4 da[4], db[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        da[i] = make_uint4(0u, 0u, 0u, 0u);
        db[i] = make_uint4(0u, 0u, 0u, 0u);
        if (i < na) da[i] = src[off[i]];
        if (i < nb) db[i] = src[off[4 + i]];
      }
      for (int sl = 0; sl < nslice; ++sl) {
        const bool more = sl + 1 < nslice;
        src += L;
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        combine_add4(acc, da, wj, na);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (i < na && more) da[i] = src[off[i]];
        combine_add4(acc, db, wj + 4, nb);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (i < nb && more) db[i] = src[off[4 + i]];
        uint4 o;
        __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
        *dst = o;
        dst += L;
      }
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
          if ((unsigned)p < n_rows) {
            wj[i] = w[(size_t)t * k + j];
            d[i] = D[(size_t)p * vec_per_row + v];
          }
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
