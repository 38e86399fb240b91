// Local candidate segment (masked), partial merge (Eq. 14) + finalize, and commit-gather.
#include "ss_internal.h"

namespace ss {
namespace {

constexpr int kWarpsPerCta = 4;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------------------------------
// Local segment: one warp per query row (b, h_q, i).  Lanes split the local keys for the
// scores and the head dim for the weighted sum.  The visible set of row i is given by the
// chain rule j <= i + (T_loc - T_q) or by bit j of the row's mask words.
// ---------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32) local_kernel(const LocalParams p) {
  constexpr int CPL = D / 32;  // columns per lane
  extern __shared__ float sc_all[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t row_id = (int64_t)blockIdx.x * kWarpsPerCta + warp;
  const int64_t n_rows = (int64_t)p.B * p.H_q * p.T_q;
  pdl_launch_dependents();
  if (row_id < n_rows) {
    float* sc = sc_all + (size_t)warp * p.T_loc;
    const int i = (int)(row_id % p.T_q);
    const int h = (int)((row_id / p.T_q) % p.H_q);
    const int b = (int)(row_id / ((int64_t)p.T_q * p.H_q));
    const int kvh = h / p.G;
    const __nv_bfloat16* q = p.Q + b * p.q_sb + (int64_t)h * p.q_sh + i * p.q_st;
    const __nv_bfloat16* Kb = p.K + b * p.k_sb + kvh * p.k_sh;
    const __nv_bfloat16* Vb = p.V + b * p.v_sb + kvh * p.v_sh;
    const uint64_t* bits =
        p.mask_bits ? p.mask_bits + ((int64_t)b * p.T_q + i) * p.mask_words : nullptr;
    const int chain_last = i + (p.T_loc - p.T_q);

    float mx = -INFINITY;
    for (int j = lane; j < p.T_loc; j += 32) {
      const bool vis = bits ? ((bits[j >> 6] >> (j & 63)) & 1ull) : (j <= chain_last);
      float s = -INFINITY;
      if (vis) {
        const uint4* kr = reinterpret_cast<const uint4*>(Kb + (int64_t)j * p.k_st);
        const uint4* qr = reinterpret_cast<const uint4*>(q);
        float dot = 0.f;
#pragma unroll 4
        for (int c8 = 0; c8 < D / 8; ++c8) {
          const uint4 kq = kr[c8], qq = qr[c8];
          const __nv_bfloat162* kh = reinterpret_cast<const __nv_bfloat162*>(&kq);
          const __nv_bfloat162* qh = reinterpret_cast<const __nv_bfloat162*>(&qq);
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const float2 kf = __bfloat1622float2(kh[t]), qf = __bfloat1622float2(qh[t]);
            dot = fmaf(qf.x, kf.x, dot);
            dot = fmaf(qf.y, kf.y, dot);
          }
        }
        s = dot * p.scale_log2;
      }
      sc[j] = s;
      mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    __syncwarp();
    float acc[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
    float l = 0.f;
    if (mx > -INFINITY) {
      for (int j = 0; j < p.T_loc; ++j) {
        const float s = sc[j];
        if (s == -INFINITY) continue;  // warp-uniform
        const float w = exp2f(s - mx);
        l += w;
        const __nv_bfloat16* vr = Vb + (int64_t)j * p.v_st + lane * CPL;
        if (CPL == 4) {
          const uint2 raw = *reinterpret_cast<const uint2*>(vr);
          const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
          const float2 c = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
          acc[0] = fmaf(w, a.x, acc[0]);
          acc[1] = fmaf(w, a.y, acc[1]);
          acc[CPL - 2] = fmaf(w, c.x, acc[CPL - 2]);
          acc[CPL - 1] = fmaf(w, c.y, acc[CPL - 1]);
        } else {
          const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(vr));
          acc[0] = fmaf(w, a.x, acc[0]);
          acc[1] = fmaf(w, a.y, acc[1]);
        }
      }
    }
    const size_t slot = (size_t)b * p.H_kv + kvh;
    const int r = (h % p.G) * p.T_q + i;
    if (lane == 0) p.part_ml[slot * p.R_stride + r] = make_float2(mx, l);
    float* out = p.part_a + (slot * p.R_stride + r) * D + lane * CPL;
    if (CPL == 4)
      *reinterpret_cast<float4*>(out) = make_float4(acc[0], acc[1], acc[CPL - 2], acc[CPL - 1]);
    else
      *reinterpret_cast<float2*>(out) = make_float2(acc[0], acc[1]);
  }
  if (blockIdx.x == 0) pdl_wait_prior();  // one CTA keeps the completion order along the stream
}

// ---------------------------------------------------------------------------------------
// Merge of every partial state of a row (Eq. 14, as one max + one rescaled sum, which is
// the same value as the serial recurrence up to rounding order), then either O = a / l
// and LSE (finalize) or the merged state itself (fold).  One warp per row.
// ---------------------------------------------------------------------------------------
// MODE 0: finalize (O, LSE); 1: fold into set 0; 2: export the merged state in row order.
template <int D, int MODE>
__global__ void __launch_bounds__(kWarpsPerCta * 32) merge_kernel(const MergeParams p) {
  constexpr bool FOLD = MODE == 1;
  constexpr int CPL = D / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t row_id = (int64_t)blockIdx.x * kWarpsPerCta + warp;
  const int64_t n_rows = (int64_t)p.B * p.H_q * p.T_q;
  if (MODE == 0) pdl_wait_prior();  // every partial of the round must be complete
  if (row_id >= n_rows) return;
  const int i = (int)(row_id % p.T_q);
  const int h = (int)((row_id / p.T_q) % p.H_q);
  const int b = (int)(row_id / ((int64_t)p.T_q * p.H_q));
  const int kvh = h / p.G;
  const int r = (h % p.G) * p.T_q + i;
  const size_t slot0 = (size_t)b * p.H_kv + kvh;
  const size_t split_stride = (size_t)p.B * p.H_kv;

  // pass 1: global maximum over partials
  const int n_total = p.n_sets + (p.has_local ? 1 : 0);
  float M = -INFINITY;
  for (int s = 0; s < n_total; ++s) {
    const int set = (s < p.n_sets) ? s : p.local_set;
    const int ns = (s < p.n_sets) ? p.splits[s] : 1;
    const float2* ml = p.part_ml + (int64_t)set * p.set_stride_ml;
    for (int k = lane; k < ns; k += 32)
      M = fmaxf(M, ml[(slot0 + k * split_stride) * p.R_stride + r].x);
  }
  M = warp_max(M);

  float acc[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
  float L = 0.f;
  if (M > -INFINITY) {
    for (int s = 0; s < n_total; ++s) {
      const int set = (s < p.n_sets) ? s : p.local_set;
      const int ns = (s < p.n_sets) ? p.splits[s] : 1;
      const float2* ml = p.part_ml + (int64_t)set * p.set_stride_ml;
      const float* pa = p.part_a + (int64_t)set * p.set_stride_a;
      for (int k = 0; k < ns; ++k) {
        const size_t idx = (slot0 + k * split_stride) * p.R_stride + r;
        const float2 st = ml[idx];
        if (st.y == 0.f || st.x == -INFINITY) continue;  // identity: a[] undefined
        const float w = exp2f(st.x - M);
        L = fmaf(w, st.y, L);
        const float* a = pa + idx * D + lane * CPL;
        if (CPL == 4) {
          const float4 v = *reinterpret_cast<const float4*>(a);
          acc[0] = fmaf(w, v.x, acc[0]);
          acc[1] = fmaf(w, v.y, acc[1]);
          acc[CPL - 2] = fmaf(w, v.z, acc[CPL - 2]);
          acc[CPL - 1] = fmaf(w, v.w, acc[CPL - 1]);
        } else {
          const float2 v = *reinterpret_cast<const float2*>(a);
          acc[0] = fmaf(w, v.x, acc[0]);
          acc[1] = fmaf(w, v.y, acc[1]);
        }
      }
    }
  }
  if (MODE == 2) {
    if (lane == 0) p.fold_ml[row_id] = make_float2(L > 0.f ? M : -INFINITY, L);
    float* out = p.fold_a + row_id * D + lane * CPL;
    if (CPL == 4)
      *reinterpret_cast<float4*>(out) = make_float4(acc[0], acc[1], acc[CPL - 2], acc[CPL - 1]);
    else
      *reinterpret_cast<float2*>(out) = make_float2(acc[0], acc[1]);
  } else if (FOLD) {
    const size_t idx = slot0 * p.R_stride + r;
    if (lane == 0) p.fold_ml[idx] = make_float2(L > 0.f ? M : -INFINITY, L);
    float* out = p.fold_a + idx * D + lane * CPL;
    if (CPL == 4)
      *reinterpret_cast<float4*>(out) = make_float4(acc[0], acc[1], acc[CPL - 2], acc[CPL - 1]);
    else
      *reinterpret_cast<float2*>(out) = make_float2(acc[0], acc[1]);
  } else {
    const float inv = (L > 0.f) ? 1.f / L : 0.f;
    __nv_bfloat16* o = p.O + row_id * D + lane * CPL;
    if (CPL == 4) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
      __nv_bfloat162 hi = __floats2bfloat162_rn(acc[CPL - 2] * inv, acc[CPL - 1] * inv);
      uint2 raw;
      raw.x = *reinterpret_cast<uint32_t*>(&lo);
      raw.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(o) = raw;
    } else {
      *reinterpret_cast<__nv_bfloat162*>(o) = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
    }
    if (p.LSE && lane == 0)
      p.LSE[row_id] = (L > 0.f) ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
  }
}

// ---------------------------------------------------------------------------------------
// Import: a merged state in row order [B, H_q, T_q] -> one partial set (split 0).
// ---------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32) import_kernel(const MergeParams p) {
  constexpr int CPL = D / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t row_id = (int64_t)blockIdx.x * kWarpsPerCta + warp;
  if (row_id >= (int64_t)p.B * p.H_q * p.T_q) return;
  const int i = (int)(row_id % p.T_q);
  const int h = (int)((row_id / p.T_q) % p.H_q);
  const int b = (int)(row_id / ((int64_t)p.T_q * p.H_q));
  const size_t idx = ((size_t)b * p.H_kv + h / p.G) * p.R_stride + (h % p.G) * p.T_q + i;
  if (lane == 0) p.fold_ml[idx] = reinterpret_cast<const float2*>(p.part_ml)[row_id];
  const float* src = p.part_a + row_id * D + lane * CPL;
  float* dst = p.fold_a + idx * D + lane * CPL;
#pragma unroll
  for (int c = 0; c < CPL; ++c) dst[c] = src[c];
}

// ---------------------------------------------------------------------------------------
// Commit-gather: one thread per 16-byte vector of one (request, accepted row, K|V, head).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gather_kernel(const GatherParams p) {
  const int vec_per_row = p.d / 8;
  const int64_t per_req = (int64_t)p.T_loc * 2 * p.H_kv * vec_per_row;
  const int64_t total = per_req * p.B;
  for (int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; id < total;
       id += (int64_t)gridDim.x * blockDim.x) {
    const int b = (int)(id / per_req);
    int64_t rem = id % per_req;
    const int vec = (int)(rem % vec_per_row);
    rem /= vec_per_row;
    const int h = (int)(rem % p.H_kv);
    rem /= p.H_kv;
    const int kv = (int)(rem & 1);
    const int k = (int)(rem >> 1);
    const int cnt = p.accept_cnt[b];
    const bool first = (vec == 0 && h == 0 && kv == 0);
    if (cnt < 0 || cnt > p.T_loc) {
      if (first && k == 0) atomicOr(p.status, SS_DEV_BAD_ACCEPT);
    }
    if (k >= min(max(cnt, 0), p.T_loc)) continue;
    const int src = p.accept_idx[(int64_t)b * p.T_loc + k];
    if (src < 0 || src >= p.T_loc) {
      if (first) atomicOr(p.status, SS_DEV_BAD_ACCEPT);
      continue;
    }
    const int64_t dst = (int64_t)p.dst_off[b] + k;
    if (dst < 0 || dst >= p.cap) {
      if (first) atomicOr(p.status, SS_DEV_DST_OVERFLOW);
      continue;
    }
    if (kv == 0) {
      const uint4 v = *reinterpret_cast<const uint4*>(p.K_loc + b * p.ks_b + h * p.ks_h +
                                                      src * p.ks_t + vec * 8);
      *reinterpret_cast<uint4*>(p.K_dst + b * p.kd_b + h * p.kd_h + dst * p.kd_t + vec * 8) = v;
    } else {
      const uint4 v = *reinterpret_cast<const uint4*>(p.V_loc + b * p.vs_b + h * p.vs_h +
                                                      src * p.vs_t + vec * 8);
      *reinterpret_cast<uint4*>(p.V_dst + b * p.vd_b + h * p.vd_h + dst * p.vd_t + vec * 8) = v;
    }
  }
}

}  // namespace

cudaError_t launch_local(const LocalParams& p, cudaStream_t s, bool pdl) {
  const int64_t rows = (int64_t)p.B * p.H_q * p.T_q;
  dim3 grid((unsigned)((rows + kWarpsPerCta - 1) / kWarpsPerCta)), block(kWarpsPerCta * 32);
  const size_t smem = (size_t)kWarpsPerCta * p.T_loc * sizeof(float);
  if (p.d == 128) return launch_kernel(local_kernel<128>, grid, block, smem, s, pdl, p);
  return launch_kernel(local_kernel<64>, grid, block, smem, s, pdl, p);
}

cudaError_t launch_finalize(const MergeParams& p, cudaStream_t s, bool pdl) {
  const int64_t rows = (int64_t)p.B * p.H_q * p.T_q;
  dim3 grid((unsigned)((rows + kWarpsPerCta - 1) / kWarpsPerCta)), block(kWarpsPerCta * 32);
  if (p.d == 128) return launch_kernel(merge_kernel<128, 0>, grid, block, 0, s, pdl, p);
  return launch_kernel(merge_kernel<64, 0>, grid, block, 0, s, pdl, p);
}

cudaError_t launch_fold(const MergeParams& p, cudaStream_t s) {
  const int64_t rows = (int64_t)p.B * p.H_q * p.T_q;
  dim3 grid((unsigned)((rows + kWarpsPerCta - 1) / kWarpsPerCta)), block(kWarpsPerCta * 32);
  if (p.d == 128) return launch_kernel(merge_kernel<128, 1>, grid, block, 0, s, false, p);
  return launch_kernel(merge_kernel<64, 1>, grid, block, 0, s, false, p);
}

cudaError_t launch_export(const MergeParams& p, cudaStream_t s) {
  const int64_t rows = (int64_t)p.B * p.H_q * p.T_q;
  dim3 grid((unsigned)((rows + kWarpsPerCta - 1) / kWarpsPerCta)), block(kWarpsPerCta * 32);
  if (p.d == 128) return launch_kernel(merge_kernel<128, 2>, grid, block, 0, s, false, p);
  return launch_kernel(merge_kernel<64, 2>, grid, block, 0, s, false, p);
}

cudaError_t launch_import(const MergeParams& p, cudaStream_t s) {
  const int64_t rows = (int64_t)p.B * p.H_q * p.T_q;
  dim3 grid((unsigned)((rows + kWarpsPerCta - 1) / kWarpsPerCta)), block(kWarpsPerCta * 32);
  if (p.d == 128) return launch_kernel(import_kernel<128>, grid, block, 0, s, false, p);
  return launch_kernel(import_kernel<64>, grid, block, 0, s, false, p);
}

cudaError_t launch_gather(const GatherParams& p, cudaStream_t s) {
  const int64_t total = (int64_t)p.B * p.T_loc * 2 * p.H_kv * (p.d / 8);
  const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
  return launch_kernel(gather_kernel, dim3(blocks > 0 ? blocks : 1), dim3(256), 0, s, false, p);
}

}  // namespace ss
