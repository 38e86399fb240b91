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
// Local segment: one warp per query row (b, h_q, i).  The lanes split the head dim (each holds
// D / 32 elements of q); the warp walks the VISIBLE local keys only - bit j of the row's mask
// words, or the chain rule j <= i + (T_loc - T_q) - four at a time so that their K (then V)
// loads are in flight together.  A tree row sees depth + 1 keys of the T_loc, so the work
// follows the mask, not T_loc.  Scores go through a per-warp shared array (two passes: maximum,
// then weights), which keeps the result independent of the order of the keys.
// ---------------------------------------------------------------------------------------
constexpr int kLocalBatch = 4;

// visible keys of row i among local keys [w0, w0 + 64)
__device__ __forceinline__ unsigned long long visible_word(const uint64_t* bits, int w0, int chain_last,
                                                           int T_loc) {
  unsigned long long vis;
  if (bits) {
    vis = bits[w0 >> 6];
  } else {
    const int n = chain_last - w0 + 1;  // keys w0 .. chain_last
    vis = n >= 64 ? ~0ull : (n <= 0 ? 0ull : ((1ull << n) - 1));
  }
  if (T_loc - w0 < 64) vis &= (1ull << (T_loc - w0)) - 1;
  return vis;
}

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
    // 32-bit index arithmetic (the row count fits: checked by the host): a 64-bit division costs
    // a hundred instructions, more than the rest of a short row
    const unsigned rid = (unsigned)row_id;
    const int i = (int)(rid % (unsigned)p.T_q);
    const int h = (int)((rid / (unsigned)p.T_q) % (unsigned)p.H_q);
    const int b = (int)(rid / ((unsigned)p.T_q * (unsigned)p.H_q));
    const int kvh = h / p.G;
    const __nv_bfloat16* Kb = p.K + b * p.k_sb + kvh * p.k_sh + lane * CPL;
    const __nv_bfloat16* Vb = p.V + b * p.v_sb + kvh * p.v_sh + lane * CPL;
    const uint64_t* bits =
        p.mask_bits ? p.mask_bits + ((int64_t)b * p.T_q + i) * p.mask_words : nullptr;
    const int chain_last = i + (p.T_loc - p.T_q);

    // this lane's CPL elements of a bf16 row as floats
    auto load_row = [&](const __nv_bfloat16* ptr, float (&v)[CPL]) {
      if (CPL == 4) {
        const uint2 raw = *reinterpret_cast<const uint2*>(ptr);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
        const float2 c = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
        v[0] = a.x;
        v[1] = a.y;
        v[CPL - 2] = c.x;
        v[CPL - 1] = c.y;
      } else {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(ptr));
        v[0] = a.x;
        v[1] = a.y;
      }
    };
    float q[CPL];
    load_row(p.Q + b * p.q_sb + (int64_t)h * p.q_sh + i * p.q_st + lane * CPL, q);

    // pass 1: scores of the visible keys and their maximum
    float mx = -INFINITY;
    for (int w0 = 0; w0 < p.T_loc; w0 += 64) {
      unsigned long long vis = visible_word(bits, w0, chain_last, p.T_loc);
      while (vis) {
        int jj[kLocalBatch];
        float dot[kLocalBatch];
#pragma unroll
        for (int u = 0; u < kLocalBatch; ++u) {
          jj[u] = vis ? w0 + __ffsll((long long)vis) - 1 : -1;
          vis &= vis - 1;  // 0 stays 0
          dot[u] = 0.f;
          if (jj[u] >= 0) {
            float k[CPL];
            load_row(Kb + (int64_t)jj[u] * p.k_st, k);
#pragma unroll
            for (int c = 0; c < CPL; ++c) dot[u] = fmaf(q[c], k[c], dot[u]);
          }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
#pragma unroll
          for (int u = 0; u < kLocalBatch; ++u) dot[u] += __shfl_xor_sync(0xffffffffu, dot[u], o);
        }
#pragma unroll
        for (int u = 0; u < kLocalBatch; ++u) {
          if (jj[u] >= 0) {
            const float sv = dot[u] * p.scale_log2;
            if (lane == 0) sc[jj[u]] = sv;
            mx = fmaxf(mx, sv);
          }
        }
      }
    }
    __syncwarp();

    // pass 2: weights, row sum and weighted V sum over the same keys
    float acc[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
    float l = 0.f;
    if (mx > -INFINITY) {
      for (int w0 = 0; w0 < p.T_loc; w0 += 64) {
        unsigned long long vis = visible_word(bits, w0, chain_last, p.T_loc);
        while (vis) {
          float wgt[kLocalBatch], v[kLocalBatch][CPL];
#pragma unroll
          for (int u = 0; u < kLocalBatch; ++u) {
            const int j = vis ? w0 + __ffsll((long long)vis) - 1 : -1;
            vis &= vis - 1;
            wgt[u] = 0.f;
#pragma unroll
            for (int c = 0; c < CPL; ++c) v[u][c] = 0.f;
            if (j >= 0) {
              load_row(Vb + (int64_t)j * p.v_st, v[u]);
              wgt[u] = exp2f(sc[j] - mx);
            }
          }
#pragma unroll
          for (int u = 0; u < kLocalBatch; ++u) {
            l += wgt[u];
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[c] = fmaf(wgt[u], v[u][c], acc[c]);
          }
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
//
// A row has one partial per (set, token split): 17 for a 16-chunk round, up to a few hundred.
// They are read with as many loads in flight as the warp can hold: the (m, l) pairs one per
// lane (32 at a time), the a[] rows eight at a time with the weight and the address of each
// broadcast from the lane that owns the partial.
constexpr int kMergeBatch = 8;

template <int D, int MODE>
__global__ void __launch_bounds__(kWarpsPerCta * 32) merge_kernel(const MergeParams p) {
  constexpr bool FOLD = MODE == 1;
  constexpr int CPL = D / 32;
  // flat partial index f -> set: first_s[s] = partials before set s (sets in launch order, the
  // local set last); built before the wait below, it depends on the launch parameters only
  __shared__ int first_s[kMaxSets + 2];
  __shared__ uint8_t set_of[(kMaxSets + 1) * kMaxSplits];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_total = p.n_sets + (p.has_local ? 1 : 0);
  if (threadIdx.x == 0) {
    int acc = 0;
    for (int s = 0; s < n_total; ++s) {
      first_s[s] = acc;
      acc += (s < p.n_sets) ? p.splits[s] : 1;
    }
    first_s[n_total] = acc;
  }
  __syncthreads();
  for (int s = threadIdx.x; s < n_total; s += kWarpsPerCta * 32)
    for (int f = first_s[s]; f < first_s[s + 1]; ++f) set_of[f] = (uint8_t)s;
  __syncthreads();
  const int64_t row_id = (int64_t)blockIdx.x * kWarpsPerCta + warp;
  const int64_t n_rows = (int64_t)p.B * p.H_q * p.T_q;
  // (finalize) the next kernel may be set up meanwhile: the first chunk kernel of the next round
  // waits for this grid's completion before it reads or writes anything
  if (MODE == 0) pdl_launch_dependents();
  if (MODE == 0) pdl_wait_prior();  // every partial of the round must be complete
  if (row_id >= n_rows) return;
  const unsigned rid = (unsigned)row_id;  // 32-bit index arithmetic: the row count fits
  const int i = (int)(rid % (unsigned)p.T_q);
  const int h = (int)((rid / (unsigned)p.T_q) % (unsigned)p.H_q);
  const int b = (int)(rid / ((unsigned)p.T_q * (unsigned)p.H_q));
  const int kvh = h / p.G;
  const int r = (h % p.G) * p.T_q + i;
  const size_t slot0 = (size_t)b * p.H_kv + kvh;
  const size_t split_stride = (size_t)p.B * p.H_kv;
  const int n_part = first_s[n_total];
  // (m, l) of partial f and the element offset of its a[] row
  auto load_ml = [&](int f, int64_t* a_off) {
    const int s = set_of[f], k = f - first_s[s];
    if (s < p.n_sets && b < kMaxListed && ((p.absent[s][b >> 6] >> (b & 63)) & 1)) {  // the call skipped this request
      *a_off = 0;
      return make_float2(-INFINITY, 0.f);
    }
    const int set = (s < p.n_sets) ? s : p.local_set;
    const size_t idx = (slot0 + k * split_stride) * p.R_stride + r;
    *a_off = (int64_t)set * p.set_stride_a + (int64_t)idx * D;
    return p.part_ml[(int64_t)set * p.set_stride_ml + idx];
  };

  // pass 1: global maximum over the partials, one per lane
  float M = -INFINITY;
  for (int f = lane; f < n_part; f += 32) {
    int64_t off;
    M = fmaxf(M, load_ml(f, &off).x);
  }
  M = warp_max(M);

  float acc[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
  float L = 0.f;
  if (M > -INFINITY) {
    for (int base = 0; base < n_part; base += 32) {
      // lane j owns partial base + j: its weight (0 for an identity state, whose a[] is
      // undefined and must not be read) and the offset of its a[] row
      float w = 0.f;
      int64_t off = 0;
      if (base + lane < n_part) {
        const float2 st = load_ml(base + lane, &off);
        if (st.y != 0.f && st.x != -INFINITY) {
          w = exp2f(st.x - M);
          L = fmaf(w, st.y, L);
        }
      }
      const int cnt = min(32, n_part - base);
      for (int j0 = 0; j0 < cnt; j0 += kMergeBatch) {
        float wj[kMergeBatch];
        float v[kMergeBatch][CPL];
#pragma unroll
        for (int u = 0; u < kMergeBatch; ++u) {
          const int j = (j0 + u) & 31;
          wj[u] = __shfl_sync(0xffffffffu, w, j);
          const int64_t oj = __shfl_sync(0xffffffffu, off, j);
#pragma unroll
          for (int c = 0; c < CPL; ++c) v[u][c] = 0.f;
          if (j0 + u < cnt && wj[u] != 0.f) {  // warp-uniform
            const float* a = p.part_a + oj + lane * CPL;
            if (CPL == 4) {
              const float4 x = *reinterpret_cast<const float4*>(a);
              v[u][0] = x.x;
              v[u][1] = x.y;
              v[u][CPL - 2] = x.z;
              v[u][CPL - 1] = x.w;
            } else {
              const float2 x = *reinterpret_cast<const float2*>(a);
              v[u][0] = x.x;
              v[u][1] = x.y;
            }
          } else {
            wj[u] = 0.f;
          }
        }
#pragma unroll
        for (int u = 0; u < kMergeBatch; ++u) {
#pragma unroll
          for (int c = 0; c < CPL; ++c) acc[c] = fmaf(wj[u], v[u][c], acc[c]);
        }
      }
    }
    L = warp_sum(L);
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
  const unsigned rid = (unsigned)row_id;  // 32-bit index arithmetic: the row count fits
  const int i = (int)(rid % (unsigned)p.T_q);
  const int h = (int)((rid / (unsigned)p.T_q) % (unsigned)p.H_q);
  const int b = (int)(rid / ((unsigned)p.T_q * (unsigned)p.H_q));
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
