// CUDA-core chunk attention: the path for shapes the tensor-core kernel does not take
// (head dim 64, few rows per kv-head) and an on-GPU cross-check of it.
//
// One CTA owns one (request, kv-head, token split, tile of <= 32 query rows) and walks its
// tokens in tiles of 64: scores for all rows of the tile against the staged K tile, the
// chunk-local row maximum / exponentials / row sum (Eq. 13, kept as a running state inside
// the CTA), and a += P V with V read straight from global memory (coalesced rows).
#include "ss_internal.h"

namespace ss {
namespace {

constexpr int kRows = 32;     // query rows per CTA
constexpr int kKeys = kTileKeys;
constexpr int kThreads = 128;

template <int D>
__global__ void __launch_bounds__(kThreads) chunk_simt_kernel(const ChunkParams p) {
  constexpr int KS = D + 8;                 // padded K row (elements)
  constexpr int CP = D / 2;                 // column pairs
  constexpr int TG = kThreads / CP;         // token groups in the PV phase
  constexpr int KPG = kKeys / TG;           // keys per token group
  __shared__ __align__(16) float q_s[kRows * D];
  __shared__ __align__(16) __nv_bfloat16 k_s[kKeys * KS];
  __shared__ float p_s[kRows * (kKeys + 1)];
  __shared__ float m_s[kRows], l_s[kRows], corr_s[kRows];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (p.wait_first) pdl_wait_prior();
  pdl_launch_dependents();
  const ChunkWork w = chunk_work(p, kRows);
  const int b = w.b, kvh = w.kvh, row0 = w.row0, nrows = w.nrows, tok0 = w.tok0, tok1 = w.tok1;
  const bool chain_cta = w.chain_cta;
  float2* out_ml = w.out_ml;
  float* out_a = w.out_a;

  if (tok0 >= tok1) {  // nothing visible here: identity state
    if (tid < nrows) out_ml[tid] = make_float2(-INFINITY, 0.f);
    if (!p.wait_first && chain_cta) pdl_wait_prior();
    return;
  }

  // Q rows of this tile -> fp32 shared memory (rows past R are zero)
  for (int i = tid; i < kRows * (D / 8); i += kThreads) {
    const int r = i / (D / 8), c8 = i % (D / 8);
    float v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (r < nrows) {
      const int rg = row0 + r, g = rg / p.T_q, t = rg % p.T_q;
      const uint4 raw = *reinterpret_cast<const uint4*>(
          p.Q + b * p.q_sb + (int64_t)(kvh * p.G + g) * p.q_sh + t * p.q_st + c8 * 8);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(h[j]);
        v[2 * j] = f.x;
        v[2 * j + 1] = f.y;
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) q_s[r * D + c8 * 8 + j] = v[j];
  }
  if (tid < kRows) {
    m_s[tid] = -INFINITY;
    l_s[tid] = 0.f;
  }

  float acc[kRows][2];
#pragma unroll
  for (int r = 0; r < kRows; ++r) acc[r][0] = acc[r][1] = 0.f;

  // row of token tok (contiguous chunk or page of a pool)
  auto k_row = [&](int tok) {
    int outer, inner;
    locate_token(p, b, tok, &outer, &inner);
    return outer == p.n_pages && p.page_table ? (const __nv_bfloat16*)nullptr
                                              : p.K + outer * p.k_sb + kvh * p.k_sh + inner * p.k_st;
  };
  auto v_row = [&](int tok) {
    int outer, inner;
    locate_token(p, b, tok, &outer, &inner);
    return outer == p.n_pages && p.page_table ? (const __nv_bfloat16*)nullptr
                                              : p.V + outer * p.v_sb + kvh * p.v_sh + inner * p.v_st;
  };
  const int cp = tid % CP, tg = tid / CP;

  for (int t0 = tok0; t0 < tok1; t0 += kKeys) {
    const int nk = min(kKeys, tok1 - t0);
    __syncthreads();
    // stage K tile (rows past nk are zero so the dot products stay finite)
    for (int i = tid; i < kKeys * (D / 8); i += kThreads) {
      const int k = i / (D / 8), c8 = i % (D / 8);
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (k < nk) {
        const __nv_bfloat16* row = k_row(t0 + k);
        if (row) raw = *reinterpret_cast<const uint4*>(row + c8 * 8);
      }
      *reinterpret_cast<uint4*>(&k_s[k * KS + c8 * 8]) = raw;
    }
    __syncthreads();
    // scores: thread = (key, half of the rows)
    {
      const int kk = tid % kKeys, rh = tid / kKeys;  // rh in {0,1}: rows rh*16..+16
      float s[16];
#pragma unroll
      for (int r = 0; r < 16; ++r) s[r] = 0.f;
      for (int c8 = 0; c8 < D / 8; ++c8) {
        const uint4 raw = *reinterpret_cast<const uint4*>(&k_s[kk * KS + c8 * 8]);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
        float kv[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(h[j]);
          kv[2 * j] = f.x;
          kv[2 * j + 1] = f.y;
        }
#pragma unroll
        for (int r = 0; r < 16; ++r) {
          const float4 qa = *reinterpret_cast<const float4*>(&q_s[(rh * 16 + r) * D + c8 * 8]);
          const float4 qb = *reinterpret_cast<const float4*>(&q_s[(rh * 16 + r) * D + c8 * 8 + 4]);
          s[r] = fmaf(qa.x, kv[0], s[r]);
          s[r] = fmaf(qa.y, kv[1], s[r]);
          s[r] = fmaf(qa.z, kv[2], s[r]);
          s[r] = fmaf(qa.w, kv[3], s[r]);
          s[r] = fmaf(qb.x, kv[4], s[r]);
          s[r] = fmaf(qb.y, kv[5], s[r]);
          s[r] = fmaf(qb.z, kv[6], s[r]);
          s[r] = fmaf(qb.w, kv[7], s[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < 16; ++r)
        p_s[(rh * 16 + r) * (kKeys + 1) + kk] = (kk < nk) ? s[r] * p.scale_log2 : -INFINITY;
    }
    __syncthreads();
    // row statistics: warp w owns rows w*8..w*8+7
    for (int rr = 0; rr < 8; ++rr) {
      const int r = warp * 8 + rr;
      float* row = &p_s[r * (kKeys + 1)];
      const float s0 = row[lane], s1 = row[lane + 32];
      float mx = fmaxf(s0, s1);
#pragma unroll
      for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_old = m_s[r];
      const float m_new = fmaxf(m_old, mx);  // finite: nk >= 1
      const float e0 = exp2f(s0 - m_new), e1 = exp2f(s1 - m_new);
      float sum = e0 + e1;
#pragma unroll
      for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      row[lane] = e0;
      row[lane + 32] = e1;
      if (lane == 0) {
        const float corr = (m_old == -INFINITY) ? 0.f : exp2f(m_old - m_new);
        corr_s[r] = corr;
        m_s[r] = m_new;
        l_s[r] = l_s[r] * corr + sum;
      }
    }
    __syncthreads();
    // a = a * corr + P V: thread = (column pair, token group)
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
      const float c = corr_s[r];
      acc[r][0] *= c;
      acc[r][1] *= c;
    }
    const int kend = min(nk, (tg + 1) * KPG);
    for (int k = tg * KPG; k < kend; ++k) {
      const __nv_bfloat16* vrow = v_row(t0 + k);
      const float2 v = vrow ? __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(vrow + 2 * cp))
                            : make_float2(0.f, 0.f);
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        const float pr = p_s[r * (kKeys + 1) + k];
        acc[r][0] = fmaf(pr, v.x, acc[r][0]);
        acc[r][1] = fmaf(pr, v.y, acc[r][1]);
      }
    }
  }
  __syncthreads();
  // reduce the token groups through shared memory (reuse q_s: kRows*D floats) and write out
  float* red = q_s;
  for (int g = 0; g < TG; ++g) {
    if (tg == g) {
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        float2* dst = reinterpret_cast<float2*>(&red[r * D + 2 * cp]);
        if (g == 0) {
          *dst = make_float2(acc[r][0], acc[r][1]);
        } else {
          float2 o = *dst;
          o.x += acc[r][0];
          o.y += acc[r][1];
          *dst = o;
        }
      }
    }
    __syncthreads();
  }
  for (int i = tid; i < nrows * (D / 4); i += kThreads) {
    const int r = i / (D / 4), c4 = i % (D / 4);
    *reinterpret_cast<float4*>(out_a + (size_t)r * D + c4 * 4) =
        *reinterpret_cast<const float4*>(&red[r * D + c4 * 4]);
  }
  if (tid < nrows) out_ml[tid] = make_float2(m_s[tid], l_s[tid]);
  // Completion order along the stream: one CTA of this grid waits for the previous grid, so
  // this grid cannot complete before it (the other CTAs leave at once and free their SM slot).
  if (!p.wait_first && chain_cta) pdl_wait_prior();
}

}  // namespace

cudaError_t launch_chunk_simt(const ChunkParams& p, cudaStream_t s, bool pdl) {
  dim3 grid(p.splits * p.row_tiles, p.H_kv, p.n_active ? p.n_active : p.B), block(kThreads);
  if (p.d == 128) return launch_kernel(chunk_simt_kernel<128>, grid, block, 0, s, pdl, p);
  return launch_kernel(chunk_simt_kernel<64>, grid, block, 0, s, pdl, p);
}

}  // namespace ss
