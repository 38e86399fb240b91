// CUDA-core chunk attention: the path for calls the tensor-core kernels do not take (tiny
// calls at head dim 64, page sizes they cannot tile, the entry point that allocates nothing),
// an on-GPU cross-check of them, and the kernel of small whole rounds (ss_verify_round).
//
// One CTA owns one (request, kv-head, token split, tile of RT query rows), RT = 8, 16 or 32
// chosen from the rows per kv-head so that a plain decode or a narrow verification does not
// pay for 32 rows.  It walks its tokens in tiles of 64: the K and the V tile of the NEXT
// tile are on their way to shared memory (cp.async, 16 bytes per request, two stages) while
// the current one is worked on: scores for all rows of the tile against the staged K tile,
// the running row maximum / exponentials / row sum (Eq. 13, kept as a running state inside
// the CTA), and a += P V from the staged V tile.
//
// The same tile loop serves two kernels:
//   chunk_simt_kernel   one chunk call: the CTA's partial state (m, l, a) goes to the call's
//                       partial set (Eq. 13), merged later (Eq. 14);
//   round_simt_kernel   a whole small round in one launch: every history chunk, then the local
//                       candidate segment under its chain or tree mask, then O = a / l and the
//                       LSE (Eq. 12) - no partial state ever leaves the SM.
#include "ss_internal.h"

namespace ss {
namespace {

constexpr int kKeys = kTileKeys;
constexpr int kThreads = 128;

template <int D, int RT>
struct Lay {
  static constexpr int KS = D + 8;                           // padded K / V row (elements)
  static constexpr int kTile = kKeys * KS * 2;               // bytes of one staged K or V tile
  static constexpr int kOffQ = 4 * kTile;                    // two stages x (K, V)
  static constexpr int kOffP = kOffQ + RT * D * 4;           // Q rows as fp32
  static constexpr int kOffSt = kOffP + RT * (kKeys + 1) * 4;  // scores / weights
  static constexpr int kBytes = kOffSt + 3 * RT * 4;         // m, l, correction per row
  static_assert(RT == 8 || RT == 16 || RT == 32, "rows per tile");
};

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  const int n = valid ? 16 : 0;  // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Where the tokens of one run come from: a contiguous [tokens][d] slice of one (request,
// kv-head), or the pages of a pool (per-token lookup).
struct Source {
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  int64_t k_st, v_st;          // element stride between tokens
  const ChunkParams* paged;    // non-null: look every token up (K, V, strides come from it)
  int b, kvh;
};

// The per-CTA state of the tile loop.
template <int D, int RT>
struct Simt {
  using L = Lay<D, RT>;
  static constexpr int KS = L::KS;
  static constexpr int CP = D / 2;            // column pairs
  static constexpr int TG = kThreads / CP;    // token groups in the PV phase
  static constexpr int KPG = kKeys / TG;      // keys per token group
  static constexpr int RH = RT / 2;           // rows per thread in the score phase
  static constexpr int RW = RT / 4;           // rows per warp in the statistics phase

  uint8_t* smem;
  float* q_s;
  float* p_s;
  float* m_s;
  float* l_s;
  float* corr_s;
  float acc[RT][2];
  int tid, lane, warp;

  __device__ __forceinline__ void init(uint8_t* base) {
    smem = base;
    q_s = reinterpret_cast<float*>(base + L::kOffQ);
    p_s = reinterpret_cast<float*>(base + L::kOffP);
    m_s = reinterpret_cast<float*>(base + L::kOffSt);
    l_s = m_s + RT;
    corr_s = l_s + RT;
    tid = threadIdx.x;
    lane = tid & 31;
    warp = tid >> 5;
#pragma unroll
    for (int r = 0; r < RT; ++r) acc[r][0] = acc[r][1] = 0.f;
  }
  __device__ __forceinline__ __nv_bfloat16* k_stage(int s) {
    return reinterpret_cast<__nv_bfloat16*>(smem + (2 * s) * L::kTile);
  }
  __device__ __forceinline__ __nv_bfloat16* v_stage(int s) {
    return reinterpret_cast<__nv_bfloat16*>(smem + (2 * s + 1) * L::kTile);
  }

  // Q rows [row0, row0 + nrows) of the kv-head -> fp32 shared memory (rows past nrows are
  // zero); identity row state.  In two steps, so that the first K/V tile's copies can be
  // started between the global loads and their first use: q_fetch only issues the loads.
  static constexpr int kQPieces = (RT * (D / 8) + kThreads - 1) / kThreads;
  uint4 qraw[kQPieces];
  __device__ __forceinline__ void q_fetch(const __nv_bfloat16* Q, int64_t q_sb, int64_t q_sh, int64_t q_st,
                                          int b, int kvh, int G, int T_q, int row0, int nrows) {
#pragma unroll
    for (int j = 0; j < kQPieces; ++j) {
      const int i = tid + j * kThreads;
      const int r = i / (D / 8), c8 = i % (D / 8);
      qraw[j] = make_uint4(0, 0, 0, 0);
      if (i < RT * (D / 8) && r < nrows) {
        const int rg = row0 + r, g = rg / T_q, t = rg % T_q;
        qraw[j] = *reinterpret_cast<const uint4*>(Q + b * q_sb + (int64_t)(kvh * G + g) * q_sh + t * q_st + c8 * 8);
      }
    }
  }
  __device__ __forceinline__ void q_store() {
#pragma unroll
    for (int j = 0; j < kQPieces; ++j) {
      const int i = tid + j * kThreads;
      if (i < RT * (D / 8)) {
        const int r = i / (D / 8), c8 = i % (D / 8);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&qraw[j]);
        const float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]);
        const float2 f2 = __bfloat1622float2(h[2]), f3 = __bfloat1622float2(h[3]);
        *reinterpret_cast<float4*>(&q_s[r * D + c8 * 8]) = make_float4(f0.x, f0.y, f1.x, f1.y);
        *reinterpret_cast<float4*>(&q_s[r * D + c8 * 8 + 4]) = make_float4(f2.x, f2.y, f3.x, f3.y);
      }
    }
    if (tid < RT) {
      m_s[tid] = -INFINITY;
      l_s[tid] = 0.f;
    }
  }

  // Start the copies of tokens [t0, t0 + nk) of `src` into stage s (keys past nk zero-filled).
  __device__ __forceinline__ void issue(const Source& src, int t0, int nk, int s) {
    __nv_bfloat16* ks = k_stage(s);
    __nv_bfloat16* vs = v_stage(s);
#pragma unroll
    for (int j = 0; j < kKeys * (D / 8) / kThreads; ++j) {
      const int i = tid + j * kThreads;
      const int k = i / (D / 8), c8 = i % (D / 8);
      const __nv_bfloat16* krow = src.K;
      const __nv_bfloat16* vrow = src.V;
      bool ok = k < nk;
      if (ok) {
        if (src.paged) {
          int outer, inner;
          locate_token(*src.paged, src.b, t0 + k, &outer, &inner);
          ok = outer != src.paged->n_pages;  // a page id outside the pool reads as zeros
          krow = src.paged->K + outer * src.paged->k_sb + src.kvh * src.paged->k_sh + inner * src.paged->k_st;
          vrow = src.paged->V + outer * src.paged->v_sb + src.kvh * src.paged->v_sh + inner * src.paged->v_st;
        } else {
          krow = src.K + (int64_t)(t0 + k) * src.k_st;
          vrow = src.V + (int64_t)(t0 + k) * src.v_st;
        }
      }
      cp_async16(&ks[k * KS + c8 * 8], ok ? krow + c8 * 8 : src.K, ok);
      cp_async16(&vs[k * KS + c8 * 8], ok ? vrow + c8 * 8 : src.V, ok);
    }
    cp_async_commit();
  }

  // One staged tile: scores, row statistics, a += P V.  `visible(r, k)` says whether row r of
  // the tile sees key k of the tile (history: always; local segment: the candidate mask).
  template <typename Vis>
  __device__ __forceinline__ void tile(int s, int nk, float scale_log2, Vis visible) {
    const __nv_bfloat16* ks = k_stage(s);
    const __nv_bfloat16* vs = v_stage(s);
    {  // scores: thread = (key, half of the rows)
      const int kk = tid % kKeys, rh = tid / kKeys;
      float sc[RH];
#pragma unroll
      for (int r = 0; r < RH; ++r) sc[r] = 0.f;
#pragma unroll 4
      for (int c8 = 0; c8 < D / 8; ++c8) {
        const uint4 raw = *reinterpret_cast<const uint4*>(&ks[kk * KS + c8 * 8]);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
        float kv[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(h[j]);
          kv[2 * j] = f.x;
          kv[2 * j + 1] = f.y;
        }
#pragma unroll
        for (int r = 0; r < RH; ++r) {
          const float4 qa = *reinterpret_cast<const float4*>(&q_s[(rh * RH + r) * D + c8 * 8]);
          const float4 qb = *reinterpret_cast<const float4*>(&q_s[(rh * RH + r) * D + c8 * 8 + 4]);
          sc[r] = fmaf(qa.x, kv[0], sc[r]);
          sc[r] = fmaf(qa.y, kv[1], sc[r]);
          sc[r] = fmaf(qa.z, kv[2], sc[r]);
          sc[r] = fmaf(qa.w, kv[3], sc[r]);
          sc[r] = fmaf(qb.x, kv[4], sc[r]);
          sc[r] = fmaf(qb.y, kv[5], sc[r]);
          sc[r] = fmaf(qb.z, kv[6], sc[r]);
          sc[r] = fmaf(qb.w, kv[7], sc[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < RH; ++r)
        p_s[(rh * RH + r) * (kKeys + 1) + kk] =
            (kk < nk && visible(rh * RH + r, kk)) ? sc[r] * scale_log2 : -INFINITY;
    }
    __syncthreads();
    // row statistics: warp w owns rows w * RW .. w * RW + RW - 1
#pragma unroll
    for (int rr = 0; rr < RW; ++rr) {
      const int r = warp * RW + rr;
      float* row = &p_s[r * (kKeys + 1)];
      const float s0 = row[lane], s1 = row[lane + 32];
      float mx = fmaxf(s0, s1);
#pragma unroll
      for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_old = m_s[r];
      const float m_new = fmaxf(m_old, mx);
      // a row that has seen nothing yet (everything masked so far) keeps the identity
      const float e0 = (m_new == -INFINITY) ? 0.f : exp2f(s0 - m_new);
      const float e1 = (m_new == -INFINITY) ? 0.f : exp2f(s1 - m_new);
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
    const int cp = tid % CP, tg = tid / CP;
#pragma unroll
    for (int r = 0; r < RT; ++r) {
      const float c = corr_s[r];
      acc[r][0] *= c;
      acc[r][1] *= c;
    }
    const int kend = min(nk, (tg + 1) * KPG);
#pragma unroll 4
    for (int k = tg * KPG; k < kend; ++k) {
      const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vs[k * KS + 2 * cp]));
#pragma unroll
      for (int r = 0; r < RT; ++r) {
        const float pr = p_s[r * (kKeys + 1) + k];
        acc[r][0] = fmaf(pr, v.x, acc[r][0]);
        acc[r][1] = fmaf(pr, v.y, acc[r][1]);
      }
    }
  }

  // Tokens [tok0, tok1) of `src`, two stages: the next tile's copies fly while this one is
  // worked on.  Ends with a CTA-wide barrier (the stages are free again).
  // `q_pending`: the Q rows are still in registers (q_fetch); they go to shared memory once the
  // first tile's copies are on their way.
  template <typename Vis>
  __device__ __forceinline__ void run(const Source& src, int tok0, int tok1, float scale_log2, Vis visible,
                                      bool& q_pending) {
    const int n = (tok1 - tok0 + kKeys - 1) / kKeys;
    if (n <= 0) return;
    issue(src, tok0, min(kKeys, tok1 - tok0), 0);
    if (q_pending) {
      q_store();
      q_pending = false;
    }
    for (int it = 0; it < n; ++it) {
      const int t0 = tok0 + it * kKeys;
      if (it + 1 < n) {
        issue(src, t0 + kKeys, min(kKeys, tok1 - t0 - kKeys), (it + 1) & 1);
        cp_async_wait<1>();
      } else {
        cp_async_wait<0>();
      }
      __syncthreads();
      const int base = t0 - tok0;
      tile(it & 1, min(kKeys, tok1 - t0), scale_log2, [&](int r, int k) { return visible(r, base + k); });
      __syncthreads();  // the stage is rewritten two tiles on, the weights by the next tile
    }
  }

  // Sum the token groups' partial outputs through shared memory (over the Q rows, which are
  // no longer needed); afterwards q_s[r * D + c] holds a[r][c].  Begins and ends synchronised.
  __device__ __forceinline__ void reduce_groups() {
    const int cp = tid % CP, tg = tid / CP;
    __syncthreads();
    for (int g = 0; g < TG; ++g) {
      if (tg == g) {
#pragma unroll
        for (int r = 0; r < RT; ++r) {
          float2* dst = reinterpret_cast<float2*>(&q_s[r * D + 2 * cp]);
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
  }
};

template <int D, int RT>
__global__ void __launch_bounds__(kThreads) chunk_simt_kernel(const __grid_constant__ ChunkParams p) {
  extern __shared__ __align__(16) uint8_t smem_simt[];
  Simt<D, RT> st;
  st.init(smem_simt);
  const int tid = threadIdx.x;
  if (p.wait_first) pdl_wait_prior();
  pdl_launch_dependents();
  const ChunkWork w = chunk_work(p, RT);
  const bool chain_cta = w.chain_cta;

  if (w.tok0 >= w.tok1) {  // nothing visible here: identity state
    if (tid < w.nrows) w.out_ml[tid] = make_float2(-INFINITY, 0.f);
    if (!p.wait_first && chain_cta) pdl_wait_prior();
    return;
  }
  st.q_fetch(p.Q, p.q_sb, p.q_sh, p.q_st, w.b, w.kvh, p.G, p.T_q, w.row0, w.nrows);
  bool q_pending = true;
  Source src;
  src.paged = p.page_table ? &p : nullptr;
  src.b = w.b;
  src.kvh = w.kvh;
  src.K = p.K + (p.page_table ? 0 : w.b * p.k_sb + w.kvh * p.k_sh);
  src.V = p.V + (p.page_table ? 0 : w.b * p.v_sb + w.kvh * p.v_sh);
  src.k_st = p.k_st;
  src.v_st = p.v_st;
  st.run(src, w.tok0, w.tok1, p.scale_log2, [](int, int) { return true; }, q_pending);
  st.reduce_groups();
  for (int i = tid; i < w.nrows * (D / 4); i += kThreads) {
    const int r = i / (D / 4), c4 = i % (D / 4);
    *reinterpret_cast<float4*>(w.out_a + (size_t)r * D + c4 * 4) =
        *reinterpret_cast<const float4*>(&st.q_s[r * D + c4 * 4]);
  }
  if (tid < w.nrows) w.out_ml[tid] = make_float2(st.m_s[tid], st.l_s[tid]);
  // Completion order along the stream: one CTA of this grid waits for the previous grid, so
  // this grid cannot complete before it (the other CTAs leave at once and free their SM slot).
  if (!p.wait_first && chain_cta) pdl_wait_prior();
}

// A whole round in one launch: grid = (row tiles x token splits, H_kv, B).  The history's
// 64-token tiles (all chunks, in order) are dealt to the splits in equal runs, the last split
// also takes the local segment.  With one split a CTA finalizes its rows itself.  With more,
// the splits of a (request, kv-head, row tile) form a thread-block cluster (p.cluster): every
// CTA leaves its partial state (m, l, a) in its own shared memory, and after a cluster barrier
// the first CTA reads all of them through distributed shared memory, merges (Eq. 14) and
// finalizes - no state goes through global memory.  Without clusters every CTA parks its state
// in scratch and takes a ticket from the unit's counter; the CTA that draws the last ticket
// merges, finalizes and leaves the counter at zero for the next round.  A round this small is
// bound by memory latency, not bandwidth: the splits are what puts enough loads in flight.
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of this CTA's shared-memory location `p` in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(const void* p, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
               : "=r"(r)
               : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(rank));
  return r;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t a) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t a) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(a)
               : "memory");
  return v;
}

template <int D, int RT>
__global__ void __launch_bounds__(kThreads) round_simt_kernel(const __grid_constant__ RoundParams p) {
  extern __shared__ __align__(16) uint8_t smem_simt[];
  __shared__ int s_last;
  Simt<D, RT> st;
  st.init(smem_simt);
  const int tid = threadIdx.x;
  const int row_tiles = gridDim.x / p.splits;   // p.splits counts the local segment's own CTA
  // (clusters run along x: the splits of a row tile are neighbours there, sp = rank in the cluster)
  const int rt = p.cluster ? blockIdx.x / p.splits : blockIdx.x % row_tiles;
  const int sp = p.cluster ? blockIdx.x % p.splits : blockIdx.x / row_tiles;
  const int b = blockIdx.z, kvh = blockIdx.y, row0 = rt * RT;
  const int R = p.T_q * p.G, nrows = min(RT, R - row0);
  // Launched with programmatic stream serialization, the grid is set up while the kernel before
  // it (typically the previous round's) is still running; nothing is read or written before
  // that kernel has completed.  The next launch is let in at once on the same terms.
  pdl_launch_dependents();
  pdl_wait_prior();
  st.q_fetch(p.Q, p.q_sb, p.q_sh, p.q_st, b, kvh, p.G, p.T_q, row0, nrows);
  bool q_pending = true;
  Source src;
  src.paged = nullptr;
  src.b = b;
  src.kvh = kvh;
  // this split's run of history tiles [g0, g1) in the concatenation of all chunks
  const int g0 = sp * p.tiles_per_split, g1 = g0 + p.tiles_per_split;
  int base = 0;  // global index of the chunk's first tile
  for (int j = 0; j < p.n_chunks; ++j) {
    const RoundChunk& c = p.chunk[j];
    const int n_t = (c.L_c + kKeys - 1) / kKeys;
    const int lo = max(g0, base), hi = min(g1, base + n_t);
    if (lo < hi) {
      int valid = c.L_c;
      if (c.valid_len) {
        valid = c.valid_len[b];
        if (valid < 0 || valid > c.L_c) {  // flagged and clamped, never trusted
          if (tid == 0 && p.status) atomicOr(p.status, SS_DEV_BAD_VALID_LEN);
          valid = max(0, min(valid, c.L_c));
        }
      }
      src.K = c.K + b * c.k_sb + kvh * c.k_sh;
      src.V = c.V + b * c.v_sb + kvh * c.v_sh;
      src.k_st = c.k_st;
      src.v_st = c.v_st;
      st.run(src, (lo - base) * kKeys, min(valid, (hi - base) * kKeys), p.scale_log2,
             [](int, int) { return true; }, q_pending);
    }
    base += n_t;
  }
  // the local segment: the last split's, or - with several splits - a CTA of its own
  if (p.T_loc > 0 && sp == p.loc_split) {
    src.K = p.K_loc + b * p.kl_sb + kvh * p.kl_sh;
    src.V = p.V_loc + b * p.vl_sb + kvh * p.vl_sh;
    src.k_st = p.kl_st;
    src.v_st = p.vl_st;
    const uint64_t* bits = p.mask_bits ? p.mask_bits + (int64_t)b * p.T_q * p.mask_words : nullptr;
    const int shift = p.T_loc - p.T_q, T_q = p.T_q, words = p.mask_words;
    st.run(src, 0, p.T_loc, p.scale_log2, [&](int r, int key) {
      if (r >= nrows) return false;
      const int i = (row0 + r) % T_q;  // candidate query of this row
      if (bits) return ((bits[(int64_t)i * words + (key >> 6)] >> (key & 63)) & 1ull) != 0;
      return key <= i + shift;
    }, q_pending);
  }
  if (q_pending) st.q_store();  // nothing to attend to here: the identity state
  st.reduce_groups();  // q_s[r][c] = a[r][c]
  if (p.splits > 1 && p.cluster) {
    // every CTA of the cluster holds its state in q_s / m_s / l_s; CTA 0 merges them (Eq. 14 over
    // all splits at once, every load of a phase independent of the others) through distributed
    // shared memory.  The second barrier keeps the other CTAs' shared memory alive until then.
    cluster_sync_all();
    if (sp == 0) {
      float* ml_all = st.p_s;  // [split][2 * RT]: the scores array is free by now
      for (int i = tid; i < p.splits * 2 * RT; i += kThreads)
        ml_all[i] = ld_cluster_f32(cluster_map(st.m_s + i % (2 * RT), i / (2 * RT)));  // (l_s follows m_s)
      __syncthreads();
      if (tid < RT) {
        float M = -INFINITY;
        for (int s2 = 0; s2 < p.splits; ++s2) M = fmaxf(M, ml_all[s2 * 2 * RT + tid]);
        float l = 0.f;
        for (int s2 = 0; s2 < p.splits; ++s2) {
          const float m2 = ml_all[s2 * 2 * RT + tid];
          const float f = m2 > -INFINITY ? exp2f(m2 - M) : 0.f;
          l += f * ml_all[s2 * 2 * RT + RT + tid];
          ml_all[s2 * 2 * RT + tid] = f;  // the split's factor for this row replaces its maximum
        }
        st.m_s[tid] = M;
        st.l_s[tid] = l;
      }
      __syncthreads();
      for (int i = tid; i < RT * D / 4; i += kThreads) {
        const int r = i / (D / 4);
        float4 v[16];
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2)
          v[s2] = s2 < p.splits ? ld_cluster_f32x4(cluster_map(st.q_s + 4 * i, s2)) : make_float4(0.f, 0.f, 0.f, 0.f);
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2) {
          const float f = s2 < p.splits ? ml_all[s2 * 2 * RT + r] : 0.f;
          if (f > 0.f) {  // a split that saw nothing holds no a[]
            a.x += f * v[s2].x;
            a.y += f * v[s2].y;
            a.z += f * v[s2].z;
            a.w += f * v[s2].w;
          }
        }
        reinterpret_cast<float4*>(st.q_s)[i] = a;   // (the thread's own piece of CTA 0's state)
      }
      __syncthreads();
    }
    cluster_sync_all();
    if (sp != 0) return;
  } else if (p.splits > 1) {
    // park the partial state, take a ticket; only the CTA with the last ticket goes on
    const int64_t unit = ((int64_t)b * p.H_kv + kvh) * row_tiles + rt;
    float* slot = p.scratch + (unit * p.splits + sp) * (int64_t)(RT * (D + 2));
    for (int i = tid; i < RT * D / 4; i += kThreads)
      reinterpret_cast<float4*>(slot + 2 * RT)[i] = reinterpret_cast<const float4*>(st.q_s)[i];
    if (tid < RT) {
      slot[tid] = st.m_s[tid];
      slot[RT + tid] = st.l_s[tid];
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const unsigned int ticket = atomicAdd(&p.counters[unit], 1u);
      s_last = ticket == (unsigned int)p.splits - 1;
      if (s_last) p.counters[unit] = 0;  // every CTA of this unit has drawn: ready for the next round
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // merge: common maximum, rescaled sums (Eq. 14 over all splits at once).  Every load of a
    // phase is independent of the others, so a phase costs one trip to L2, not one per split.
    const float* first = p.scratch + unit * p.splits * (int64_t)(RT * (D + 2));
    constexpr int kSlot = RT * (D + 2);
    float* ml_all = st.p_s;  // [split][2 * RT]: the scores array is free by now
    static_assert(16 * 2 * RT <= RT * (kKeys + 1), "all (m, l) pairs fit the scores array");
    for (int i = tid; i < p.splits * 2 * RT; i += kThreads)
      ml_all[i] = __ldcg(first + (int64_t)(i / (2 * RT)) * kSlot + i % (2 * RT));
    __syncthreads();
    if (tid < RT) {
      float M = -INFINITY;
      for (int s2 = 0; s2 < p.splits; ++s2) M = fmaxf(M, ml_all[s2 * 2 * RT + tid]);
      float l = 0.f;
      for (int s2 = 0; s2 < p.splits; ++s2) {
        const float m2 = ml_all[s2 * 2 * RT + tid];
        const float f = m2 > -INFINITY ? exp2f(m2 - M) : 0.f;
        l += f * ml_all[s2 * 2 * RT + RT + tid];
        ml_all[s2 * 2 * RT + tid] = f;  // the split's factor for this row replaces its maximum
      }
      st.m_s[tid] = M;
      st.l_s[tid] = l;
    }
    __syncthreads();
    for (int i = tid; i < RT * D / 4; i += kThreads) {
      const int r = i / (D / 4);
      float4 v[16];
#pragma unroll
      for (int s2 = 0; s2 < 16; ++s2)
        v[s2] = s2 < p.splits ? __ldcg(reinterpret_cast<const float4*>(first + (int64_t)s2 * kSlot + 2 * RT) + i)
                              : make_float4(0.f, 0.f, 0.f, 0.f);
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s2 = 0; s2 < 16; ++s2) {
        const float f = s2 < p.splits ? ml_all[s2 * 2 * RT + r] : 0.f;
        if (f > 0.f) {  // a split that saw nothing holds no a[]
          a.x += f * v[s2].x;
          a.y += f * v[s2].y;
          a.z += f * v[s2].z;
          a.w += f * v[s2].w;
        }
      }
      reinterpret_cast<float4*>(st.q_s)[i] = a;
    }
    __syncthreads();
  }
  // O = a / l as bf16 (a row that saw nothing: O = 0), LSE = (m + log2 l) ln 2
  for (int i = tid; i < nrows * (D / 2); i += kThreads) {
    const int r = i / (D / 2), c2 = i % (D / 2);
    const int rg = row0 + r, g = rg / p.T_q, t = rg % p.T_q;
    const float l = st.l_s[r];
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const float2 a = *reinterpret_cast<const float2*>(&st.q_s[r * D + 2 * c2]);
    __nv_bfloat16* o = p.O + (((int64_t)b * p.H_q + kvh * p.G + g) * p.T_q + t) * D;
    *reinterpret_cast<__nv_bfloat162*>(o + 2 * c2) = __floats2bfloat162_rn(a.x * inv, a.y * inv);
  }
  if (p.LSE && tid < nrows) {
    const int rg = row0 + tid, g = rg / p.T_q, t = rg % p.T_q;
    const float l = st.l_s[tid];
    p.LSE[((int64_t)b * p.H_q + kvh * p.G + g) * p.T_q + t] =
        l > 0.f ? (st.m_s[tid] + log2f(l)) * 0.6931471805599453f : -INFINITY;
  }
}

template <int D, int RT>
cudaError_t prepare_one() {
  cudaError_t e = cudaFuncSetAttribute(chunk_simt_kernel<D, RT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       Lay<D, RT>::kBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(round_simt_kernel<D, RT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Lay<D, RT>::kBytes);
  if (e == cudaSuccess)  // clusters of up to 16 CTAs (more than the portable 8)
    e = cudaFuncSetAttribute(round_simt_kernel<D, RT>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  return e;
}

}  // namespace

// Rows per CTA tile for R rows per kv-head: the smallest of 8 / 16 / 32 that holds them (32
// with several row tiles above that).
int simt_rows_per_tile(int R) { return R <= 8 ? 8 : (R <= 16 ? 16 : 32); }

cudaError_t chunk_simt_prepare() {
  cudaError_t e = prepare_one<64, 8>();
  if (e == cudaSuccess) e = prepare_one<64, 16>();
  if (e == cudaSuccess) e = prepare_one<64, 32>();
  if (e == cudaSuccess) e = prepare_one<128, 8>();
  if (e == cudaSuccess) e = prepare_one<128, 16>();
  if (e == cudaSuccess) e = prepare_one<128, 32>();
  return e;
}

#define SS_SIMT_DISPATCH(KERNEL, D_, RT_, ...)                                                   \
  ((D_) == 128 ? ((RT_) == 8    ? launch_kernel(KERNEL<128, 8>, __VA_ARGS__)                      \
                  : (RT_) == 16 ? launch_kernel(KERNEL<128, 16>, __VA_ARGS__)                     \
                                : launch_kernel(KERNEL<128, 32>, __VA_ARGS__))                    \
               : ((RT_) == 8    ? launch_kernel(KERNEL<64, 8>, __VA_ARGS__)                       \
                  : (RT_) == 16 ? launch_kernel(KERNEL<64, 16>, __VA_ARGS__)                      \
                                : launch_kernel(KERNEL<64, 32>, __VA_ARGS__)))

static size_t simt_smem(int d, int rt) {
  if (d == 128) return rt == 8 ? Lay<128, 8>::kBytes : (rt == 16 ? Lay<128, 16>::kBytes : Lay<128, 32>::kBytes);
  return rt == 8 ? Lay<64, 8>::kBytes : (rt == 16 ? Lay<64, 16>::kBytes : Lay<64, 32>::kBytes);
}

// p.rows_per_tile must be simt_rows_per_tile(p.R) and p.row_tiles the matching tile count.
cudaError_t launch_chunk_simt(const ChunkParams& p, cudaStream_t s, bool pdl) {
  dim3 grid(p.splits * p.row_tiles, p.H_kv, p.n_active ? p.n_active : p.B), block(kThreads);
  const size_t smem = simt_smem(p.d, p.rows_per_tile);
  return SS_SIMT_DISPATCH(chunk_simt_kernel, p.d, p.rows_per_tile, grid, block, smem, s, pdl, p);
}

#define SS_SIMT_DISPATCH_CLUSTER(KERNEL, D_, RT_, ...)                                           \
  ((D_) == 128 ? ((RT_) == 8    ? launch_kernel_cluster(KERNEL<128, 8>, __VA_ARGS__)              \
                  : (RT_) == 16 ? launch_kernel_cluster(KERNEL<128, 16>, __VA_ARGS__)             \
                                : launch_kernel_cluster(KERNEL<128, 32>, __VA_ARGS__))            \
               : ((RT_) == 8    ? launch_kernel_cluster(KERNEL<64, 8>, __VA_ARGS__)               \
                  : (RT_) == 16 ? launch_kernel_cluster(KERNEL<64, 16>, __VA_ARGS__)              \
                                : launch_kernel_cluster(KERNEL<64, 32>, __VA_ARGS__)))

// p.cluster: the p.splits (2 to 16) CTAs of a unit are launched as one cluster along x.
cudaError_t launch_round_simt(const RoundParams& p, cudaStream_t s, bool pdl) {
  const int R = p.T_q * p.G, rt = p.rows_per_tile;
  dim3 grid(((R + rt - 1) / rt) * p.splits, p.H_kv, p.B), block(kThreads);
  const size_t smem = simt_smem(p.d, rt);
  if (p.cluster) {
    if (p.splits < 2 || p.splits > 16) return cudaErrorInvalidValue;
    return SS_SIMT_DISPATCH_CLUSTER(round_simt_kernel, p.d, rt, grid, block, smem, s, pdl, (unsigned)p.splits, p);
  }
  return SS_SIMT_DISPATCH(round_simt_kernel, p.d, rt, grid, block, smem, s, pdl, p);
}

}  // namespace ss
