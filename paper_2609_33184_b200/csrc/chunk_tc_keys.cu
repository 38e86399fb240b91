// Tensor-core chunk attention for few rows per kv-head (R <= 32): keys on the MMA's M axis.
//
// With R = T_q * G <= 32 query rows per kv-head, putting the rows on the 128-wide M axis wastes
// three quarters of every MMA.  Here the contraction is transposed instead:
//
//   S^T = K Q^T   M = 128 keys of the tile, N = 32 rows, K = d = 128   (8 x k16, smem x smem)
//   O^T = V^T P^T M = 128 head dims,        N = 32 rows, K = 128 keys  (8 x k16, smem x smem)
//
// so the tensor work is proportional to the rows that exist.  One CTA = one (request, kv-head,
// token split); 192 threads: warps 0-3 softmax, warp 4 TMA producer, warp 5 MMA issuer.
//
//  * K and V tiles of 128 tokens (two [128][64] bf16 boxes each, 128-byte swizzle) go through
//    a ring of three 32 KB units in the order K0 V0 K1 V1 ...; a K unit is released when its
//    score MMAs retire, a V unit after its output MMAs.  V^T is fed as an MN-major A operand
//    straight from the [token][d] tile.
//  * S^T sits in tensor memory, double buffered (2 x 32 columns): thread L of the softmax
//    warps owns TMEM lane L = key L of the tile and sees that key's scores against all rows.
//    Ragged tails are a per-thread select (key >= valid -> weight 0).
//  * The row reference m[r] is shared by all keys, so it cannot follow each tile's maximum
//    without a cross-lane reduction.  It is kept lazily: weights are exp2(x - m[r]) with the
//    current m[r]; only if some x - m[r] exceeds 16 (always on the first tile, where
//    m = -inf) do the 128 threads agree (one named barrier per tile) to take the exact tile
//    maxima (warp shuffles + shared memory), raise m, and rescale O^T and the row sums.
//    Any common reference gives the same a / l (Eq. 17), so this is exact.
//  * Row sums l[r] accumulate per thread (per key lane) in registers and are reduced across
//    the 128 lanes once, when the CTA ends.
//  * P^T goes to shared memory as the MN-major B operand (unswizzled 8x8 core matrices: each
//    thread writes four 16-byte pieces, a warp's pieces are contiguous).
//  * O^T accumulates in tensor memory (32 columns); at the end thread L holds head dim L of
//    every row and writes a[r][L], coalesced over L.
//
// 112 KB of shared memory and 128 TMEM columns per CTA: two CTAs per SM, so one CTA's ramp-up
// and tail overlap the other's steady state (also across consecutive chunk kernels).
// Every mbarrier wait is bounded; on expiry the CTA raises SS_DEV_WAIT_EXPIRED, lets its own
// copies land (bounded), frees its tensor memory and returns.
#include <cstddef>

#include "ss_internal.h"
#include "tc_ptx.cuh"

namespace ss {
namespace {

using namespace ss::tc;

constexpr int kThreads = 192;
constexpr int kD = 128;
constexpr int kKeys = 128;                     // keys per tile = MMA M
constexpr int kN = 32;                         // padded query rows = MMA N
constexpr int kUnits = 3;                      // ring of K / V tiles
constexpr int kHalf = kKeys * 64 * 2;          // 16 KB: [128 keys][64 d] bf16
constexpr int kUnitBytes = 2 * kHalf;          // 32 KB: one K tile or one V tile
constexpr int kQHalf = kN * 64 * 2;            // 4 KB: [32 rows][64 d]
constexpr int kQBytes = 2 * kQHalf;            // 8 KB
constexpr int kPBytes = kKeys * kN * 2;        // 8 KB: P^T
constexpr int kOffQ = kUnits * kUnitBytes;     // 96 KB
constexpr int kOffP = kOffQ + kQBytes;
constexpr int kOffCtl = kOffP + kPBytes;       // 112 KB
constexpr int kCtlBytes = 1024;
constexpr int kSmemTotal = kOffCtl + kCtlBytes;
constexpr uint32_t kTmemCols = 128;
constexpr uint32_t kColS = 0, kColO = 2 * kN;  // S^T buffers at 0 and 32, O^T at 64
constexpr float kLazyThreshold = 16.f;

struct Ctl {
  uint64_t ufull[kUnits], uempty[kUnits];
  uint64_t sfull[2], pready, pfree;
  uint32_t tmem_base;
  volatile uint32_t abort;
  volatile uint32_t flag[3];
  alignas(16) float m_ref[kN];  // read as float4
  alignas(16) float smax[4][kN];
};
static_assert(offsetof(Ctl, m_ref) % 16 == 0, "m_ref is read with 16-byte loads");
static_assert(sizeof(Ctl) <= kCtlBytes, "control block");

__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Ctl* ctl, uint32_t* status) {
  return mbar_wait_abortable(bar, parity, &ctl->abort, status);
}
__device__ __forceinline__ void trace(unsigned long long* tr, int role, int it, int ev) {
  if (tr && it < kTraceTiles) tr[(role * kTraceTiles + it) * 8 + ev] = clock64();
}

__global__ void __launch_bounds__(kThreads, 2)
chunk_tc_keys_kernel(const ChunkParams p, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Ctl* ctl = reinterpret_cast<Ctl*>(smem + kOffCtl);
  uint8_t* q_s = smem + kOffQ;
  uint8_t* p_s = smem + kOffP;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.x;
  const int kvh = blockIdx.y, b = blockIdx.z;
  const int nrows = p.R;  // <= kN
  unsigned long long* tr = (blockIdx.x | blockIdx.y | blockIdx.z) ? nullptr : p.trace;

  const bool chain_cta = (blockIdx.x | blockIdx.y | blockIdx.z) == 0;
  if (p.wait_first) pdl_wait_prior();
  pdl_launch_dependents();

  int valid = p.L_c;
  if (p.valid_len) {
    valid = p.valid_len[b];
    if (valid < 0 || valid > p.L_c) {
      if (tid == 0) atomicOr(p.status, SS_DEV_BAD_VALID_LEN);
      valid = max(0, min(valid, p.L_c));
    }
  }
  // splits are given in 64-token tiles by the host; this kernel walks 128-token tiles
  const int tok0 = split * p.tiles_per_split * kTileKeys;
  const int tok1 = min(valid, tok0 + p.tiles_per_split * kTileKeys);
  const int n_tiles = (tok1 > tok0) ? (tok1 - tok0 + kKeys - 1) / kKeys : 0;

  const size_t slot = ((size_t)split * p.B + b) * p.H_kv + kvh;
  float2* out_ml = p.part_ml + slot * p.R_stride;
  float* out_a = p.part_a + slot * p.R_stride * kD;

  if (n_tiles == 0 || (smem_u32(smem) & 1023u)) {
    // nothing visible here (identity state, no tensor memory taken); a misaligned shared
    // memory window would break the swizzled layouts and is reported instead of run
    if (n_tiles && tid == 0) atomicOr(p.status, SS_DEV_WAIT_EXPIRED);
    if (tid < nrows) out_ml[tid] = make_float2(-INFINITY, 0.f);
    if (!p.wait_first && chain_cta) pdl_wait_prior();
    return;
  }

  // ---- set-up ------------------------------------------------------------------------------
  // use j of the ring: K of tile t is j = 2t, V of tile t is j = 2t + 1; unit j % 3
  auto issue_use = [&](int j, uint64_t pol) {
    const int u = j % kUnits;
    const int tok = tok0 + (j >> 1) * kKeys;
    const uint32_t dst = smem_u32(smem + u * kUnitBytes);
    const CUtensorMap* tm = (j & 1) ? &tmV : &tmK;
    mbar_expect_tx(&ctl->ufull[u], kUnitBytes);
    tma_load_4d(dst, tm, 0, tok, kvh, b, &ctl->ufull[u], pol);
    tma_load_4d(dst + kHalf, tm, 64, tok, kvh, b, &ctl->ufull[u], pol);
  };
  const int n_uses = 2 * n_tiles;
  const int n_pre = min(n_uses, kUnits);
  if (warp == 4) {
    if (lane == 0) {
      for (int u = 0; u < kUnits; ++u) {
        mbar_init(&ctl->ufull[u], 1);
        mbar_init(&ctl->uempty[u], 1);
      }
      mbar_init(&ctl->sfull[0], 1);
      mbar_init(&ctl->sfull[1], 1);
      mbar_init(&ctl->pready, 128);
      mbar_init(&ctl->pfree, 1);
      ctl->abort = 0;
      ctl->flag[0] = ctl->flag[1] = ctl->flag[2] = 0;
      fence_barrier_init();
      const uint64_t pol = l2_evict_first_policy();
      for (int j = 0; j < n_pre; ++j) issue_use(j, pol);  // first loads before the rest is set up
    }
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&ctl->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else if (warp < 4) {
    // Q rows -> shared memory as the K-major B operand (128-byte swizzle), zero padding rows
    for (int i = tid; i < kN * (kD / 8); i += 128) {
      const int n = i / (kD / 8), c8 = i % (kD / 8);
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (n < nrows) {
        const int g = n / p.T_q, t = n % p.T_q;
        raw = *reinterpret_cast<const uint4*>(p.Q + b * p.q_sb + (int64_t)(kvh * p.G + g) * p.q_sh +
                                              t * p.q_st + c8 * 8);
      }
      const int half = c8 >> 3, j = c8 & 7;
      *reinterpret_cast<uint4*>(q_s + half * kQHalf + n * 128 + ((j ^ (n & 7)) << 4)) = raw;
    }
    if (tid < kN) ctl->m_ref[tid] = -INFINITY;
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  unsigned long long* trl = lane == 0 ? tr : nullptr;

  if (warp == 4) {
    // ===== TMA producer =====
    if (lane == 0) {
      const uint64_t pol = l2_evict_first_policy();
      int issued = n_pre;
      for (int j = n_pre; j < n_uses; ++j) {
        const int u = j % kUnits;
        const uint32_t ph = (j / kUnits) & 1;
        trace(tr, 0, j >> 1, (j & 1) * 2);
        if (!mbar_wait(&ctl->uempty[u], ph ^ 1, ctl, p.status)) break;
        trace(tr, 0, j >> 1, (j & 1) * 2 + 1);
        issue_use(j, pol);
        issued = j + 1;
      }
      if (ctl->abort) {
        // let the copies this thread started land before the CTA leaves (bounded)
        const unsigned long long t0 = gtime_ns();
        for (int j = max(0, issued - kUnits); j < issued; ++j)
          while (!mbar_try_wait(&ctl->ufull[j % kUnits], (j / kUnits) & 1) &&
                 gtime_ns() - t0 < kWaitNs) {
          }
      }
    }
  } else if (warp == 5) {
    // ===== MMA issuer: the whole warp walks the loop, one elected lane issues =====
    constexpr uint32_t idesc_qk = make_idesc_major(128, kN, false, false);
    constexpr uint32_t idesc_pv = make_idesc_major(128, kN, true, true);
    const bool leader = elect_one();
    const uint32_t base = smem_u32(smem);
    const uint32_t q_addr = smem_u32(q_s), p_addr = smem_u32(p_s);
    auto issue_qk = [&](int t) {  // S^T[t & 1] = K(t) Q^T
      const uint32_t k_addr = base + ((2 * t) % kUnits) * kUnitBytes;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint32_t off = (kk & 3) * 32;
          mma_ss(tmem + kColS + (t & 1) * kN, desc_kmajor(k_addr + (kk >> 2) * kHalf + off),
                 desc_kmajor(q_addr + (kk >> 2) * kQHalf + off), idesc_qk, kk > 0);
        }
        tc_commit(&ctl->uempty[(2 * t) % kUnits]);
        tc_commit(&ctl->sfull[t & 1]);
      }
      __syncwarp();
    };
    bool ok = mbar_wait(&ctl->ufull[0], 0, ctl, p.status);
    if (ok) {
      tc_fence_after();
      issue_qk(0);
    }
    for (int t = 0; ok && t < n_tiles; ++t) {
      trace(trl, 1, t, 0);
      if (t + 1 < n_tiles) {
        // scores of the next tile go out first: its softmax overlaps this tile's output MMAs.
        // S^T[(t+1) & 1] was last read for tile t-1, whose pready was awaited in iteration t-1.
        const int j = 2 * (t + 1);
        ok = mbar_wait(&ctl->ufull[j % kUnits], (j / kUnits) & 1, ctl, p.status);
        if (!ok) break;
        trace(trl, 1, t, 1);
        tc_fence_after();
        issue_qk(t + 1);
        trace(trl, 1, t, 2);
      }
      const int jv = 2 * t + 1;
      ok = mbar_wait(&ctl->pready, t & 1, ctl, p.status);
      trace(trl, 1, t, 3);
      ok = ok && mbar_wait(&ctl->ufull[jv % kUnits], (jv / kUnits) & 1, ctl, p.status);
      if (!ok) break;
      trace(trl, 1, t, 4);
      tc_fence_after();
      const uint32_t v_addr = base + (jv % kUnits) * kUnitBytes;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < kKeys / 16; ++kk) {
          // A = V^T: MN-major, 64 head dims (128 bytes) per token row, 8-token atoms 1024 bytes
          // apart, the other 64 head dims one half-tile away.  B = P^T: plain 8x8 core matrices.
          mma_ss(tmem + kColO, desc_mnmajor(v_addr + kk * 2048, kHalf),
                 desc_mnmajor_plain(p_addr + kk * 256, 128, kKeys * 16), idesc_pv,
                 (t > 0 || kk > 0));
        }
        tc_commit(&ctl->uempty[jv % kUnits]);
        tc_commit(&ctl->pfree);
      }
      __syncwarp();
      trace(trl, 1, t, 5);
    }
  } else {
    // ===== softmax warps: thread L = TMEM lane L = key L of the tile =====
    // A wait that gives up makes the whole warp `dead`: it keeps walking the loop and the
    // named barriers (so nobody is left waiting) but touches nothing else.
    const int L = tid;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    bool dead = false;
    auto wait = [&](uint64_t* bar, uint32_t parity) {
      if (!dead && !mbar_wait(bar, parity, ctl, p.status)) dead = true;
      dead = __any_sync(0xffffffffu, dead);
    };
    float lsum[kN];
#pragma unroll
    for (int r = 0; r < kN; ++r) lsum[r] = 0.f;
    for (int t = 0; t < n_tiles; ++t) {
      if (L == 0) trace(tr, 2, t, 0);
      wait(&ctl->sfull[t & 1], (t >> 1) & 1);
      tc_fence_after();
      if (L == 0) trace(tr, 2, t, 1);
      const int n_valid = min(kKeys, tok1 - (tok0 + t * kKeys));
      const bool key_ok = L < n_valid;
      if (n_valid < kKeys) {
        // ragged tail: tokens past the valid length may hold anything; their weights are 0, so
        // V must be finite there: clear those rows of the staged V tile (both halves)
        const int jv = 2 * t + 1;
        wait(&ctl->ufull[jv % kUnits], (jv / kUnits) & 1);
        if (!dead) {
          uint8_t* v_s = smem + (jv % kUnits) * kUnitBytes;
          const int n_vec = (kKeys - n_valid) * 16;
          for (int i = L; i < n_vec; i += 128) {
            const int row = n_valid + (i >> 4), half = (i >> 3) & 1, ch = i & 7;
            *reinterpret_cast<uint4*>(v_s + half * kHalf + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
          }
        }
        // made visible to the tensor core by the proxy fence before pready below
      }
      uint32_t raw[2][16];
      float x[kN];
      bool over = false;
      if (!dead) {
        tmem_ld16(tmem + lane_off + kColS + (t & 1) * kN, raw[0]);
        tmem_ld16(tmem + lane_off + kColS + (t & 1) * kN + 16, raw[1]);
        tc_wait_ld();
        float mx = -INFINITY;
#pragma unroll
        for (int r4 = 0; r4 < kN / 4; ++r4) {
          const float4 mr = *reinterpret_cast<const float4*>(&ctl->m_ref[r4 * 4]);
          const float mm[4] = {mr.x, mr.y, mr.z, mr.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int r = r4 * 4 + e;
            const float s2 = __uint_as_float(raw[r / 16][r % 16]) * p.scale_log2;
            x[r] = s2 - mm[e];  // +inf while m_ref is -inf
            mx = fmaxf(mx, x[r]);
          }
        }
        over = key_ok && (mx > kLazyThreshold);
      }
      if (L == 0) ctl->flag[(t + 1) % 3] = 0;
      if (__any_sync(0xffffffffu, over) && lane == 0) ctl->flag[t % 3] = 1;
      named_bar_sync(1, 128);
      if (ctl->flag[t % 3]) {
        // ---- raise the row references to the exact tile maxima (rare after the first tile) ----
        if (!dead) {
#pragma unroll
          for (int r = 0; r < kN; ++r) {
            float v = key_ok ? __uint_as_float(raw[r / 16][r % 16]) * p.scale_log2 : -INFINITY;
            v = warp_max_f(v);
            if (lane == 0) ctl->smax[warp][r] = v;
          }
        }
        named_bar_sync(1, 128);
        if (t > 0) {  // O^T must be at rest: the output MMAs of tile t-1 have retired
          wait(&ctl->pfree, (t - 1) & 1);
          tc_fence_after();
        }
        if (!dead) {
          float f[kN];
#pragma unroll
          for (int r = 0; r < kN; ++r) {
            const float m_old = ctl->m_ref[r];
            const float m_new = fmaxf(fmaxf(m_old, ctl->smax[0][r]),
                                      fmaxf(fmaxf(ctl->smax[1][r], ctl->smax[2][r]), ctl->smax[3][r]));
            f[r] = (m_old == -INFINITY) ? 0.f : exp2f(m_old - m_new);
            lsum[r] *= f[r];
            x[r] = __uint_as_float(raw[r / 16][r % 16]) * p.scale_log2 - m_new;
          }
          if (t > 0) {
#pragma unroll
            for (int q = 0; q < kN / 16; ++q) {
              uint32_t o[16];
              tmem_ld16(tmem + lane_off + kColO + q * 16, o);
              tc_wait_ld();
#pragma unroll
              for (int c = 0; c < 16; ++c)
                o[c] = __float_as_uint(__uint_as_float(o[c]) * f[q * 16 + c]);
              tmem_st16(tmem + lane_off + kColO + q * 16, o);
            }
            tc_wait_st();
          }
        }
        named_bar_sync(1, 128);  // every thread has read the old references
        if (L < kN && !dead) {
          const float m_old = ctl->m_ref[L];
          ctl->m_ref[L] = fmaxf(fmaxf(m_old, ctl->smax[0][L]),
                                fmaxf(fmaxf(ctl->smax[1][L], ctl->smax[2][L]), ctl->smax[3][L]));
        }
        named_bar_sync(1, 128);
      }
      // weights, row sums, P^T as bf16
      uint32_t pk[kN / 2];
      if (!dead) {
#pragma unroll
        for (int r = 0; r < kN; r += 2) {
          const float p0 = key_ok ? exp2f(x[r]) : 0.f;
          const float p1 = key_ok ? exp2f(x[r + 1]) : 0.f;
          lsum[r] += p0;
          lsum[r + 1] += p1;
          __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);  // low half = even row
          pk[r / 2] = *reinterpret_cast<uint32_t*>(&h);
        }
      }
      if (t > 0) wait(&ctl->pfree, (t - 1) & 1);  // the output MMAs of tile t-1 consumed P^T
      if (!dead) {
#pragma unroll
        for (int c = 0; c < kN / 8; ++c)  // rows 8c..8c+7 of key L: one 16-byte piece
          *reinterpret_cast<uint4*>(p_s + c * (kKeys * 16) + L * 16) =
              make_uint4(pk[c * 4], pk[c * 4 + 1], pk[c * 4 + 2], pk[c * 4 + 3]);
        fence_proxy_async();
        tc_fence_before();
      }
      mbar_arrive(&ctl->pready);
      if (L == 0) trace(tr, 2, t, 2);
    }
    wait(&ctl->pfree, (n_tiles - 1) & 1);
    named_bar_sync(1, 128);
    if (ctl->abort == 0) {  // uniform over the 128 threads after the barrier
      tc_fence_after();
      // ---- row sums across the 128 key lanes, then the partial state ----
      float* red = reinterpret_cast<float*>(smem);  // [128][33] over the free ring
#pragma unroll
      for (int r = 0; r < kN; ++r) red[L * (kN + 1) + r] = lsum[r];
      named_bar_sync(1, 128);
      if (L < nrows) {
        float lt = 0.f;
        for (int k = 0; k < kKeys; ++k) lt += red[k * (kN + 1) + L];
        out_ml[L] = make_float2(lt > 0.f ? ctl->m_ref[L] : -INFINITY, lt);
      }
      // thread L holds head dim L of every row
      uint32_t o[2][16];
      tmem_ld16(tmem + lane_off + kColO, o[0]);
      tmem_ld16(tmem + lane_off + kColO + 16, o[1]);
      tc_wait_ld();
#pragma unroll
      for (int r = 0; r < kN; ++r)
        if (r < nrows) out_a[(size_t)r * kD + L] = __uint_as_float(o[r / 16][r % 16]);
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
  }
  // Completion order along the stream: one CTA of this grid waits for the previous grid, so
  // this grid cannot complete before it (the other CTAs leave at once and free their SM slot).
  if (!p.wait_first && chain_cta) pdl_wait_prior();
}

}  // namespace

cudaError_t chunk_tc_keys_prepare() {
  return cudaFuncSetAttribute(chunk_tc_keys_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmemTotal);
}

cudaError_t launch_chunk_tc_keys(const ChunkParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                 cudaStream_t s, bool pdl) {
  dim3 grid(p.splits, p.H_kv, p.B), block(kThreads);
  return launch_kernel(chunk_tc_keys_kernel, grid, block, kSmemTotal, s, pdl, p, tmK, tmV);
}

}  // namespace ss
