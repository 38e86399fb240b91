// Tensor-core chunk attention with the keys on the MMA's M axis.
//
// The rows of a kv-head (T_q candidate queries x G query heads) are few compared with the
// 128-wide M axis of tcgen05.mma, so the contraction is transposed:
//
//   S^T = K Q^T   M = 128 keys of the tile, N = rows (16..128), K = d = 128   (8 x k16)
//   O^T = V^T P^T M = 128 head dims,        N = rows,           K = 128 keys  (8 x k16)
//
// and the tensor work is proportional to the rows that exist (no padding of M).  One CTA =
// one (request, kv-head, token split, group of <= 128 rows); kv-heads with more rows use
// several row groups (their CTAs are adjacent in the grid and share K/V through L2).
//
//  * Warps: 4*WG softmax warps, one TMA producer warp, one MMA issuer warp.
//  * K and V tiles of 128 tokens (two [128][64] bf16 boxes each, 128-byte swizzle, evict-first)
//    go through a ring of 32 KB units in the order K0 V0 K1 V1 ...; a K unit is released when
//    its score MMAs retire, a V unit after its output MMAs.  V^T is fed as an MN-major A
//    operand straight from the [token][d] tile.
//  * S^T sits in tensor memory, double buffered: a softmax thread owns TMEM lane L = key L of
//    the tile and a block of the score columns (= rows); with WG = 2 two threads share a lane
//    and split the columns.  Ragged tails are a per-thread select (key >= valid -> weight 0).
//  * The row reference m[r] is shared by all keys, so it cannot follow each tile's maximum
//    without a cross-lane reduction.  It is kept lazily: it starts as the exact maxima of the
//    first tile; weights are exp2(s - m[r]) with the current m[r]; only if some s - m[r] exceeds
//    16 do the softmax threads agree (one named barrier per tile) to take the exact tile maxima
//    (warp shuffles + shared memory), raise m, and rescale O^T and the row sums.  Any common
//    reference gives the same a / l (Eq. 17), so this is exact.
//  * Row sums l[r] accumulate per thread in registers and are reduced across the 128 key
//    lanes once, when the CTA ends.
//  * P^T goes to shared memory as the MN-major B operand (unswizzled 8x8 core matrices: a
//    thread writes 16-byte pieces, a warp's pieces are contiguous).
//  * O^T accumulates in tensor memory; at the end a thread holds head dim L of its rows and
//    writes a[r][L], coalesced over L.
//
// Rows <= 32: 3 ring units, 113 KB shared memory, 128 TMEM columns -> two CTAs per SM, so one
// CTA's ramp-up and tail overlap the other's steady state (also across consecutive kernels).
// Rows up to 64 / 128: 6 / 5 ring units, one CTA per SM, 8 / 16 softmax warps (the latency of
// tensor-memory loads is hidden by warps, not by holding more columns per thread).
// Every mbarrier wait is bounded; on expiry the CTA raises SS_DEV_WAIT_EXPIRED, lets its own
// copies land (bounded), frees its tensor memory and returns.
#include <cstddef>

#include "ss_internal.h"
#include "tc_ptx.cuh"

namespace ss {
namespace {

using namespace ss::tc;

constexpr int kKeys = 128;                  // keys per tile = MMA M
constexpr int kHalf = kKeys * 64 * 2;       // 16 KB: [128 keys][64 d] bf16, one TMA box
constexpr float kLazyThreshold = 16.f;
constexpr int kMaxHistChunksKeys = kMaxHistChunks;   // chunks one launch over a list of chunks takes (table in the control block)

template <int N>
struct alignas(16) Ctl {
  uint64_t ufull[8], uempty[8];
  uint64_t sfull[2], pready, pfree;
  uint32_t tmem_base;
  volatile uint32_t abort;
  volatile uint32_t flag[3];
  alignas(16) float nm_ref[N];    // NEGATED row references -m[r] (+inf = none yet); read as float4
  alignas(16) float smax[4][N];   // per lane quadrant
  // launch over a list of chunks: 128-token tiles of the request before chunk j (a request has
  // fewer than 65,536 of them: checked by the host), valid tokens of chunk j's last tile (1..128)
  uint16_t hist_prefix[kMaxHistChunksKeys + 1];
  uint8_t hist_last[kMaxHistChunksKeys];
};

// NC = score columns per softmax thread, WG = softmax warpgroups (threads sharing a TMEM lane),
// UNITS = ring units, D = head dim (64 or 128).  N = NC * WG is the widest row group the
// instantiation takes.  A K or V tile is D / 64 boxes of [128 keys][64 d].
// Head dim 64: the output MMA still runs with M = 128; the upper 64 rows of its A operand
// (V^T) are whatever lies one box further in shared memory, their results land in TMEM lanes
// 64..127 and are never read.  kSmem keeps that box inside the CTA's window.
template <int NC, int WG, int UNITS, int D>
struct Cfg {
  static constexpr int N = NC * WG;
  static constexpr int kHalves = D / 64;
  static constexpr int kUnitBytes = kHalves * kHalf;  // one K tile or one V tile
  static constexpr int kSoft = 128 * WG;              // softmax threads
  static constexpr int kThreads = kSoft + 64;
  static constexpr int kQHalf = N * 64 * 2;           // [N rows][64 d]
  static constexpr int kOffQ = UNITS * kUnitBytes;
  static constexpr int kOffP = kOffQ + kHalves * kQHalf;
  static constexpr int kOffCtl = kOffP + kKeys * N * 2;
  static constexpr int kCtlBytes = (sizeof(Ctl<N>) + 1023) / 1024 * 1024;
  static constexpr int kSmemUsed = kOffCtl + kCtlBytes;
  static constexpr int kSmem = (D == 64 && kSmemUsed < kOffQ + kHalf) ? kOffQ + kHalf : kSmemUsed;
  static constexpr uint32_t kTmemCols = (3 * N <= 128) ? 128 : (3 * N <= 256 ? 256 : 512);
  static constexpr uint32_t kColO = 2 * N;            // S^T buffers at 0 and N, O^T at 2N
  static constexpr int kMinBlocks = (kSmem <= 113 * 1024 && kTmemCols <= 256 && WG == 1) ? 2 : 1;
  static_assert(kSmem <= 227 * 1024, "shared memory");
  static_assert(NC % 16 == 0 && UNITS <= 8 && (D == 64 || D == 128), "shape");
};


// HIST = 1: the launch covers a list of chunks (HistParams; see ss_internal.h): the CTA walks an
// equal share of its request's 128-token tiles, counted chunk by chunk, with one accumulator.
// HIST = 2: the same for ragged batches: the CTAs of a kv-head walk equal shares of ALL its requests'
// tiles laid end to end; a CTA runs the kernel's body once per request its share touches (a new Q
// tile, a new accumulator, a partial state of its own), the barriers set up anew each time.
template <int NC, int WG, int UNITS, int D, int HIST>
__global__ void __launch_bounds__(Cfg<NC, WG, UNITS, D>::kThreads, Cfg<NC, WG, UNITS, D>::kMinBlocks)
chunk_tc_keys_kernel(const ChunkParams p, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const __grid_constant__ HistParams h) {
  using C = Cfg<NC, WG, UNITS, D>;
  constexpr int N = C::N;
  constexpr int kD = D, kUnitBytes = C::kUnitBytes;
  extern __shared__ __align__(1024) uint8_t smem[];
  Ctl<N>* ctl = reinterpret_cast<Ctl<N>*>(smem + C::kOffCtl);
  uint8_t* q_s = smem + C::kOffQ;
  uint8_t* p_s = smem + C::kOffP;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 32 * (4 * WG)) {  // the producer lane: fetch the tensor maps while the work item is read
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmV) : "memory");
  }
  const unsigned long long t_cta0 = p.cta_log ? cta_log_now() : 0ull;
  if (p.wait_first) pdl_wait_prior();
  pdl_launch_dependents();
  constexpr bool WALK = HIST == 2;
  const ChunkWork w = chunk_work(p, p.rows_per_tile);
  const int kvh = w.kvh, row0 = w.row0, nrows = w.nrows, tok0 = w.tok0, tok1 = w.tok1;  // nrows <= N
  const bool chain_cta = w.chain_cta;
  const int n_mma = (nrows + 15) & ~15;                 // MMA N of this CTA
  unsigned long long* tr = chain_cta ? p.trace : nullptr;
  // (ragged batches) this CTA's share [share_lo, share_hi) of the kv-head's tiles by the host's lengths
  long long share_lo = 0, share_hi = 0;
  int req = w.b, req_end = w.b + 1;  // requests to run the body for: [req, req_end) as long as they overlap the share
  if (WALK) {
    const long long all = h.req_prefix[h.n_req];
    share_lo = all * blockIdx.x / gridDim.x;
    share_hi = all * (blockIdx.x + 1) / gridDim.x;
    req = 0;
    while (req < h.n_req && h.req_prefix[req + 1] <= share_lo) ++req;
    req_end = h.n_req;
  }
  bool tmem_held = false;
  int tiles_walked = 0;
  uint32_t tmem = 0;
  for (; req < req_end && (!WALK || h.req_prefix[req] < share_hi); ++req) {
  const int b = req;
  int piece = w.split;        // which of the request's partial states this pass writes
  bool last_piece = false;    // (ragged batches) no CTA after this one has tiles of the request
  long long hint_a = 0, hint_e = 0, hint_n = 1;
  if (WALK) {
    const long long p0 = h.req_prefix[b], p1 = h.req_prefix[b + 1];
    hint_n = p1 - p0;
    hint_a = (share_lo > p0 ? share_lo : p0) - p0;
    hint_e = (share_hi < p1 ? share_hi : p1) - p0;
    last_piece = share_hi >= p1;
    int first = blockIdx.x;   // the first CTA of the kv-head whose share reaches into this request
    const long long all = h.req_prefix[h.n_req];
    while (first > 0 && all * first / gridDim.x > p0) --first;
    piece = blockIdx.x - first;
  }
  auto state_ml = [&](int k) {  // (m, l) rows of the request's partial state number k
    return p.part_ml + (((size_t)k * p.B + b) * p.H_kv + kvh) * p.R_stride + row0;
  };
  float2* out_ml = WALK ? state_ml(piece) : w.out_ml;
  float* out_a = WALK ? p.part_a + ((((size_t)piece * p.B + b) * p.H_kv + kvh) * p.R_stride + row0) * p.d : w.out_a;
  // the states nobody computes (the request has fewer pieces than the launch has splits) are the identity
  auto fill_unused = [&]() {
    if (WALK && last_piece && tid < nrows)
      for (int k = piece + 1; k < p.splits; ++k) state_ml(k)[tid] = make_float2(-INFINITY, 0.f);
  };
  // splits are given in 64-token tiles by the host; this kernel walks 128-token tiles
  int n_tiles = (tok1 > tok0) ? (tok1 - tok0 + kKeys - 1) / kKeys : 0;
  int g0 = 0;  // (list of chunks) the CTA's first tile in the request's numbering
  if (HIST) {
    if (warp == 0) {
      int v = 0;
      if (lane < h.n_chunks) {
        const int Lc = h.L_c[lane];
        v = h.valid_len[lane] ? h.valid_len[lane][b] : Lc;
        if (v < 0 || v > Lc) {  // flagged and clamped, never trusted
          atomicOr(p.status, SS_DEV_BAD_VALID_LEN);
          v = max(0, min(v, Lc));
        }
      }
      int incl = (v + kKeys - 1) / kKeys;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      if (lane < h.n_chunks) {
        ctl->hist_prefix[lane + 1] = (uint16_t)incl;
        ctl->hist_last[lane] = (uint8_t)(v ? v - (v - 1) / kKeys * kKeys : 0);
      }
      if (lane == 0) ctl->hist_prefix[0] = 0;
      const int total = __shfl_sync(0xffffffffu, incl, 31);
      if (lane >= h.n_chunks && lane < kMaxHistChunksKeys) ctl->hist_prefix[lane + 1] = (uint16_t)total;
    }
    __syncthreads();
    const int total = ctl->hist_prefix[h.n_chunks];
    if (WALK) {  // the share of the request by the host's lengths, scaled to the tiles it really has
      g0 = (int)((long long)total * hint_a / hint_n);
      n_tiles = (int)((long long)total * hint_e / hint_n) - g0;
    } else {
      g0 = (int)((int64_t)total * w.split / p.splits);
      n_tiles = (int)((int64_t)total * (w.split + 1) / p.splits) - g0;
    }
  }
  // (list of chunks) chunk of the CTA's tile t and the tile's first token in it; tiles are asked
  // for in ascending order, `cur` is the caller's own cursor
  auto hist_locate = [&](int t, int& cur, int* tok) {
    const int g = g0 + t;
    while (g >= ctl->hist_prefix[cur + 1]) ++cur;
    *tok = (g - ctl->hist_prefix[cur]) * kKeys;
    return cur;
  };

  if (n_tiles == 0 || (smem_u32(smem) & 1023u)) {
    // nothing visible here (identity state, no tensor memory taken); a misaligned shared
    // memory window would break the swizzled layouts and is reported instead of run
    if (n_tiles && tid == 0) atomicOr(p.status, SS_DEV_WAIT_EXPIRED);
    if (tid < nrows) out_ml[tid] = make_float2(-INFINITY, 0.f);
    fill_unused();
    if (WALK) {
      __syncthreads();  // (the table in the control block is rebuilt for the next request)
      continue;
    }
    if (!p.wait_first && chain_cta) pdl_wait_prior();
    return;
  }
  auto mwait = [&](uint64_t* bar, uint32_t parity) {
    return mbar_wait_abortable(bar, parity, &ctl->abort, p.status);
  };

  // ---- set-up ------------------------------------------------------------------------------
  // use j of the ring: K of tile t is j = 2t, V of tile t is j = 2t + 1; unit j % UNITS
  // both 64-column halves of `rows` tokens starting at (outer, tok) -> dst (K when !is_v)
  auto load_rows = [&](bool is_v, uint32_t dst, int tok, int outer, uint64_t* bar, uint64_t pol) {
    if (is_v) {  // (no runtime-selected pointer: the tensor maps stay in the parameter space)
      tma_load_4d(dst, &tmV, 0, tok, kvh, outer, bar, pol);
      if (D == 128) tma_load_4d(dst + kHalf, &tmV, 64, tok, kvh, outer, bar, pol);
    } else {
      tma_load_4d(dst, &tmK, 0, tok, kvh, outer, bar, pol);
      if (D == 128) tma_load_4d(dst + kHalf, &tmK, 64, tok, kvh, outer, bar, pol);
    }
  };
  // Pages smaller than a tile (8 to 64 tokens): the tile is gathered page by page by the
  // whole producer warp, see below; this path is for contiguous chunks and pages of a tile or more.
  const bool small_pages = p.page_table && p.page_size < kKeys;
  int prod_chunk = 0;  // (list of chunks) the producer's cursor
  auto issue_use = [&](int j, uint64_t pol) {
    const int u = j % UNITS;
    mbar_expect_tx(&ctl->ufull[u], kUnitBytes);
    if (HIST) {
      int tok;
      const int c = hist_locate(j >> 1, prod_chunk, &tok);
      const CUtensorMap* m = h.maps + 2 * c + (j & 1);  // in device memory
      const uint32_t dst = smem_u32(smem + u * kUnitBytes);
      tma_load_4d(dst, m, 0, tok, kvh, b, &ctl->ufull[u], pol);
      if (D == 128) tma_load_4d(dst + kHalf, m, 64, tok, kvh, b, &ctl->ufull[u], pol);
      return;
    }
    int outer, tok;
    locate_token(p, b, tok0 + (j >> 1) * kKeys, &outer, &tok);
    load_rows(j & 1, smem_u32(smem + u * kUnitBytes), tok, outer, &ctl->ufull[u], pol);
  };
  const int n_uses = 2 * n_tiles;
  const int n_pre = small_pages ? 0 : min(n_uses, UNITS);  // small pages: all copies go out below
  constexpr int kProducerWarp = 4 * WG, kMmaWarp = 4 * WG + 1;
  if (warp == kProducerWarp) {
    if (lane == 0) {
      if (tmem_held) {  // a later request of the share: the barriers start over
        for (int u = 0; u < UNITS; ++u) {
          mbar_inval(&ctl->ufull[u]);
          mbar_inval(&ctl->uempty[u]);
        }
        mbar_inval(&ctl->sfull[0]);
        mbar_inval(&ctl->sfull[1]);
        mbar_inval(&ctl->pready);
        mbar_inval(&ctl->pfree);
      }
      // the first loads go out as early as possible: only their own barriers exist yet
      for (int u = 0; u < UNITS; ++u) mbar_init(&ctl->ufull[u], 1);
      fence_barrier_init();
      // streamed once: evict first; shared by the row groups of a kv-head through L2: keep
      const uint64_t pol = p.row_tiles > 1 ? l2_evict_normal_policy() : l2_evict_first_policy();
      for (int j = 0; j < n_pre; ++j) issue_use(j, pol);
      for (int u = 0; u < UNITS; ++u) mbar_init(&ctl->uempty[u], 1);
      mbar_init(&ctl->sfull[0], 1);
      mbar_init(&ctl->sfull[1], 1);
      mbar_init(&ctl->pready, C::kSoft);
      mbar_init(&ctl->pfree, 1);
      ctl->abort = 0;
      ctl->flag[0] = ctl->flag[1] = ctl->flag[2] = 0;
      fence_barrier_init();
    }
    __syncwarp();
    if (!tmem_held) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                       smem_u32(&ctl->tmem_base)),
                   "r"(C::kTmemCols)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  } else if (warp < 4 * WG) {
    // Q rows -> shared memory as the K-major B operand (128-byte swizzle), zero padding rows
    // (N rows x 16 pieces of 16 bytes over 128 * WG threads = 4 pieces per thread: all four
    // global loads go out before the first store, one memory latency instead of four)
    constexpr int kQPieces = N * (kD / 8) / C::kSoft;
    static_assert(kQPieces * C::kSoft == N * (kD / 8), "Q pieces per thread");
    uint4 qraw[kQPieces];
#pragma unroll
    for (int u = 0; u < kQPieces; ++u) {
      const int i = tid + u * C::kSoft;
      const int n = i / (kD / 8), c8 = i % (kD / 8);
      qraw[u] = make_uint4(0, 0, 0, 0);
      if (n < nrows) {
        const int rg = row0 + n, g = rg / p.T_q, t = rg % p.T_q;
        qraw[u] = *reinterpret_cast<const uint4*>(p.Q + b * p.q_sb + (int64_t)(kvh * p.G + g) * p.q_sh +
                                                  t * p.q_st + c8 * 8);
      }
    }
#pragma unroll
    for (int u = 0; u < kQPieces; ++u) {
      const int i = tid + u * C::kSoft;
      const int n = i / (kD / 8), c8 = i % (kD / 8);
      const int half = c8 >> 3, j = c8 & 7;
      if (n < n_mma)
        *reinterpret_cast<uint4*>(q_s + half * C::kQHalf + n * 128 + ((j ^ (n & 7)) << 4)) = qraw[u];
    }
    if (tid < N) ctl->nm_ref[tid] = INFINITY;
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  tmem = ctl->tmem_base;
  tmem_held = true;
  unsigned long long* trl = lane == 0 ? tr : nullptr;

  if (warp == kProducerWarp && small_pages) {
    // ===== TMA producer, pages smaller than a tile =====
    // The tensor map's box is one page; page i of a tile lands at row i * page_size of the ring
    // unit, which keeps the swizzled layout of a single 128-token box.  Lane l copies 64-column
    // half l % 2 of page l / 2 of the tile, so a unit's 4 to 32 copies and their page look-ups
    // go out side by side; each lane fetches the page id of the next tile right after a tile's
    // V copy, off the path of the next copy.  Pages that start at or past the valid length are
    // not looked up (index n_pages is outside the pool and reads as zeros).  Lane 0 waits for
    // the unit (bounded) and arms its barrier; the outcome is shared through a shuffle.
    const uint64_t pol = p.row_tiles > 1 ? l2_evict_normal_policy() : l2_evict_first_policy();
    const int ps = p.page_size, n_sub = kKeys / ps;  // 2 to 16 pages per tile (pages of 64 to 8 tokens)
    const int sub = lane / C::kHalves, half = lane % C::kHalves;
    const bool mine = lane < C::kHalves * n_sub;
    auto lane_page = [&](int tile) {  // page id of this lane's page of `tile`; -2: not looked up
      const int tk = tok0 + tile * kKeys + sub * ps;
      if (!mine || tk >= tok1) return -2;
      const int pg = tk / ps;
      return pg < p.pages_per_req ? p.page_table[(int64_t)b * p.pages_per_req + pg] : -1;
    };
    int page = lane_page(0), issued = 0;
    for (int j = 0; j < n_uses; ++j) {
      const int u = j % UNITS;
      const uint32_t ph = (j / UNITS) & 1;
      int ok = 1;
      if (lane == 0) {
        ok = mwait(&ctl->uempty[u], ph ^ 1);
        if (ok) mbar_expect_tx(&ctl->ufull[u], kUnitBytes);
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);  // also orders the arming before the copies
      if (!ok) break;
      if (mine) {
        int id = page;
        if (id == -2) {
          id = p.n_pages;
        } else if (id < 0 || id >= p.n_pages) {
          atomicOr(p.status, SS_DEV_BAD_PAGE);
          id = p.n_pages;
        }
        const uint32_t dst = smem_u32(smem + u * kUnitBytes) + half * kHalf + sub * ps * 128;
        if (j & 1) tma_load_4d(dst, &tmV, half * 64, 0, kvh, id, &ctl->ufull[u], pol);
        else tma_load_4d(dst, &tmK, half * 64, 0, kvh, id, &ctl->ufull[u], pol);
      }
      if (j & 1) page = lane_page((j >> 1) + 1);
      issued = j + 1;
    }
    if (lane == 0 && ctl->abort) {
      // let the copies the warp started land before the CTA leaves (bounded)
      const unsigned long long t0 = gtime_ns();
      for (int j = max(0, issued - UNITS); j < issued; ++j)
        while (!mbar_try_wait(&ctl->ufull[j % UNITS], (j / UNITS) & 1) && gtime_ns() - t0 < kWaitNs) {
        }
    }
  } else if (warp == kProducerWarp) {
    // ===== TMA producer =====
    if (lane == 0) {
      // streamed once: evict first; shared by the row groups of a kv-head through L2: keep
      const uint64_t pol = p.row_tiles > 1 ? l2_evict_normal_policy() : l2_evict_first_policy();
      int issued = n_pre;
      for (int j = n_pre; j < n_uses; ++j) {
        const int u = j % UNITS;
        const uint32_t ph = (j / UNITS) & 1;
        trace(tr, 0, j >> 1, (j & 1) * 2);
        if (!mwait(&ctl->uempty[u], ph ^ 1)) break;
        trace(tr, 0, j >> 1, (j & 1) * 2 + 1);
        issue_use(j, pol);
        issued = j + 1;
      }
      if (ctl->abort) {
        // let the copies this thread started land before the CTA leaves (bounded)
        const unsigned long long t0 = gtime_ns();
        for (int j = max(0, issued - UNITS); j < issued; ++j)
          while (!mbar_try_wait(&ctl->ufull[j % UNITS], (j / UNITS) & 1) && gtime_ns() - t0 < kWaitNs) {
          }
      }
    }
  } else if (warp == kMmaWarp) {
    // ===== MMA issuer: the whole warp walks the loop, one elected lane issues =====
    const uint32_t idesc_qk = make_idesc_major(128, n_mma, false, false);
    const uint32_t idesc_pv = make_idesc_major(128, n_mma, true, true);
    const bool leader = elect_one();
    const uint32_t base = smem_u32(smem);
    const uint32_t q_addr = smem_u32(q_s), p_addr = smem_u32(p_s);
    auto issue_qk = [&](int t) {  // S^T[t & 1] = K(t) Q^T
      const uint32_t k_addr = base + ((2 * t) % UNITS) * kUnitBytes;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint32_t off = (kk & 3) * 32;
          mma_ss(tmem + (t & 1) * N, desc_kmajor(k_addr + (kk >> 2) * kHalf + off),
                 desc_kmajor(q_addr + (kk >> 2) * C::kQHalf + off), idesc_qk, kk > 0);
        }
        tc_commit(&ctl->uempty[(2 * t) % UNITS]);
        tc_commit(&ctl->sfull[t & 1]);
      }
      __syncwarp();
    };
    // The issuer polls for whichever of its two next operations can go: the score MMAs of tile
    // qi (K landed; its score buffer free, i.e. the output MMAs of tile qi - 2 issued) or the
    // output MMAs of tile pi (weights ready, V landed).  Walking them in a fixed order would
    // hold back an output MMA - and the release of its V unit - behind a K tile that is late.
    auto issue_pv = [&](int t) {
      const int jv = 2 * t + 1;
      const uint32_t v_addr = base + (jv % UNITS) * kUnitBytes;
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < kKeys / 16; ++kk) {
          // A = V^T: MN-major, 64 head dims (128 bytes) per token row, 8-token atoms 1024 bytes
          // apart, the other 64 head dims one half-tile away.  B = P^T: plain 8x8 core matrices.
          mma_ss(tmem + C::kColO, desc_mnmajor(v_addr + kk * 2048, kHalf),
                 desc_mnmajor_plain(p_addr + kk * 256, 128, kKeys * 16), idesc_pv, (t > 0 || kk > 0));
        }
        tc_commit(&ctl->uempty[jv % UNITS]);
        tc_commit(&ctl->pfree);
      }
      __syncwarp();
    };
    int qi = 0, pi = 0;
    unsigned long long t0 = gtime_ns();
    uint32_t spins = 0;
    while (pi < n_tiles) {
      bool did = false;
      if (qi < n_tiles && qi < pi + 2) {
        const int j = 2 * qi;
        if (__all_sync(0xffffffffu, mbar_test(&ctl->ufull[j % UNITS], (j / UNITS) & 1))) {
          trace(trl, 1, qi, 0);  // the tile's first stamp: its K has landed
          tc_fence_after();
          trace(trl, 1, qi, 1);
          issue_qk(qi);
          trace(trl, 1, qi, 2);
          ++qi;
          did = true;
        }
      }
      if (pi < qi) {
        const int jv = 2 * pi + 1;
        if (__all_sync(0xffffffffu, mbar_test(&ctl->pready, pi & 1) &&
                                        mbar_test(&ctl->ufull[jv % UNITS], (jv / UNITS) & 1))) {
          tc_fence_after();
          trace(trl, 1, pi, 4);
          issue_pv(pi);
          trace(trl, 1, pi, 5);
          ++pi;
          did = true;
        }
      }
      if (did) {
        spins = 0;
        t0 = gtime_ns();
      } else if ((++spins & 255u) == 0) {  // bounded like every other wait
        const bool stop = ctl->abort != 0 || gtime_ns() - t0 > kWaitNs;
        if (__any_sync(0xffffffffu, stop)) {
          if (lane == 0 && ctl->abort == 0) {
            ctl->abort = 1;
            atomicOr(p.status, SS_DEV_WAIT_EXPIRED);
          }
          break;
        }
      }
    }
    if (WALK && lane == 0 && n_uses >= 2) {
      // the barriers are set up anew for the share's next request: the last two releases of ring
      // units (asynchronous arrivals of the tensor core) must have landed
      mwait(&ctl->uempty[(n_uses - 2) % UNITS], ((n_uses - 2) / UNITS) & 1);
      mwait(&ctl->uempty[(n_uses - 1) % UNITS], ((n_uses - 1) / UNITS) & 1);
    }
  } else {
    // ===== softmax warps: TMEM lane L = key L of the tile; columns [c0, c0 + cn) = rows =====
    // A wait that gives up makes the whole warp `dead`: it keeps walking the loop and the
    // named barriers (so nobody is left waiting) but touches nothing else.
    // tensor-memory loads in flight per wait: with 16 softmax warps the load latency is hidden
    // by the other warps and registers are scarce; with fewer warps two loads go out together
    constexpr int kBatch = (WG >= 4) ? 1 : 2;
    const int L = (warp & 3) * 32 + lane;
    const int cg = (WG == 1) ? 0 : (warp >> 2);                // column group (0..WG-1)
    const int cpg = ((n_mma / WG) + 15) & ~15;                 // columns per group
    const int c0 = cg * cpg;
    const int cn = max(0, min(cpg, n_mma - c0));               // multiple of 16, <= NC
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    bool dead = false;
    const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
    auto wait = [&](uint64_t* bar, uint32_t parity) {
      if (!dead && !mwait(bar, parity)) dead = true;
      dead = __any_sync(0xffffffffu, dead);
    };
    float2 lsum[NC / 2];  // row sums of this key lane, two rows per packed add
#pragma unroll
    for (int r = 0; r < NC / 2; ++r) lsum[r] = make_float2(0.f, 0.f);
    int soft_chunk = 0;  // (list of chunks) this thread's cursor
    for (int t = 0; t < n_tiles; ++t) {
      if (tid == 0) trace(tr, 2, t, 0);
      wait(&ctl->sfull[t & 1], (t >> 1) & 1);
      tc_fence_after();
      if (tid == 0) trace(tr, 2, t, 1);
      int n_valid;
      if (HIST) {
        int tok;
        const int c = hist_locate(t, soft_chunk, &tok);
        n_valid = (g0 + t + 1 == ctl->hist_prefix[c + 1]) ? ctl->hist_last[c] : kKeys;   // the chunk's last tile?
      } else {
        n_valid = min(kKeys, tok1 - (tok0 + t * kKeys));
      }
      const bool key_ok = L < n_valid;
      if (n_valid < kKeys) {
        // ragged tail: tokens past the valid length may hold anything; their weights are 0, so
        // V must be finite there: clear those rows of the staged V tile (both halves)
        const int jv = 2 * t + 1;
        wait(&ctl->ufull[jv % UNITS], (jv / UNITS) & 1);
        if (!dead) {
          uint8_t* v_s = smem + (jv % UNITS) * kUnitBytes;
          constexpr int kVecRow = 8 * C::kHalves;  // 16-byte pieces per token row
          const int n_vec = (kKeys - n_valid) * kVecRow;
          for (int i = tid; i < n_vec; i += C::kSoft) {
            const int row = n_valid + i / kVecRow, half = (i % kVecRow) >> 3, ch = i & 7;
            *reinterpret_cast<uint4*>(v_s + half * kHalf + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
          }
        }
        // made visible to the tensor core by the proxy fence before pready below
      }
      // The scores are read from tensor memory twice (first for the overflow test, then for the
      // weights) instead of being held in registers across the barrier below.
      const uint32_t t_s = tmem + lane_off + (t & 1) * N + c0;
      if (t == 0) {
        // First references: the exact maxima of the first tile, which keeps its largest weight at
        // exactly 1.  Done here without the bookkeeping of the general path below (nothing to
        // rescale yet), which would cost three tiles' time while the CTA's ring sits full.
        if (!dead) {
#pragma unroll
          for (int q = 0; q < NC / 16; ++q) {
            if (q * 16 < cn) {
              uint32_t raw[16];
              tmem_ld16(t_s + q * 16, raw);
              tc_wait_ld();
#pragma unroll
              for (int c = 0; c < 16; ++c) {
                float v = key_ok ? __uint_as_float(raw[c]) * p.scale_log2 : -INFINITY;
                v = warp_max_f(v);
                if (lane == 0) ctl->smax[warp & 3][c0 + q * 16 + c] = v;
              }
            }
          }
        }
        named_bar_sync(1, C::kSoft);
        if (tid < n_mma && !dead)  // the tile's first key is valid, so the maximum is finite
          ctl->nm_ref[tid] = -fmaxf(fmaxf(ctl->smax[0][tid], ctl->smax[1][tid]),
                                    fmaxf(ctl->smax[2][tid], ctl->smax[3][tid]));
        named_bar_sync(1, C::kSoft);
      }
      bool over = false;
      if (!dead) {
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // independent chains
#pragma unroll
        for (int q0 = 0; q0 < NC / 16; q0 += kBatch) {  // kBatch loads, one wait
          uint32_t raw[kBatch][16];
#pragma unroll
          for (int h = 0; h < kBatch; ++h)
            if ((q0 + h) * 16 < cn) tmem_ld16(t_s + (q0 + h) * 16, raw[h]);
          tc_wait_ld();
#pragma unroll
          for (int h = 0; h < kBatch; ++h) {
            const int q = q0 + h;
            if (q * 16 < cn) {
#pragma unroll
              for (int c4 = 0; c4 < 4; ++c4) {
                // s * scale - m for four rows as two packed FMAs (+inf while there is no reference)
                const float4 nm = *reinterpret_cast<const float4*>(&ctl->nm_ref[c0 + q * 16 + c4 * 4]);
                const float2 x01 = fma2_f(make_float2(__uint_as_float(raw[h][c4 * 4 + 0]),
                                                      __uint_as_float(raw[h][c4 * 4 + 1])),
                                          sc2, make_float2(nm.x, nm.y));
                const float2 x23 = fma2_f(make_float2(__uint_as_float(raw[h][c4 * 4 + 2]),
                                                      __uint_as_float(raw[h][c4 * 4 + 3])),
                                          sc2, make_float2(nm.z, nm.w));
                mx4[c4 & 1] = max3_f(mx4[c4 & 1], x01.x, x01.y);
                mx4[2 + (c4 & 1)] = max3_f(mx4[2 + (c4 & 1)], x23.x, x23.y);
              }
            }
          }
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        over = key_ok && (mx > kLazyThreshold);
      }
      if (tid == 0) trace(tr, 2, t, 3);
      if (tid == 0) ctl->flag[(t + 1) % 3] = 0;
      if (__any_sync(0xffffffffu, over) && lane == 0) ctl->flag[t % 3] = 1;
      named_bar_sync(1, C::kSoft);
      if (tid == 0) trace(tr, 2, t, 4);
      if (ctl->flag[t % 3]) {
        // ---- raise the row references to the exact tile maxima (rare after the first tile) ----
        if (!dead) {
#pragma unroll
          for (int q = 0; q < NC / 16; ++q) {
            if (q * 16 < cn) {
              uint32_t raw[16];
              tmem_ld16(t_s + q * 16, raw);
              tc_wait_ld();
#pragma unroll
              for (int c = 0; c < 16; ++c) {
                float v = key_ok ? __uint_as_float(raw[c]) * p.scale_log2 : -INFINITY;
                v = warp_max_f(v);
                if (lane == 0) ctl->smax[warp & 3][c0 + q * 16 + c] = v;
              }
            }
          }
        }
        named_bar_sync(1, C::kSoft);
        if (t > 0) {  // O^T must be at rest: the output MMAs of tile t-1 have retired
          wait(&ctl->pfree, (t - 1) & 1);
          tc_fence_after();
        }
        if (!dead) {
#pragma unroll
          for (int q = 0; q < NC / 16; ++q) {
            if (q * 16 < cn) {
              float f[16];
#pragma unroll
              for (int c = 0; c < 16; ++c) {
                const int r = c0 + q * 16 + c;
                const float m_old = -ctl->nm_ref[r];
                const float m_new = fmaxf(fmaxf(m_old, ctl->smax[0][r]),
                                          fmaxf(fmaxf(ctl->smax[1][r], ctl->smax[2][r]), ctl->smax[3][r]));
                f[c] = (m_old == -INFINITY) ? 0.f : exp2f(m_old - m_new);
              }
#pragma unroll
              for (int c = 0; c < 16; c += 2) {
                lsum[q * 8 + c / 2].x *= f[c];
                lsum[q * 8 + c / 2].y *= f[c + 1];
              }
              if (t > 0) {
                uint32_t o[16];
                tmem_ld16(tmem + lane_off + C::kColO + c0 + q * 16, o);
                tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f[c]);
                tmem_st16(tmem + lane_off + C::kColO + c0 + q * 16, o);
              }
            }
          }
          tc_wait_st();
        }
        named_bar_sync(1, C::kSoft);  // every thread has read the old references
        if (tid < n_mma && !dead) {
          const float m_old = -ctl->nm_ref[tid];
          ctl->nm_ref[tid] = -fmaxf(fmaxf(m_old, ctl->smax[0][tid]),
                                    fmaxf(fmaxf(ctl->smax[1][tid], ctl->smax[2][tid]), ctl->smax[3][tid]));
        }
        named_bar_sync(1, C::kSoft);
      }
      if (t > 0) wait(&ctl->pfree, (t - 1) & 1);  // the output MMAs of tile t-1 consumed P^T
      if (tid == 0) trace(tr, 2, t, 5);
      if (!dead) {
        // weights, row sums, P^T as bf16: rows c0+8c .. c0+8c+7 of key L form one 16-byte piece
#pragma unroll
        for (int q0 = 0; q0 < NC / 16; q0 += kBatch) {  // kBatch loads, one wait
          uint32_t raw2[kBatch][16];
#pragma unroll
          for (int h = 0; h < kBatch; ++h)
            if ((q0 + h) * 16 < cn) tmem_ld16(t_s + (q0 + h) * 16, raw2[h]);
          tc_wait_ld();
#pragma unroll
          for (int h = 0; h < kBatch; ++h) {
          const int q = q0 + h;
          const uint32_t (&raw)[16] = raw2[h];
          if (q * 16 < cn) {
            // staged so that the 16 exponentials of a chunk are independent instructions;
            // two rows per packed fp32 instruction
            float pv[16];
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
              const float4 nm = *reinterpret_cast<const float4*>(&ctl->nm_ref[c0 + q * 16 + c4 * 4]);
              const float2 x01 = fma2_f(make_float2(__uint_as_float(raw[c4 * 4 + 0]),
                                                    __uint_as_float(raw[c4 * 4 + 1])),
                                        sc2, make_float2(nm.x, nm.y));
              const float2 x23 = fma2_f(make_float2(__uint_as_float(raw[c4 * 4 + 2]),
                                                    __uint_as_float(raw[c4 * 4 + 3])),
                                        sc2, make_float2(nm.z, nm.w));
              pv[c4 * 4 + 0] = x01.x;
              pv[c4 * 4 + 1] = x01.y;
              pv[c4 * 4 + 2] = x23.x;
              pv[c4 * 4 + 3] = x23.y;
            }
#pragma unroll
            for (int c = 0; c < 16; ++c) pv[c] = ex2_ftz(pv[c]);
            if (n_valid < kKeys) {  // only the tile that straddles the valid length (warp-uniform)
#pragma unroll
              for (int c = 0; c < 16; ++c) pv[c] = key_ok ? pv[c] : 0.f;
            }
#pragma unroll
            for (int c = 0; c < 16; c += 2)
              lsum[q * 8 + c / 2] = add2_f(lsum[q * 8 + c / 2], make_float2(pv[c], pv[c + 1]));
            uint32_t pk[8];
#pragma unroll
            for (int c = 0; c < 16; c += 2) {
              __nv_bfloat162 hh = __floats2bfloat162_rn(pv[c], pv[c + 1]);  // low half = even row
              pk[c / 2] = *reinterpret_cast<uint32_t*>(&hh);
            }
#pragma unroll
            for (int h8 = 0; h8 < 2; ++h8)
              *reinterpret_cast<uint4*>(p_s + ((c0 >> 3) + q * 2 + h8) * (kKeys * 16) + L * 16) =
                  make_uint4(pk[h8 * 4], pk[h8 * 4 + 1], pk[h8 * 4 + 2], pk[h8 * 4 + 3]);
          }
          }
        }
        fence_proxy_async();
        tc_fence_before();
      }
      mbar_arrive(&ctl->pready);
      if (tid == 0) trace(tr, 2, t, 2);
    }
    wait(&ctl->pfree, (n_tiles - 1) & 1);
    named_bar_sync(1, C::kSoft);
    if (ctl->abort == 0) {  // uniform over the softmax threads after the barrier
      tc_fence_after();
      // ---- row sums across the 128 key lanes, then the partial state ----
      float* red = reinterpret_cast<float*>(smem);  // [128][N + 1] over the free ring
#pragma unroll
      for (int r = 0; r < NC; ++r)
        if (r < cn) red[L * (N + 1) + c0 + r] = (r & 1) ? lsum[r / 2].y : lsum[r / 2].x;
      named_bar_sync(1, C::kSoft);
      // four threads per row, each over a quarter of the key lanes (kSoft / N = 4), then one
      // thread per row over the four partial sums
      float* red4 = red + kKeys * (N + 1);  // [4][N]
      {
        const int row = tid % N, part = tid / N;
        float ps = 0.f;
#pragma unroll 8
        for (int k = part * (kKeys / 4); k < (part + 1) * (kKeys / 4); ++k) ps += red[k * (N + 1) + row];
        red4[part * N + row] = ps;
      }
      named_bar_sync(1, C::kSoft);
      if (tid < nrows) {
        const float lt = (red4[tid] + red4[N + tid]) + (red4[2 * N + tid] + red4[3 * N + tid]);
        out_ml[tid] = make_float2(lt > 0.f ? -ctl->nm_ref[tid] : -INFINITY, lt);
      }
      // thread (L, cg) holds head dim L of its rows
#pragma unroll
      for (int q = 0; q < NC / 16; ++q) {
        if (q * 16 < cn) {
          uint32_t o[16];
          tmem_ld16(tmem + lane_off + C::kColO + c0 + q * 16, o);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const int r = c0 + q * 16 + c;
            if (r < nrows && L < kD) out_a[(size_t)r * kD + L] = __uint_as_float(o[c]);
          }
        }
      }
    }
  }

  if (warp < 4 * WG) {
    fill_unused();
    if (WALK) fence_proxy_async();  // the ring served as scratch; bulk copies write it next
  }
  tiles_walked += n_tiles;
  // every role is done with this request: the ring, the barriers and the tensor memory are free
  tc_fence_before();
  __syncthreads();
  if (ctl->abort) break;
  }  // for each request of the CTA's share

  // ---- teardown ----
  if (tmem_held && warp == 4 * WG) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols)
                 : "memory");
  }
  if (tid == 0) cta_log_write(p, t_cta0, tiles_walked);
  // Completion order along the stream: one CTA of this grid waits for the previous grid, so
  // this grid cannot complete before it (the other CTAs leave at once and free their SM slot).
  if (!p.wait_first && chain_cta) pdl_wait_prior();
}

template <int NC, int WG, int UNITS, int D, int HIST>
cudaError_t launch_hist_cfg(const ChunkParams& p, const HistParams& h, const CUtensorMap& any_map, dim3 grid,
                            cudaStream_t s, bool pdl) {
  using C = Cfg<NC, WG, UNITS, D>;
  return launch_kernel(chunk_tc_keys_kernel<NC, WG, UNITS, D, HIST>, grid, dim3(C::kThreads), C::kSmem, s, pdl, p,
                       any_map, any_map, h);
}

template <int NC, int WG, int UNITS, int D, int HIST>
cudaError_t prepare_hist() {
  return cudaFuncSetAttribute(chunk_tc_keys_kernel<NC, WG, UNITS, D, HIST>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<NC, WG, UNITS, D>::kSmem);
}

template <int NC, int WG, int UNITS, int D>
cudaError_t launch_cfg(const ChunkParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       cudaStream_t s, bool pdl) {
  using C = Cfg<NC, WG, UNITS, D>;
  dim3 grid(p.splits * p.row_tiles, p.H_kv, p.n_active ? p.n_active : p.B), block(C::kThreads);
  static const HistParams none = {};
  return launch_kernel(chunk_tc_keys_kernel<NC, WG, UNITS, D, 0>, grid, block, C::kSmem, s, pdl, p, tmK, tmV, none);
}

template <int NC, int WG, int UNITS, int D>
cudaError_t prepare_cfg() {
  return cudaFuncSetAttribute(chunk_tc_keys_kernel<NC, WG, UNITS, D, 0>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<NC, WG, UNITS, D>::kSmem);
}

}  // namespace

cudaError_t chunk_tc_keys_prepare() {
  cudaError_t e = prepare_cfg<32, 1, 3, 128>();
  if (e == cudaSuccess) e = prepare_cfg<32, 2, 6, 128>();
  if (e == cudaSuccess) e = prepare_cfg<32, 4, 5, 128>();
  if (e == cudaSuccess) e = prepare_cfg<32, 1, 6, 64>();
  if (e == cudaSuccess) e = prepare_cfg<32, 2, 8, 64>();
  if (e == cudaSuccess) e = prepare_cfg<32, 4, 8, 64>();
  if (e == cudaSuccess) e = prepare_hist<32, 1, 3, 128, 1>();
  if (e == cudaSuccess) e = prepare_hist<32, 1, 3, 128, 2>();
  if (e == cudaSuccess) e = prepare_hist<32, 1, 6, 64, 1>();
  if (e == cudaSuccess) e = prepare_hist<32, 1, 6, 64, 2>();
  return e;
}

// A list of chunks in one launch: up to 32 rows per kv-head (two CTAs per SM).
cudaError_t launch_chunk_tc_keys_hist(const ChunkParams& p, const HistParams& h, const CUtensorMap& any_map,
                                      cudaStream_t s, bool pdl) {
  if (h.n_chunks < 1 || h.n_chunks > kMaxHistChunksKeys || !h.maps || p.n_active || p.page_table ||
      p.rows_per_tile > 32)
    return cudaErrorInvalidValue;
  // (the K/V map parameters are not used by these instantiations: any valid map will do)
  if (h.n_req) {
    // ragged batch: h.walk_ctas CTAs per kv-head share all requests' tiles (one row tile)
    if (p.row_tiles != 1 || h.n_req != p.B || h.walk_ctas < 1) return cudaErrorInvalidValue;
    dim3 grid(h.walk_ctas, p.H_kv, 1);
    return p.d == 64 ? launch_hist_cfg<32, 1, 6, 64, 2>(p, h, any_map, grid, s, pdl)
                     : launch_hist_cfg<32, 1, 3, 128, 2>(p, h, any_map, grid, s, pdl);
  }
  dim3 grid(p.splits * p.row_tiles, p.H_kv, p.B);
  return p.d == 64 ? launch_hist_cfg<32, 1, 6, 64, 1>(p, h, any_map, grid, s, pdl)
                   : launch_hist_cfg<32, 1, 3, 128, 1>(p, h, any_map, grid, s, pdl);
}

// Rows per CTA (p.rows_per_tile): <= 32 -> two CTAs per SM with 4 softmax warps; <= 64 and
// <= 128 -> one CTA per SM with 8 and 16 softmax warps (32 score columns per thread each).
// Head dim 64 halves a tile's bytes, so its rings have twice the units.
cudaError_t launch_chunk_tc_keys(const ChunkParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                 cudaStream_t s, bool pdl) {
  if (p.d == 64) {
    if (p.rows_per_tile <= 32) return launch_cfg<32, 1, 6, 64>(p, tmK, tmV, s, pdl);
    if (p.rows_per_tile <= 64) return launch_cfg<32, 2, 8, 64>(p, tmK, tmV, s, pdl);
    return launch_cfg<32, 4, 8, 64>(p, tmK, tmV, s, pdl);
  }
  if (p.rows_per_tile <= 32) return launch_cfg<32, 1, 3, 128>(p, tmK, tmV, s, pdl);
  if (p.rows_per_tile <= 64) return launch_cfg<32, 2, 6, 128>(p, tmK, tmV, s, pdl);
  return launch_cfg<32, 4, 5, 128>(p, tmK, tmV, s, pdl);
}

}  // namespace ss
