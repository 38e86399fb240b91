// Tensor-core chunk attention for sm_100a: TMA-staged K/V tiles, tcgen05 MMAs with the query
// tile Q, the score tile S, the probabilities P and the unnormalised output O all held in
// tensor memory.
//
// One CTA owns one (request, kv-head, token split, tile of <= 128 query rows).  All rows of
// the kv-head (T_q candidate queries x G query heads) ride in the M dimension of the MMAs,
// so every K/V byte is fetched from HBM once and serves the whole query group.
//
// The kernel is a template over the head dim (64 or 128); the figures below are for 128.  At 64
// a tile is one [64][64] box per operand, the rings hold six K and six V slots, the score
// MMA takes four k-steps, the output MMA has N = 64, and tensor memory has room for a second
// score buffer (see Tm below), so the score MMAs run two tiles ahead instead of the register
// double-buffering described next.
//
//   warp 4 (one lane)  TMA producer: K tiles and V tiles of 64 tokens, three K slots and four V
//                      slots, 128-byte swizzle, evict-first L2 policy (the history is
//                      streamed).  A K slot is released as soon as its score MMAs retire, a V
//                      slot after its output MMAs.
//   warp 5 (one lane)  MMA issuer:   S = Q K_t^T     (M=128, N=64,  K=d=128: 8 x k16, tmem x smem)
//                                    O += P_t V_t    (M=128, N=128, K=64:    4 x k16, tmem x smem)
//                      Both A operands come from tensor memory, so an MMA reads only its B
//                      operand from shared memory (2 KB and 4 KB per k-step).  With Q in shared
//                      memory a score MMA read 6 KB per k-step and ran at the shared-memory
//                      bandwidth (48 instead of 32 cycles, measured), which made the tensor
//                      pipe's queue the bound of the many-rows workloads.
//   warps 0-3          softmax: each thread owns one TMEM lane (= one MMA row): per tile it
//                      computes P from the scores it holds in registers, reads the NEXT tile's
//                      scores from the score buffer into registers, and only then writes P as
//                      packed bf16 over the leading columns of the same buffer.
//
// One score buffer is enough because the double buffering happens in registers.  Arrival k of
// the softmax threads means "S(k) is in registers and P(k-1) is in the buffer"; on it the
// issuer runs PV(k-1) and then QK(k+1), which overwrites the buffer.  While the threads work on
// tile k (about a thousand cycles) the tensor pipe finishes PV(k-1) and QK(k+1), so neither
// side waits for the other in steady state.
//
// Tensor memory (256 columns): [0,64) S (fp32; P of a tile as bf16 pairs over its first 32
// columns); [64,128) Q as bf16 pairs (column j of lane r = head dims 2j, 2j+1 of row r);
// [128,256) O (fp32).  Shared memory: three K slots and four V slots (112 KB) and 256 bytes of
// barriers, so that two CTAs fit per SM (the window must be 1024-byte aligned; checked at run
// time).
//
// When the row tile has <= 32 (<= 64) rows the Q rows are replicated 4x (2x) along M and
// each replica takes a quarter (half) of the tile's keys: lane L holds row L % R_pad and
// key group L / R_pad.  All four softmax warps then work on every tile, and the four
// replicas are four independent online-softmax states that are merged when the CTA ends.
//
// Running maximum: a row's reference maximum m only moves when the tile maximum exceeds it
// by more than 8 (base-2 domain), which keeps exp2(s - m) <= 256 and makes the rescale of O
// in tensor memory rare.  Because PV(t-1) may still be accumulating into O while the softmax
// of tile t runs, a rescale first waits for the commit of PV(t-1).
//
// Every wait on an mbarrier is bounded; on expiry the CTA raises SS_DEV_WAIT_EXPIRED, lets
// its own copies land (bounded), frees its tensor memory and returns.
#include "ss_internal.h"
#include "tc_ptx.cuh"

namespace ss {
namespace {

constexpr int kThreads = 192;
constexpr int kHalfTile = kTileKeys * 64 * 2;       // 8 KB: [64 keys][64 d] bf16, one TMA box
constexpr int kSmemCtl = 512;   // barriers (<= 256 bytes), then the chunk table of a launch over a list of chunks
constexpr uint32_t kTmemCols = 256;
// Tensor-memory columns for head dim D: NS score buffers of 64 columns, Q as bf16 pairs (D / 2
// columns), O (D columns).  Head dim 128: one score buffer (64 + 64 + 128 = 256 columns, what a
// CTA can take with two CTAs per SM).  Head dim 64: room for two (128 + 32 + 64 = 224), so the
// scores of tile t+1 can be computed while tile t is still in its buffer.
template <int D>
struct Tm {
  static constexpr int NS = D == 64 ? 2 : 1;
  static constexpr uint32_t kColS = 0, kColQ = NS * 64, kColO = NS * 64 + D / 2;
  static_assert(kColO + D <= 256, "tensor-memory columns");
};
constexpr float kRescaleThreshold = 8.f;

// Shared-memory layout for head dim D (64 or 128): the K slots, then the V slots, D / 64 boxes
// of 64 columns each.  Head dim 64 halves a tile's bytes, so it takes about twice the slots.
template <int D>
struct Lay {
  static constexpr int kHalves = D / 64;
  static constexpr int kKStages = D == 128 ? 3 : 6, kVStages = D == 128 ? 4 : 6;
  static constexpr int kTileBytes = kHalves * kHalfTile;      // one K tile or one V tile
  static constexpr int kOffK = 0;                             // K slots
  static constexpr int kOffV = kOffK + kKStages * kTileBytes; // V slots
  static constexpr int kSmemData = kOffV + kVStages * kTileBytes;  // 112 KB (d = 128), 96 KB (64)
  static constexpr int kSmemTotal = kSmemData + kSmemCtl;
  // two CTAs per SM: 227 KB per SM less 1 KB reserved per CTA
  static_assert(2 * (kSmemTotal + 1024) <= 227 * 1024, "two CTAs per SM");
  // the write-out stages 128 rows x D floats and 128 (m, l) pairs over the idle slots
  static_assert(kSmemData >= 128 * D * 4 + 128 * 8, "write-out staging");
  static_assert(D == 64 || D == 128, "head dim");
};

template <int KS, int VS>
struct CtlT {
  uint64_t kfull[KS], kempty[KS], vfull[VS], vempty[VS];
  uint64_t qready;               // the Q rows are in tensor memory
  uint64_t sfull[2];             // S(t) = Q K_t^T has retired: one score buffer -> sfull[0], one phase per
                                 // tile; two score buffers -> sfull[t % 2]
  uint64_t pready[2];            // arrival k of the softmax threads (S(k) in registers, P(k-1) stored)
                                 // goes to pready[k % 2]: a thread may make its last arrival before the
                                 // issuer has looked at the one before it, and one barrier's parity
                                 // could not tell the two phases apart
  uint64_t odone;                // one phase per tile: PV(t) has retired
  uint64_t pvdone;               // the last PV has retired
  uint32_t tmem_base;
  volatile uint32_t abort;
};
static_assert(sizeof(CtlT<3, 4>) <= kSmemCtl && sizeof(CtlT<6, 6>) <= kSmemCtl, "control block");


using namespace ss::tc;
template <typename C>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, C* ctl, uint32_t* status) {
  return mbar_wait_abortable(bar, parity, &ctl->abort, status);
}

// P (bf16 pairs) over the 32 leading score columns in 4 blocks of 8: blocks
// [FIRST, FIRST + NC/16) hold this lane's keys, the others are zero.
template <int NC, int FIRST>
__device__ __forceinline__ void store_p(uint32_t t_s, const uint32_t (&pk)[NC / 16][8]) {
  const uint32_t zero[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (q >= FIRST && q < FIRST + NC / 16)
      tmem_st8(t_s + q * 8, pk[(q >= FIRST && q < FIRST + NC / 16) ? q - FIRST : 0]);
    else
      tmem_st8(t_s + q * 8, zero);
  }
}

// ---- softmax of one tile for one TMEM lane --------------------------------------------------
// NC = number of key columns this lane owns in a 64-key tile (columns [c0, c0 + NC)).
template <int NC>
__device__ __forceinline__ void load_scores(uint32_t t_s, int c0, uint32_t (&raw)[NC / 16][16]) {
#pragma unroll
  for (int q = 0; q < NC / 16; ++q) tmem_ld16(t_s + c0 + q * 16, raw[q]);
  tc_wait_ld();
}

// From the scores in `raw` to P as packed bf16 pairs in `pk`, updating the row state (m, l).
// MASK = the tile straddles the valid length (columns >= n_valid are invisible).  The scale is
// positive (checked at ss_verify_begin), so the maximum is taken on the raw scores and the
// scaling rides in the FMA that subtracts the reference.
// Returns false when the wait for PV(it - 1) in the rescale path gave up.
template <int NC, bool MASK, int D, typename C>
__device__ __forceinline__ bool softmax_compute(uint32_t (&raw)[NC / 16][16], uint32_t t_o, int c0,
                                                int n_valid, int it, float scale_log2, float& m,
                                                float& l, C* ctl, uint32_t* status,
                                                uint32_t (&pk)[NC / 16][8]) {
  const bool have_o = it > 0;
  float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // independent chains
  if (MASK) {
#pragma unroll
    for (int c = 0; c < NC; ++c)
      if (c0 + c >= n_valid) raw[c / 16][c % 16] = __float_as_uint(-INFINITY);
  }
#pragma unroll
  for (int c = 0; c < NC; c += 2)
    mx4[(c >> 1) & 3] = max3_f(mx4[(c >> 1) & 3], __uint_as_float(raw[c / 16][c % 16]),
                               __uint_as_float(raw[(c + 1) / 16][(c + 1) % 16]));
  const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
  float f = 1.f;
  if (mx > m + kRescaleThreshold) {  // also the first finite maximum (m = -inf)
    f = (m == -INFINITY) ? 0.f : exp2f(m - mx);
    l *= f;
    m = mx;
  }
  const bool need = have_o && (f != 1.f);
  if (__any_sync(0xffffffffu, need)) {
    // rare: move this lane's O row to the new reference maximum, once PV(it - 1) has retired
    // (its phase is the latest the barrier can have completed: PV(it) needs this tile's P)
    if (!mbar_wait(&ctl->odone, (it - 1) & 1, ctl, status)) return false;
    tc_fence_after();
#pragma unroll 1
    for (int q = 0; q < D / 16; ++q) {
      uint32_t o[16];
      tmem_ld16(t_o + q * 16, o);
      tc_wait_ld();
#pragma unroll
      for (int c = 0; c < 16; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
      tmem_st16(t_o + q * 16, o);
    }
  }
  const float neg_m = (m == -INFINITY) ? 0.f : -m;
  // two keys per packed fp32 instruction: x = s * scale - m, then the row sum
  float2 sum2[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
  const float2 sc2 = make_float2(scale_log2, scale_log2), nm2 = make_float2(neg_m, neg_m);
#pragma unroll
  for (int c = 0; c < NC; c += 2) {
    const float2 x = fma2_f(make_float2(__uint_as_float(raw[c / 16][c % 16]),
                                        __uint_as_float(raw[(c + 1) / 16][(c + 1) % 16])),
                            sc2, nm2);
    const float2 pp = make_float2(ex2_ftz(x.x), ex2_ftz(x.y));
    sum2[(c >> 1) & 3] = add2_f(sum2[(c >> 1) & 3], pp);
    __nv_bfloat162 h = __floats2bfloat162_rn(pp.x, pp.y);  // low half = even key
    pk[c / 16][(c / 2) % 8] = *reinterpret_cast<uint32_t*>(&h);
  }
  const float2 s01 = add2_f(sum2[0], sum2[1]), s23 = add2_f(sum2[2], sum2[3]);
  l += (s01.x + s01.y) + (s23.x + s23.y);
  return true;
}

// P of this lane's keys -> the leading 32 columns of the score buffer (zeros for the other
// lanes' key groups), then wait for every tensor-memory store of this thread.
template <int NC>
__device__ __forceinline__ void store_p_at(uint32_t t_s, int c0, const uint32_t (&pk)[NC / 16][8]) {
  // c0 is uniform across a warp; dispatching on it keeps pk[] in registers
  if (NC == 64) {
    store_p<NC, 0>(t_s, pk);
  } else if (NC == 32) {
    if (c0 == 0) store_p<NC, 0>(t_s, pk);
    else store_p<NC, 2>(t_s, pk);
  } else {
    switch (c0 / 16) {
      case 0: store_p<NC, 0>(t_s, pk); break;
      case 1: store_p<NC, 1>(t_s, pk); break;
      case 2: store_p<NC, 2>(t_s, pk); break;
      default: store_p<NC, 3>(t_s, pk); break;
    }
  }
  tc_wait_st();
}

// Which tokens the CTA's tile `it` holds.  One chunk: tokens [tok0, tok1) in tiles of 64.  A list
// of chunks: the CTA's tiles are numbers [g0, g0 + n_tiles) of the request's tiles counted chunk
// by chunk; prefix[j] = tiles before chunk j, valid[j] = the request's tokens in chunk j (a table
// in shared memory); a role walks the tiles in order and keeps the chunk it is in.
template <bool HIST>
struct TileMap {
  int tok0, tok1;
  __device__ __forceinline__ int n_valid(int it) { return min(kTileKeys, tok1 - (tok0 + it * kTileKeys)); }
};
template <>
struct TileMap<true> {
  const uint16_t* prefix;
  const int* valid;
  int g0, j;
  // chunk of tile `it` (tiles are asked for in ascending order) and the tile's first token in it
  __device__ __forceinline__ int locate(int it, int* tok) {
    const int g = g0 + it;
    while (g >= prefix[j + 1]) ++j;
    *tok = (g - prefix[j]) * kTileKeys;
    return j;
  }
  __device__ __forceinline__ int n_valid(int it) {
    int tok;
    const int c = locate(it, &tok);
    return min(kTileKeys, valid[c] - tok);
  }
};

// The tile loop of one softmax thread (TMEM lane L, key columns [c0, c0 + NC) of every tile).
// Arrival k on `pready` says: S(k) is in this thread's registers and P(k-1) is in the buffer.
// Returns false when a bounded wait gave up.
template <int NC, int D, typename C, typename TM>
__device__ __forceinline__ bool softmax_loop(const ChunkParams& p, C* ctl, uint32_t tmem_lane, int c0,
                                             int n_tiles, TM tm, uint8_t* v_s0, int L,
                                             float& m, float& l, unsigned long long* tr) {
  constexpr int kVStages = Lay<D>::kVStages, kTileBytes = Lay<D>::kTileBytes;
  const uint32_t t_s = tmem_lane + Tm<D>::kColS, t_o = tmem_lane + Tm<D>::kColO;
  uint32_t raw[NC / 16][16];
  if (!mbar_wait(&ctl->sfull[0], 0, ctl, p.status)) return false;
  tc_fence_after();
  load_scores<NC>(t_s, c0, raw);
  tc_fence_before();
  mbar_arrive(&ctl->pready[0]);  // arrival 0: the issuer may overwrite the buffer with S(1)
  for (int it = 0; it < n_tiles; ++it) {
    if (L == 0) trace(tr, 2, it, 0);
    const int n_valid = tm.n_valid(it);
    if (n_valid < kTileKeys) {
      // ragged tail: rows past the valid length may hold anything; P is 0 there, so V must
      // be finite: clear those rows of the staged V tile (whole 128-byte rows, both halves)
      const int s = it % kVStages;
      if (!mbar_wait(&ctl->vfull[s], (it / kVStages) & 1, ctl, p.status)) return false;
      uint8_t* v_s = v_s0 + s * kTileBytes;
      constexpr int kVecRow = D / 8;  // 16-byte pieces per token row
      const int n_vec = (kTileKeys - n_valid) * kVecRow;
      for (int i = L; i < n_vec; i += 128) {
        const int row = n_valid + i / kVecRow, half = (i % kVecRow) >> 3, ch = i & 7;
        *reinterpret_cast<uint4*>(v_s + half * kHalfTile + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
      }
      fence_proxy_async();
    }
    uint32_t pk[NC / 16][8];
    const bool ok = (n_valid < kTileKeys)
                        ? softmax_compute<NC, true, D>(raw, t_o, c0, n_valid, it, p.scale_log2, m, l, ctl, p.status, pk)
                        : softmax_compute<NC, false, D>(raw, t_o, c0, n_valid, it, p.scale_log2, m, l, ctl, p.status, pk);
    if (!ok) return false;
    if (L == 0) trace(tr, 2, it, 1);
    if (it + 1 < n_tiles) {
      // the next tile's scores move into registers before P takes their place
      if (!mbar_wait(&ctl->sfull[0], (it + 1) & 1, ctl, p.status)) return false;
      tc_fence_after();
      load_scores<NC>(t_s, c0, raw);
      if (L == 0) trace(tr, 2, it, 3);
    } else if (it > 0) {
      // Last tile: no new scores to wait for.  PV(it - 1) still reads P(it - 1) from the columns
      // P(it) is about to take (S(it + 1) having retired implies it in the other iterations).
      if (!mbar_wait(&ctl->odone, (it - 1) & 1, ctl, p.status)) return false;
      tc_fence_after();
    }
    store_p_at<NC>(t_s, c0, pk);
    tc_fence_before();
    mbar_arrive(&ctl->pready[(it + 1) & 1]);  // arrival it + 1
    if (L == 0) trace(tr, 2, it, 2);
  }
  return true;
}

// The same loop with two score buffers (head dim 64): tile t lives in buffer t % 2, its P goes
// over the leading columns of the same buffer, and the issuer runs the score MMAs two tiles
// ahead, so a thread finds S(t) ready when it gets there and needs no second set of registers.
template <int NC, int D, typename C, typename TM>
__device__ __forceinline__ bool softmax_loop2(const ChunkParams& p, C* ctl, uint32_t tmem_lane, int c0,
                                              int n_tiles, TM tm, uint8_t* v_s0, int L,
                                              float& m, float& l, unsigned long long* tr) {
  constexpr int kVStages = Lay<D>::kVStages, kTileBytes = Lay<D>::kTileBytes;
  const uint32_t t_o = tmem_lane + Tm<D>::kColO;
  for (int it = 0; it < n_tiles; ++it) {
    const uint32_t t_s = tmem_lane + Tm<D>::kColS + (it & 1) * 64;
    if (L == 0) trace(tr, 2, it, 0);
    if (!mbar_wait(&ctl->sfull[it & 1], (it >> 1) & 1, ctl, p.status)) return false;
    tc_fence_after();
    uint32_t raw[NC / 16][16];
    load_scores<NC>(t_s, c0, raw);
    if (L == 0) trace(tr, 2, it, 3);
    const int n_valid = tm.n_valid(it);
    if (n_valid < kTileKeys) {
      // ragged tail: clear the rows of the staged V tile past the valid length (see softmax_loop)
      const int s = it % kVStages;
      if (!mbar_wait(&ctl->vfull[s], (it / kVStages) & 1, ctl, p.status)) return false;
      uint8_t* v_s = v_s0 + s * kTileBytes;
      constexpr int kVecRow = D / 8;
      const int n_vec = (kTileKeys - n_valid) * kVecRow;
      for (int i = L; i < n_vec; i += 128) {
        const int row = n_valid + i / kVecRow, half = (i % kVecRow) >> 3, ch = i & 7;
        *reinterpret_cast<uint4*>(v_s + half * kHalfTile + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
      }
      fence_proxy_async();
    }
    uint32_t pk[NC / 16][8];
    const bool ok = (n_valid < kTileKeys)
                        ? softmax_compute<NC, true, D>(raw, t_o, c0, n_valid, it, p.scale_log2, m, l, ctl, p.status, pk)
                        : softmax_compute<NC, false, D>(raw, t_o, c0, n_valid, it, p.scale_log2, m, l, ctl, p.status, pk);
    if (!ok) return false;
    if (L == 0) trace(tr, 2, it, 1);
    store_p_at<NC>(t_s, c0, pk);
    tc_fence_before();
    mbar_arrive(&ctl->pready[it & 1]);
    if (L == 0) trace(tr, 2, it, 2);
  }
  return true;
}

template <int D, bool HIST>
__global__ void __launch_bounds__(kThreads, 2)
chunk_tc_kernel(const ChunkParams p, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmA,
                const __grid_constant__ HistParams h) {
  using L_ = Lay<D>;
  constexpr int kD = D, kHalves = L_::kHalves, kKStages = L_::kKStages, kVStages = L_::kVStages;
  constexpr int kTileBytes = L_::kTileBytes, kOffK = L_::kOffK, kOffV = L_::kOffV, kSmemData = L_::kSmemData;
  using Ctl = CtlT<kKStages, kVStages>;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* k_s = smem + kOffK;     // K slots
  uint8_t* v_s0 = smem + kOffV;    // V slots
  Ctl* ctl = reinterpret_cast<Ctl*>(smem + kSmemData);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned long long t_cta0 = p.cta_log ? cta_log_now() : 0ull;
  if (p.wait_first) pdl_wait_prior();
  pdl_launch_dependents();
  const ChunkWork w = chunk_work(p, p.rows_per_tile);
  const int b = w.b, kvh = w.kvh, row0 = w.row0, nrows = w.nrows;
  int tok0 = w.tok0, tok1 = w.tok1;
  const bool chain_cta = w.chain_cta;
  float2* out_ml = w.out_ml;
  // key groups sharing the 128 lanes: the Q rows are replicated when the tile has few rows
  const int groups = nrows <= 32 ? 4 : (nrows <= 64 ? 2 : 1);
  const int r_pad = 128 / groups;
  unsigned long long* tr = chain_cta ? p.trace : nullptr;
  int n_tiles = (tok1 > tok0) ? (tok1 - tok0 + kTileKeys - 1) / kTileKeys : 0;
  // a list of chunks: the table of the request's tiles per chunk, then this CTA's share of them
  // (16-bit tile counts: the host keeps a request's tiles below 65,536; 256 + 128 + 66 bytes end
  // inside the control block's 512)
  int* const hist_valid = reinterpret_cast<int*>(smem + kSmemData + 256);                      // [kMaxHistChunks]
  uint16_t* const hist_prefix = reinterpret_cast<uint16_t*>(hist_valid + kMaxHistChunks);      // [kMaxHistChunks + 1]
  static_assert(256 + kMaxHistChunks * 4 + (kMaxHistChunks + 1) * 2 <= kSmemCtl, "chunk table");
  int g0 = 0;
  if (HIST) {
    if (warp == 0) {
      int v = 0;
      if (lane < h.n_chunks) {
        const int L = h.L_c[lane];
        v = h.valid_len[lane] ? h.valid_len[lane][b] : L;
        if (v < 0 || v > L) {  // flagged and clamped, never trusted
          atomicOr(p.status, SS_DEV_BAD_VALID_LEN);
          v = max(0, min(v, L));
        }
      }
      int incl = (v + kTileKeys - 1) / kTileKeys;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      if (lane < h.n_chunks) {
        hist_prefix[lane + 1] = (uint16_t)incl;
        hist_valid[lane] = v;
      }
      if (lane == 0) hist_prefix[0] = 0;
      // (entries past the last chunk repeat the total, so a walk never runs off the table)
      const int total = __shfl_sync(0xffffffffu, incl, 31);
      if (lane >= h.n_chunks) hist_prefix[lane + 1] = (uint16_t)total;
    }
    __syncthreads();
    const int total = hist_prefix[h.n_chunks];
    g0 = (int)((int64_t)total * w.split / p.splits);
    n_tiles = (int)((int64_t)total * (w.split + 1) / p.splits) - g0;
  }

  if (n_tiles == 0 || (smem_u32(smem) & 1023u)) {
    // nothing visible here (identity state, no tensor memory taken); a misaligned shared
    // memory window would break the swizzled layouts and is reported instead of run
    if (n_tiles && tid == 0) atomicOr(p.status, SS_DEV_WAIT_EXPIRED);
    if (tid < nrows) out_ml[tid] = make_float2(-INFINITY, 0.f);
    if (!p.wait_first && chain_cta) pdl_wait_prior();
    return;
  }

  // ---- set-up: barriers, first loads, tensor memory, the Q tile --------------------------------
  // both 64-column halves of a box of tokens starting at (outer, tok) -> dst (K when !is_v)
  auto load_rows = [&](bool is_v, uint32_t dst, int tok, int outer, uint64_t* bar, uint64_t pol) {
    if (is_v) {  // (no runtime-selected pointer: the tensor maps stay in the parameter space)
      tma_load_4d(dst, &tmV, 0, tok, kvh, outer, bar, pol);
      if (D == 128) tma_load_4d(dst + kHalfTile, &tmV, 64, tok, kvh, outer, bar, pol);
    } else {
      tma_load_4d(dst, &tmK, 0, tok, kvh, outer, bar, pol);
      if (D == 128) tma_load_4d(dst + kHalfTile, &tmK, 64, tok, kvh, outer, bar, pol);
    }
  };
  // Pages smaller than a tile (8, 16 or 32 tokens): the tile is gathered page by page by the whole
  // producer warp, see below; this path is for contiguous chunks and pages of a tile or more.
  const bool small_pages = p.page_table && p.page_size < kTileKeys;
  TileMap<true> map_k = {hist_prefix, hist_valid, g0, 0}, map_v = map_k;  // (list of chunks) the producer's two walks
  auto issue_tile = [&](bool is_v, int it, uint32_t dst, uint64_t* bar, uint64_t pol) {
    mbar_expect_tx(bar, kTileBytes);
    if (HIST) {
      int tok;
      const int c = is_v ? map_v.locate(it, &tok) : map_k.locate(it, &tok);
      const CUtensorMap* m = h.maps + 2 * c + (is_v ? 1 : 0);  // in device memory
      tma_load_4d(dst, m, 0, tok, kvh, b, bar, pol);
      if (D == 128) tma_load_4d(dst + kHalfTile, m, 64, tok, kvh, b, bar, pol);
      return;
    }
    int outer, tok;
    locate_token(p, b, tok0 + it * kTileKeys, &outer, &tok);
    load_rows(is_v, dst, tok, outer, bar, pol);
  };
  auto issue_k = [&](int it, uint64_t pol) {
    const int s = it % kKStages;
    issue_tile(false, it, smem_u32(k_s + s * kTileBytes), &ctl->kfull[s], pol);
  };
  auto issue_v = [&](int it, uint64_t pol) {
    const int s = it % kVStages;
    issue_tile(true, it, smem_u32(v_s0 + s * kTileBytes), &ctl->vfull[s], pol);
  };
  // (small pages: all copies go out from the producer warp's loop)
  const int n_pre_k = small_pages ? 0 : min(n_tiles, kKStages), n_pre_v = small_pages ? 0 : min(n_tiles, kVStages);
  uint4 qreg[kD / 8];  // softmax threads: this lane's Q row on its way to tensor memory
  if (warp == 4) {
    if (lane == 0) {
      for (int s = 0; s < kKStages; ++s) {
        mbar_init(&ctl->kfull[s], 1);
        mbar_init(&ctl->kempty[s], 1);
      }
      for (int s = 0; s < kVStages; ++s) {
        mbar_init(&ctl->vfull[s], 1);
        mbar_init(&ctl->vempty[s], 1);
      }
      mbar_init(&ctl->qready, 128);
      mbar_init(&ctl->sfull[0], 1);
      mbar_init(&ctl->sfull[1], 1);
      mbar_init(&ctl->pready[0], 128);
      mbar_init(&ctl->pready[1], 128);
      mbar_init(&ctl->odone, 1);
      mbar_init(&ctl->pvdone, 1);
      ctl->abort = 0;
      fence_barrier_init();
      // the first tiles go out before the rest of the CTA is set up (K first: the score
      // MMAs of both tiles come before the first output MMAs)
      // streamed once: evict first; shared by the row groups of a kv-head through L2: keep
      const uint64_t pol = p.row_tiles > 1 ? l2_evict_normal_policy() : l2_evict_first_policy();
      for (int it = 0; it < n_pre_k; ++it) issue_k(it, pol);
      for (int it = 0; it < n_pre_v; ++it) issue_v(it, pol);
    }
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&ctl->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  } else if (warp < 4) {
    // this lane's Q row, fetched while the barriers and the tensor memory are being set up
    const int r = tid % r_pad;
    const uint4* src = nullptr;
    if (r < nrows) {
      const int rg = row0 + r, g = rg / p.T_q, t = rg % p.T_q;
      src = reinterpret_cast<const uint4*>(p.Q + b * p.q_sb + (int64_t)(kvh * p.G + g) * p.q_sh +
                                           t * p.q_st);
    }
#pragma unroll
    for (int v = 0; v < kD / 8; ++v) qreg[v] = src ? src[v] : make_uint4(0, 0, 0, 0);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  unsigned long long* trl = lane == 0 ? tr : nullptr;

  if (warp == 4 && small_pages) {
    // ===== TMA producer, pages smaller than a tile =====
    // The tensor map's box is one page; page i of a tile lands at row i * page_size of the slot,
    // which keeps the swizzled layout of a single 64-token box.  Lane l copies 64-column half
    // l % 2 of page l / 2 of the tile, so a tile's 4 to 16 copies and their page look-ups go out
    // side by side; each lane fetches the page id of a ring's next tile right after its copy,
    // off the path of the next one.  Pages that start at or past the valid length are not
    // looked up (index n_pages is outside the pool and reads as zeros).  Lane 0 polls the two
    // rings as in the loop below, arms the barriers and shares what to issue through a shuffle.
    const uint64_t pol = p.row_tiles > 1 ? l2_evict_normal_policy() : l2_evict_first_policy();
    const int ps = p.page_size, n_sub = kTileKeys / ps;  // 2 to 8 pages per tile (pages of 32 to 8 tokens)
    const int sub = lane / kHalves, half = lane % kHalves;
    const bool mine = lane < kHalves * n_sub;
    auto lane_page = [&](int tile) {  // page id of this lane's page of `tile`; -2: not looked up
      const int tk = tok0 + tile * kTileKeys + sub * ps;
      if (!mine || tk >= tok1) return -2;
      const int pg = tk / ps;
      return pg < p.pages_per_req ? p.page_table[(int64_t)b * p.pages_per_req + pg] : -1;
    };
    auto checked = [&](int id) {
      if (id == -2) return p.n_pages;
      if (id < 0 || id >= p.n_pages) {
        atomicOr(p.status, SS_DEV_BAD_PAGE);
        return p.n_pages;
      }
      return id;
    };
    int issued_k = 0, issued_v = 0;
    int page_k = lane_page(0), page_v = page_k;
    unsigned long long t0 = gtime_ns();
    uint32_t spins = 0;
    while (issued_k < n_tiles || issued_v < n_tiles) {
      int act = 0;  // bit 0: K tile, bit 1: V tile, bit 2: give up
      if (lane == 0) {
        if (issued_k < n_tiles &&
            mbar_test(&ctl->kempty[issued_k % kKStages], ((issued_k / kKStages) & 1) ^ 1)) {
          mbar_expect_tx(&ctl->kfull[issued_k % kKStages], kTileBytes);
          act |= 1;
        }
        if (issued_v < n_tiles &&
            mbar_test(&ctl->vempty[issued_v % kVStages], ((issued_v / kVStages) & 1) ^ 1)) {
          mbar_expect_tx(&ctl->vfull[issued_v % kVStages], kTileBytes);
          act |= 2;
        }
        if (act) {
          spins = 0;
          t0 = gtime_ns();
        } else if ((++spins & 255u) == 0) {  // bounded like every other wait
          if (ctl->abort) {
            act = 4;
          } else if (gtime_ns() - t0 > kWaitNs) {
            ctl->abort = 1;
            atomicOr(p.status, SS_DEV_WAIT_EXPIRED);
            act = 4;
          }
        }
      }
      act = __shfl_sync(0xffffffffu, act, 0);  // also orders the arming before the copies
      if (act & 4) break;
      if (act & 1) {
        const int s = issued_k % kKStages;
        if (mine)
          tma_load_4d(smem_u32(k_s + s * kTileBytes) + half * kHalfTile + sub * ps * 128, &tmK, half * 64, 0,
                      kvh, checked(page_k), &ctl->kfull[s], pol);
        ++issued_k;
        page_k = lane_page(issued_k);
      }
      if (act & 2) {
        const int s = issued_v % kVStages;
        if (mine)
          tma_load_4d(smem_u32(v_s0 + s * kTileBytes) + half * kHalfTile + sub * ps * 128, &tmV, half * 64, 0,
                      kvh, checked(page_v), &ctl->vfull[s], pol);
        ++issued_v;
        page_v = lane_page(issued_v);
      }
    }
    if (lane == 0 && ctl->abort) {
      // let the copies the warp started land before the CTA leaves (bounded)
      const unsigned long long t1 = gtime_ns();
      for (int it = max(0, issued_k - kKStages); it < issued_k; ++it)
        while (!mbar_try_wait(&ctl->kfull[it % kKStages], (it / kKStages) & 1) && gtime_ns() - t1 < kWaitNs) {
        }
      for (int it = max(0, issued_v - kVStages); it < issued_v; ++it)
        while (!mbar_try_wait(&ctl->vfull[it % kVStages], (it / kVStages) & 1) && gtime_ns() - t1 < kWaitNs) {
        }
    }
  } else if (warp == 4) {
    // ===== TMA producer =====
    if (lane == 0) {
      // streamed once: evict first; shared by the row groups of a kv-head through L2: keep
      const uint64_t pol = p.row_tiles > 1 ? l2_evict_normal_policy() : l2_evict_first_policy();
      // A K slot frees when its score MMAs retire, a V slot when its output MMAs do, and the
      // issuer runs them in a fixed order: QK(0), then QK(j), PV(j - 1) for j = 1, 2, ...  The
      // producer follows that order with blocking (bounded) waits - K(j + 3) after QK(j), V(j + 3)
      // after PV(j - 1) - so that it sleeps in the barrier instead of taking issue slots from
      // the softmax warp on its scheduler.
      int issued_k = n_pre_k, issued_v = n_pre_v;
      for (int j = 0; issued_k < n_tiles || issued_v < n_tiles; ++j) {
        if (issued_k < n_tiles) {
          if (!mbar_wait(&ctl->kempty[issued_k % kKStages], ((issued_k / kKStages) & 1) ^ 1, ctl, p.status)) break;
          trace(tr, 0, issued_k, 1);
          issue_k(issued_k, pol);
          ++issued_k;
        }
        if (j >= 1 && issued_v < n_tiles) {
          if (!mbar_wait(&ctl->vempty[issued_v % kVStages], ((issued_v / kVStages) & 1) ^ 1, ctl, p.status)) break;
          trace(tr, 0, issued_v, 2);
          issue_v(issued_v, pol);
          ++issued_v;
        }
      }
      if (ctl->abort) {
        // let the copies this thread started land before the CTA leaves (bounded)
        const unsigned long long t0 = gtime_ns();
        for (int it = max(0, issued_k - kKStages); it < issued_k; ++it) {
          while (!mbar_try_wait(&ctl->kfull[it % kKStages], (it / kKStages) & 1) &&
                 gtime_ns() - t0 < kWaitNs) {
          }
        }
        for (int it = max(0, issued_v - kVStages); it < issued_v; ++it) {
          while (!mbar_try_wait(&ctl->vfull[it % kVStages], (it / kVStages) & 1) &&
                 gtime_ns() - t0 < kWaitNs) {
          }
        }
      }
    }
  } else if (warp == 5) {
    // ===== MMA issuer: the whole warp walks the loop (uniform descriptors), one elected
    // lane issues =====
    constexpr uint32_t idesc_qk = make_idesc(128, kTileKeys, false);
    constexpr uint32_t idesc_pv = make_idesc(128, kD, true);
    constexpr int kNS = Tm<D>::NS;
    const bool leader = elect_one();
    const uint32_t k_base = smem_u32(k_s), v_base = smem_u32(v_s0);
    // The operand descriptors of one slot differ only in their address field (bits 0-13, the
    // shared-memory address / 16): they are built once and advanced by constants, which keeps
    // the issue loop to a few instructions per MMA.  (All operand addresses are below 256 KB,
    // so the field never carries.)
    const uint64_t k_desc0 = desc_kmajor(k_base);
    const uint64_t v_desc0 = desc_mnmajor(v_base, kHalfTile);
    // S = Q K_it^T (A = Q from tensor memory); releases the K slot and signals the softmax warps
    auto issue_qk = [&](int it) {
      const int s = it % kKStages;
      const uint64_t k_desc = k_desc0 + (uint64_t)(s * (kTileBytes >> 4));
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint32_t koff = (kk >> 2) * kHalfTile + (kk & 3) * 32;
          mma_ts(tmem + Tm<D>::kColS + (kNS == 2 ? (it & 1) * 64 : 0), tmem + Tm<D>::kColQ + kk * 8,
                 k_desc + (koff >> 4), idesc_qk, kk > 0);
        }
        tc_commit(&ctl->kempty[s]);
        tc_commit(&ctl->sfull[kNS == 2 ? (it & 1) : 0]);
      }
      __syncwarp();
    };
    // O += P_it V_it (A = P from the score buffer); releases the V slot, counts the tile on odone
    auto issue_pv = [&](int it) {
      const int s = it % kVStages;
      const uint64_t v_desc = v_desc0 + (uint64_t)(s * (kTileBytes >> 4));
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < kTileKeys / 16; ++kk) {
          mma_ts(tmem + Tm<D>::kColO, tmem + Tm<D>::kColS + (kNS == 2 ? (it & 1) * 64 : 0) + kk * 8,
                 v_desc + (kk * 2048 >> 4), idesc_pv,
                 (it > 0 || kk > 0));
        }
        tc_commit(&ctl->vempty[s]);
        tc_commit(&ctl->odone);
        if (it + 1 == n_tiles) tc_commit(&ctl->pvdone);
      }
      __syncwarp();
    };
    // every lane waits (bounded); the outcome is made uniform
    auto wwait = [&](uint64_t* bar, uint32_t parity) {
      const bool ok = mbar_wait(bar, parity, ctl, p.status);
      return __all_sync(0xffffffffu, ok);
    };
    if (kNS == 2) {
      // Two score buffers: QK(0), QK(1) go out as their K tiles land; arrival t of the softmax
      // threads (P(t) stored in buffer t % 2) lets PV(t) and then QK(t+2), which overwrites that
      // buffer, go: the pipe runs one thread's MMAs in issue order.
      bool ok = wwait(&ctl->qready, 0);
      for (int it = 0; ok && it < min(2, n_tiles); ++it) {
        ok = wwait(&ctl->kfull[it % kKStages], (it / kKStages) & 1);
        if (!ok) break;
        trace(trl, 1, it, 0);
        tc_fence_after();
        issue_qk(it);
        trace(trl, 1, it, 5);
      }
      for (int t = 0; ok && t < n_tiles; ++t) {
        ok = wwait(&ctl->pready[t & 1], (t >> 1) & 1) && wwait(&ctl->vfull[t % kVStages], (t / kVStages) & 1);
        if (!ok) break;
        trace(trl, 1, t, 2);
        tc_fence_after();
        issue_pv(t);
        trace(trl, 1, t, 3);
        if (t + 2 < n_tiles) {
          const int it = t + 2;
          ok = wwait(&ctl->kfull[it % kKStages], (it / kKStages) & 1);
          if (!ok) break;
          trace(trl, 1, it, 0);
          tc_fence_after();
          issue_qk(it);
          trace(trl, 1, it, 5);
        }
      }
    } else {
      // Arrival k of the softmax threads (S(k) in their registers, P(k-1) in the buffer) lets
      // PV(k-1) and then QK(k+1) go: the tensor pipe runs one thread's MMAs in issue order, so
      // PV(k-1) has consumed P before the new scores overwrite it.
      bool ok = wwait(&ctl->qready, 0) && wwait(&ctl->kfull[0], 0);
      if (ok) {
        trace(trl, 1, 0, 0);
        tc_fence_after();
        issue_qk(0);
        trace(trl, 1, 0, 5);
      }
      for (int k = 0; ok && k <= n_tiles; ++k) {
        ok = wwait(&ctl->pready[k & 1], (k >> 1) & 1);
        if (!ok) break;
        if (k >= 1) {
          const int it = k - 1;
          ok = wwait(&ctl->vfull[it % kVStages], (it / kVStages) & 1);
          if (!ok) break;
          trace(trl, 1, it, 2);
          tc_fence_after();
          issue_pv(it);
          trace(trl, 1, it, 3);
        }
        if (k + 1 < n_tiles) {
          const int it = k + 1;
          ok = wwait(&ctl->kfull[it % kKStages], (it / kKStages) & 1);
          if (!ok) break;
          trace(trl, 1, it, 0);
          tc_fence_after();
          issue_qk(it);
          trace(trl, 1, it, 5);
        }
      }
    }
  } else {
    // ===== softmax warps: thread = TMEM lane =====
    const int L = tid;  // 0..127
    const int r = L % r_pad;
    const int grp = L / r_pad;
    const int nc = kTileKeys / groups;
    const int c0 = grp * nc;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    const uint32_t t_o = tmem + lane_off + Tm<D>::kColO;
    // the Q row -> tensor memory as the A operand of the score MMAs: column j of this lane
    // holds head dims 2j and 2j + 1 (the pair's memory order)
#pragma unroll
    for (int q = 0; q < kD / 32; ++q) {
      uint32_t wq[16];
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        wq[v * 4 + 0] = qreg[q * 4 + v].x;
        wq[v * 4 + 1] = qreg[q * 4 + v].y;
        wq[v * 4 + 2] = qreg[q * 4 + v].z;
        wq[v * 4 + 3] = qreg[q * 4 + v].w;
      }
      tmem_st16(tmem + lane_off + Tm<D>::kColQ + q * 16, wq);
    }
    tc_wait_st();
    tc_fence_before();
    mbar_arrive(&ctl->qready);
    float m = -INFINITY, l = 0.f;
    bool ok;
    TileMap<HIST> tmap;
    if constexpr (HIST) tmap = {hist_prefix, hist_valid, g0, 0};
    else tmap = {tok0, tok1};
#define SS_LOOP(NC_)                                                                                        \
  (Tm<D>::NS == 2 ? softmax_loop2<NC_, D>(p, ctl, tmem + lane_off, c0, n_tiles, tmap, v_s0, L, m, l, tr) \
                  : softmax_loop<NC_, D>(p, ctl, tmem + lane_off, c0, n_tiles, tmap, v_s0, L, m, l, tr))
    if (nc == 16)
      ok = SS_LOOP(16);
    else if (nc == 32)
      ok = SS_LOOP(32);
    else
      ok = SS_LOOP(64);
#undef SS_LOOP
    // all output MMAs have retired (a barrier of its own: by now odone may be one or two
    // phases past the last one this thread looked at, which a parity cannot tell apart)
    ok = ok && mbar_wait(&ctl->pvdone, 0, ctl, p.status);
    named_bar_sync(2, 128);
    if (ctl->abort == 0) {  // uniform over the 128 threads after the barrier
      tc_fence_after();
      // ---- merge the key groups of each row and write the partial state ----
      // Everything below lives over the idle K/V slots.  The 128 lanes' O rows are
      // staged as fp32 in the layout a TMA store with the 128-byte swizzle reads: four blocks
      // of [128 rows][32 floats], 16-byte chunk c of a row at chunk c ^ (row % 8) (so a warp's
      // 16-byte accesses, one row per lane, spread over all banks); the lanes' (m, l) sit
      // behind them.
      float* o_s = reinterpret_cast<float*>(smem);
      float2* ml_s = reinterpret_cast<float2*>(smem + 128 * kD * 4);
      auto o_at = [&](int row, int c4) {  // float4 number c4 (0..31) of a staged row
        return reinterpret_cast<float4*>(o_s + (c4 >> 3) * (128 * 32) + row * 32 +
                                         (((c4 & 7) ^ (row & 7)) << 2));
      };
      ml_s[L] = make_float2(m, l);
      named_bar_sync(1, 128);
      float M = -INFINITY;
      for (int g = 0; g < groups; ++g) M = fmaxf(M, ml_s[g * r_pad + r].x);
      const float f = (m == -INFINITY) ? 0.f : exp2f(m - M);
#pragma unroll 1
      for (int q = 0; q < kD / 32; ++q) {
        uint32_t o[2][16];
        tmem_ld16(t_o + q * 32, o[0]);
        tmem_ld16(t_o + q * 32 + 16, o[1]);
        tc_wait_ld();
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          float4 v;
          v.x = __uint_as_float(o[c4 >> 2][(c4 & 3) * 4 + 0]) * f;
          v.y = __uint_as_float(o[c4 >> 2][(c4 & 3) * 4 + 1]) * f;
          v.z = __uint_as_float(o[c4 >> 2][(c4 & 3) * 4 + 2]) * f;
          v.w = __uint_as_float(o[c4 >> 2][(c4 & 3) * 4 + 3]) * f;
          *o_at(L, q * 8 + c4) = v;
        }
      }
      if (L < nrows) {
        float lt = 0.f;
        for (int g = 0; g < groups; ++g) {
          const float2 st = ml_s[g * r_pad + r];
          if (st.x > -INFINITY) lt += exp2f(st.x - M) * st.y;
        }
        out_ml[L] = make_float2(lt > 0.f ? M : -INFINITY, lt);
      }
      if (groups > 1) {
        // lane (r, grp) sums columns [grp * 128/groups, (grp + 1) * 128/groups) of row r over
        // the row's `groups` staged copies and puts them back over the first copy
        named_bar_sync(1, 128);
        const int n4 = (kD / 4) / groups, c40 = grp * n4;
        for (int c = 0; c < n4; c += 4) {
          float4 acc[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) acc[k] = *o_at(r, c40 + c + k);
          for (int g = 1; g < groups; ++g) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float4 v = *o_at(g * r_pad + r, c40 + c + k);
              acc[k].x += v.x;
              acc[k].y += v.y;
              acc[k].z += v.z;
              acc[k].w += v.w;
            }
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) *o_at(r, c40 + c + k) = acc[k];
        }
      }
      // Four TMA stores move rows [row0, row0 + 128) of the slot.  Rows past `nrows` carry
      // padding lanes (or the other groups' copies): they land in rows >= R of this slot, which
      // nothing reads, or past the slot's last row, where the hardware clips the box.
      fence_proxy_async();  // generic-proxy writes -> visible to the TMA store
      named_bar_sync(1, 128);
      if (L == 0) {
#pragma unroll
        for (int j = 0; j < kD / 32; ++j)
          tma_store_3d(&tmA, smem_u32(o_s + j * (128 * 32)), j * 32, row0, p.a_slot0 + w.slot);
        bulk_commit();
        bulk_wait_read();  // shared memory is released when the CTA leaves
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
  }
  if (tid == 0) cta_log_write(p, t_cta0, n_tiles);
  // Completion order along the stream: one CTA of this grid waits for the previous grid, so
  // this grid cannot complete before it (the other CTAs leave at once and free their SM slot).
  if (!p.wait_first && chain_cta) pdl_wait_prior();
}

}  // namespace

namespace {
template <int D, bool HIST>
cudaError_t prepare_one() {
  return cudaFuncSetAttribute(chunk_tc_kernel<D, HIST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Lay<D>::kSmemTotal);
}
}  // namespace

cudaError_t chunk_tc_prepare() {
  cudaError_t e = prepare_one<128, false>();
  if (e == cudaSuccess) e = prepare_one<64, false>();
  if (e == cudaSuccess) e = prepare_one<128, true>();
  if (e == cudaSuccess) e = prepare_one<64, true>();
  return e;
}

cudaError_t launch_chunk_tc(const ChunkParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            const CUtensorMap& tmA, cudaStream_t s, bool pdl) {
  dim3 grid(p.splits * p.row_tiles, p.H_kv, p.n_active ? p.n_active : p.B), block(kThreads);
  static const HistParams none = {};
  if (p.d == 64)
    return launch_kernel(chunk_tc_kernel<64, false>, grid, block, Lay<64>::kSmemTotal, s, pdl, p, tmK, tmV, tmA, none);
  return launch_kernel(chunk_tc_kernel<128, false>, grid, block, Lay<128>::kSmemTotal, s, pdl, p, tmK, tmV, tmA, none);
}

cudaError_t launch_chunk_tc_hist(const ChunkParams& p, const HistParams& h, const CUtensorMap& tmA,
                                 cudaStream_t s, bool pdl) {
  if (h.n_chunks < 1 || h.n_chunks > kMaxHistChunks || !h.maps || p.n_active || p.page_table)
    return cudaErrorInvalidValue;
  dim3 grid(p.splits * p.row_tiles, p.H_kv, p.B), block(kThreads);
  // (the K/V map parameters are not used by this instantiation: any valid map will do)
  if (p.d == 64)
    return launch_kernel(chunk_tc_kernel<64, true>, grid, block, Lay<64>::kSmemTotal, s, pdl, p, tmA, tmA, tmA, h);
  return launch_kernel(chunk_tc_kernel<128, true>, grid, block, Lay<128>::kSmemTotal, s, pdl, p, tmA, tmA, tmA, h);
}

}  // namespace ss
