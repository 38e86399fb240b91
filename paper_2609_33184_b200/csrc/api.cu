// Host side of libspecstream: argument validation, round state machine, workspace layout,
// tensor-map cache and kernel launches.  Allocates no device memory.
#include <chrono>
#include <cstdlib>
#include <cstring>
#include <new>

#include "ss_internal.h"

struct ss_ctx {
  ss_config cfg;
  int G, R_max, R_stride;
  int slots_per_set;       // (split, b, kvh) slots of one partial set
  int slots_chunk_call;    // of which a single chunk call may use (its split policy's limit)
  int n_set_cap;           // chunk sets (the local set is one more)
  uint8_t* ws;
  size_t ws_bytes;
  uint32_t* status;        // device status word
  float2* part_ml;
  float* part_a;
  int64_t set_stride_ml, set_stride_a;
  bool tc_ok;              // device can run the tensor-core kernel
  // round state
  enum { IDLE, OPEN } state;
  ss_tensor Q;
  int B, T_q;
  float scale;
  int n_sets;
  uint8_t splits[ss::kMaxSets];
  uint64_t absent[ss::kMaxSets][ss::kMaxListed / 64];  // per chunk set: requests (bits) the call skipped
  bool has_local;
  bool first_launch;       // next kernel is the first of the round (or follows a fold)
  cudaStream_t stream;
  int32_t last_cuda;
  int64_t launches;
  const char* last_kernel;
  int force_splits;        // SS_SPLITS env override (0 = automatic)
  bool force_rows_kernel;  // SS_CHUNK_KERNEL=rows: rows-on-M tensor-core kernel even for few rows
  bool force_keys_kernel;  // SS_CHUNK_KERNEL=keys: keys-on-M tensor-core kernel for any row count
  int target_ctas;
  bool target_forced;      // SS_TARGET_CTAS is set: used as given for every call
  // tensor-map cache
  struct TmEntry {
    const void* ptr;
    int64_t sb, sh, st;
    int B, L_c, box_tokens;
    CUtensorMap map;
    uint64_t age;
  } tm[64];
  int tm_n;
  uint64_t tm_clock;
  CUtensorMap tm_a;         // all partial a[]: [sets * slots][R_stride][d] fp32, box [128 rows][32]
  // pipeline resources (created lazily by ss_stream_round)
  cudaStream_t copy_stream, attn_stream;
  cudaEvent_t ev_ready[2], ev_free[2], ev_t0, ev_t1;
  bool pipe_ready;
  bool no_overlap;          // set while ss_stream_round drives the context
  unsigned long long* trace;  // device trace region (in the workspace)
  unsigned int* round_counters;  // ticket counters of split small rounds (zero between rounds)
  bool round_clusters;           // split small rounds merge inside a thread-block cluster (until a launch refuses)
  bool trace_on;
  unsigned long long* cta_log;  // caller's per-CTA log buffer (ss_cta_log_set) or null
  int cta_log_cap;
  ss_stats stats;           // counters (launches is filled in when they are read)
  // tensor maps of a whole-history launch: kHistSlots lists in the workspace, their host mirrors
  CUtensorMap* hist_maps;   // device [kHistSlots][2 * kMaxHistChunks]
  CUtensorMap hist_host[4][2 * ss::kMaxHistChunks];
  int hist_n[4];            // maps in use per slot (0 = empty)
  uint64_t hist_age[4];
  bool hist_pinned[4];      // the list was used under a stream capture: a graph may replay the launch, never evicted
  cudaEvent_t* ev_pool;     // timing events of the streamed round (SS_FLAG_STREAM_TIMING)
  int ev_pool_n;
};

namespace ss {
void ctx_pipeline_release(ss_ctx* c);
}

namespace {

using ss::kMaxSets;
using ss::kMaxSplits;
using ss::kTileKeys;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool cfg_valid(const ss_config* c) {
  if (!c) return false;
  if (c->max_B <= 0 || c->H_q <= 0 || c->H_kv <= 0 || c->max_Tq <= 0 || c->max_Tloc < 0 ||
      c->max_Lc <= 0)
    return false;
  if (c->H_q % c->H_kv) return false;
  if (c->d != 64 && c->d != 128) return false;
  if (c->max_Tloc > 1024) return false;
  if (c->max_chunks < 0 || c->max_chunks > kMaxSets) return false;
  if ((int64_t)c->max_Tq * (c->H_q / c->H_kv) > 4096) return false;
  // query rows per round: the row-per-warp kernels index them with 32-bit arithmetic
  if ((int64_t)c->max_B * c->H_q * c->max_Tq >= (1ll << 31)) return false;
  return true;
}

// partial sets for chunk calls: at least two, so that a fold (all sets -> set 0) leaves one free
int set_cap(const ss_config* c) { return c->max_chunks ? (c->max_chunks < 2 ? 2 : c->max_chunks) : 64; }

int target_ctas_default() {
  const char* e = getenv("SS_TARGET_CTAS");
  int v = e ? atoi(e) : 0;
  return v > 0 ? v : ss::kNumSM;
}

// (split, b, kvh) slots one chunk call may use: about one CTA per SM at the largest batch
// (successive chunk kernels overlap, so a second CTA per SM comes from the next launch).
int slots_for(const ss_config* c) {
  const int pairs = c->max_B * c->H_kv;
  int s = target_ctas_default() / pairs;
  if (s < 1) s = 1;
  if (s > kMaxSplits) s = kMaxSplits;
  return pairs * s;
}
// Slots a partial set holds: room for two CTAs per SM (a launch over a list of chunks has all of
// its CTAs resident at once), at least what a chunk call may use.
int slot_capacity_for(const ss_config* c) {
  const int pairs = c->max_B * c->H_kv;
  int s = 2 * ss::kNumSM / pairs;
  if (s < 1) s = 1;
  if (s > kMaxSplits) s = kMaxSplits;
  const int cap = pairs * s, use = slots_for(c);
  return cap > use ? cap : use;
}

constexpr int kHistSlots = 4;
struct Layout {
  size_t off_hist, off_ml, off_a, total;
  int64_t set_stride_ml, set_stride_a;
  int R_stride;
};

Layout layout_for(const ss_config* c) {
  Layout L;
  const int G = c->H_q / c->H_kv;
  L.R_stride = c->max_Tq * G;
  const int64_t rows = (int64_t)slot_capacity_for(c) * L.R_stride;
  L.set_stride_ml = rows;                 // float2 elements
  L.set_stride_a = rows * c->d;           // float elements
  const int sets = set_cap(c) + 1;
  L.off_hist = 256 + align_up(ss::kTraceWords * sizeof(unsigned long long), 256) +
               ss::kRoundCounters * sizeof(unsigned int);   // status, trace region, round counters
  L.off_ml = L.off_hist + kHistSlots * 2 * ss::kMaxHistChunks * sizeof(CUtensorMap);  // lists of tensor maps
  L.off_a = align_up(L.off_ml + (size_t)sets * rows * sizeof(float2), 256);
  L.total = align_up(L.off_a + (size_t)sets * rows * c->d * sizeof(float), 256);
  return L;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }
bool tensor_ok(const ss_tensor& t) {
  return aligned16(t.ptr) && (t.stride_b % 8 == 0) && (t.stride_h % 8 == 0) && (t.stride_t % 8 == 0);
}

ss_status cuda_fail(ss_ctx* c, cudaError_t e) {
  c->last_cuda = (int32_t)e;
  return SS_ERR_CUDA;
}

// Tensor map over K or V [B, H_kv, L_c, d] with a [box_tokens][64 d] box and 128-byte swizzle.
bool get_tensor_map(ss_ctx* c, const ss_tensor& t, int B, int L_c, int box_tokens, CUtensorMap* out) {
  for (int i = 0; i < c->tm_n; ++i) {
    ss_ctx::TmEntry& e = c->tm[i];
    if (e.ptr == t.ptr && e.sb == t.stride_b && e.sh == t.stride_h && e.st == t.stride_t &&
        e.B == B && e.L_c == L_c && e.box_tokens == box_tokens) {
      e.age = ++c->tm_clock;
      *out = e.map;
      return true;
    }
  }
  if (!g_encode) return false;
  const int H_kv = c->cfg.H_kv, d = c->cfg.d;
  cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)L_c, (cuuint64_t)H_kv, (cuuint64_t)B};
  // unused outer strides still have to be positive multiples of 16 bytes
  const int64_t st = t.stride_t, sh = (H_kv > 1 || t.stride_h > 0) ? t.stride_h : (int64_t)L_c * st;
  const int64_t sb = (B > 1 || t.stride_b > 0) ? t.stride_b : (int64_t)H_kv * sh;
  if (st <= 0 || sh <= 0 || sb <= 0) return false;
  cuuint64_t strides[3] = {(cuuint64_t)st * 2, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)box_tokens, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUtensorMap m;
  CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(t.ptr), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  int slot = c->tm_n;
  if (c->tm_n < 64) {
    ++c->tm_n;
  } else {
    slot = 0;
    for (int i = 1; i < 64; ++i)
      if (c->tm[i].age < c->tm[slot].age) slot = i;
  }
  c->tm[slot] = {t.ptr, t.stride_b, t.stride_h, t.stride_t, B, L_c, box_tokens, m, ++c->tm_clock};
  *out = m;
  return true;
}

// Tensor map over every partial a[] of the workspace, [sets * slots][R_stride][d] fp32, for the
// rows-on-M kernel's write-out: boxes of 128 rows x 32 floats, 128-byte swizzle.  A box that
// reaches past row R_stride of its slot is clipped there by the hardware.
bool encode_partials_map(ss_ctx* c) {
  if (!g_encode) return false;
  const uint64_t d = (uint64_t)c->cfg.d, rows = (uint64_t)c->R_stride;
  const uint64_t slots = (uint64_t)(c->n_set_cap + 1) * c->slots_per_set;
  cuuint64_t dims[3] = {d, rows, slots};
  cuuint64_t strides[2] = {d * 4, rows * d * 4};
  cuuint32_t box[3] = {32, (cuuint32_t)(rows < 128 ? rows : 128), 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return g_encode(&c->tm_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, c->part_a, dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool use_pdl(ss_ctx* c) {
  return (c->cfg.flags & SS_FLAG_OVERLAP_CHUNKS) && !c->first_launch && !c->no_overlap;
}
// Chunk kernels (and the one-launch small round) can also be the FIRST kernel of a round under
// programmatic stream serialization: with wait_first they do nothing before the kernel in front of
// them (the previous round's finalize, a fold, anything else) has completed, so only their launch
// and set-up overlap it.
bool use_pdl_first(ss_ctx* c) { return (c->cfg.flags & SS_FLAG_OVERLAP_CHUNKS) && !c->no_overlap; }

void fill_merge(ss_ctx* c, ss::MergeParams* m) {
  memset(m, 0, sizeof(*m));
  m->part_ml = c->part_ml;
  m->part_a = c->part_a;
  m->set_stride_ml = c->set_stride_ml;
  m->set_stride_a = c->set_stride_a;
  m->n_sets = c->n_sets;
  m->has_local = c->has_local ? 1 : 0;
  m->local_set = c->n_set_cap;
  m->B = c->B;
  m->H_q = c->cfg.H_q;
  m->H_kv = c->cfg.H_kv;
  m->G = c->G;
  m->T_q = c->T_q;
  m->d = c->cfg.d;
  m->R_stride = c->R_stride;
  memcpy(m->splits, c->splits, sizeof(m->splits));
  memcpy(m->absent, c->absent, sizeof(m->absent));
}

// All partial sets in use: fold them into set 0 (Eq. 14 is associative).
cudaError_t fold_sets(ss_ctx* c, cudaStream_t s) {
  ss::MergeParams m;
  fill_merge(c, &m);
  m.has_local = 0;
  m.fold_ml = c->part_ml;
  m.fold_a = c->part_a;
  cudaError_t e = ss::launch_fold(m, s);
  if (e != cudaSuccess) return e;
  ++c->launches;
  c->n_sets = 1;
  c->splits[0] = 1;
  memset(c->absent[0], 0, sizeof(c->absent[0]));  // the folded set holds every request
  c->first_launch = true;  // the next kernel must not overlap the fold
  return cudaSuccess;
}


// What the host copy of the valid lengths says about a chunk call.
struct HintScan {
  int active;         // requests with tokens in this chunk (>= 1; all B without a host copy)
  int longest;        // tokens of the longest of them (>= 1; L_c without a host copy)
  int n_listed;       // > 0: the launch covers only the requests in listed[] (batches of <= 256)
  uint8_t listed[ss::kMaxListed];
  uint64_t absent[ss::kMaxListed / 64];  // bit b: request b is not in listed[]
};

// Requests without tokens in this chunk (by the host copy) get no CTAs at all when the batch
// has at most 256 requests: the launch covers the listed requests only and the merge skips this
// call's set for the others.
HintScan scan_hint(const ss_ctx* c, const int32_t* valid_len_host, int L_c) {
  HintScan h;
  h.active = c->B;
  h.longest = L_c;
  h.n_listed = 0;
  memset(h.absent, 0, sizeof(h.absent));
  if (!valid_len_host) return h;
  const bool can_list = c->B <= ss::kMaxListed;
  int active = 0, longest = 0;
  for (int b = 0; b < c->B; ++b) {
    int v = valid_len_host[b];
    v = v < 0 ? 0 : (v > L_c ? L_c : v);
    if (v > 0) {
      ++active;
      if (can_list) h.listed[h.n_listed++] = (uint8_t)b;
    } else if (can_list) {
      h.absent[b >> 6] |= 1ull << (b & 63);
    }
    if (v > longest) longest = v;
  }
  if (can_list && h.n_listed == 0) {  // nobody has tokens: one request keeps the launch well-formed
    h.listed[h.n_listed++] = 0;
    h.absent[0] &= ~1ull;
  }
  if (h.n_listed == c->B) h.n_listed = 0;  // everybody is in: plain launch
  h.active = active > 0 ? active : 1;
  h.longest = longest > 0 ? longest : 1;
  return h;
}

// Token splits of a chunk call: `ctas1` CTAs have work with one split, `used_tiles` 64-token
// tiles reach the longest request's last token.
int pick_splits(ss_ctx* c, bool tensor_core, bool whole_waves, int pairs, int ctas1, int used_tiles) {
  // tensor-core CTAs amortise their set-up over at least 256 tokens; CUDA-core CTAs take one tile
  const int min_tiles = tensor_core ? 4 : 1;
  int max_splits = c->slots_chunk_call / pairs;
  if (max_splits > kMaxSplits) max_splits = kMaxSplits;
  if (max_splits > (used_tiles + min_tiles - 1) / min_tiles) max_splits = (used_tiles + min_tiles - 1) / min_tiles;
  if (max_splits < 1) max_splits = 1;
  int splits;
  if (c->force_splits > 0) {
    splits = c->force_splits;
  } else if (whole_waves) {
    // one CTA per SM and no co-residency with the next launch: pick the split count whose CTA
    // count fills whole waves of SMs best (smallest such count: fewer partial states)
    double best = 0.0;
    splits = 1;
    for (int sp = 1; sp <= max_splits; ++sp) {
      const int ctas = ctas1 * sp;
      const int waves = (ctas + ss::kNumSM - 1) / ss::kNumSM;
      const double eff = (double)ctas / ((double)waves * ss::kNumSM);
      if (eff > best + 0.05) {
        best = eff;
        splits = sp;
      }
    }
  } else {
    // About one CTA per SM for the first chunk call of a round.  A later call whose kernel
    // overlaps the one before it (programmatic dependent launch) finds the SMs partly taken and
    // more launches on their way: half as many CTAs, each with twice the tiles, leave less
    // set-up and fewer partial states per byte (measured on the ragged 7B-shaped workload,
    // 64 kv-head groups per call: 6.39 -> 6.68 TB/s; unchanged where a call has 128 groups or
    // more).  The choice depends on the position in the round only, so results stay
    // reproducible bit for bit.
    int target = c->target_ctas;
    if (!c->target_forced && use_pdl(c)) target = target / 2 > 0 ? target / 2 : 1;
    splits = target / ctas1;
  }
  if (splits > max_splits) splits = max_splits;
  if (splits < 1) splits = 1;
  return splits;
}

}  // namespace

extern "C" {

size_t ss_workspace_bytes(const ss_config* cfg) {
  if (!cfg_valid(cfg)) return 0;
  return layout_for(cfg).total;
}

ss_status ss_create(ss_ctx** out, const ss_config* cfg, void* workspace, size_t workspace_bytes) {
  if (!out || !cfg || !workspace) return SS_ERR_ARG;
  if (!cfg_valid(cfg)) return SS_ERR_SHAPE;
  if ((uintptr_t)workspace & 255) return SS_ERR_ALIGN;
  const Layout L = layout_for(cfg);
  if (workspace_bytes < L.total) return SS_ERR_CAPACITY;
  cudaDeviceProp prop;
  cudaError_t e = cudaGetDeviceProperties(&prop, cfg->device);
  if (e != cudaSuccess) return SS_ERR_CUDA;
  if (prop.major != 10) return SS_ERR_UNSUPPORTED;
  e = cudaSetDevice(cfg->device);
  if (e != cudaSuccess) return SS_ERR_CUDA;

  ss_ctx* c = new (std::nothrow) ss_ctx();
  if (!c) return SS_ERR_ARG;
  memset(c, 0, sizeof(*c));
  c->cfg = *cfg;
  c->G = cfg->H_q / cfg->H_kv;
  c->R_max = cfg->max_Tq * c->G;
  c->R_stride = L.R_stride;
  c->slots_per_set = slot_capacity_for(cfg);
  c->slots_chunk_call = slots_for(cfg);
  c->n_set_cap = set_cap(cfg);
  c->ws = (uint8_t*)workspace;
  c->ws_bytes = workspace_bytes;
  c->status = (uint32_t*)c->ws;
  c->trace = (unsigned long long*)(c->ws + 256);
  c->round_counters = (unsigned int*)(c->ws + 256 + align_up(ss::kTraceWords * sizeof(unsigned long long), 256));
  c->hist_maps = (CUtensorMap*)(c->ws + L.off_hist);
  c->part_ml = (float2*)(c->ws + L.off_ml);
  c->part_a = (float*)(c->ws + L.off_a);
  c->set_stride_ml = L.set_stride_ml;
  c->set_stride_a = L.set_stride_a;
  c->state = ss_ctx::IDLE;
  c->last_kernel = "none";
  c->target_ctas = target_ctas_default();
  c->target_forced = getenv("SS_TARGET_CTAS") != nullptr && atoi(getenv("SS_TARGET_CTAS")) > 0;
  const char* fs = getenv("SS_SPLITS");
  c->force_splits = fs ? atoi(fs) : 0;
  const char* rc = getenv("SS_ROUND_CLUSTER");
  c->round_clusters = !(rc && strcmp(rc, "never") == 0);
  const char* ck = getenv("SS_CHUNK_KERNEL");
  c->force_rows_kernel = (ck && strcmp(ck, "rows") == 0) || (cfg->flags & SS_FLAG_ROWS_ON_M);
  c->force_keys_kernel = (ck && strcmp(ck, "keys") == 0) || (cfg->flags & SS_FLAG_KEYS_ON_M);

  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) ==
            cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      g_encode = (EncodeTiledFn)fn;
  }
  if (ss::chunk_simt_prepare() != cudaSuccess) {
    delete c;
    return SS_ERR_CUDA;
  }
  c->tc_ok = (g_encode != nullptr) && !(cfg->flags & SS_FLAG_FORCE_SIMT);
  if (c->tc_ok) c->tc_ok = encode_partials_map(c);
  if (c->tc_ok) {
    e = ss::chunk_tc_prepare();
    if (e == cudaSuccess) e = ss::chunk_tc_keys_prepare();
    if (e != cudaSuccess) {
      delete c;
      return SS_ERR_CUDA;
    }
  }
  e = cudaMemset(c->status, 0, 256);
  if (e == cudaSuccess) e = cudaMemset(c->round_counters, 0, ss::kRoundCounters * sizeof(unsigned int));
  if (e != cudaSuccess) {
    delete c;
    return SS_ERR_CUDA;
  }
  *out = c;
  return SS_OK;
}

ss_status ss_destroy(ss_ctx* c) {
  if (!c) return SS_ERR_ARG;
  ss::ctx_pipeline_release(c);
  delete c;
  return SS_OK;
}

ss_status ss_verify_begin(ss_ctx* c, ss_tensor Q, int32_t B, int32_t T_q, float scale,
                          void* stream) {
  if (!c || !Q.ptr) return SS_ERR_ARG;
  if (B <= 0 || T_q <= 0) return SS_ERR_ARG;
  if (!(scale > 0.f) || !(scale < 3.0e38f)) return SS_ERR_ARG;  // positive and finite
  if (B > c->cfg.max_B || T_q > c->cfg.max_Tq) return SS_ERR_SHAPE;
  if (!tensor_ok(Q)) return SS_ERR_ALIGN;
  if (c->state != ss_ctx::IDLE) return SS_ERR_STATE;
  // The identity state (m, l, a) = (-inf, 0, 0) of every row is represented by an empty
  // list of partial sets: finalize starts its merge from the identity.
  c->Q = Q;
  c->B = B;
  c->T_q = T_q;
  c->scale = scale;
  c->n_sets = 0;
  c->has_local = false;
  c->first_launch = true;
  c->stream = (cudaStream_t)stream;
  c->state = ss_ctx::OPEN;
  return SS_OK;
}

struct PagedArgs {
  int32_t n_pages, page_size, pages_per_req;
  const int32_t* page_table;
};
static ss_status chunk_impl(ss_ctx* c, ss_tensor K, ss_tensor V, int32_t L_c, const int32_t* valid_len,
                            const int32_t* valid_len_host, void* stream, const PagedArgs* pg = nullptr);

ss_status ss_verify_chunk(ss_ctx* c, ss_tensor K, ss_tensor V, int32_t L_c,
                          const int32_t* valid_len, void* stream) {
  return chunk_impl(c, K, V, L_c, valid_len, nullptr, stream);
}

ss_status ss_verify_chunk_hinted(ss_ctx* c, ss_tensor K, ss_tensor V, int32_t L_c,
                                 const int32_t* valid_len, const int32_t* valid_len_host,
                                 void* stream) {
  return chunk_impl(c, K, V, L_c, valid_len, valid_len_host, stream);
}

ss_status ss_verify_chunk_paged(ss_ctx* c, ss_tensor K_pool, ss_tensor V_pool, int32_t n_pages,
                                int32_t page_size, const int32_t* page_table, int32_t pages_per_req,
                                const int32_t* valid_len, const int32_t* valid_len_host, void* stream) {
  if (!page_table || n_pages <= 0 || page_size <= 0 || pages_per_req <= 0) return SS_ERR_ARG;
  if ((uintptr_t)page_table & 3) return SS_ERR_ALIGN;
  if ((int64_t)page_size * pages_per_req > 0x7fffffff) return SS_ERR_SHAPE;
  const PagedArgs pg = {n_pages, page_size, pages_per_req, page_table};
  return chunk_impl(c, K_pool, V_pool, page_size * pages_per_req, valid_len, valid_len_host, stream, &pg);
}

static ss_status chunk_impl(ss_ctx* c, ss_tensor K, ss_tensor V, int32_t L_c, const int32_t* valid_len,
                            const int32_t* valid_len_host, void* stream, const PagedArgs* pg) {
  if (!c || !K.ptr || !V.ptr) return SS_ERR_ARG;
  if (L_c <= 0) return SS_ERR_ARG;
  if (L_c > c->cfg.max_Lc) return SS_ERR_SHAPE;
  if (!tensor_ok(K) || !tensor_ok(V)) return SS_ERR_ALIGN;
  if (valid_len && ((uintptr_t)valid_len & 3)) return SS_ERR_ALIGN;
  if (c->state != ss_ctx::OPEN || (cudaStream_t)stream != c->stream) return SS_ERR_STATE;
  cudaStream_t s = c->stream;

  if (c->n_sets == c->n_set_cap) {
    cudaError_t e = fold_sets(c, s);
    if (e != cudaSuccess) return cuda_fail(c, e);
  }

  const int R = c->T_q * c->G;
  const int pairs = c->B * c->cfg.H_kv;
  const int n_tiles = (L_c + kTileKeys - 1) / kTileKeys;
  // host copy of the valid lengths (a hint): which requests have tokens here, how far they reach
  const HintScan hint = scan_hint(c, valid_len ? valid_len_host : nullptr, L_c);
  const int active_pairs = hint.active * c->cfg.H_kv;
  const int used_tiles = (hint.longest + kTileKeys - 1) / kTileKeys;
  CUtensorMap tmK, tmV;
  bool tc = c->tc_ok;
  // paged chunks: a tile is one page, a whole number of pages (8, 16, 32 or 64 tokens each,
  // gathered page by page: a page of 8 tokens is one 1024-byte swizzle atom, the smallest box
  // that keeps the tile's layout) or part of a page; anything else takes the CUDA-core kernel
  const auto pages_fit = [&](int tile) {
    const int ps = pg->page_size;
    return ps % tile == 0 || (ps >= 8 && tile % ps == 0);
  };
  // up to 32 rows per kv-head the keys ride the MMA's M axis (tiles of 128 tokens); with more
  // rows the kernel with the rows on M is faster (measured).  SS_FLAG_ROWS_ON_M /
  // SS_FLAG_KEYS_ON_M (or SS_CHUNK_KERNEL=rows|keys) force one of them.
  // Head dim 64, tiny call (a few tiles in all): the CUDA-core kernel's small CTAs finish sooner
  // than one tensor-core CTA gets going (measured on the 1,024-token chain workload: 43 vs 46 us
  // per round).  SS_FLAG_KEYS_ON_M / SS_FLAG_ROWS_ON_M override.
  if (c->cfg.d == 64 && !c->force_keys_kernel && !c->force_rows_kernel && (int64_t)pairs * n_tiles <= 8)
    tc = false;
  // (At head dim 64 a tile has half the bytes for the same softmax work and the rows-on-M kernel
  // already wins above 16 rows: 4.8 vs 4.5 TB/s at 32 rows, 4.9 vs 5.1 at 16.)
  const int keys_max_rows = c->cfg.d == 64 ? 16 : 32;
  const bool keys_on_m = tc && !c->force_rows_kernel && (R <= keys_max_rows || c->force_keys_kernel) &&
                         (!pg || pages_fit(128));
  if (pg && !keys_on_m && !pages_fit(kTileKeys)) tc = false;
  int box = keys_on_m ? 128 : kTileKeys;
  if (pg && pg->page_size < box) box = pg->page_size;
  // tensor map over [outer, H_kv, tokens, d]: (requests, chunk tokens) or (pages, page tokens)
  const int tm_outer = pg ? pg->n_pages : c->B, tm_tokens = pg ? pg->page_size : L_c;
  if (tc)
    tc = get_tensor_map(c, K, tm_outer, tm_tokens, box, &tmK) &&
         get_tensor_map(c, V, tm_outer, tm_tokens, box, &tmV);

  ss::ChunkParams p;
  memset(&p, 0, sizeof(p));
  if (tc && keys_on_m) {
    p.row_tiles = (R + 127) / 128;
    p.rows_per_tile = R < 128 ? R : 128;
  } else if (tc) {
    // row tiles of 128 rows and a remainder tile; a tile with <= 64 (<= 32) rows replicates its
    // rows 2x (4x) along M, so no lane computes padding
    p.row_tiles = (R + 127) / 128;
    p.rows_per_tile = R < 128 ? R : 128;
  } else {
    // a call of a few CTAs in all is latency bound: tiles of 8 rows spread a kv-head's rows over
    // more SMs (K/V are re-read through L2, which such a call fits into)
    p.rows_per_tile = ((int64_t)pairs * ((R + 7) / 8) * n_tiles <= 2 * ss::kNumSM) ? 8 : ss::simt_rows_per_tile(R);
    p.row_tiles = (R + p.rows_per_tile - 1) / p.rows_per_tile;
  }
  const int ctas1 = active_pairs * p.row_tiles;  // CTAs with work when splits = 1
  int splits = pick_splits(c, tc, tc && keys_on_m && R > 32, pairs, ctas1, used_tiles);
  p.tiles_per_split = (used_tiles + splits - 1) / splits;
  if (tc && keys_on_m) p.tiles_per_split += p.tiles_per_split & 1;  // whole 128-token tiles
  splits = (used_tiles + p.tiles_per_split - 1) / p.tiles_per_split;
  p.splits = splits;

  p.Q = (const __nv_bfloat16*)c->Q.ptr;
  p.q_sb = c->Q.stride_b;
  p.q_sh = c->Q.stride_h;
  p.q_st = c->Q.stride_t;
  p.K = (const __nv_bfloat16*)K.ptr;
  p.V = (const __nv_bfloat16*)V.ptr;
  p.k_sb = K.stride_b;
  p.k_sh = K.stride_h;
  p.k_st = K.stride_t;
  p.v_sb = V.stride_b;
  p.v_sh = V.stride_h;
  p.v_st = V.stride_t;
  p.valid_len = valid_len;
  p.B = c->B;
  p.H_kv = c->cfg.H_kv;
  p.G = c->G;
  p.T_q = c->T_q;
  p.R = R;
  p.d = c->cfg.d;
  p.L_c = L_c;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.part_ml = c->part_ml + (int64_t)c->n_sets * c->set_stride_ml;
  p.part_a = c->part_a + (int64_t)c->n_sets * c->set_stride_a;
  p.R_stride = c->R_stride;
  p.n_active = hint.n_listed;
  if (hint.n_listed) memcpy(p.active_b, hint.listed, (size_t)hint.n_listed);
  p.a_slot0 = c->n_sets * c->slots_per_set;
  p.status = c->status;
  p.wait_first = c->first_launch ? 1 : 0;
  p.trace = c->trace_on ? c->trace : nullptr;
  p.cta_log = c->cta_log;
  p.cta_log_cap = c->cta_log_cap;
  p.launch_seq = (unsigned int)c->launches;
  if (pg) {
    p.page_table = pg->page_table;
    p.pages_per_req = pg->pages_per_req;
    p.page_size = pg->page_size;
    p.n_pages = pg->n_pages;
  }

  const bool pdl = use_pdl_first(c);
  cudaError_t e = !tc ? ss::launch_chunk_simt(p, s, pdl)
                  : keys_on_m ? ss::launch_chunk_tc_keys(p, tmK, tmV, s, pdl)
                              : ss::launch_chunk_tc(p, tmK, tmV, c->tm_a, s, pdl);
  if (e != cudaSuccess) return cuda_fail(c, e);
  c->last_kernel = !tc ? "simt" : keys_on_m ? "tcgen05-keys" : "tcgen05";
  ++c->launches;
  ++c->stats.chunk_calls;
  {
    int64_t tokens = (int64_t)c->B * L_c;  // no lengths, or lengths only the device knows
    if (valid_len && valid_len_host) {
      tokens = 0;
      for (int b = 0; b < c->B; ++b) {
        const int v = valid_len_host[b];
        tokens += v < 0 ? 0 : (v > L_c ? L_c : v);
      }
    }
    c->stats.kv_bytes += tokens * c->cfg.H_kv * c->cfg.d * 4;  // K and V, 2 bytes each
  }
  c->splits[c->n_sets] = (uint8_t)splits;
  if (hint.n_listed) memcpy(c->absent[c->n_sets], hint.absent, sizeof(hint.absent));
  else memset(c->absent[c->n_sets], 0, sizeof(hint.absent));
  ++c->n_sets;
  c->first_launch = false;
  return SS_OK;
}

ss_status ss_verify_local(ss_ctx* c, ss_tensor K_loc, ss_tensor V_loc, int32_t T_loc,
                          ss_mask_kind kind, const uint64_t* mask_bits, void* stream) {
  if (!c || !K_loc.ptr || !V_loc.ptr) return SS_ERR_ARG;
  if (T_loc <= 0) return SS_ERR_ARG;
  if (T_loc > c->cfg.max_Tloc) return SS_ERR_SHAPE;
  if (kind != SS_MASK_CHAIN && kind != SS_MASK_TREE_BITS) return SS_ERR_ARG;
  if (kind == SS_MASK_TREE_BITS && !mask_bits) return SS_ERR_ARG;
  if (!tensor_ok(K_loc) || !tensor_ok(V_loc)) return SS_ERR_ALIGN;
  if (mask_bits && ((uintptr_t)mask_bits & 7)) return SS_ERR_ALIGN;
  if (c->state != ss_ctx::OPEN || (cudaStream_t)stream != c->stream || c->has_local)
    return SS_ERR_STATE;
  // chain rule j <= i + (T_loc - T_q): with fewer local tokens than queries the leading rows
  // would see nothing of the local segment, which no caller means
  if (kind == SS_MASK_CHAIN && T_loc < c->T_q) return SS_ERR_ARG;
  ss::LocalParams p;
  memset(&p, 0, sizeof(p));
  p.Q = (const __nv_bfloat16*)c->Q.ptr;
  p.q_sb = c->Q.stride_b;
  p.q_sh = c->Q.stride_h;
  p.q_st = c->Q.stride_t;
  p.K = (const __nv_bfloat16*)K_loc.ptr;
  p.V = (const __nv_bfloat16*)V_loc.ptr;
  p.k_sb = K_loc.stride_b;
  p.k_sh = K_loc.stride_h;
  p.k_st = K_loc.stride_t;
  p.v_sb = V_loc.stride_b;
  p.v_sh = V_loc.stride_h;
  p.v_st = V_loc.stride_t;
  p.mask_bits = (kind == SS_MASK_TREE_BITS) ? mask_bits : nullptr;
  p.B = c->B;
  p.H_q = c->cfg.H_q;
  p.H_kv = c->cfg.H_kv;
  p.G = c->G;
  p.T_q = c->T_q;
  p.T_loc = T_loc;
  p.d = c->cfg.d;
  p.mask_words = (T_loc + 63) / 64;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.part_ml = c->part_ml + (int64_t)c->n_set_cap * c->set_stride_ml;
  p.part_a = c->part_a + (int64_t)c->n_set_cap * c->set_stride_a;
  p.R_stride = c->R_stride;
  cudaError_t e = ss::launch_local(p, c->stream, use_pdl(c));
  if (e != cudaSuccess) return cuda_fail(c, e);
  ++c->launches;
  c->has_local = true;
  c->first_launch = false;
  return SS_OK;
}

ss_status ss_verify_export_state(ss_ctx* c, float* ml, float* a, void* stream) {
  if (!c || !ml || !a) return SS_ERR_ARG;
  if (((uintptr_t)ml & 7) || !aligned16(a)) return SS_ERR_ALIGN;
  if (c->state != ss_ctx::OPEN || (cudaStream_t)stream != c->stream) return SS_ERR_STATE;
  ss::MergeParams m;
  fill_merge(c, &m);
  m.fold_ml = (float2*)ml;
  m.fold_a = a;
  cudaError_t e = ss::launch_export(m, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e);
  ++c->launches;
  c->first_launch = true;  // reads every partial: the next kernel must not overlap it
  return SS_OK;
}

ss_status ss_verify_import_state(ss_ctx* c, const float* ml, const float* a, void* stream) {
  if (!c || !ml || !a) return SS_ERR_ARG;
  if (((uintptr_t)ml & 7) || !aligned16(a)) return SS_ERR_ALIGN;
  if (c->state != ss_ctx::OPEN || (cudaStream_t)stream != c->stream) return SS_ERR_STATE;
  if (c->n_sets == c->n_set_cap) {
    cudaError_t e = fold_sets(c, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
  }
  ss::MergeParams m;
  fill_merge(c, &m);
  m.part_ml = (const float2*)ml;
  m.part_a = a;
  m.fold_ml = c->part_ml + (int64_t)c->n_sets * c->set_stride_ml;
  m.fold_a = c->part_a + (int64_t)c->n_sets * c->set_stride_a;
  cudaError_t e = ss::launch_import(m, c->stream);
  if (e != cudaSuccess) return cuda_fail(c, e);
  ++c->launches;
  c->splits[c->n_sets] = 1;
  memset(c->absent[c->n_sets], 0, sizeof(c->absent[0]));
  ++c->n_sets;
  c->first_launch = true;
  return SS_OK;
}

ss_status ss_verify_finalize(ss_ctx* c, void* O, float* LSE, void* stream) {
  if (!c || !O) return SS_ERR_ARG;
  if (!aligned16(O) || (LSE && ((uintptr_t)LSE & 3))) return SS_ERR_ALIGN;
  if (c->state != ss_ctx::OPEN || (cudaStream_t)stream != c->stream) return SS_ERR_STATE;
  ss::MergeParams m;
  fill_merge(c, &m);
  m.O = (__nv_bfloat16*)O;
  m.LSE = LSE;
  cudaError_t e = ss::launch_finalize(m, c->stream, use_pdl(c));
  if (e != cudaSuccess) return cuda_fail(c, e);
  ++c->launches;
  ++c->stats.rounds;
  c->stats.rows += (int64_t)c->B * c->cfg.H_q * c->T_q;
  c->state = ss_ctx::IDLE;
  c->Q.ptr = nullptr;
  return SS_OK;
}

// The whole history of a round in ONE launch of the rows-on-M kernel (Section 4.2: the chunks of a
// request are reduced into one running state; Eq. 13-14).  Taken when that kernel would run every
// chunk anyway and one CTA per (request, kv-head, row tile, split) fills the GPU at most once:
// the CTAs are equally long, keep their accumulator across chunk boundaries and leave `splits`
// partial states per row instead of one per chunk.  Returns SS_OK with *taken = false when the
// round does not qualify (nothing has been enqueued then).
static ss_status hist_chunks(ss_ctx* c, const ss_chunk_desc* chunks, int n_chunks, bool* taken) {
  *taken = false;
  if (!c->tc_ok || n_chunks < 2 || n_chunks > ss::kMaxHistChunks) return SS_OK;
  // SS_HISTORY_LAUNCH=never / always overrides the routing below (not the limits of the launch)
  const char* hl = getenv("SS_HISTORY_LAUNCH");
  if (hl && strcmp(hl, "never") == 0) return SS_OK;
  const bool always = hl && strcmp(hl, "always") == 0;
  const int R = c->T_q * c->G, pairs = c->B * c->cfg.H_kv;
  const int keys_max_rows = c->cfg.d == 64 ? 16 : 32;
  const bool keys_on_m = !c->force_rows_kernel && (R <= keys_max_rows || c->force_keys_kernel);
  // What the host knows about the requests' history lengths: every chunk without lengths or with a
  // host copy of them -> the totals; otherwise unknown.
  const int row_tiles = (R + 127) / 128;
  bool known = c->B <= ss::kMaxListed;
  int64_t len[ss::kMaxListed], lo = INT64_MAX, hi = 0;
  for (int b = 0; b < c->B && known; ++b) {
    len[b] = 0;
    for (int j = 0; j < n_chunks && known; ++j) {
      const ss_chunk_desc& d = chunks[j];
      if (!d.valid_len) len[b] += d.L_c;
      else if (d.valid_len_host) len[b] += d.valid_len_host[b] < 0 ? 0 : (d.valid_len_host[b] > d.L_c ? d.L_c : d.valid_len_host[b]);
      else known = false;
    }
    lo = len[b] < lo ? len[b] : lo;
    hi = len[b] > hi ? len[b] : hi;
  }
  const bool uniform = known && hi <= lo + lo / 10;
  // The keys-on-M kernel (up to 32 rows per kv-head) runs at the HBM ceiling, and a CTA that walks
  // a request's whole history instead of one chunk call's 2,048 tokens pays set-up, ring fill and
  // drain once instead of sixteen times (measured on the Qwen3-8B-shaped workload: +9 %).  The CTAs
  // of the launch should end together, so the host has to know that the histories are about equally
  // long.  A batch it knows to be ragged gets equally long CTAs another way (below): the tiles of a
  // kv-head's requests are laid end to end and cut into one share per CTA, whatever request a share
  // starts or ends in (streamed workload's batch, 8,192 to 65,536 tokens, resident: 6.39 -> 6.93 TB/s;
  // per-request pieces of equal length in two or three waves of CTAs had measured 6.0-6.4).
  // The rows-on-M kernel: with more than 128 rows per kv-head at head dim 128 the tile's arithmetic
  // bounds it and the one launch pays off whatever the host knows (+5 % at 192 rows, +22 % at 256,
  // +8-13 % on the 320-row tree workload), unless it knows the batch to be ragged; with up to 128
  // rows it is taken for histories known to be equally long (B = 16, 16,384 tokens each, head dim
  // 128: +3 / +4 / +7 / +12 % at 48 / 64 / 96 / 128 rows; head dim 64: +12-15 % at 24-64 rows, +7-10 %
  // at 96-128; -2 % / +1 % at 192 / 320 rows, where it is not taken).
  // Ragged batches on the keys-on-M kernel whose lengths the host knows (no request empty): the CTAs
  // of a kv-head walk equal shares of all its requests' tiles laid end to end (HistParams::n_req).
  // SS_HISTORY_WALK=never leaves such batches to the separate calls.
  const char* wk = getenv("SS_HISTORY_WALK");
  // (The rows-on-M kernel was given the same mode per (kv-head, row tile) and lost to the separate
  // calls on ragged batches at every row count but one: not kept.)
  const bool walk = keys_on_m && R <= 32 && known && lo > 0 && (!uniform || (wk && strcmp(wk, "always") == 0)) &&
                    !(wk && strcmp(wk, "never") == 0);
  if (keys_on_m) {
    if (R > 32) return SS_OK;
    if (!uniform && !always && !walk) return SS_OK;
  } else if (!always) {
    if (known && !uniform) return SS_OK;
    if (row_tiles >= 2 ? c->cfg.d != 128 : !uniform) return SS_OK;
  }
  const int64_t units = (int64_t)pairs * row_tiles;
  const int wave = 2 * ss::kNumSM;                                  // two CTAs per SM
  if (units > wave) return SS_OK;
  int64_t tiles = 0;
  for (int j = 0; j < n_chunks; ++j) {
    const ss_chunk_desc& d = chunks[j];
    if (!d.K.ptr || !d.V.ptr || d.L_c <= 0) return SS_ERR_ARG;
    if (d.L_c > c->cfg.max_Lc) return SS_ERR_SHAPE;
    if (!tensor_ok(d.K) || !tensor_ok(d.V) || (d.valid_len && ((uintptr_t)d.valid_len & 3))) return SS_ERR_ALIGN;
    tiles += (d.L_c + kTileKeys - 1) / kTileKeys;
    if (keys_on_m && d.L_c < 128) return SS_OK;   // (a box of 128 tokens)
  }
  if ((keys_on_m ? tiles / 2 : tiles) > 65000) return SS_OK;   // (the kernels' 16-bit tile tables)
  // a history of a few tiles per request is latency bound: the separate calls (CUDA-core kernel for
  // tiny ones) or the one-launch small round of ss_verify_round do better (measured on the
  // 1,024-token chain workload)
  if (tiles < 64 && !always) return SS_OK;
  if (c->n_sets == c->n_set_cap) {  // every partial set is in use: fold them into one first
    cudaError_t e = fold_sets(c, c->stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
  }
  // the launch's partial states may take the room of several sets (they are contiguous): the
  // highest split number it may use
  int64_t split_cap = (int64_t)(c->n_set_cap - c->n_sets) * c->slots_per_set / pairs;
  if (split_cap > kMaxSplits) split_cap = kMaxSplits;
  int splits = (int)(wave / units);
  if (splits > split_cap) splits = (int)split_cap;
  if (splits > tiles / 8) splits = (int)(tiles / 8);               // at least eight tiles per CTA
  if (c->force_splits > 0 && c->force_splits < splits) splits = c->force_splits;
  if (splits < 1) splits = 1;
  ss::HistParams h;
  memset(&h, 0, sizeof(h));
  if (walk) {
    // 128-token tiles of each request by the host's lengths; the shares and the largest number of
    // pieces a request is cut into (= partial states per row), with the kernel's own arithmetic
    const int tile_tokens = 128;
    h.n_req = c->B;
    for (int b = 0; b < c->B; ++b) {
      int64_t t128 = 0;
      for (int j = 0; j < n_chunks; ++j) {
        const ss_chunk_desc& d = chunks[j];
        int64_t v = d.valid_len ? d.valid_len_host[b] : d.L_c;
        v = v < 0 ? 0 : (v > d.L_c ? d.L_c : v);
        t128 += (v + tile_tokens - 1) / tile_tokens;
      }
      h.req_prefix[b + 1] = h.req_prefix[b] + (int)t128;
    }
    const int64_t all = h.req_prefix[c->B];
    int ctas = wave / c->cfg.H_kv;
    if (ctas > all / 8) ctas = (int)(all / 8);                     // at least eight tiles per CTA
    if (ctas < 1) ctas = 1;
    h.walk_ctas = ctas;
    int most = 1;
    for (int b = 0; b < c->B; ++b) {
      const int64_t p0 = h.req_prefix[b], p1 = h.req_prefix[b + 1];
      int first = 0, last = ctas - 1;
      while (all * (first + 1) / ctas <= p0) ++first;               // the first share that reaches past p0
      while (last > first && all * last / ctas >= p1) --last;       // the last share that starts before p1
      if (last - first + 1 > most) most = last - first + 1;
    }
    if (most > split_cap) return SS_OK;
    splits = most;
  }
  const int sets_taken = (int)(((int64_t)splits * pairs + c->slots_per_set - 1) / c->slots_per_set);
  // the chunks' tensor maps, K and V alternating, in one of the workspace's lists
  CUtensorMap maps[2 * ss::kMaxHistChunks];
  for (int j = 0; j < n_chunks; ++j)
    if (!get_tensor_map(c, chunks[j].K, c->B, chunks[j].L_c, keys_on_m ? 128 : kTileKeys, &maps[2 * j]) ||
        !get_tensor_map(c, chunks[j].V, c->B, chunks[j].L_c, keys_on_m ? 128 : kTileKeys, &maps[2 * j + 1]))
      return SS_OK;
  int slot = -1;
  for (int i = 0; i < kHistSlots && slot < 0; ++i)
    if (c->hist_n[i] == 2 * n_chunks && memcmp(c->hist_host[i], maps, (size_t)2 * n_chunks * sizeof(CUtensorMap)) == 0)
      slot = i;
  cudaStream_t s = c->stream;
  // Under a stream capture the launch may be replayed from a graph for as long as the context
  // lives, reading its list of tensor maps every time: a list that is already on the device is kept
  // for good; a list that would have to be sent now (a copy from pageable memory, and whose slot
  // could be reused later) is not taken: the chunks go out one by one, their maps as parameters.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) {
    (void)cudaGetLastError();
    cap = cudaStreamCaptureStatusNone;
  }
  const bool capturing = cap != cudaStreamCaptureStatusNone;
  if (slot < 0) {
    if (capturing) return SS_OK;
    for (int i = 0; i < kHistSlots; ++i)
      if (!c->hist_pinned[i] && (slot < 0 || c->hist_age[i] < c->hist_age[slot])) slot = i;
    if (slot < 0) return SS_OK;  // every list belongs to a captured launch
    memcpy(c->hist_host[slot], maps, (size_t)2 * n_chunks * sizeof(CUtensorMap));
    c->hist_n[slot] = 0;  // (not valid until the copy has been enqueued)
    // stream order: the copy runs after every kernel already enqueued, which may still read the list
    cudaError_t e = cudaMemcpyAsync(c->hist_maps + (size_t)slot * 2 * ss::kMaxHistChunks, c->hist_host[slot],
                                    (size_t)2 * n_chunks * sizeof(CUtensorMap), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->hist_n[slot] = 2 * n_chunks;
  }
  if (capturing) c->hist_pinned[slot] = true;
  c->hist_age[slot] = ++c->tm_clock;

  ss::ChunkParams p;
  memset(&p, 0, sizeof(p));
  h.n_chunks = n_chunks;
  h.maps = c->hist_maps + (size_t)slot * 2 * ss::kMaxHistChunks;
  int64_t tokens = 0;
  for (int j = 0; j < n_chunks; ++j) {
    h.valid_len[j] = chunks[j].valid_len;
    h.L_c[j] = chunks[j].L_c;
    if (chunks[j].valid_len && chunks[j].valid_len_host) {
      for (int b = 0; b < c->B; ++b) {
        const int v = chunks[j].valid_len_host[b];
        tokens += v < 0 ? 0 : (v > chunks[j].L_c ? chunks[j].L_c : v);
      }
    } else {
      tokens += (int64_t)c->B * chunks[j].L_c;
    }
  }
  p.row_tiles = row_tiles;
  p.rows_per_tile = R < 128 ? R : 128;
  p.splits = splits;
  p.tiles_per_split = 0;
  p.Q = (const __nv_bfloat16*)c->Q.ptr;
  p.q_sb = c->Q.stride_b;
  p.q_sh = c->Q.stride_h;
  p.q_st = c->Q.stride_t;
  p.B = c->B;
  p.H_kv = c->cfg.H_kv;
  p.G = c->G;
  p.T_q = c->T_q;
  p.R = R;
  p.d = c->cfg.d;
  p.L_c = 0;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.part_ml = c->part_ml + (int64_t)c->n_sets * c->set_stride_ml;
  p.part_a = c->part_a + (int64_t)c->n_sets * c->set_stride_a;
  p.R_stride = c->R_stride;
  p.a_slot0 = c->n_sets * c->slots_per_set;
  p.status = c->status;
  p.trace = c->trace_on ? c->trace : nullptr;
  p.cta_log = c->cta_log;
  p.cta_log_cap = c->cta_log_cap;
  p.launch_seq = (unsigned int)c->launches;
  p.wait_first = c->first_launch ? 1 : 0;
  cudaError_t e = keys_on_m ? ss::launch_chunk_tc_keys_hist(p, h, c->tm_a, s, use_pdl_first(c))
                            : ss::launch_chunk_tc_hist(p, h, c->tm_a, s, use_pdl_first(c));
  if (e != cudaSuccess) return cuda_fail(c, e);
  c->last_kernel = keys_on_m ? "tcgen05-keys-round" : "tcgen05-round";
  ++c->launches;
  c->stats.chunk_calls += n_chunks;
  c->stats.kv_bytes += tokens * c->cfg.H_kv * c->cfg.d * 4;
  for (int k = 0; k < sets_taken; ++k) {  // (the sets whose room the launch's states run into hold none of their own)
    c->splits[c->n_sets] = k == 0 ? (uint8_t)splits : 0;
    memset(c->absent[c->n_sets], 0, sizeof(c->absent[0]));
    ++c->n_sets;
  }
  c->first_launch = false;
  *taken = true;
  return SS_OK;
}

ss_status ss_verify_chunks(ss_ctx* c, const ss_chunk_desc* chunks, int32_t n_chunks, void* stream) {
  if (!c || n_chunks < 0 || (n_chunks > 0 && !chunks)) return SS_ERR_ARG;
  if (c->state != ss_ctx::OPEN || (cudaStream_t)stream != c->stream) return SS_ERR_STATE;
  bool one_launch = false;
  ss_status st = hist_chunks(c, chunks, n_chunks, &one_launch);
  for (int j = 0; !one_launch && j < n_chunks && st == SS_OK; ++j)
    st = chunk_impl(c, chunks[j].K, chunks[j].V, chunks[j].L_c, chunks[j].valid_len,
                    chunks[j].valid_len_host, stream);
  return st;
}

ss_status ss_verify_round(ss_ctx* c, ss_tensor Q, int32_t B, int32_t T_q, float scale,
                          const ss_chunk_desc* chunks, int32_t n_chunks, ss_tensor K_loc, ss_tensor V_loc,
                          int32_t T_loc, ss_mask_kind kind, const uint64_t* mask_bits, void* O, float* LSE,
                          void* stream) {
  if (!c || !O || n_chunks < 0 || (n_chunks > 0 && !chunks) || T_loc < 0) return SS_ERR_ARG;
  if (c->state != ss_ctx::IDLE) return SS_ERR_STATE;
  // A round of a few tiles in all takes one launch: chunks, local segment and finalize in one
  // CUDA-core kernel, no partial state in HBM.  Everything is checked as the separate calls do.
  int64_t tiles = 0;
  bool small = n_chunks <= ss::kMaxRoundChunks && T_loc <= 64 && !(c->cfg.flags & (SS_FLAG_ROWS_ON_M | SS_FLAG_KEYS_ON_M));
  for (int j = 0; small && j < n_chunks; ++j) {
    if (chunks[j].L_c <= 0) return SS_ERR_ARG;
    tiles += (chunks[j].L_c + kTileKeys - 1) / kTileKeys;
  }
  if (small && tiles <= 32 && B > 0 && T_q > 0) {
    if (!Q.ptr) return SS_ERR_ARG;
    if (!(scale > 0.f) || !(scale < 3.0e38f)) return SS_ERR_ARG;
    if (B > c->cfg.max_B || T_q > c->cfg.max_Tq || T_loc > c->cfg.max_Tloc) return SS_ERR_SHAPE;
    if (!tensor_ok(Q) || !aligned16(O) || (LSE && ((uintptr_t)LSE & 3))) return SS_ERR_ALIGN;
    ss::RoundParams p;
    memset(&p, 0, sizeof(p));
    for (int j = 0; j < n_chunks; ++j) {
      const ss_chunk_desc& d = chunks[j];
      if (!d.K.ptr || !d.V.ptr) return SS_ERR_ARG;
      if (d.L_c > c->cfg.max_Lc) return SS_ERR_SHAPE;
      if (!tensor_ok(d.K) || !tensor_ok(d.V) || (d.valid_len && ((uintptr_t)d.valid_len & 3))) return SS_ERR_ALIGN;
      p.chunk[j] = {(const __nv_bfloat16*)d.K.ptr, (const __nv_bfloat16*)d.V.ptr, d.K.stride_b, d.K.stride_h,
                    d.K.stride_t, d.V.stride_b, d.V.stride_h, d.V.stride_t, d.valid_len, d.L_c};
    }
    if (T_loc > 0) {
      if (!K_loc.ptr || !V_loc.ptr) return SS_ERR_ARG;
      if (kind != SS_MASK_CHAIN && kind != SS_MASK_TREE_BITS) return SS_ERR_ARG;
      if (kind == SS_MASK_TREE_BITS && !mask_bits) return SS_ERR_ARG;
      if (kind == SS_MASK_CHAIN && T_loc < T_q) return SS_ERR_ARG;
      if (!tensor_ok(K_loc) || !tensor_ok(V_loc) || (mask_bits && ((uintptr_t)mask_bits & 7))) return SS_ERR_ALIGN;
    }
    p.Q = (const __nv_bfloat16*)Q.ptr;
    p.q_sb = Q.stride_b;
    p.q_sh = Q.stride_h;
    p.q_st = Q.stride_t;
    p.B = B;
    p.H_q = c->cfg.H_q;
    p.H_kv = c->cfg.H_kv;
    p.G = c->G;
    p.T_q = T_q;
    p.d = c->cfg.d;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.n_chunks = n_chunks;
    p.K_loc = (const __nv_bfloat16*)K_loc.ptr;
    p.V_loc = (const __nv_bfloat16*)V_loc.ptr;
    p.kl_sb = K_loc.stride_b;
    p.kl_sh = K_loc.stride_h;
    p.kl_st = K_loc.stride_t;
    p.vl_sb = V_loc.stride_b;
    p.vl_sh = V_loc.stride_h;
    p.vl_st = V_loc.stride_t;
    p.T_loc = T_loc;
    p.mask_bits = (T_loc > 0 && kind == SS_MASK_TREE_BITS) ? mask_bits : nullptr;
    p.mask_words = (T_loc + 63) / 64;
    // few CTAs in all: tiles of 8 rows spread a kv-head's rows over more SMs (K/V are re-read
    // through L2, which a round this small fits into)
    const int R = T_q * c->G;
    p.rows_per_tile = ((int64_t)B * c->cfg.H_kv * ((R + 7) / 8) <= 2 * ss::kNumSM) ? 8 : ss::simt_rows_per_tile(R);
    // token splits: about two CTAs per SM in all, at most 16 and at most one per tile; the
    // partial states go to the (otherwise idle) partial-set area of the workspace
    const int64_t units = (int64_t)B * c->cfg.H_kv * ((R + p.rows_per_tile - 1) / p.rows_per_tile);
    int splits = (int)((2 * ss::kNumSM) / units);
    if (splits > (T_loc > 0 ? 15 : 16)) splits = T_loc > 0 ? 15 : 16;  // the local segment's CTA makes 16
    if (splits > tiles) splits = (int)tiles;
    const int64_t slot_floats = (int64_t)p.rows_per_tile * (c->cfg.d + 2);
    if (units > ss::kRoundCounters ||
        units * (splits + 1) * slot_floats * (int64_t)sizeof(float) >
            (int64_t)(c->ws_bytes - ((uint8_t*)c->part_a - c->ws)))
      splits = 1;
    if (splits < 1) splits = 1;
    p.tiles_per_split = tiles ? (int)((tiles + splits - 1) / splits) : 0;
    p.splits = tiles ? (int)((tiles + p.tiles_per_split - 1) / p.tiles_per_split) : 1;
    p.loc_split = p.splits - 1;
    if (splits > 1 && p.splits > 1 && T_loc > 0 && p.splits < 16) p.loc_split = p.splits++;  // a CTA of its own
    p.scratch = c->part_a;
    p.counters = c->round_counters;
    p.O = (__nv_bfloat16*)O;
    p.LSE = LSE;
    p.status = c->status;
    const bool pdl = (c->cfg.flags & SS_FLAG_OVERLAP_CHUNKS) && !c->no_overlap;
    // the splits of a unit as one thread-block cluster: the states are merged through distributed
    // shared memory instead of scratch, a ticket and two trips to L2
    p.cluster = (p.splits > 1 && c->round_clusters) ? 1 : 0;
    cudaError_t e = ss::launch_round_simt(p, (cudaStream_t)stream, pdl);
    if (e != cudaSuccess && p.cluster) {  // (a device or driver that does not take the cluster: the ticket path)
      (void)cudaGetLastError();
      c->round_clusters = false;
      p.cluster = 0;
      e = ss::launch_round_simt(p, (cudaStream_t)stream, pdl);
    }
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->last_kernel = "simt-round";
    ++c->launches;
    ++c->stats.rounds;
    c->stats.rows += (int64_t)B * c->cfg.H_q * T_q;
    c->stats.chunk_calls += n_chunks;
    for (int j = 0; j < n_chunks; ++j)
      c->stats.kv_bytes += (int64_t)B * chunks[j].L_c * c->cfg.H_kv * c->cfg.d * 4;
    return SS_OK;
  }
  // the general case: the separate calls, enqueued from here
  ss_status st = ss_verify_begin(c, Q, B, T_q, scale, stream);
  if (st != SS_OK) return st;
  st = ss_verify_chunks(c, chunks, n_chunks, stream);
  if (st == SS_OK && T_loc > 0) st = ss_verify_local(c, K_loc, V_loc, T_loc, kind, mask_bits, stream);
  if (st == SS_OK) st = ss_verify_finalize(c, O, LSE, stream);
  if (st != SS_OK) ss_verify_abort(c);  // kernels already enqueued finish; nothing is merged
  return st;
}

ss_status ss_time_rounds(ss_ctx* c, ss_tensor Q, int32_t B, int32_t T_q, float scale,
                         const ss_chunk_desc* chunks, int32_t n_chunks, int32_t n_sets, ss_tensor K_loc,
                         ss_tensor V_loc, int32_t T_loc, ss_mask_kind kind, const uint64_t* mask_bits, void* O,
                         float* LSE, void* stream, int32_t n_rounds, int32_t single_call, float* ms_total) {
  if (!c || !ms_total || n_rounds <= 0 || n_sets <= 0 || n_chunks < 0 || (n_chunks > 0 && !chunks))
    return SS_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess) return SS_ERR_CUDA;
  if (cudaEventCreate(&e1) != cudaSuccess) {
    cudaEventDestroy(e0);
    return SS_ERR_CUDA;
  }
  ss_status st = SS_OK;
  cudaError_t e = cudaEventRecord(e0, s);
  for (int i = 0; i < n_rounds && st == SS_OK && e == cudaSuccess; ++i) {
    const ss_chunk_desc* set = chunks + (size_t)(i % n_sets) * n_chunks;   // round i's history buffers
    if (single_call) {
      st = ss_verify_round(c, Q, B, T_q, scale, set, n_chunks, K_loc, V_loc, T_loc, kind, mask_bits, O, LSE, stream);
    } else {
      st = ss_verify_begin(c, Q, B, T_q, scale, stream);
      for (int j = 0; j < n_chunks && st == SS_OK; ++j)
        st = chunk_impl(c, set[j].K, set[j].V, set[j].L_c, set[j].valid_len, set[j].valid_len_host, stream);
      if (st == SS_OK && T_loc > 0) st = ss_verify_local(c, K_loc, V_loc, T_loc, kind, mask_bits, stream);
      if (st == SS_OK) st = ss_verify_finalize(c, O, LSE, stream);
      if (st != SS_OK) ss_verify_abort(c);
    }
  }
  if (e == cudaSuccess) e = cudaEventRecord(e1, s);
  if (e == cudaSuccess) e = cudaEventSynchronize(e1);
  if (e == cudaSuccess) e = cudaEventElapsedTime(ms_total, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (st != SS_OK) return st;
  return e == cudaSuccess ? SS_OK : cuda_fail(c, e);
}

ss_status ss_verify_abort(ss_ctx* c) {
  if (!c) return SS_ERR_ARG;
  // Kernels already enqueued finish on their own; their partial states are simply never merged.
  c->state = ss_ctx::IDLE;
  c->Q.ptr = nullptr;
  c->n_sets = 0;
  c->has_local = false;
  return SS_OK;
}

ss_status ss_commit_gather(ss_ctx* c, ss_tensor K_loc, ss_tensor V_loc, int32_t B, int32_t T_loc,
                           const int32_t* accept_idx, const int32_t* accept_cnt, ss_tensor K_dst,
                           ss_tensor V_dst, int32_t cap, const int32_t* dst_off, void* stream) {
  if (!c || !K_loc.ptr || !V_loc.ptr || !K_dst.ptr || !V_dst.ptr || !accept_idx || !accept_cnt ||
      !dst_off)
    return SS_ERR_ARG;
  if (B <= 0 || T_loc <= 0 || cap <= 0) return SS_ERR_ARG;
  if (B > c->cfg.max_B || T_loc > c->cfg.max_Tloc) return SS_ERR_SHAPE;
  if (!tensor_ok(K_loc) || !tensor_ok(V_loc) || !tensor_ok(K_dst) || !tensor_ok(V_dst))
    return SS_ERR_ALIGN;
  ss::GatherParams p;
  memset(&p, 0, sizeof(p));
  p.K_loc = (const uint16_t*)K_loc.ptr;
  p.V_loc = (const uint16_t*)V_loc.ptr;
  p.ks_b = K_loc.stride_b;
  p.ks_h = K_loc.stride_h;
  p.ks_t = K_loc.stride_t;
  p.vs_b = V_loc.stride_b;
  p.vs_h = V_loc.stride_h;
  p.vs_t = V_loc.stride_t;
  p.K_dst = (uint16_t*)K_dst.ptr;
  p.V_dst = (uint16_t*)V_dst.ptr;
  p.kd_b = K_dst.stride_b;
  p.kd_h = K_dst.stride_h;
  p.kd_t = K_dst.stride_t;
  p.vd_b = V_dst.stride_b;
  p.vd_h = V_dst.stride_h;
  p.vd_t = V_dst.stride_t;
  p.accept_idx = accept_idx;
  p.accept_cnt = accept_cnt;
  p.dst_off = dst_off;
  p.B = B;
  p.H_kv = c->cfg.H_kv;
  p.T_loc = T_loc;
  p.d = c->cfg.d;
  p.cap = cap;
  p.status = c->status;
  cudaError_t e = ss::launch_gather(p, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(c, e);
  ++c->launches;
  return SS_OK;
}

ss_status ss_poll_status(ss_ctx* c, void* stream, int32_t timeout_ms, uint32_t* dev_bits) {
  if (!c) return SS_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (timeout_ms > 0) {
    const auto t0 = std::chrono::steady_clock::now();
    for (;;) {
      cudaError_t q = cudaStreamQuery(s);
      if (q == cudaSuccess) break;
      if (q != cudaErrorNotReady) return cuda_fail(c, q);
      const auto ms = std::chrono::duration_cast<std::chrono::milliseconds>(
                          std::chrono::steady_clock::now() - t0)
                          .count();
      if (ms > timeout_ms) return SS_ERR_TIMEOUT;
    }
  } else {
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(c, e);
  }
  uint32_t bits = 0;
  cudaError_t e = cudaMemcpy(&bits, c->status, 4, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(c, e);
  if (dev_bits) *dev_bits = bits;
  if (bits) {
    e = cudaMemset(c->status, 0, 4);
    if (e != cudaSuccess) return cuda_fail(c, e);
    return SS_ERR_DEVICE_FLAG;
  }
  return SS_OK;
}

const char* ss_strerror(ss_status s) {
  switch (s) {
    case SS_OK: return "ok";
    case SS_ERR_ARG: return "invalid argument";
    case SS_ERR_SHAPE: return "shape outside the configured limits";
    case SS_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case SS_ERR_STATE: return "call order violated";
    case SS_ERR_CAPACITY: return "workspace too small";
    case SS_ERR_UNSUPPORTED: return "device is not sm_100";
    case SS_ERR_CUDA: return "CUDA call failed";
    case SS_ERR_DEVICE_FLAG: return "device status word set";
    case SS_ERR_TIMEOUT: return "timed out";
  }
  return "unknown";
}

size_t ss_sizeof_stream_desc(void) { return sizeof(ss_stream_desc); }
int32_t ss_last_cuda_error(ss_ctx* c) { return c ? c->last_cuda : 0; }
ss_status ss_trace_enable(ss_ctx* c, int32_t on) {
  if (!c) return SS_ERR_ARG;
  c->trace_on = on != 0;
  if (on) {
    cudaError_t e = cudaMemset(c->trace, 0, ss::kTraceWords * sizeof(unsigned long long));
    if (e != cudaSuccess) return cuda_fail(c, e);
  }
  return SS_OK;
}

int32_t ss_trace_read(ss_ctx* c, uint64_t* out, int32_t max_words) {
  if (!c || !out || max_words <= 0) return 0;
  const int n = max_words < ss::kTraceWords ? max_words : ss::kTraceWords;
  if (cudaMemcpy(out, c->trace, (size_t)n * sizeof(uint64_t), cudaMemcpyDeviceToHost) != cudaSuccess)
    return 0;
  return n;
}

ss_status ss_cta_log_set(ss_ctx* c, uint64_t* log, int32_t capacity) {
  if (!c || capacity < 0 || (log && capacity == 0)) return SS_ERR_ARG;
  if ((uintptr_t)log & 7) return SS_ERR_ALIGN;
  c->cta_log = (unsigned long long*)log;
  c->cta_log_cap = log ? capacity : 0;
  return SS_OK;
}

ss_status ss_get_stats(ss_ctx* c, ss_stats* out) {
  if (!c || !out) return SS_ERR_ARG;
  *out = c->stats;
  out->launches = c->launches;
  return SS_OK;
}

int64_t ss_launch_count(ss_ctx* c) { return c ? c->launches : 0; }
const char* ss_last_chunk_kernel(ss_ctx* c) { return c ? c->last_kernel : "none"; }

}  // extern "C"

// accessors for the pipeline translation unit
namespace ss {
struct PipeRes {
  cudaStream_t copy_stream, attn_stream;
  cudaEvent_t *ev_ready, *ev_free, ev_t0, ev_t1;
};
namespace {
// Releases whatever pipeline resources exist (handles are null until created).
void pipeline_release(ss_ctx* c) {
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->attn_stream) cudaStreamDestroy(c->attn_stream);
  for (int i = 0; i < 2; ++i) {
    if (c->ev_ready[i]) cudaEventDestroy(c->ev_ready[i]);
    if (c->ev_free[i]) cudaEventDestroy(c->ev_free[i]);
  }
  if (c->ev_t0) cudaEventDestroy(c->ev_t0);
  if (c->ev_t1) cudaEventDestroy(c->ev_t1);
  for (int i = 0; i < c->ev_pool_n; ++i) cudaEventDestroy(c->ev_pool[i]);
  delete[] c->ev_pool;
  c->ev_pool = nullptr;
  c->ev_pool_n = 0;
  c->copy_stream = c->attn_stream = nullptr;
  c->ev_ready[0] = c->ev_ready[1] = c->ev_free[0] = c->ev_free[1] = c->ev_t0 = c->ev_t1 = nullptr;
  c->pipe_ready = false;
}
}  // namespace
void ctx_pipeline_release(ss_ctx* c) { pipeline_release(c); }
cudaError_t ctx_pipeline(ss_ctx* c, PipeRes* out) {
  if (!c->pipe_ready) {
    cudaError_t e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->attn_stream, cudaStreamNonBlocking);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
      e = cudaEventCreateWithFlags(&c->ev_ready[i], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_free[i], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreate(&c->ev_t0);
    if (e == cudaSuccess) e = cudaEventCreate(&c->ev_t1);
    if (e != cudaSuccess) {
      pipeline_release(c);  // nothing half-built stays behind
      return e;
    }
    c->pipe_ready = true;
  }
  out->copy_stream = c->copy_stream;
  out->attn_stream = c->attn_stream;
  out->ev_ready = c->ev_ready;
  out->ev_free = c->ev_free;
  out->ev_t0 = c->ev_t0;
  out->ev_t1 = c->ev_t1;
  return cudaSuccess;
}
// Timing events for the streamed round: at least n of them, or null when the context was
// created without SS_FLAG_STREAM_TIMING (or they cannot be had).  Grown on demand, kept.
cudaEvent_t* ctx_timing_events(ss_ctx* c, int n) {
  if (!(c->cfg.flags & SS_FLAG_STREAM_TIMING)) return nullptr;
  if (n <= c->ev_pool_n) return c->ev_pool;
  cudaEvent_t* grown = new (std::nothrow) cudaEvent_t[n];
  if (!grown) return nullptr;
  for (int i = 0; i < c->ev_pool_n; ++i) grown[i] = c->ev_pool[i];
  int have = c->ev_pool_n;
  for (; have < n; ++have)
    if (cudaEventCreate(&grown[have]) != cudaSuccess) break;
  delete[] c->ev_pool;
  c->ev_pool = grown;
  c->ev_pool_n = have;
  return have >= n ? c->ev_pool : nullptr;
}
void ctx_set_stream_times(ss_ctx* c, int64_t round_ns, int64_t transfer_ns, int64_t chunk_ns, int64_t tail_ns) {
  c->stats.last_round_ns = round_ns;
  c->stats.last_transfer_ns = transfer_ns;
  c->stats.last_chunk_ns = chunk_ns;
  c->stats.last_tail_ns = tail_ns;
  const int64_t w = round_ns - chunk_ns - tail_ns;
  c->stats.last_wait_ns = w > 0 ? w : 0;
}
int ctx_dims(ss_ctx* c, int* H_q, int* H_kv, int* d) {
  *H_q = c->cfg.H_q;
  *H_kv = c->cfg.H_kv;
  *d = c->cfg.d;
  return c->cfg.max_B;
}
void ctx_set_cuda_error(ss_ctx* c, cudaError_t e) { c->last_cuda = (int32_t)e; }
uint32_t* ctx_status_word(ss_ctx* c) { return c->status; }
bool ctx_round_open(ss_ctx* c) { return c->state != ss_ctx::IDLE; }
// The streamed entry points refuse to start while the caller has a round open, so a round
// that is open when they finish is one of their own (error path) and is dropped.
void ctx_pipeline_mode(ss_ctx* c, bool on) {
  c->no_overlap = on;
  if (!on) c->state = ss_ctx::IDLE;
}
// Error path of the pipeline: what was enqueued before the failing call still reads the caller's
// buffers, so wait for it before the error is returned.
void ctx_pipeline_drain(ss_ctx* c) {
  if (!c->pipe_ready) return;
  cudaStreamSynchronize(c->copy_stream);
  cudaStreamSynchronize(c->attn_stream);
}
}  // namespace ss
