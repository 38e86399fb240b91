// Internal declarations shared by the host API and the kernels of libspecstream.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "specstream.h"

namespace ss {

constexpr int kMaxSets = 128;      // chunk-call partial sets a finalize launch can take
constexpr int kMaxSplits = 16;     // token splits of one chunk call
constexpr int kTileKeys = 64;      // keys per shared-memory tile of the tensor-core kernel
constexpr int kMaxListed = 256;    // largest batch whose requests a chunk call can list one by one
constexpr int kNumSM = 148;
constexpr int kTraceTiles = 32;    // tiles of CTA (0,0,0) a trace records
constexpr int kTraceWords = 3 * kTraceTiles * 8;  // [role][tile][event] clock64 stamps

// Partial state of one (set, split, request, kv-head): for each of its R rows the pair
// (m, l) and the unnormalised output a[d].  m is the row maximum of
// score * scale * log2(e) (base-2 domain), l = sum exp2(s2 - m), a = sum exp2(s2 - m) v.
// An untouched or empty row is the identity (m = -inf, l = 0); its a[] is never read.
struct PartialView {
  float2* ml;        // [slots][R_stride]
  float* a;          // [slots][R_stride][d]
};

struct ChunkParams {
  const __nv_bfloat16* Q;
  int64_t q_sb, q_sh, q_st;
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  int64_t k_sb, k_sh, k_st, v_sb, v_sh, v_st;
  const int32_t* valid_len;  // device [B] or null
  int B, H_kv, G, T_q, R, d, L_c;
  int splits;           // token splits (grid.x / row_tiles)
  int tiles_per_split;  // kTileKeys-token tiles per split
  int row_tiles;        // tiles of query rows per (b, kvh)
  int rows_per_tile;    // rows in each row tile but possibly the last
  float scale_log2;     // scale * log2(e)
  float2* part_ml;      // partial set of this call
  float* part_a;
  int R_stride;
  int a_slot0;          // index of the call's first (split, b, kvh) slot along the outermost axis of
                        // the tensor map over all partial a[] (tensor-core kernel with rows on M)
  uint32_t* status;
  int wait_first;       // 1: wait for the preceding kernel before reading inputs
  unsigned long long* trace;  // optional: per-tile clock stamps of CTA (0,0,0), see ss_trace_read
  // requests this launch covers: 0 = all B (grid.z = B, b = blockIdx.z); otherwise grid.z =
  // n_active and b = active_b[blockIdx.z] (the host knew which requests have tokens in this chunk)
  int n_active;
  uint8_t active_b[kMaxListed];
  // paged chunk (null = contiguous): token tok of request b lives in page
  // page_table[b][tok / page_size] of the pool, at token offset tok % page_size
  const int32_t* page_table;
  int pages_per_req, page_size, n_pages;
  // optional per-CTA log (ss_cta_log_set): word 0 counts entries, entry i = 4 words from word
  // 4 * (i + 1): start ns, end ns, (SM id << 32 | launch number), (linear block id << 32 | tiles)
  unsigned long long* cta_log;
  int cta_log_cap;
  unsigned int launch_seq;
};

// A round's history as a list of contiguous chunks, for ONE launch of the rows-on-M kernel over all
// of them: a CTA takes an equal share of its request's 64-token tiles (counted chunk by chunk from
// the valid lengths), keeps one accumulator across the chunk boundaries and writes one partial state,
// so a round has `splits` partial states per row instead of one per chunk call, and its CTAs are as
// many as the GPU holds at once and equally long.
constexpr int kMaxHistChunks = 32;
struct HistParams {
  int n_chunks;                               // 0: an ordinary one-chunk launch (ChunkParams alone)
  const CUtensorMap* maps;                    // device memory: chunk j's K map at [2j], its V map at [2j + 1]
  const int32_t* valid_len[kMaxHistChunks];   // per chunk: device [B], or null (= L_c[j])
  // Ragged batches (keys-on-M kernel): the CTAs of a kv-head walk equal shares of ALL its requests'
  // tiles laid end to end, so a CTA may finish one request and start the next (one partial state
  // per request it touches).  The shares are cut on the host's copy of the lengths: req_prefix[b] =
  // 128-token tiles (by that copy, at least one per request) before request b; a CTA's share of a
  // request is scaled to the tiles the device's lengths give.  n_req = 0: not used.
  int n_req;
  int walk_ctas;                              // CTAs per kv-head (grid.x) of that mode
  int req_prefix[kMaxListed + 1];
  int L_c[kMaxHistChunks];
};

// A whole small round for round_simt_kernel: every history chunk, the local segment, outputs.
constexpr int kMaxRoundChunks = 16;
constexpr int kRoundCounters = 1024;  // ticket counters in the workspace (units of a split round)
struct RoundChunk {
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  int64_t k_sb, k_sh, k_st, v_sb, v_sh, v_st;
  const int32_t* valid_len;  // device [B] or null
  int L_c;
};
struct RoundParams {
  const __nv_bfloat16* Q;
  int64_t q_sb, q_sh, q_st;
  int B, H_q, H_kv, G, T_q, d;
  float scale_log2;
  int n_chunks;
  RoundChunk chunk[kMaxRoundChunks];
  const __nv_bfloat16* K_loc;  // T_loc == 0: no local segment
  const __nv_bfloat16* V_loc;
  int64_t kl_sb, kl_sh, kl_st, vl_sb, vl_sh, vl_st;
  int T_loc;
  const uint64_t* mask_bits;   // null for chain
  int mask_words;
  int rows_per_tile;           // 8, 16 or 32
  int splits, tiles_per_split; // CTAs per (b, kvh, row tile): token splits over the history's 64-token
                               // tiles (all chunks), plus one for the local segment when it has its own
  int loc_split;               // the split that takes the local segment
  float* scratch;              // splits > 1: [unit][split][(m, l)[RT], a[RT][d]], unit = (b, kvh, row tile)
  unsigned int* counters;      // splits > 1: one ticket counter per unit, zero between rounds
  int cluster;                 // 1: the splits of a unit are one thread-block cluster (grid.x = row tile x
                               // split, split fastest) and merge through distributed shared memory
  __nv_bfloat16* O;
  float* LSE;                  // may be null
  uint32_t* status;            // may be null
};

struct LocalParams {
  const __nv_bfloat16* Q;
  int64_t q_sb, q_sh, q_st;
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  int64_t k_sb, k_sh, k_st, v_sb, v_sh, v_st;
  const uint64_t* mask_bits;  // null for chain
  int B, H_q, H_kv, G, T_q, T_loc, d, mask_words;
  float scale_log2;
  float2* part_ml;  // local set: slot = b * H_kv + kvh
  float* part_a;
  int R_stride;
};

struct MergeParams {
  const float2* part_ml;  // set 0
  const float* part_a;
  int64_t set_stride_ml;  // elements between sets
  int64_t set_stride_a;
  int n_sets;
  int has_local;
  int local_set;          // index of the local set
  int B, H_q, H_kv, G, T_q, d, R_stride;
  uint8_t splits[kMaxSets];
  // bit b of absent[s] (kMaxListed bits): chunk set s holds no partial of request b.  (With
  // this table the structure is larger than 4 KB: it relies on the large kernel parameter
  // space of CUDA 12.1+ on sm_70 and later.)
  uint64_t absent[kMaxSets][kMaxListed / 64];
  // finalize outputs
  __nv_bfloat16* O;
  float* LSE;
  // fold output (set 0, split 0)
  float2* fold_ml;
  float* fold_a;
};

struct GatherParams {
  const uint16_t* K_loc;
  const uint16_t* V_loc;
  int64_t ks_b, ks_h, ks_t, vs_b, vs_h, vs_t;
  uint16_t* K_dst;
  uint16_t* V_dst;
  int64_t kd_b, kd_h, kd_t, vd_b, vd_h, vd_t;
  const int32_t* accept_idx;
  const int32_t* accept_cnt;
  const int32_t* dst_off;
  int B, H_kv, T_loc, d, cap;
  uint32_t* status;
};

// launchers (each returns the cudaError_t of the launch)
cudaError_t launch_chunk_simt(const ChunkParams& p, cudaStream_t s, bool pdl);
cudaError_t launch_round_simt(const RoundParams& p, cudaStream_t s, bool pdl);
cudaError_t chunk_simt_prepare();    // one-time function attributes
int simt_rows_per_tile(int R);       // rows per CTA tile of the CUDA-core chunk kernel
cudaError_t launch_chunk_tc(const ChunkParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            const CUtensorMap& tmA, cudaStream_t s, bool pdl);
// The keys-on-M kernel over a list of chunks (head dim 128, up to 32 rows per kv-head, fewer than
// 65,536 tiles of 128 tokens per request).
cudaError_t launch_chunk_tc_keys_hist(const ChunkParams& p, const HistParams& h, const CUtensorMap& any_map,
                                      cudaStream_t s, bool pdl);
// The same kernel over a list of chunks (HistParams); p.splits = CTAs per (request, kv-head, row tile).
cudaError_t launch_chunk_tc_hist(const ChunkParams& p, const HistParams& h, const CUtensorMap& tmA,
                                 cudaStream_t s, bool pdl);
cudaError_t chunk_tc_prepare();  // one-time function attributes
cudaError_t launch_chunk_tc_keys(const ChunkParams& p, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                 cudaStream_t s, bool pdl);
cudaError_t chunk_tc_keys_prepare();
cudaError_t launch_local(const LocalParams& p, cudaStream_t s, bool pdl);
cudaError_t launch_finalize(const MergeParams& p, cudaStream_t s, bool pdl);
cudaError_t launch_fold(const MergeParams& p, cudaStream_t s);
cudaError_t launch_export(const MergeParams& p, cudaStream_t s);  // fold_ml/fold_a = caller buffers
cudaError_t launch_import(const MergeParams& p, cudaStream_t s);  // part_ml/part_a = caller buffers
cudaError_t launch_gather(const GatherParams& p, cudaStream_t s);

// Launch helper: optional programmatic stream serialization attribute.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t s, bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The same with thread-block clusters of cluster_x CTAs along x.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                         cudaStream_t s, bool pdl, unsigned cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster_x;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Device-side programmatic-dependent-launch controls (no-ops when the kernel was
// launched without the attribute).
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait_prior() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Optional trace of the tensor-core chunk kernels: CTA (0,0,0) stamps clock64 at fixed points
// of each role's tile loop.  role 0 = TMA producer, 1 = MMA issuer, 2 = softmax thread 0.
__device__ __forceinline__ void trace(unsigned long long* tr, int role, int it, int ev) {
  if (tr && it < kTraceTiles) tr[(role * kTraceTiles + it) * 8 + ev] = clock64();
}

// Per-CTA log entry, written by one thread when the CTA leaves (no-op without a log buffer).
__device__ __forceinline__ unsigned long long cta_log_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void cta_log_write(const ChunkParams& p, unsigned long long t_start, int n_tiles) {
  if (!p.cta_log) return;
  const unsigned long long i = atomicAdd(p.cta_log, 1ull);
  if (i >= (unsigned long long)p.cta_log_cap) return;
  unsigned int smid;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
  const unsigned long long lin = blockIdx.x + (unsigned long long)gridDim.x * (blockIdx.y + (unsigned long long)gridDim.y * blockIdx.z);
  unsigned long long* e = p.cta_log + 4 * (i + 1);
  e[0] = t_start;
  e[1] = cta_log_now();
  e[2] = ((unsigned long long)smid << 32) | p.launch_seq;
  e[3] = (lin << 32) | (unsigned int)n_tiles;
}

// What one CTA of a chunk kernel owns: a tile of query rows of one (request, kv-head) and a
// range of the chunk's tokens (its token split), plus where its partial state goes.  Shared
// by the three chunk kernels; `tile_rows` is the kernel's rows per row tile.
struct ChunkWork {
  int b, kvh, split;
  int slot;             // (split, b, kvh) slot of the call's partial set
  int row0, nrows;      // query rows [row0, row0 + nrows) of the kv-head
  int tok0, tok1;       // visible tokens [tok0, tok1) of the chunk (tok1 <= tok0: nothing to do)
  float2* out_ml;       // partial state of the CTA's rows
  float* out_a;
  bool chain_cta;       // the one CTA of the grid that keeps the completion order (see below)
};
__device__ __forceinline__ ChunkWork chunk_work(const ChunkParams& p, int tile_rows) {
  ChunkWork w;
  const int rt = blockIdx.x % p.row_tiles;
  w.split = blockIdx.x / p.row_tiles;
  w.kvh = blockIdx.y;
  w.b = p.n_active ? p.active_b[blockIdx.z] : blockIdx.z;
  w.row0 = rt * tile_rows;
  w.nrows = min(tile_rows, p.R - w.row0);
  w.chain_cta = (blockIdx.x | blockIdx.y | blockIdx.z) == 0;
  int valid = p.L_c;
  if (p.valid_len) {
    valid = p.valid_len[w.b];
    if (valid < 0 || valid > p.L_c) {  // flagged and clamped, never trusted
      if (threadIdx.x == 0) atomicOr(p.status, SS_DEV_BAD_VALID_LEN);
      valid = max(0, min(valid, p.L_c));
    }
  }
  w.tok0 = w.split * p.tiles_per_split * kTileKeys;
  w.tok1 = min(valid, w.tok0 + p.tiles_per_split * kTileKeys);
  const size_t slot = ((size_t)w.split * p.B + w.b) * p.H_kv + w.kvh;
  w.slot = (int)slot;
  w.out_ml = p.part_ml + slot * p.R_stride + w.row0;
  w.out_a = p.part_a + (slot * p.R_stride + w.row0) * p.d;
  return w;
}

// Where token `tok` of request b lives: (index along the tensor's outermost axis, token within
// it).  Contiguous chunks: (b, tok).  Paged chunks: (page id, offset); a page id outside the pool
// raises SS_DEV_BAD_PAGE and maps to index n_pages, which loads read as zeros.
__device__ __forceinline__ void locate_token(const ChunkParams& p, int b, int tok, int* outer,
                                             int* inner) {
  if (!p.page_table) {
    *outer = b;
    *inner = tok;
    return;
  }
  const int pg = tok / p.page_size;
  int id = (pg < p.pages_per_req) ? p.page_table[(int64_t)b * p.pages_per_req + pg] : -1;
  if (id < 0 || id >= p.n_pages) {
    atomicOr(p.status, SS_DEV_BAD_PAGE);
    id = p.n_pages;
  }
  *outer = id;
  *inner = tok - pg * p.page_size;
}

}  // namespace ss
