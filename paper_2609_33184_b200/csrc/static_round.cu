// A whole verification round for callers that cannot allocate device memory.
//
// Some callers of this library may not call cudaMalloc (or any allocating routine) at the
// point where they need attention: code running inside a stream-ordered region that must
// not synchronise the device, plug-ins loaded into a host process whose memory pool they do
// not own, or start-up paths that run before the host framework's allocator exists.  The
// regular entry points need a caller-allocated workspace for the per-row partial states
// (m, l, a).  This entry point keeps that scratch in a fixed array inside the library's
// device image instead, so a round needs nothing but its inputs and outputs.
//
// The scratch is one file-scope array per loaded device image: every GPU that loads the
// library holds SS_STATIC_SCRATCH_BYTES of it until the process exits, all calls share it
// and it keeps the previous call's contents.  The words that must start at zero are cleared
// on the caller's stream at the start of every call; every partial state the final merge
// reads is rewritten by the call itself.  Two calls whose kernels can overlap on the GPU
// (different streams) race on the array: callers serialise them.
#include <cstring>
#include <mutex>

#include "ss_internal.h"

namespace {

// Scratch for the partial states of one round.  In host code this name is only a stand-in
// for the symbol, not a device address: the address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[SS_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
struct DeviceSlot {
  bool ready;
  unsigned char* base;  // device address of g_static_scratch on this device
};
DeviceSlot g_slots[kMaxDevices];
std::mutex g_slots_mutex;  // host threads may make their first calls on a device at the same time

// First call on a device: resolve the array's device address (no allocation involved).
ss_status scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_slots_mutex);
  DeviceSlot& s = g_slots[dev];
  if (!s.ready) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return SS_ERR_CUDA;
    if (major != 10) return SS_ERR_UNSUPPORTED;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr)
      return SS_ERR_CUDA;
    if (ss::chunk_simt_prepare() != cudaSuccess) return SS_ERR_CUDA;  // function attributes only
    s.base = static_cast<unsigned char*>(p);
    s.ready = true;
  }
  *out = s.base;
  return SS_OK;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }
bool tensor_ok(const ss_tensor& t) {
  return t.ptr && aligned16(t.ptr) && t.stride_b % 8 == 0 && t.stride_h % 8 == 0 && t.stride_t % 8 == 0;
}

}  // namespace

extern "C" ss_status ss_verify_round_static(const ss_static_round* r, void* stream) {
  // The set-up (address of the scratch array on the current device) comes first, so that any
  // call - even one rejected for its arguments, e.g. with r == NULL - serves as the warm-up
  // call that has to precede a stream capture.  Its own error is reported after the argument
  // checks, which need no device.
  unsigned char* base = nullptr;
  const ss_status setup = scratch_for_current_device(&base);
  if (!r || !r->O) return SS_ERR_ARG;
  if (r->B <= 0 || r->H_q <= 0 || r->H_kv <= 0 || r->T_q <= 0 || r->L_c < 0 || r->T_loc < 0)
    return SS_ERR_ARG;
  if (r->H_q % r->H_kv || (r->d != 64 && r->d != 128) || r->T_loc > 1024) return SS_ERR_SHAPE;
  // the limits of the regular entry points: the row-per-warp kernels index query rows with
  // 32-bit arithmetic and a kv-head carries at most 4096 rows
  if ((int64_t)r->T_q * (r->H_q / r->H_kv) > 4096) return SS_ERR_SHAPE;
  if ((int64_t)r->B * r->H_q * r->T_q >= (1ll << 31)) return SS_ERR_SHAPE;
  if (r->L_c == 0 && r->T_loc == 0) return SS_ERR_ARG;
  if (!(r->scale > 0.f) || !(r->scale < 3.0e38f)) return SS_ERR_ARG;
  if (r->T_loc > 0 && r->mask_kind != SS_MASK_CHAIN && r->mask_kind != SS_MASK_TREE_BITS) return SS_ERR_ARG;
  if (r->T_loc > 0 && r->mask_kind == SS_MASK_CHAIN && r->T_loc < r->T_q) return SS_ERR_ARG;
  if (!tensor_ok(r->Q) || !aligned16(r->O)) return SS_ERR_ALIGN;
  if (r->L_c > 0 && (!tensor_ok(r->K) || !tensor_ok(r->V))) return SS_ERR_ALIGN;
  if (r->T_loc > 0 && (!tensor_ok(r->K_loc) || !tensor_ok(r->V_loc))) return SS_ERR_ALIGN;
  if (r->T_loc > 0 && r->mask_kind == SS_MASK_TREE_BITS && !r->mask_bits) return SS_ERR_ARG;

  const int G = r->H_q / r->H_kv;
  const int R = r->T_q * G;                                  // <= 4096
  const int64_t pairs = (int64_t)r->B * r->H_kv;
  const int rows_per_tile = ss::simt_rows_per_tile(R);
  const int64_t row_tiles = (R + rows_per_tile - 1) / rows_per_tile;
  const int n_tiles = (r->L_c + ss::kTileKeys - 1) / ss::kTileKeys;
  int splits = 1;
  if (n_tiles > 0) {
    splits = (int)(ss::kNumSM / (pairs * row_tiles));   // pairs * row_tiles >= 1
    if (splits > ss::kMaxSplits) splits = ss::kMaxSplits;
    if (splits > (n_tiles + 1) / 2) splits = (n_tiles + 1) / 2;
    if (splits < 1) splits = 1;
  }
  const int tiles_per_split = n_tiles ? (n_tiles + splits - 1) / splits : 0;
  if (n_tiles) splits = (n_tiles + tiles_per_split - 1) / tiles_per_split;

  // layout inside the scratch: [256 B header: status word] [ml: sets x slots x R] [a: ... x d]
  // (rows of one set: at most 16 * 2^31 / T_q, far inside 64 bits; a set that large fails the
  // capacity check below)
  const size_t rows_per_set = (size_t)splits * (size_t)pairs * (size_t)R;   // set 0 = history chunk, set 1 = local
  if (rows_per_set > SS_STATIC_SCRATCH_BYTES) return SS_ERR_CAPACITY;
  const size_t ml_bytes = 2 * rows_per_set * sizeof(float2);
  const size_t off_a = 256 + ((ml_bytes + 255) / 256) * 256;
  const size_t need = off_a + 2 * rows_per_set * r->d * sizeof(float);
  if (need > SS_STATIC_SCRATCH_BYTES) return SS_ERR_CAPACITY;
  if (setup != SS_OK) return setup;
  cudaStream_t s = (cudaStream_t)stream;
  uint32_t* status = r->status ? r->status : reinterpret_cast<uint32_t*>(base);
  // the shared array keeps the last call's contents: clear the word that must start at zero
  if (cudaMemsetAsync(base, 0, 256, s) != cudaSuccess) return SS_ERR_CUDA;
  float2* part_ml = reinterpret_cast<float2*>(base + 256);
  float* part_a = reinterpret_cast<float*>(base + off_a);
  const float scale_log2 = r->scale * 1.4426950408889634f;

  if (n_tiles) {
    ss::ChunkParams p;
    memset(&p, 0, sizeof(p));
    p.Q = (const __nv_bfloat16*)r->Q.ptr;
    p.q_sb = r->Q.stride_b;
    p.q_sh = r->Q.stride_h;
    p.q_st = r->Q.stride_t;
    p.K = (const __nv_bfloat16*)r->K.ptr;
    p.V = (const __nv_bfloat16*)r->V.ptr;
    p.k_sb = r->K.stride_b;
    p.k_sh = r->K.stride_h;
    p.k_st = r->K.stride_t;
    p.v_sb = r->V.stride_b;
    p.v_sh = r->V.stride_h;
    p.v_st = r->V.stride_t;
    p.valid_len = r->valid_len;
    p.B = r->B;
    p.H_kv = r->H_kv;
    p.G = G;
    p.T_q = r->T_q;
    p.R = R;
    p.d = r->d;
    p.L_c = r->L_c;
    p.splits = splits;
    p.tiles_per_split = tiles_per_split;
    p.row_tiles = (int)row_tiles;
    p.rows_per_tile = rows_per_tile;
    p.scale_log2 = scale_log2;
    p.part_ml = part_ml;
    p.part_a = part_a;
    p.R_stride = R;
    p.status = status;
    if (ss::launch_chunk_simt(p, s, false) != cudaSuccess) return SS_ERR_CUDA;
  }
  if (r->T_loc > 0) {
    ss::LocalParams p;
    memset(&p, 0, sizeof(p));
    p.Q = (const __nv_bfloat16*)r->Q.ptr;
    p.q_sb = r->Q.stride_b;
    p.q_sh = r->Q.stride_h;
    p.q_st = r->Q.stride_t;
    p.K = (const __nv_bfloat16*)r->K_loc.ptr;
    p.V = (const __nv_bfloat16*)r->V_loc.ptr;
    p.k_sb = r->K_loc.stride_b;
    p.k_sh = r->K_loc.stride_h;
    p.k_st = r->K_loc.stride_t;
    p.v_sb = r->V_loc.stride_b;
    p.v_sh = r->V_loc.stride_h;
    p.v_st = r->V_loc.stride_t;
    p.mask_bits = (r->mask_kind == SS_MASK_TREE_BITS) ? r->mask_bits : nullptr;
    p.B = r->B;
    p.H_q = r->H_q;
    p.H_kv = r->H_kv;
    p.G = G;
    p.T_q = r->T_q;
    p.T_loc = r->T_loc;
    p.d = r->d;
    p.mask_words = (r->T_loc + 63) / 64;
    p.scale_log2 = scale_log2;
    p.part_ml = part_ml + rows_per_set;
    p.part_a = part_a + rows_per_set * r->d;
    p.R_stride = R;
    if (ss::launch_local(p, s, false) != cudaSuccess) return SS_ERR_CUDA;
  }
  ss::MergeParams m;
  memset(&m, 0, sizeof(m));
  m.part_ml = part_ml;
  m.part_a = part_a;
  m.set_stride_ml = (int64_t)rows_per_set;
  m.set_stride_a = (int64_t)rows_per_set * r->d;
  m.n_sets = n_tiles ? 1 : 0;
  m.has_local = r->T_loc > 0 ? 1 : 0;
  m.local_set = 1;
  m.B = r->B;
  m.H_q = r->H_q;
  m.H_kv = r->H_kv;
  m.G = G;
  m.T_q = r->T_q;
  m.d = r->d;
  m.R_stride = R;
  m.splits[0] = (uint8_t)splits;
  m.O = (__nv_bfloat16*)r->O;
  m.LSE = r->LSE;
  if (ss::launch_finalize(m, s, false) != cudaSuccess) return SS_ERR_CUDA;
  return SS_OK;
}
