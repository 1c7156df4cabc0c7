// Host side of the dKV-Cache step library: handles, arena layout, the
// per-step launch sequence, and the extern "C" entry points of dkv.h.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <unordered_set>
#include <vector>

#include "../../include/dkv.h"
#include "attn_mma.cuh"
#include "attn_simt.cuh"
#include "gemm_f32.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "attn_tc.cuh"
#include "index_kernels.cuh"
#include "stream_probe.cuh"
#include "ptx.cuh"
#include "row_kernels.cuh"

using namespace dkv;

namespace {

constexpr int NUM_SMS = 148;            // B200; the cost models are calibrated for it
constexpr int MAX_TILE_COUNTERS = 256;  // arrival counters of the fused GEMM tails (one per weight tile x row tile)
constexpr int N_BOX = 16;   // row boxes of 16, 32, ..., 256 rows
inline int box_rows(int i) { return 16 * (i + 1); }

enum ProfClass {
  PC_COMPACT = 0, PC_EMBED, PC_GEMM_QKV, PC_QKV_POST, PC_ATTN, PC_GEMM_O, PC_RESID_NORM, PC_GEMM_GU, PC_SWIGLU,
  PC_GEMM_DOWN, PC_GEMM_HEAD, PC_HEAD_STATS, PC_SELECT, PC_COUNT
};
const char* const PROF_NAMES[PC_COUNT] = {"compact", "embed_norm", "gemm_qkv", "qkv_rope_scatter", "attention",
                                          "gemm_o", "resid_norm", "gemm_gateup", "swiglu", "gemm_down",
                                          "gemm_head", "head_stats", "select_unmask"};

// Launch with programmatic dependent launch allowed: the kernel may start while
// its predecessor in the stream drains; every kernel calls pdl_wait() before it
// touches anything a predecessor wrote.  DKV_PDL=0 switches the attribute off.
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  static const bool use_pdl = []() {
    const char* e = getenv("DKV_PDL");
    return !(e && atoi(e) == 0);
  }();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = use_pdl ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// SMs of the current device (looked up once per device): what bounds a launch whose CTAs wait for each other.
inline int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
  if (!cached[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 1;
    cached[dev] = n;
  }
  return cached[dev];
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// K-major 16-bit matrix [rows, k] -> boxes of 64 columns x box_rows rows, 128-byte swizzle.
int make_tmap(CUtensorMap* tm, const void* base, long long rows, long long k, int box_rows, bool fp16 = false) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return DKV_E_CUDA;
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(k), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstride[1] = {static_cast<cuuint64_t>(k) * 2};
  cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? DKV_OK : DKV_E_CUDA;
}

// Tensor map of a weight matrix stored in blocks of 128 rows x 64 columns ([ceil(rows / 128)][ceil(k / 64)]
// blocks of 16 KB each, zero-padded): the box the GEMM loads per weight half and k-block is then one
// contiguous piece of memory instead of 128 pieces of 128 bytes a row pitch apart.
int make_tmap_blocked(CUtensorMap* tm, const void* base, long long rows, long long k) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return DKV_E_CUDA;
  const long long blocks = ((rows + GEMM_BM - 1) / GEMM_BM) * ((k + GEMM_BK - 1) / GEMM_BK);
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(GEMM_BK), static_cast<cuuint64_t>(blocks * GEMM_BM)};
  cuuint64_t gstride[1] = {static_cast<cuuint64_t>(GEMM_BK) * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(GEMM_BK), static_cast<cuuint32_t>(GEMM_BM)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? DKV_OK : DKV_E_CUDA;
}
inline size_t blocked_bytes(long long rows, long long k) {
  return static_cast<size_t>((rows + GEMM_BM - 1) / GEMM_BM) * ((k + GEMM_BK - 1) / GEMM_BK) * GEMM_BM * GEMM_BK * 2;
}

// 16-bit tensor with 128-byte rows of 64 elements innermost, up to 3 dimensions (dims / box innermost
// first, strides in bytes for dimensions 1..rank-1), 128-byte swizzle.
int make_tmap_nd(CUtensorMap* tm, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
                 const cuuint32_t* box, bool fp16) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return DKV_E_CUDA;
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(tm, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank,
                  const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? DKV_OK : DKV_E_CUDA;
}

// The opt-in to large dynamic shared memory is a per-device property of a kernel: one flag per
// (call site, device), so that a process that drives several GPUs sets it on each of them.
struct PerDeviceOnce {
  bool done[64] = {};
  bool need() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
    if (done[dev]) return false;
    done[dev] = true;
    return true;
  }
};

struct AttnMaps {
  CUtensorMap q, k, v;      // K/V boxes of 128 slots (one CTA per SM, two softmax warpgroups)
  CUtensorMap k64, v64;     // K/V boxes of 64 slots (two CTAs per SM)
  int group, rows_q;
};
// Tensor maps of the tcgen05 attention kernel (head_dim 128): queries [rows][H_q][128] with a box of
// (64 columns, the KV head's query heads, rows_q rows);
// K and V slots as a 3-D tensor [KV heads of all layers and sequences][kv_len slots][128]: a slot tile that
// reaches past kv_len is zero-filled by the copy engine instead of running into the next head's (or the
// next layer's, possibly unwritten) slots.  kv_stride = slots per head in memory (>= kv_len).
int make_attn_maps(AttnMaps* am, const void* q, long long q_rows, const void* k_slots, const void* v_slots,
                   long long kv_heads_total, int kv_len, int kv_stride, int hq, int hkv, bool fp16) {
  am->group = hq / hkv;
  am->rows_q = ATC_M / am->group;
  if (am->rows_q < 1) return DKV_E_UNSUPPORTED;
  cuuint64_t qd[3] = {static_cast<cuuint64_t>(ATC_DH), static_cast<cuuint64_t>(hq), static_cast<cuuint64_t>(q_rows)};
  cuuint64_t qs[2] = {static_cast<cuuint64_t>(ATC_DH) * 2, static_cast<cuuint64_t>(hq) * ATC_DH * 2};
  cuuint32_t qb[3] = {64, static_cast<cuuint32_t>(am->group), static_cast<cuuint32_t>(am->rows_q)};
  int rc = make_tmap_nd(&am->q, q, 3, qd, qs, qb, fp16);
  cuuint64_t kd[3] = {static_cast<cuuint64_t>(ATC_DH), static_cast<cuuint64_t>(kv_len),
                      static_cast<cuuint64_t>(kv_heads_total)};
  cuuint64_t ks[2] = {static_cast<cuuint64_t>(ATC_DH) * 2, static_cast<cuuint64_t>(kv_stride) * ATC_DH * 2};
  cuuint32_t kb[3] = {64, ATC_BKV, 1};
  if (!rc) rc = make_tmap_nd(&am->k, k_slots, 3, kd, ks, kb, fp16);
  if (!rc) rc = make_tmap_nd(&am->v, v_slots, 3, kd, ks, kb, fp16);
  cuuint32_t kb64[3] = {64, 64, 1};
  if (!rc) rc = make_tmap_nd(&am->k64, k_slots, 3, kd, ks, kb64, fp16);
  if (!rc) rc = make_tmap_nd(&am->v64, v_slots, 3, kd, ks, kb64, fp16);
  return rc;
}

// kv_len: the slots every query attends = the slot extent of am's K/V maps; kv_head0: first KV head of
// this layer inside the maps.
int attention_tc(const AttnMaps& am, void* o, const int32_t* row_off, int batch, int rows_bound, int kv_len, int hq,
                 int hkv, int kv_head0, bool bf16, int* status, cudaStream_t st) {
  static PerDeviceOnce attr_once;
  if (attr_once.need()) {
    if (cudaFuncSetAttribute(k_attn_tc<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_tc_smem<128, 2>()) !=
            cudaSuccess ||
        cudaFuncSetAttribute(k_attn_tc<64, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_tc_smem<64, 1>()) !=
            cudaSuccess)
      return DKV_E_CUDA;
  }
  AttnTcParams p;
  p.o = o;
  p.row_off = row_off;
  p.seq_len = kv_len;
  p.n_q_heads = hq;
  p.n_kv_heads = hkv;
  p.group = am.group;
  p.rows_q = am.rows_q;
  p.kv_head0 = kv_head0;
  p.scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(ATC_DH));
  p.bf16 = bf16 ? 1 : 0;
  p.status = status;
  dim3 grid(ceil_div(rows_bound, am.rows_q), hkv, batch);
  // Two resident CTAs per SM keep the units busy; with at most one CTA per SM to hand out, the
  // 128-slot shape has half the iterations and the shorter latency.
  const long long ctas = static_cast<long long>(grid.x) * grid.y * grid.z;
  if (ctas > 148)
    launch_k((k_attn_tc<64, 1>), grid, 192, attn_tc_smem<64, 1>(), st, am.q, am.k64, am.v64, p);
  else
    launch_k((k_attn_tc<128, 2>), grid, 320, attn_tc_smem<128, 2>(), st, am.q, am.k, am.v, p);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

struct LayerMaps {
  CUtensorMap wqkv, wo, wgu, wd;
};

}  // namespace

struct dkv_model {
  dkv_model_desc desc;
  std::vector<dkv_layer_weights> layers;
  const void* embed;
  const void* head;
  const float* final_norm;
  std::vector<LayerMaps> maps;
  CUtensorMap head_map;
  int d_q, d_kv, n_qkv;
  size_t esize;   // bytes per weight element
  size_t asize;   // bytes per activation / cache element
  bool w_blocked; // the layers' fp16 weight copies are stored in 128 x 64 blocks (make_tmap_blocked)
  int gu_blk;     // 128: the gate/up copy is regrouped [128 gate | 128 up] per 256 rows (SwiGLU in the GEMM epilogue); 0: not
  bool gu_pair;   // the standalone SwiGLU launch runs on CTA pairs (d_ffn a multiple of 256)
};

namespace {

enum XBuf { XB_XN = 0, XB_AO, XB_U, XB_XH, XB_COUNT };

struct Arena {
  // K/V slots
  void* k_slots;
  void* v_slots;
  float2* rope_tab;
  uint8_t* mask_buf[2];
  int32_t* d_buf[2];
  int32_t* written_step;
  int32_t* act_idx;
  int32_t* row_off;
  int32_t* inv;
  int32_t* head_row;
  int32_t* head_pos;
  int32_t* head_off;
  int* status;
  float* h;
  void* xn;
  void* qb;
  void* ao;
  void* ub;
  void* xh;
  float* logits;
  float* st_max;                 // head statistics per 32 token ids: [ceil(V/32)][h_cap]
  float* st_sum;
  int* st_arg;
  float* st_m2;
  float* st_t;
  float* part;
  float* ssq;                    // [ceil(d_model / 128)][r_cap]: partial sums of squares of the residual rows
  float* head_rs;                // [h_cap]: 1 / RMS of each head row
  unsigned int* tile_cnt;        // [2][MAX_TILE_COUNTERS]: arrival counters of the fused GEMM tails, two sets used in turn
  float* conf_i;
  int32_t* pred_i;
  int32_t* tok_stage;
  uint8_t* mask_stage;
  int32_t* chosen_stage;
  int32_t* dpos_stage;
  size_t total;
};

struct Dims {
  int B, L, P, G, kmax, hmax;
  long long r_cap, h_cap, part_rows, n_max;
};

Dims make_dims(const dkv_model* m, int B, int L, int P, const dkv_policy* pol) {
  Dims d;
  d.B = B;
  d.L = L;
  d.P = P;
  d.G = L - P;
  d.kmax = (pol && pol->max_k > 0) ? pol->max_k : 1;
  int hm = (pol && pol->max_head_rows > 0) ? pol->max_head_rows : (L - P);
  d.hmax = std::max(1, std::min(hm, L));
  d.r_cap = std::max<long long>(256, align_up(static_cast<size_t>(B) * L, 16));
  d.h_cap = std::max<long long>(256, align_up(static_cast<size_t>(B) * d.hmax, 16));
  d.part_rows = std::max<long long>(d.r_cap, 2048);
  d.n_max = std::max<long long>(std::max<long long>(m->n_qkv, 2LL * m->desc.d_ffn), m->desc.d_model);
  return d;
}

// Walk the arena layout; with base == nullptr only the size is computed.
void carve(const dkv_model* m, const Dims& d, uint8_t* base, Arena* a) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> uint8_t* {
    off = align_up(off, 256);
    uint8_t* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  };
  const dkv_model_desc& md = m->desc;
  const size_t es = m->asize;
  const size_t BL = static_cast<size_t>(d.B) * d.L;
  const size_t slots = static_cast<size_t>(md.n_layers) * d.B * md.n_kv_heads * d.L * md.head_dim * es;
  a->k_slots = take(slots);
  a->v_slots = take(slots);
  a->rope_tab = reinterpret_cast<float2*>(take(static_cast<size_t>(d.L) * (md.head_dim / 2) * sizeof(float2)));
  a->mask_buf[0] = take(BL);
  a->mask_buf[1] = take(BL);
  a->d_buf[0] = reinterpret_cast<int32_t*>(take(static_cast<size_t>(d.B) * d.kmax * 4));
  a->d_buf[1] = reinterpret_cast<int32_t*>(take(static_cast<size_t>(d.B) * d.kmax * 4));
  a->written_step = reinterpret_cast<int32_t*>(take(BL * 4));
  a->act_idx = reinterpret_cast<int32_t*>(take(BL * 4));
  a->row_off = reinterpret_cast<int32_t*>(take((d.B + 1) * 4));
  a->inv = reinterpret_cast<int32_t*>(take(BL * 4));
  a->head_row = reinterpret_cast<int32_t*>(take(BL * 4));
  a->head_pos = reinterpret_cast<int32_t*>(take(BL * 4));
  a->head_off = reinterpret_cast<int32_t*>(take((d.B + 1) * 4));
  a->status = reinterpret_cast<int*>(take(256));
  a->h = reinterpret_cast<float*>(take(d.r_cap * md.d_model * 4));
  a->xn = take(d.r_cap * md.d_model * es);
  a->qb = take(d.r_cap * m->d_q * es);
  a->ao = take(d.r_cap * m->d_q * es);
  a->ub = take(d.r_cap * md.d_ffn * es);
  a->xh = take(d.h_cap * md.d_model * es);
  a->logits = reinterpret_cast<float*>(take(d.h_cap * static_cast<size_t>(md.vocab) * 4));
  {
    const size_t groups = (static_cast<size_t>(md.vocab) + 31) / 32 + 8;   // + the tail of the last weight tile
    a->st_max = reinterpret_cast<float*>(take(groups * d.h_cap * 4));
    a->st_sum = reinterpret_cast<float*>(take(groups * d.h_cap * 4));
    a->st_arg = reinterpret_cast<int*>(take(groups * d.h_cap * 4));
    a->st_m2 = reinterpret_cast<float*>(take(groups * d.h_cap * 4));
    a->st_t = reinterpret_cast<float*>(take(groups * d.h_cap * 4));
  }
  a->part = reinterpret_cast<float*>(take(d.part_rows * d.n_max * 4));
  a->ssq = reinterpret_cast<float*>(take(static_cast<size_t>((md.d_model + 127) / 128) * d.r_cap * 4));
  a->head_rs = reinterpret_cast<float*>(take(d.h_cap * 4));
  a->tile_cnt = reinterpret_cast<unsigned int*>(take(2 * MAX_TILE_COUNTERS * 4));
  a->conf_i = reinterpret_cast<float*>(take(BL * 4));
  a->pred_i = reinterpret_cast<int32_t*>(take(BL * 4));
  a->tok_stage = reinterpret_cast<int32_t*>(take(BL * 4));
  a->mask_stage = take(BL);
  a->chosen_stage = reinterpret_cast<int32_t*>(take(static_cast<size_t>(d.B) * d.kmax * 4));
  a->dpos_stage = reinterpret_cast<int32_t*>(take(static_cast<size_t>(d.B) * d.kmax * 4));
  a->total = align_up(off, 256);
}

struct ProfEvent {
  cudaEvent_t a, b;
  int cls;
  double bytes, flops;
};

}  // namespace

struct dkv_cache {
  const dkv_model* model;
  Dims dims;
  dkv_policy policy;
  Arena ar;
  CUtensorMap xmaps[XB_COUNT][N_BOX];
  CUtensorMap xmaps_half[XB_COUNT][N_BOX];   // the same operands in boxes of half the rows, for the CTA-pair GEMM
  AttnMaps attn_maps;            // tcgen05 attention (head_dim 128, 16-bit modes): all seq_len slots attended
  AttnMaps attn_maps_prompt;     // the same buffers with the slot extent cut at the prompt (isolated prefill pass)
  bool attn_tc;
  int fuse_tails;        // bit 0: RoPE / K/V scatter inside the QKV GEMM; bit 1: residual / norm statistics inside
                         // the O and down GEMMs (one-wave launches)
  long long tail_wait_cycles;   // bound of the fused tails' cross-CTA wait; dkv_debug_tail_wait shortens it
  int tail_extra;               // arrivals the tails expect beyond the real ones (0; 1 under dkv_debug_tail_wait)
  int tail_cnt_set;             // which of the two sets of tile counters the next fused launch uses
  int step;              // steps run so far
  int last_refresh;      // step number of the last full / generation-only step
  int pending_refresh;   // -1 none, else DKV_REFRESH_*
  int prev_rows_bound;   // bound on #M_{t-1} per sequence
  bool have_dprev;
  int prev_k;            // k of the step that stored D_{t-1}
  cudaStream_t last_stream;
  dkv_stats stats;
  bool profiling;
  std::vector<ProfEvent> events;
  size_t ev_used;
  dkv_profile_entry prof[PC_COUNT];
};

namespace {

// Live handles: every entry point checks its handle against these sets, so that a destroyed,
// never-created or foreign pointer yields DKV_E_STATE instead of undefined behaviour.
std::mutex g_live_mu;
std::unordered_set<const void*> g_live_models, g_live_caches;
bool live_model(const dkv_model* m) {
  std::lock_guard<std::mutex> lk(g_live_mu);
  return g_live_models.count(m) != 0;
}
bool live_cache(const dkv_cache* c) {
  std::lock_guard<std::mutex> lk(g_live_mu);
  return g_live_caches.count(c) != 0 && g_live_models.count(c->model) != 0;
}
void set_live(std::unordered_set<const void*>& set, const void* h, bool on) {
  std::lock_guard<std::mutex> lk(g_live_mu);
  if (on) set.insert(h);
  else set.erase(h);
}
// NULL -> INVALID_ARG, not a live handle (or its model was destroyed) -> STATE
#define DKV_CHECK_CACHE(c)             \
  do {                                 \
    if (!(c)) return DKV_E_INVALID_ARG; \
    if (!live_cache(c)) return DKV_E_STATE; \
  } while (0)

// --------------------------------------------------------------- profiling
void prof_flush(dkv_cache* c) {
  for (size_t i = 0; i < c->ev_used; ++i) {
    ProfEvent& e = c->events[i];
    cudaEventSynchronize(e.b);
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e.a, e.b);
    c->prof[e.cls].launches += 1;
    c->prof[e.cls].ms += ms;
    c->prof[e.cls].bytes += e.bytes;
    c->prof[e.cls].flops += e.flops;
  }
  c->ev_used = 0;
}

struct Launch {
  dkv_cache* c;
  cudaStream_t st;
  ProfEvent* ev;
  Launch(dkv_cache* cache, cudaStream_t s, int cls, double bytes, double flops) : c(cache), st(s), ev(nullptr) {
    if (c) c->stats.kernel_launches += 1;
    if (c && c->profiling) {
      if (c->ev_used == c->events.size()) {
        if (c->events.size() >= 4096) {
          prof_flush(c);
        } else {
          ProfEvent e;
          cudaEventCreate(&e.a);
          cudaEventCreate(&e.b);
          c->events.push_back(e);
        }
      }
      ev = &c->events[c->ev_used++];
      ev->cls = cls;
      ev->bytes = bytes;
      ev->flops = flops;
      cudaEventRecord(ev->a, st);
    }
  }
  ~Launch() {
    if (ev) cudaEventRecord(ev->b, st);
  }
};

// ------------------------------------------------------------------- GEMM
int pick_box(int r_bound) {
  // smallest multiple of 16 that holds the rows; more than 256 rows are tiled evenly
  int tiles = ceil_div(r_bound, 256);
  int per = ceil_div(r_bound, tiles);
  int i = ceil_div(per, 16) - 1;
  return std::min(std::max(i, 0), N_BOX - 1);
}

// More than one row tile (> 256 rows): the launch is bound by the tensor pipe or by the operand bytes
// an SM takes in, and by how evenly the units fall into waves of NUM_SMS.  Estimated time in SM
// clocks of a launch with `t` row tiles and `s` K splits (constants calibrated on sweeps of the four
// LLaDA-shaped projections at 512-2048 rows): per k-block the slower of the MMAs (4 * br clocks for
// two 128-row halves) and the operand ingest (52 bytes per clock), an epilogue of br * 1 KB at 64
// bytes per clock per unit, whole waves, and the fp32 partials read back by the next kernel.
double est_clocks_multi_tile(int n, int k, int r_bound, int t, int s) {
  const int per = ceil_div(r_bound, t);
  const int br = 16 * ceil_div(per, 16);
  const int kb_total = ceil_div(k, GEMM_BK);
  const double kbu = std::ceil(kb_total / static_cast<double>(s));
  const double cyc_kb = std::max(4.0 * br, (2.0 * GEMM_A_BYTES + 128.0 * br) / 52.0);
  const double unit = kbu * cyc_kb + br * 1024.0 / 64.0;
  const double units = static_cast<double>(ceil_div(n, 2 * GEMM_BM)) * t * s;
  const double waves = std::ceil(units / NUM_SMS);
  const double partials = s > 1 ? 4.0 * s * r_bound * static_cast<double>(n) / (4.0e12 / 1.85e9) : 0.0;
  return waves * unit + partials;
}

// Row tiles and K splits for more than 256 rows: the usual ceil(rows / 256) tiles or one more
// (narrower tiles can fill the last wave better), each with its best split count.
void choose_multi_tile(int n, int k, int r_bound, long long part_rows, int* tiles_out, int* splits_out) {
  const int kb_total = ceil_div(k, GEMM_BK);
  int s_max = std::min(8, std::max(1, kb_total / 4));
  s_max = static_cast<int>(std::min<long long>(s_max, std::max<long long>(1, part_rows / std::max(1, r_bound))));
  const int t_min = ceil_div(r_bound, 256);
  double best = 1e300;
  *tiles_out = t_min;
  *splits_out = 1;
  for (int t = t_min; t <= t_min + 1; ++t) {
    for (int s = 1; s <= s_max; ++s) {
      if (s > 1 && (s - 1) * ceil_div(kb_total, s) >= kb_total) continue;
      const double c = est_clocks_multi_tile(n, k, r_bound, t, s);
      if (c < best * 0.97) {      // prefer fewer tiles and splits unless clearly better
        best = c;
        *tiles_out = t;
        *splits_out = s;
      }
    }
  }
}

// The same estimate for a launch on CTA pairs (k_gemm_tc2): a unit is 512 weight rows x br rows on two
// SMs, each CTA takes in 32 KB of weights and br / 2 rows per k-block, and the units run in waves of
// NUM_SMS / 2 pairs.
double est_clocks_pairs(int n, int k, int r_bound, int t, int s) {
  const int per = ceil_div(r_bound, t);
  const int br = 16 * ceil_div(per, 16);
  const int kb_total = ceil_div(k, GEMM_BK);
  const double kbu = std::ceil(kb_total / static_cast<double>(s));
  const double cyc_kb = std::max(4.0 * br, (2.0 * GEMM_A_BYTES + 64.0 * br) / 52.0);
  const double unit = kbu * cyc_kb + br * 1024.0 / 64.0;
  const double units = static_cast<double>(ceil_div(n, 512)) * t * s;
  const double waves = std::ceil(units / (NUM_SMS / 2));
  const double partials = s > 1 ? 4.0 * s * r_bound * static_cast<double>(n) / (4.0e12 / 1.85e9) : 0.0;
  return waves * unit + partials;
}
// Row tiles and K splits of a pair launch; `one_wave`: only plans whose units are all resident at once
// (what the fused row tails need).  Zero tiles: no such plan.
double choose_pairs(int n, int k, int r_bound, long long part_rows, bool one_wave, int* tiles_out, int* splits_out) {
  const int kb_total = ceil_div(k, GEMM_BK);
  int s_max = std::min(8, std::max(1, kb_total / 4));
  s_max = static_cast<int>(std::min<long long>(s_max, std::max<long long>(1, part_rows / std::max(1, r_bound))));
  const int t_min = ceil_div(r_bound, 256);
  double best = 1e300;
  *tiles_out = 0;
  *splits_out = 0;
  for (int t = t_min; t <= t_min + 2; ++t) {
    for (int s = 1; s <= s_max; ++s) {
      if (s > 1 && (s - 1) * ceil_div(kb_total, s) >= kb_total) continue;
      if (one_wave && ceil_div(n, 512) * t * s > NUM_SMS / 2) continue;
      const double c = est_clocks_pairs(n, k, r_bound, t, s);
      if (c < best * 0.97) {
        best = c;
        *tiles_out = t;
        *splits_out = s;
      }
    }
  }
  return best;
}

int env_int(const char* name, int dflt) {
  const char* s = getenv(name);
  return s ? atoi(s) : dflt;
}

// Number of K splits.  Cost model in bytes: the weight bytes divided by the
// fraction of CTA slots the units fill in their last wave, plus the fp32
// partials written and read back (they mostly stay in L2, hence the weight 1/2).
// Sweeps over the four LLaDA-shaped projections showed total time (GEMM plus
// the reduction of the partials) flat within 10 % around this choice.
int choose_splits(int n, int k, int r_bound, const GemmTcPlan& plan, long long part_rows) {
  const int tiles = ceil_div(n, GEMM_BM * plan.halves) * ceil_div(r_bound, plan.br);
  const int kb_total = ceil_div(k, GEMM_BK);
  int s_max = std::min(16, std::max(1, kb_total / 4));
  s_max = static_cast<int>(std::min<long long>(s_max, std::max<long long>(1, part_rows / std::max(1, r_bound))));
  const double slots = static_cast<double>(plan.ctas_per_sm) * NUM_SMS;
  const double w_bytes = 2.0 * n * static_cast<double>(k);
  int best = 1;
  double best_cost = 1e300;
  for (int s = 1; s <= s_max; ++s) {
    if (s > 1 && (s - 1) * ceil_div(kb_total, s) >= kb_total) continue;   // would leave an empty split
    const double units = static_cast<double>(tiles) * s;
    const double eff = units / (std::ceil(units / slots) * slots);
    const double cost = w_bytes / eff + (s > 1 ? 4.0 * s * r_bound * static_cast<double>(n) : 0.0);
    if (cost < best_cost * 0.98) {   // prefer fewer splits unless clearly better
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

struct HeadStats {   // vocabulary-head mode of the GEMM epilogue
  int mask_id;
  float* st_max;
  float* st_sum;
  int* st_arg;
  float* st_m2;   // NULL unless the score needs the second maximum / the entropy sum
  float* st_t;
  mutable int n_groups = 0;   // out: entries per row the launch writes (4 per CTA)
};

// Per-row scale of a GEMM's result: the RMSNorm of its operand, applied after the product.
struct RowScale {
  const float* src = nullptr;   // NULL: no scale
  int parts = 0;                // > 0: src = [parts][ld] partial sums of squares; 0: src = ready factors
  long long ld = 0;
  int d = 1;
  float eps = 0.f;
};

// Row epilogue fused into the GEMM across the CTAs of a weight tile (FUSE_RESID / FUSE_QKV).
struct FusedTail {
  int mode = FUSE_NONE;
  unsigned int* tile_cnt = nullptr;   // [2][MAX_TILE_COUNTERS]
  int* cnt_set = nullptr;             // which set the next fused launch counts on (flipped by every fused launch)
  long long wait_cycles = GEMM_WAIT_CYCLES;
  int extra = 0;
  float* h = nullptr;
  const float* gain = nullptr;
  void* xn_out = nullptr;
  float* ssq_out = nullptr;
  long long ssq_ld = 0;
  const int32_t* act_idx = nullptr;
  const float2* rope_tab = nullptr;
  int seq_len = 0, n_q_heads = 0, n_kv_heads = 0, head_dim = 0;
  void* q_out = nullptr;
  void* k_slots = nullptr;
  void* v_slots = nullptr;
};

struct GemmOpts {
  int forced_splits = 0;
  bool w_static = true;
  bool w_blocked = false;                    // tw is a make_tmap_blocked map
  const HeadStats* head = nullptr;
  void* swiglu_out = nullptr;
  int ld_u = 0;
  const CUtensorMap* xmaps_half = nullptr;   // [N_BOX] boxes of half the rows: run on CTA pairs
  int row_tiles = 0;                         // > 0: this many row tiles instead of ceil(rows / 256)
  RowScale scale;
  FusedTail tail;                            // applied only when the launch is one wave (see *fused_out)
};

void set_tail(GemmTcParams& p, const FusedTail& t) {
  p.fuse_mode = t.mode;
  p.tile_cnt = t.tile_cnt + *t.cnt_set * MAX_TILE_COUNTERS;
  p.tile_cnt_next = t.tile_cnt + (1 - *t.cnt_set) * MAX_TILE_COUNTERS;
  *t.cnt_set ^= 1;
  p.tail_wait_cycles = t.wait_cycles;
  p.tail_extra = t.extra;
  p.h = t.h;
  p.gain = t.gain;
  p.xn_out = t.xn_out;
  p.ssq_out = t.ssq_out;
  p.ssq_ld = t.ssq_ld;
  p.act_idx = t.act_idx;
  p.rope_tab = t.rope_tab;
  p.seq_len = t.seq_len;
  p.n_q_heads = t.n_q_heads;
  p.n_kv_heads = t.n_kv_heads;
  p.head_dim = t.head_dim;
  p.q_out = t.q_out;
  p.k_slots = t.k_slots;
  p.v_slots = t.v_slots;
}

// out (fp32 partials) [splits][r_bound * n]; returns splits and stride through the pointers.  When a
// fused tail is asked for and every unit gets a CTA of its own (units <= SMs, so that the CTAs of a
// tile can wait for each other), the kernel runs it and *fused_out is true; otherwise the partials
// are left in `out` for a row kernel.
int gemm_tc(const CUtensorMap& tw, const CUtensorMap* xmaps /*[N_BOX]*/, int n, int k, int r_bound,
            const int* r_dev, float* out, long long part_rows, int* status, bool x_bf16, cudaStream_t st,
            int* splits_out, long long* stride_out, const GemmOpts& o = GemmOpts(), bool* fused_out = nullptr) {
  static PerDeviceOnce attr_once;
  if (attr_once.need()) {
    if (cudaFuncSetAttribute(k_gemm_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(k_gemm_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(k_gemm_tc2, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return DKV_E_CUDA;
  }
  if (fused_out) *fused_out = false;
  GemmTcParams p;
  memset(&p, 0, sizeof(p));
  p.n = n;
  p.r_bound = r_bound;
  p.r_dev = r_dev;
  p.out = out;
  p.split_stride = static_cast<long long>(r_bound) * n;
  p.ldo = n;
  p.status = status;
  p.x_bf16 = x_bf16 ? 1 : 0;
  p.w_static = o.w_static ? 1 : 0;
  p.w_blocked = o.w_blocked ? 1 : 0;
  p.swiglu_out = o.swiglu_out;
  p.ld_u = o.ld_u;
  p.mask_id = -1;
  p.rs_src = o.scale.src;
  p.rs_parts = o.scale.parts;
  p.rs_ld = o.scale.ld;
  p.rs_inv_d = 1.f / static_cast<float>(o.scale.d);
  p.rs_eps = o.scale.eps;
  const int kb_total = ceil_div(k, GEMM_BK);
  p.kb_total = kb_total;
  if (o.xmaps_half) {
    // CTA pairs (cta_group::2): 512-row weight tiles, each CTA stages half of the row tile.  Used for
    // the unsplit SwiGLU launch, whose few CTAs are bound by the operand bytes an SM can take in.
    const int bi = o.row_tiles > 0 ? std::min(std::max(ceil_div(ceil_div(r_bound, o.row_tiles), 16) - 1, 0), N_BOX - 1)
                                   : pick_box(r_bound);
    const int br = box_rows(bi);
    GemmTcPlan plan = gemm_tc2_plan(br);
    const int splits = std::max(1, std::min(o.forced_splits, kb_total));
    p.kb_per_split = ceil_div(kb_total, splits);
    p.splits = splits;
    p.br = br;
    p.halves = 2;
    p.stages = plan.stages;
    p.stage_bytes = plan.stage_bytes;
    p.col_stride = plan.col_stride;
    p.n_bufs = plan.n_bufs;
    p.tmem_cols = plan.tmem_cols;
    p.r_tiles = ceil_div(r_bound, br);
    p.units = ceil_div(n, GEMM2_TILE_ROWS) * p.r_tiles * splits;
    const int grid = 2 * std::min(p.units, NUM_SMS / 2);
    // fused row tails: each CTA of a pair is a 256-column tile of its own; all units resident at once
    if (o.tail.mode != FUSE_NONE && !o.swiglu_out && p.units <= NUM_SMS / 2 &&
        2 * ceil_div(n, GEMM2_TILE_ROWS) * p.r_tiles <= MAX_TILE_COUNTERS) {
      set_tail(p, o.tail);
      if (fused_out) *fused_out = true;
    }
    launch_k(k_gemm_tc2, grid, GEMM_THREADS, plan.smem_bytes, st, tw, o.xmaps_half[bi], p);
    *splits_out = splits;
    *stride_out = p.split_stride;
    return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
  }
  int halves = 2;
  if (n <= GEMM_BM) halves = 1;
  int bi = pick_box(r_bound);
  int multi_splits = 0;
  if (r_bound > 256 && halves == 2 && o.forced_splits <= 0 && !o.head && !o.swiglu_out) {
    int t = 0;
    choose_multi_tile(n, k, r_bound, part_rows, &t, &multi_splits);
    bi = std::min(std::max(ceil_div(ceil_div(r_bound, t), 16) - 1, 0), N_BOX - 1);
  }
  const int br = box_rows(bi);
  GemmTcPlan plan = gemm_tc_plan(br, halves, 1);
  if (plan.smem_bytes < 116 * 1024) plan.smem_bytes = 116 * 1024;  // keep the SM to one CTA
  int splits = o.forced_splits > 0 ? o.forced_splits
                                   : (multi_splits > 0 ? multi_splits : choose_splits(n, k, r_bound, plan, part_rows));
  splits = std::min(splits, kb_total);
  while (splits > 1 && (splits - 1) * ceil_div(kb_total, splits) >= kb_total) --splits;
  p.kb_per_split = ceil_div(kb_total, splits);
  p.splits = splits;
  p.br = br;
  p.halves = plan.halves;
  p.stages = plan.stages;
  p.stage_bytes = plan.stage_bytes;
  p.col_stride = plan.col_stride;
  p.n_bufs = plan.n_bufs;
  p.tmem_cols = plan.tmem_cols;
  p.r_tiles = ceil_div(r_bound, br);
  p.units = ceil_div(n, GEMM_BM * plan.halves) * p.r_tiles * splits;
  p.head_mode = o.head ? 1 : 0;
  p.mask_id = o.head ? o.head->mask_id : -1;
  p.st_max = o.head ? o.head->st_max : nullptr;
  p.st_sum = o.head ? o.head->st_sum : nullptr;
  p.st_arg = o.head ? o.head->st_arg : nullptr;
  p.st_m2 = o.head ? o.head->st_m2 : nullptr;
  p.st_t = o.head ? o.head->st_t : nullptr;
  const int sms = sm_count();
  const int grid = std::min(p.units, sms);
  if (o.head) {
    // a CTA keeps the statistics of one row tile across its weight tiles
    if (p.r_tiles != 1 || splits != 1) return DKV_E_SHAPE;
    o.head->n_groups = 4 * grid;
  }
  // the CTAs of a tile wait for each other in the fused tail: every unit needs a resident CTA of its own
  if (o.tail.mode != FUSE_NONE && p.units <= sms && p.units <= MAX_TILE_COUNTERS) {
    set_tail(p, o.tail);
    if (fused_out) *fused_out = true;
  }
  if (plan.halves == 2) launch_k(k_gemm_tc<2>, grid, GEMM_THREADS, plan.smem_bytes, st, tw, xmaps[bi], p);
  else launch_k(k_gemm_tc<1>, grid, GEMM_THREADS, plan.smem_bytes, st, tw, xmaps[bi], p);
  *splits_out = splits;
  *stride_out = p.split_stride;
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

int gemm_f32(const float* x, const float* w, int n, int k, int r_bound, const int* r_dev, float* out,
             cudaStream_t st) {
  dim3 grid(ceil_div(n, F32_TILE), ceil_div(r_bound, F32_TILE));
  launch_k(k_gemm_f32, grid, 256, 0, st, x, w, out, r_bound, r_dev, n, k, n);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

// ------------------------------------------------------------- attention
template <typename T>
int attention_simt(const T* q, const T* ks, const T* vs, T* o, const int32_t* row_off, int batch, int rows_bound,
                   int seq_len, int hq, int hkv, int dh, cudaStream_t st, int kv_stride = 0) {
  const size_t smem = static_cast<size_t>(dh + seq_len) * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k_attn_simt<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return DKV_E_CUDA;
  }
  dim3 grid(rows_bound, hq, batch);
  launch_k((k_attn_simt<T>), grid, 128, smem, st, q, ks, vs, o, row_off, seq_len, hq, hkv, dh,
                                           1.0f / sqrtf(static_cast<float>(dh)), kv_stride > 0 ? kv_stride : seq_len);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

template <int DH, typename T>
int attention_mma_dh(const T* q, const T* ks, const T* vs, T* o, const int32_t* row_off, int batch, int rows_bound,
                     int seq_len, int hq, int hkv, cudaStream_t st, int kv_stride) {
  static PerDeviceOnce attr_once;
  if (attr_once.need()) {
    if (cudaFuncSetAttribute(k_attn_mma<DH, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnSmem<DH>::BYTES) !=
        cudaSuccess)
      return DKV_E_CUDA;
  }
  dim3 grid(ceil_div(rows_bound, ATT_BQ), hq, batch);
  const float scale_log2 = 1.4426950408889634f / sqrtf(static_cast<float>(DH));
  launch_k((k_attn_mma<DH, T>), grid, ATT_THREADS, AttnSmem<DH>::BYTES, st, q, ks, vs, o, row_off, seq_len, hq, hkv, scale_log2,
           kv_stride > 0 ? kv_stride : seq_len);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

// 16-bit activations: the tensor-core flash kernel
template <typename T>
int attention_16(const T* q, const T* ks, const T* vs, T* o, const int32_t* row_off, int batch, int rows_bound,
                 int seq_len, int hq, int hkv, int dh, cudaStream_t st, int kv_stride = 0) {
  if (dh == 128) return attention_mma_dh<128, T>(q, ks, vs, o, row_off, batch, rows_bound, seq_len, hq, hkv, st, kv_stride);
  if (dh == 64) return attention_mma_dh<64, T>(q, ks, vs, o, row_off, batch, rows_bound, seq_len, hq, hkv, st, kv_stride);
  return DKV_E_UNSUPPORTED;
}
inline int attention_any(const float* q, const float* ks, const float* vs, float* o, const int32_t* row_off,
                         int batch, int rows_bound, int seq_len, int hq, int hkv, int dh, cudaStream_t st, int kv_stride) {
  return attention_simt<float>(q, ks, vs, o, row_off, batch, rows_bound, seq_len, hq, hkv, dh, st, kv_stride);
}
inline int attention_any(const __nv_bfloat16* q, const __nv_bfloat16* ks, const __nv_bfloat16* vs, __nv_bfloat16* o,
                         const int32_t* row_off, int batch, int rows_bound, int seq_len, int hq, int hkv, int dh,
                         cudaStream_t st, int kv_stride) {
  return attention_16<__nv_bfloat16>(q, ks, vs, o, row_off, batch, rows_bound, seq_len, hq, hkv, dh, st, kv_stride);
}
inline int attention_any(const __half* q, const __half* ks, const __half* vs, __half* o, const int32_t* row_off,
                         int batch, int rows_bound, int seq_len, int hq, int hkv, int dh, cudaStream_t st, int kv_stride) {
  return attention_16<__half>(q, ks, vs, o, row_off, batch, rows_bound, seq_len, hq, hkv, dh, st, kv_stride);
}

// ----------------------------------------------------------- one forward
struct StepPlan {
  int mode;         // ACT_*
  int na_bound;     // per-sequence bound on active rows
  int nh_bound;     // per-sequence bound on head rows
  bool refresh;
  int kv_count;     // slots each query attends (the first kv_count of a sequence); 0 = all
};

// TW = weight element type, T = activation / cache element type
template <typename TW, typename T>
int run_forward(dkv_cache* c, const StepPlan& plan, const int32_t* tokens, float* conf, int32_t* pred,
                float* logits_dbg, cudaStream_t st) {
  const dkv_model* m = c->model;
  const dkv_model_desc& md = m->desc;
  const Dims& dm = c->dims;
  Arena& a = c->ar;
  const bool bf16 = md.dtype == DKV_BF16;
  const int R = dm.B * plan.na_bound;   // host bound on total active rows
  const int H = dm.B * plan.nh_bound;
  const int d = md.d_model, f = md.d_ffn, dq = m->d_q, dkv = m->d_kv, nqkv = m->n_qkv;
  const int* r_dev = a.row_off + dm.B;
  const int* h_dev = a.head_off + dm.B;
  const double es = static_cast<double>(m->esize);
  const bool x_bf16 = md.act_dtype == DKV_BF16;
  if (R <= 0) return DKV_OK;
  const int kv_count = plan.kv_count > 0 ? plan.kv_count : dm.L;
  int rc;

  // 16-bit modes: the operand of a projection that follows an RMSNorm is h .* gain, and the GEMM divides
  // by the row's RMS in its epilogue (`sc`: where the sums of squares of the current operand rows are).
  // The check mode keeps the normalised operand (its plain FMA GEMM has no epilogue).
  RowScale sc;
  float* const ssq = bf16 ? a.ssq : nullptr;
  const long long ssq_ld = dm.r_cap;
  auto scale_from = [&](int parts) {
    sc.src = a.ssq;
    sc.parts = parts;
    sc.ld = ssq_ld;
    sc.d = d;
    sc.eps = md.rms_eps;
  };

  auto gemm = [&](int cls, const void* w, const CUtensorMap* tw, XBuf xb, const void* x, int n, int k, int rb,
                  const int* rdev, float* out, int* splits, long long* stride, const GemmOpts& o = GemmOpts(),
                  bool* fused = nullptr) -> int {
    const double bytes = (static_cast<double>(n) * k + static_cast<double>(rb) * k) * es + 4.0 * rb * n;
    Launch l(c, st, cls, bytes, 2.0 * rb * n * static_cast<double>(k));
    if (fused) *fused = false;
    if (bf16) {
      GemmOpts ob = o;
      ob.w_blocked = m->w_blocked;
      return gemm_tc(*tw, c->xmaps[xb], n, k, rb, rdev, out, dm.part_rows, a.status, x_bf16, st, splits, stride, ob, fused);
    }
    *splits = 1;
    *stride = 0;
    return gemm_f32(static_cast<const float*>(x), static_cast<const float*>(w), n, k, rb, rdev, out, st);
  };
  // residual + norm around the O and down projections: fused into the GEMM when the launch is one wave
  auto resid_opts = [&](const float* gain) {
    GemmOpts o;
    if (c->fuse_tails & 2) {
      o.tail.mode = FUSE_RESID;
      o.tail.tile_cnt = a.tile_cnt;
      o.tail.cnt_set = &c->tail_cnt_set;
      o.tail.wait_cycles = c->tail_wait_cycles;
      o.tail.extra = c->tail_extra;
      o.tail.h = a.h;
      o.tail.gain = gain;
      o.tail.xn_out = a.xn;
      o.tail.ssq_out = a.ssq;
      o.tail.ssq_ld = ssq_ld;
    }
    return o;
  };
  auto resid_after = [&](bool fused, int splits, long long stride, const float* gain) {
    if (fused) {
      scale_from(ceil_div(d, d <= GEMM_BM ? GEMM_BM : 2 * GEMM_BM));   // one partial sum per weight tile
      return;
    }
    Launch lk(c, st, PC_RESID_NORM, R * d * (4.0 * splits + 8.0 + es), 0);
    launch_k((k_resid_norm<T>), R, 256, 0, st, a.h, a.part, splits, stride, r_dev, gain, md.rms_eps, d,
             static_cast<T*>(a.xn), ssq);
    scale_from(1);
  };

  // More than one row tile (the full steps): the launch is bound by the operand bytes an SM takes in
  // and by the power cap, and a CTA pair (each CTA stages half of the row tile) takes in a quarter
  // less per flop: QKV 57 -> 55 us, O 42 -> 40, down 65 -> 62 at 512 LLaDA-shaped rows.  Row tiles and
  // K splits from the estimate for pairs; `one_wave`: prefer a plan that leaves every unit resident,
  // so that the residual tail can be fused.
  auto pair_plan = [&](GemmOpts& o, XBuf xb, int n, int k, bool one_wave) {
    if (!bf16 || R <= 256 || !m->gu_pair) return;
    int t = 0, sp = 0;
    choose_pairs(n, k, R, dm.part_rows, one_wave, &t, &sp);
    if (t == 0 && one_wave) choose_pairs(n, k, R, dm.part_rows, false, &t, &sp);
    if (t == 0) return;
    o.xmaps_half = c->xmaps_half[xb];
    o.row_tiles = t;
    o.forced_splits = sp;
  };

  {
    Launch l(c, st, PC_EMBED, R * d * (es + 4.0 + es), 0);
    launch_k((k_embed_norm<TW, T>), R, 256, 0, st, static_cast<const TW*>(m->embed), tokens, a.act_idx, r_dev,
                                        m->layers[0].attn_norm, md.rms_eps, d, a.h, static_cast<T*>(a.xn), ssq);
    scale_from(1);
  }
  if (!bf16) sc = RowScale();
  const size_t slot_layer = static_cast<size_t>(dm.B) * md.n_kv_heads * dm.L * md.head_dim;
  auto qkv_opts = [&](int l) {
    GemmOpts o;
    o.scale = sc;
    // (with several row tiles the launch is unsplit and compute-bound; there a tail through scratch
    // costs more than the row kernel that overlaps with the next launch's weight prefetch)
    if ((c->fuse_tails & 1) && R <= 256) {
      o.tail.mode = FUSE_QKV;
      o.tail.tile_cnt = a.tile_cnt;
      o.tail.cnt_set = &c->tail_cnt_set;
      o.tail.wait_cycles = c->tail_wait_cycles;
      o.tail.extra = c->tail_extra;
      o.tail.act_idx = a.act_idx;
      o.tail.rope_tab = a.rope_tab;
      o.tail.seq_len = dm.L;
      o.tail.n_q_heads = md.n_q_heads;
      o.tail.n_kv_heads = md.n_kv_heads;
      o.tail.head_dim = md.head_dim;
      o.tail.q_out = a.qb;
      o.tail.k_slots = static_cast<T*>(a.k_slots) + l * slot_layer;
      o.tail.v_slots = static_cast<T*>(a.v_slots) + l * slot_layer;
    }
    return o;
  };
  for (int l = 0; l < md.n_layers; ++l) {
    const dkv_layer_weights& lw = m->layers[l];
    const LayerMaps* lm = bf16 ? &m->maps[l] : nullptr;
    T* ks = static_cast<T*>(a.k_slots) + l * slot_layer;
    T* vs = static_cast<T*>(a.v_slots) + l * slot_layer;
    int splits;
    long long stride;
    bool fused;
    GemmOpts oq = qkv_opts(l);
    pair_plan(oq, XB_XN, nqkv, d, false);
    rc = gemm(PC_GEMM_QKV, lw.wqkv, lm ? &lm->wqkv : nullptr, XB_XN, a.xn, nqkv, d, R, r_dev, a.part, &splits, &stride,
              oq, &fused);
    if (rc) return rc;
    if (!fused) {
      Launch lk(c, st, PC_QKV_POST, R * (nqkv * 4.0 * splits + nqkv * es), 0);
      const int units = (md.n_q_heads + md.n_kv_heads) * (md.head_dim / 8) + dkv / 4;
      // few enough blocks that the whole grid is resident at once: a kernel launched behind it with
      // programmatic dependent launch can then start (and prefetch weights) while this one runs
      dim3 grid(R, std::max(1, std::min(ceil_div(units, 256), 1024 / std::max(R, 1))));
      launch_k((k_qkv_rope_scatter<T>), grid, 256, 0, st, a.part, splits, stride, r_dev, a.act_idx, a.rope_tab, dm.L,
                                                   md.n_q_heads, md.n_kv_heads, md.head_dim, static_cast<T*>(a.qb),
                                                   ks, vs);
    }
    {
      const double fl = 4.0 * R * dm.L * dq;
      const double by = 2.0 * dm.B * dm.L * dkv * es + 2.0 * R * dq * es;
      Launch lk(c, st, PC_ATTN, by, fl);
      if (bf16 && c->attn_tc)
        rc = attention_tc(kv_count < dm.L ? c->attn_maps_prompt : c->attn_maps, a.ao, a.row_off, dm.B, plan.na_bound,
                          kv_count, md.n_q_heads, md.n_kv_heads, l * dm.B * md.n_kv_heads, x_bf16, a.status, st);
      else
        rc = attention_any(static_cast<const T*>(a.qb), static_cast<const T*>(ks), static_cast<const T*>(vs),
                           static_cast<T*>(a.ao), a.row_off, dm.B, plan.na_bound, kv_count, md.n_q_heads, md.n_kv_heads,
                           md.head_dim, st, dm.L);
      if (rc) return rc;
    }
    const float* next_gain = (l + 1 < md.n_layers) ? m->layers[l + 1].attn_norm : m->final_norm;
    GemmOpts oo = resid_opts(lw.ffn_norm);
    pair_plan(oo, XB_AO, d, dq, oo.tail.mode != FUSE_NONE);
    rc = gemm(PC_GEMM_O, lw.wo, lm ? &lm->wo : nullptr, XB_AO, a.ao, d, dq, R, r_dev, a.part, &splits, &stride, oo, &fused);
    if (rc) return rc;
    resid_after(fused, splits, stride, lw.ffn_norm);
    // The SwiGLU epilogue needs the whole K range in one unit (no split-K).  With one row tile that
    // wins although the 2f/256 units may fill the SMs badly (no partials, one launch less); with more
    // row tiles only when the units come out as nearly whole waves.
    const int gu_workers = m->gu_pair ? NUM_SMS / 2 : NUM_SMS;                  // CTA pairs or CTAs
    const int gu_tiles_n = ceil_div(2 * f, m->gu_pair ? GEMM2_TILE_ROWS : 2 * GEMM_BM);
    int gu_rt = ceil_div(R, 256);                                              // row tiles of the fused launch
    double gu_fill = 0.0;
    for (int t = ceil_div(R, 256); t <= ceil_div(R, 256) + (m->gu_pair && R > 256 ? 1 : 0); ++t) {
      const int units = gu_tiles_n * t;                                        // one more, narrower tile may
      const double fill = units / (std::ceil(units / static_cast<double>(gu_workers)) * gu_workers);   // fill the waves
      if (fill > gu_fill + 0.1) {
        gu_fill = fill;
        gu_rt = t;
      }
    }
    if (bf16 && m->gu_blk && (R <= 256 || gu_fill >= 0.85)) {
      // gate and up rows of a feature sit in the two halves of one weight tile: no split-K, SwiGLU in
      // the epilogue, the product written once as 16-bit
      const double bytes = (2.0 * f * d + static_cast<double>(R) * d) * es + static_cast<double>(R) * f * es;
      Launch lk(c, st, PC_GEMM_GU, bytes, 4.0 * R * f * static_cast<double>(d));
      GemmOpts o;
      o.forced_splits = 1;
      o.scale = sc;
      o.swiglu_out = a.ub;
      o.ld_u = f;
      o.xmaps_half = m->gu_pair ? c->xmaps_half[XB_XN] : nullptr;
      o.row_tiles = R > 256 ? gu_rt : 0;
      o.w_blocked = m->w_blocked;
      rc = gemm_tc(lm->wgu, c->xmaps[XB_XN], 2 * f, d, R, r_dev, a.part, dm.part_rows, a.status, x_bf16, st, &splits,
                   &stride, o);
      if (rc) return rc;
    } else {
      GemmOpts o;
      o.scale = sc;
      rc = gemm(PC_GEMM_GU, lw.wgu, lm ? &lm->wgu : nullptr, XB_XN, a.xn, 2 * f, d, R, r_dev, a.part, &splits, &stride, o);
      if (rc) return rc;
      Launch lk(c, st, PC_SWIGLU, R * f * (8.0 * splits + es), 0);
      dim3 grid(R, std::max(1, std::min(ceil_div(f / 4, 256), 1024 / std::max(R, 1))));
      launch_k((k_swiglu<T>), grid, 256, 0, st, a.part, splits, stride, r_dev, f, bf16 ? m->gu_blk : 0,
               static_cast<T*>(a.ub));
    }
    GemmOpts od = resid_opts(next_gain);
    pair_plan(od, XB_U, d, f, od.tail.mode != FUSE_NONE);
    rc = gemm(PC_GEMM_DOWN, lw.wd, lm ? &lm->wd : nullptr, XB_U, a.ub, d, f, R, r_dev, a.part, &splits, &stride, od, &fused);
    if (rc) return rc;
    resid_after(fused, splits, stride, next_gain);
  }
  if (H <= 0) return DKV_OK;
  {
    Launch lk(c, st, PC_HEAD_STATS, 2.0 * H * d * es, 0);
    launch_k((k_head_gather<T>), H, 256, 0, st, static_cast<const T*>(a.xn), a.head_row, h_dev, d, static_cast<T*>(a.xh),
             static_cast<const float*>(bf16 ? sc.src : nullptr), sc.parts, sc.ld, md.rms_eps, a.head_rs);
  }
  RowScale head_sc;
  if (bf16) {
    head_sc.src = a.head_rs;     // ready factors, one per head row
    head_sc.d = d;
  }
  // 16-bit modes, no logits requested: the head GEMM's epilogue reduces every 32 token ids to
  // (max, argmax, sum exp) with warp shuffles, joins them over the weight tiles of a CTA, and a small
  // kernel combines the CTAs' entries; the logits are never written.  Otherwise (check mode, or the caller wants the logits) they are materialised.
  // (the warp-shuffle reduction costs time in proportion to the head rows: with many of them the
  // GEMM is compute-bound and writing the logits is the cheaper way)
  if (bf16 && !logits_dbg && H <= 128) {
    int splits;
    long long stride;
    const int score = c->policy.score;
    HeadStats hs;
    hs.mask_id = md.mask_id;
    hs.st_max = a.st_max;
    hs.st_sum = a.st_sum;
    hs.st_arg = a.st_arg;
    hs.st_m2 = score ? a.st_m2 : nullptr;
    hs.st_t = score ? a.st_t : nullptr;
    {
      const double bytes = (static_cast<double>(md.vocab) * d + static_cast<double>(H) * d) * es;
      Launch lk(c, st, PC_GEMM_HEAD, bytes, 2.0 * H * md.vocab * static_cast<double>(d));
      GemmOpts o;
      o.forced_splits = 1;
      o.head = &hs;
      o.scale = head_sc;
      o.w_blocked = m->w_blocked;
      rc = gemm_tc(m->head_map, c->xmaps[XB_XH], md.vocab, d, H, h_dev, nullptr, dm.part_rows, a.status, x_bf16, st,
                   &splits, &stride, o);
      if (rc) return rc;
    }
    Launch lk(c, st, PC_HEAD_STATS, 24.0 * H * hs.n_groups, 0);
    static PerDeviceOnce comb_once;
    if (comb_once.need() &&
        cudaFuncSetAttribute(k_head_combine, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024) != cudaSuccess)
      return DKV_E_CUDA;
    launch_k(k_head_combine, H, 256, 100 * 1024, st, static_cast<const float*>(a.st_max), static_cast<const float*>(a.st_sum),
             static_cast<const int*>(a.st_arg), static_cast<const float*>(a.st_m2), static_cast<const float*>(a.st_t),
             score, hs.n_groups, H, h_dev, a.head_pos, conf, pred);
    return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
  }
  float* logits = logits_dbg ? logits_dbg : a.logits;
  {
    int splits;
    long long stride;
    const double bytes = (static_cast<double>(md.vocab) * d + static_cast<double>(H) * d) * es + 4.0 * H * md.vocab;
    Launch lk(c, st, PC_GEMM_HEAD, bytes, 2.0 * H * md.vocab * static_cast<double>(d));
    if (bf16) {
      GemmOpts o;
      o.forced_splits = 1;
      o.scale = head_sc;
      o.w_blocked = m->w_blocked;
      rc = gemm_tc(m->head_map, c->xmaps[XB_XH], md.vocab, d, H, h_dev, logits, dm.part_rows, a.status, x_bf16, st,
                   &splits, &stride, o);
    } else {
      rc = gemm_f32(static_cast<const float*>(a.xh), static_cast<const float*>(m->head), md.vocab, d, H, h_dev,
                    logits, st);
    }
    if (rc) return rc;
  }
  {
    Launch lk(c, st, PC_HEAD_STATS, 8.0 * H * md.vocab, 0);
    launch_k(k_head_stats, H, 512, 0, st, logits, h_dev, a.head_pos, md.vocab, md.mask_id, c->policy.score, conf, pred);
  }
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

StepPlan plan_step(dkv_cache* c, int k, int cand_lo, int cand_hi, int rows_bound) {
  const dkv_policy& pol = c->policy;
  const Dims& dm = c->dims;
  const int t = c->step + 1;
  const int rb = rows_bound < 0 ? dm.L : std::min(rows_bound, dm.L);
  StepPlan p;
  bool interval_hit = false;
  if (pol.refresh_interval > 0 && pol.kind != DKV_POLICY_PREFILL && t > 1)
    interval_hit = ((t - c->last_refresh) % pol.refresh_interval) == 0;
  int scope = -1;
  p.kv_count = 0;
  if (t == 1 && pol.isolated_prefill && dm.P > 0) scope = DKV_REFRESH_DECODED_ONLY;   // the prompt had its own pass
  else if (pol.kind == DKV_POLICY_NONE || t == 1) scope = DKV_REFRESH_ALL;
  else if (c->pending_refresh >= 0) scope = c->pending_refresh;
  else if (interval_hit) scope = (pol.kind == DKV_POLICY_PD) ? DKV_REFRESH_DECODED_ONLY : DKV_REFRESH_ALL;
  p.refresh = scope >= 0;
  if (scope == DKV_REFRESH_ALL) {
    p.mode = ACT_FULL;
    p.na_bound = dm.L;
  } else if (scope == DKV_REFRESH_DECODED_ONLY || pol.kind == DKV_POLICY_PREFILL) {
    p.mode = ACT_GEN_ONLY;
    p.na_bound = dm.G;
    p.refresh = scope >= 0;
  } else if (pol.kind == DKV_POLICY_GREEDY) {
    p.mode = ACT_GREEDY;
    p.na_bound = std::min(dm.L, 2 * k + k * (pol.window + 1));
  } else {
    p.mode = ACT_FROM_MASK;
    p.na_bound = pol.delay ? c->prev_rows_bound : rb;
    p.na_bound = std::min(std::max(p.na_bound, 0), dm.L);
  }
  if (pol.kind == DKV_POLICY_GREEDY) p.nh_bound = k;
  else p.nh_bound = std::min(std::min(rb, std::max(0, cand_hi - cand_lo)), pol.shift ? dm.L : p.na_bound);
  if (pol.shift == 2) p.na_bound = std::min(dm.L, 2 * p.na_bound);        // each active row brings its left neighbour
  if (pol.shift) p.na_bound = std::min(dm.L, p.na_bound + p.nh_bound);   // the rows left of the candidates join
  return p;
}

int do_step(dkv_cache* c, const int32_t* tokens, const uint8_t* masked, const int32_t* next_pos, int k, int cand_lo,
            int cand_hi, int rows_bound, float* conf, int32_t* pred, float* logits_dbg, cudaStream_t st) {
  const dkv_policy& pol = c->policy;
  const Dims& dm = c->dims;
  Arena& a = c->ar;
  if (k < 1 || k > dm.kmax) return DKV_E_SHAPE;
  if (cand_lo < 0 || cand_hi > dm.L || cand_lo > cand_hi) return DKV_E_SHAPE;
  if (pol.kind == DKV_POLICY_GREEDY && !next_pos) return DKV_E_INVALID_ARG;
  // D_{t-1} was stored as [batch, k] with the previous step's k: the window rule reads it with the same k
  if (pol.kind == DKV_POLICY_GREEDY && c->have_dprev && k != c->prev_k) return DKV_E_SHAPE;
  if (pol.shift && cand_lo < 1) return DKV_E_SHAPE;   // position 0 has no row to its left
  StepPlan plan = plan_step(c, k, cand_lo, cand_hi, rows_bound);
  if (plan.nh_bound > dm.hmax) return DKV_E_SHAPE;
  const int t = c->step + 1;
  const dkv_model_desc& mdesc = c->model->desc;

  // one pass = compaction of the pass's rows, then the forward over them
  auto run_pass = [&](const StepPlan& pl, int lo, int hi) -> int {
    CompactParams cp;
    memset(&cp, 0, sizeof(cp));
    cp.mode = pl.mode;
    cp.batch = dm.B;
    cp.seq_len = dm.L;
    cp.prompt_len = dm.P;
    cp.mask_src = (pl.mode == ACT_FROM_MASK) ? (pol.delay ? a.mask_buf[(t - 1) & 1] : masked) : nullptr;
    cp.mask_cur = masked;
    cp.mask_store = a.mask_buf[t & 1];
    cp.d_cur = next_pos;
    cp.d_prev = c->have_dprev ? a.d_buf[(t - 1) & 1] : nullptr;
    cp.d_store = next_pos ? a.d_buf[t & 1] : nullptr;
    cp.k = k;
    cp.w_lo = (pol.window + 1) / 2;   // ceil(w/2)
    cp.w_hi = pol.window / 2;         // floor(w/2)
    cp.center_cur = pol.window_center == DKV_CENTER_CUR;
    cp.head_from_d = pol.kind == DKV_POLICY_GREEDY;
    cp.shift = pol.shift ? 1 : 0;
    cp.right = pol.shift == 2;
    cp.cand_lo = lo;
    cp.cand_hi = hi;
    cp.step = t;
    cp.rows_bound = pl.na_bound;
    cp.head_bound = pl.nh_bound;
    cp.act_idx = a.act_idx;
    cp.row_off = a.row_off;
    cp.inv = a.inv;
    cp.head_row = a.head_row;
    cp.head_pos = a.head_pos;
    cp.head_off = a.head_off;
    cp.written_step = a.written_step;
    cp.conf = conf;
    cp.pred = pred;
    cp.status = a.status;
    cp.active_total = reinterpret_cast<unsigned long long*>(a.status + 2);
    {
      Launch l(c, st, PC_COMPACT, dm.B * dm.L * 20.0, 0);
      launch_k(k_compact, dm.B, 256, 0, st, cp);
    }
    if (cudaGetLastError() != cudaSuccess) return DKV_E_CUDA;
    if (mdesc.dtype == DKV_F32) return run_forward<float, float>(c, pl, tokens, conf, pred, logits_dbg, st);
    if (mdesc.act_dtype == DKV_F16) return run_forward<__nv_bfloat16, __half>(c, pl, tokens, conf, pred, logits_dbg, st);
    return run_forward<__nv_bfloat16, __nv_bfloat16>(c, pl, tokens, conf, pred, logits_dbg, st);
  };

  int rc;
  if (t == 1 && pol.isolated_prefill && dm.P > 0) {
    // Prefill phase on its own (Sec. 3.3): the prompt rows attend to the prompt slots only and
    // write their K/V; no head.  The generation rows follow in the step's regular pass.
    StepPlan pre;
    pre.mode = ACT_PROMPT_ONLY;
    pre.na_bound = dm.P;
    pre.nh_bound = 0;
    pre.refresh = true;
    pre.kv_count = dm.P;
    rc = run_pass(pre, 0, 0);
    if (rc) return rc;
  }
  rc = run_pass(plan, cand_lo, cand_hi);
  if (rc) return rc;
  c->step = t;
  if (plan.refresh) c->last_refresh = t;
  c->pending_refresh = -1;
  c->prev_rows_bound = rows_bound < 0 ? dm.L : std::min(rows_bound, dm.L);
  c->have_dprev = next_pos != nullptr;
  c->prev_k = k;
  c->last_stream = st;
  c->stats.steps += 1;
  if (plan.refresh) c->stats.refresh_steps += 1;
  c->stats.total_rows += static_cast<int64_t>(dm.B) * dm.L;
  return DKV_OK;
}

}  // namespace

// =========================================================================
// C ABI
// =========================================================================
extern "C" {

const char* dkv_strerror(int status) {
  switch (status) {
    case DKV_OK: return "ok";
    case DKV_E_INVALID_ARG: return "invalid argument";
    case DKV_E_SHAPE: return "unsupported or inconsistent shape";
    case DKV_E_STATE: return "handle in the wrong state";
    case DKV_E_NOMEM: return "arena too small";
    case DKV_E_CUDA: return "CUDA call failed";
    case DKV_E_UNSUPPORTED: return "unsupported configuration";
    case DKV_E_DEVICE: return "a kernel reported a problem (see the status word)";
    default: return "unknown status";
  }
}

size_t dkv_model_bytes(const dkv_model_desc* desc) {
  if (!desc || desc->dtype != DKV_BF16 || desc->act_dtype != DKV_F16) return 0;
  const size_t d = desc->d_model, f = desc->d_ffn;
  const size_t dq = static_cast<size_t>(desc->n_q_heads) * desc->head_dim;
  const size_t dkv = static_cast<size_t>(desc->n_kv_heads) * desc->head_dim;
  size_t per_layer = 0;
  per_layer += align_up(blocked_bytes(dq + 2 * dkv, d), 256) + align_up(blocked_bytes(d, dq), 256) +
               align_up(blocked_bytes(2 * f, d), 256) + align_up(blocked_bytes(d, f), 256);
  return per_layer * desc->n_layers + align_up(blocked_bytes(desc->vocab, d), 256) + 256;
}

int dkv_model_create(const dkv_model_desc* desc, const dkv_weights* w, void* arena, size_t arena_bytes, void* stream,
                     dkv_model** out) {
  if (!desc || !w || !out || !w->layers || !w->embed || !w->head || !w->final_norm) return DKV_E_INVALID_ARG;
  if (desc->dtype != DKV_F32 && desc->dtype != DKV_BF16) return DKV_E_UNSUPPORTED;
  if (desc->dtype == DKV_F32 && desc->act_dtype != DKV_F32) return DKV_E_UNSUPPORTED;
  if (desc->dtype == DKV_BF16 && desc->act_dtype != DKV_BF16 && desc->act_dtype != DKV_F16) return DKV_E_UNSUPPORTED;
  if (desc->n_layers < 1 || desc->d_model < 8 || desc->n_q_heads < 1 || desc->n_kv_heads < 1 || desc->d_ffn < 8 ||
      desc->vocab < 2)
    return DKV_E_SHAPE;
  if (desc->head_dim != 64 && desc->head_dim != 128) return DKV_E_SHAPE;
  if (desc->n_q_heads % desc->n_kv_heads) return DKV_E_SHAPE;
  if (desc->d_model % 8 || desc->d_ffn % 8) return DKV_E_SHAPE;
  if (desc->mask_id < 0 || desc->mask_id >= desc->vocab) return DKV_E_SHAPE;
  const bool f16 = desc->act_dtype == DKV_F16;
  if (f16) {
    if (!arena || reinterpret_cast<uintptr_t>(arena) % 256) return DKV_E_INVALID_ARG;
    if (arena_bytes < dkv_model_bytes(desc)) return DKV_E_NOMEM;
  }
  dkv_model* m = new (std::nothrow) dkv_model();
  if (!m) return DKV_E_NOMEM;
  m->desc = *desc;
  m->embed = w->embed;
  m->head = w->head;
  m->final_norm = w->final_norm;
  m->d_q = desc->n_q_heads * desc->head_dim;
  m->d_kv = desc->n_kv_heads * desc->head_dim;
  m->n_qkv = m->d_q + 2 * m->d_kv;
  m->esize = desc->dtype == DKV_BF16 ? 2 : 4;
  m->asize = desc->act_dtype == DKV_F32 ? 4 : 2;
  m->layers.assign(w->layers, w->layers + desc->n_layers);
  for (const dkv_layer_weights& lw : m->layers) {
    if (!lw.wqkv || !lw.wo || !lw.wgu || !lw.wd || !lw.attn_norm || !lw.ffn_norm) {
      delete m;
      return DKV_E_INVALID_ARG;
    }
  }
  if (desc->dtype == DKV_BF16) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* cur = static_cast<uint8_t*>(arena);
    // fp16 mode: the GEMMs read an fp16 copy of each matrix (tcgen05 wants both operands in one format)
    m->gu_blk = (f16 && desc->d_ffn % 128 == 0) ? 128 : 0;
    m->gu_pair = m->gu_blk && desc->d_ffn % 256 == 0;
    m->w_blocked = f16;
    m->maps.resize(desc->n_layers);
    int rc = DKV_OK;
    const long long d = desc->d_model, f = desc->d_ffn;
    // fp16 mode: the layers' matrices and the head are copied into 128 x 64 blocks (gate/up regrouped on the way);
    // bf16 activations: the caller's row-major matrices are read in place
    auto layer_map = [&](CUtensorMap* tm, const void* src, long long rows, long long k, int gu_f, int gu_blk) -> int {
      if (!f16) return make_tmap(tm, src, rows, k, GEMM_BM, false);
      __half* dst = reinterpret_cast<__half*>(cur);
      cur += align_up(blocked_bytes(rows, k), 256);
      dim3 grid(static_cast<unsigned>(ceil_div(static_cast<int>(k), GEMM_BK)), static_cast<unsigned>(ceil_div(static_cast<int>(rows), GEMM_BM)));
      k_block_f16<<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src), dst, static_cast<int>(rows),
                                        static_cast<int>(k), gu_f, gu_blk);
      return make_tmap_blocked(tm, dst, rows, k);
    };
    for (int l = 0; l < desc->n_layers && rc == DKV_OK; ++l) {
      const dkv_layer_weights& lw = m->layers[l];
      rc = layer_map(&m->maps[l].wqkv, lw.wqkv, m->n_qkv, d, 0, 0);
      if (!rc) rc = layer_map(&m->maps[l].wo, lw.wo, d, m->d_q, 0, 0);
      if (!rc) rc = layer_map(&m->maps[l].wgu, lw.wgu, 2 * f, d, static_cast<int>(f), m->gu_blk);
      if (!rc) rc = layer_map(&m->maps[l].wd, lw.wd, d, f, 0, 0);
    }
    if (!rc) rc = layer_map(&m->head_map, m->head, desc->vocab, d, 0, 0);   // (blocked too: 181 -> 173 us per launch)
    if (!rc && cudaGetLastError() != cudaSuccess) rc = DKV_E_CUDA;
    if (rc) {
      delete m;
      return rc;
    }
  }
  set_live(g_live_models, m, true);
  *out = m;
  return DKV_OK;
}

int dkv_model_destroy(dkv_model* m) {
  if (!m) return DKV_OK;
  if (!live_model(m)) return DKV_E_STATE;
  set_live(g_live_models, m, false);
  delete m;
  return DKV_OK;
}

size_t dkv_cache_bytes(const dkv_model* m, int batch, int seq_len, const dkv_policy* policy) {
  if (!m || !live_model(m) || batch < 1 || seq_len < 1) return 0;
  Dims d = make_dims(m, batch, seq_len, 0, policy);
  Arena a;
  carve(m, d, nullptr, &a);
  return a.total;
}

int dkv_init_cache(const dkv_model* m, int batch, int seq_len, int prompt_len, const dkv_policy* policy, void* arena,
                   size_t arena_bytes, void* stream, dkv_cache** out) {
  if (!m || !policy || !arena || !out) return DKV_E_INVALID_ARG;
  if (!live_model(m)) return DKV_E_STATE;
  if (batch < 1 || seq_len < 1 || prompt_len < 0 || prompt_len > seq_len) return DKV_E_SHAPE;
  if (policy->kind < DKV_POLICY_NONE || policy->kind > DKV_POLICY_GREEDY) return DKV_E_INVALID_ARG;
  if (policy->refresh_interval < 0 || policy->window < 0) return DKV_E_INVALID_ARG;
  if (policy->score < DKV_SCORE_MAXPROB || policy->score > DKV_SCORE_NEG_ENTROPY) return DKV_E_INVALID_ARG;
  if (policy->shift < 0 || policy->shift > 2) return DKV_E_INVALID_ARG;
  if (policy->isolated_prefill && policy->kind != DKV_POLICY_PREFILL && policy->kind != DKV_POLICY_PD)
    return DKV_E_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(arena) % 256) return DKV_E_INVALID_ARG;
  if (static_cast<long long>(batch) * seq_len > (1LL << 30)) return DKV_E_SHAPE;
  dkv_cache* c = new (std::nothrow) dkv_cache();
  if (!c) return DKV_E_NOMEM;
  c->model = m;
  c->policy = *policy;
  c->dims = make_dims(m, batch, seq_len, prompt_len, policy);
  carve(m, c->dims, static_cast<uint8_t*>(arena), &c->ar);
  if (c->ar.total > arena_bytes) {
    delete c;
    return DKV_E_NOMEM;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dkv_model_desc& md = m->desc;
  Arena& a = c->ar;
  if (md.dtype == DKV_BF16) {
    int rc = DKV_OK;
    for (int i = 0; i < N_BOX && !rc; ++i) {
      const bool h = md.act_dtype == DKV_F16;
      rc = make_tmap(&c->xmaps[XB_XN][i], a.xn, c->dims.r_cap, md.d_model, box_rows(i), h);
      if (!rc) rc = make_tmap(&c->xmaps_half[XB_XN][i], a.xn, c->dims.r_cap, md.d_model, box_rows(i) / 2, h);
      if (!rc) rc = make_tmap(&c->xmaps[XB_AO][i], a.ao, c->dims.r_cap, m->d_q, box_rows(i), h);
      if (!rc) rc = make_tmap(&c->xmaps_half[XB_AO][i], a.ao, c->dims.r_cap, m->d_q, box_rows(i) / 2, h);
      if (!rc) rc = make_tmap(&c->xmaps[XB_U][i], a.ub, c->dims.r_cap, md.d_ffn, box_rows(i), h);
      if (!rc) rc = make_tmap(&c->xmaps_half[XB_U][i], a.ub, c->dims.r_cap, md.d_ffn, box_rows(i) / 2, h);
      if (!rc) rc = make_tmap(&c->xmaps[XB_XH][i], a.xh, c->dims.h_cap, md.d_model, box_rows(i), h);
    }
    c->attn_tc = false;
    if (!rc && md.head_dim == ATC_DH && md.n_q_heads / md.n_kv_heads <= ATC_M) {
      const long long kv_heads = static_cast<long long>(md.n_layers) * batch * md.n_kv_heads;
      const bool h16 = md.act_dtype == DKV_F16;
      rc = make_attn_maps(&c->attn_maps, a.qb, c->dims.r_cap, a.k_slots, a.v_slots, kv_heads, seq_len, seq_len,
                          md.n_q_heads, md.n_kv_heads, h16);
      if (!rc && policy->isolated_prefill && prompt_len > 0 && prompt_len < seq_len)
        rc = make_attn_maps(&c->attn_maps_prompt, a.qb, c->dims.r_cap, a.k_slots, a.v_slots, kv_heads, prompt_len,
                            seq_len, md.n_q_heads, md.n_kv_heads, h16);
      c->attn_tc = rc == DKV_OK;
    }
    if (rc) {
      delete c;
      return rc;
    }
  }
  const size_t BL = static_cast<size_t>(batch) * seq_len;
  cudaMemsetAsync(a.status, 0, 256, st);
  cudaMemsetAsync(a.tile_cnt, 0, 2 * MAX_TILE_COUNTERS * 4, st);
  cudaMemsetAsync(a.written_step, 0, BL * 4, st);
  cudaMemsetAsync(a.mask_buf[0], 0, BL, st);
  cudaMemsetAsync(a.mask_buf[1], 0, BL, st);
  cudaMemsetAsync(a.row_off, 0, (batch + 1) * 4, st);
  cudaMemsetAsync(a.head_off, 0, (batch + 1) * 4, st);
  // activation buffers feed TMA boxes that may cover rows no kernel wrote yet
  cudaMemsetAsync(a.xn, 0, c->dims.r_cap * md.d_model * m->asize, st);
  cudaMemsetAsync(a.ao, 0, c->dims.r_cap * m->d_q * m->asize, st);
  cudaMemsetAsync(a.ub, 0, c->dims.r_cap * md.d_ffn * m->asize, st);
  cudaMemsetAsync(a.xh, 0, c->dims.h_cap * md.d_model * m->asize, st);
  {
    const int half = md.head_dim / 2;
    const int n = seq_len * half;
    k_rope_table<<<ceil_div(n, 256), 256, 0, st>>>(a.rope_tab, seq_len, half, static_cast<double>(md.rope_theta));
  }
  if (cudaGetLastError() != cudaSuccess) {
    delete c;
    return DKV_E_CUDA;
  }
  // read per handle (not once per process), so that a test can build handles of both kinds
  c->fuse_tails = env_int("DKV_FUSE_TAILS", 3);
  c->tail_wait_cycles = GEMM_WAIT_CYCLES;
  c->tail_extra = 0;
  c->tail_cnt_set = 0;
  c->step = 0;
  c->last_refresh = 1;
  c->pending_refresh = -1;
  c->prev_rows_bound = seq_len;
  c->have_dprev = false;
  c->prev_k = 0;
  c->last_stream = st;
  memset(&c->stats, 0, sizeof(c->stats));
  c->stats.cache_bytes = 2LL * md.n_layers * batch * md.n_kv_heads * seq_len * md.head_dim * m->asize;
  c->profiling = false;
  c->ev_used = 0;
  memset(c->prof, 0, sizeof(c->prof));
  for (int i = 0; i < PC_COUNT; ++i) strncpy(c->prof[i].name, PROF_NAMES[i], sizeof(c->prof[i].name) - 1);
  set_live(g_live_caches, c, true);
  *out = c;
  return DKV_OK;
}

int dkv_cache_destroy(dkv_cache* c) {
  if (!c) return DKV_OK;
  {
    std::lock_guard<std::mutex> lk(g_live_mu);
    if (!g_live_caches.count(c)) return DKV_E_STATE;
    g_live_caches.erase(c);
  }
  for (ProfEvent& e : c->events) {
    cudaEventDestroy(e.a);
    cudaEventDestroy(e.b);
  }
  delete c;
  return DKV_OK;
}

int dkv_step(dkv_cache* c, const int32_t* tokens, const uint8_t* masked, const int32_t* next_pos, int k, int cand_lo,
             int cand_hi, int rows_bound, float* conf, int32_t* pred, float* logits_dbg, void* stream) {
  if (!c || !tokens || !masked || !conf || !pred) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  return do_step(c, tokens, masked, next_pos, k, cand_lo, cand_hi, rows_bound, conf, pred, logits_dbg,
                 static_cast<cudaStream_t>(stream));
}

int dkv_refresh(dkv_cache* c, int scope) {
  DKV_CHECK_CACHE(c);
  if (scope != DKV_REFRESH_ALL && scope != DKV_REFRESH_DECODED_ONLY) return DKV_E_INVALID_ARG;
  c->pending_refresh = scope;
  return DKV_OK;
}

int dkv_select_unmask(const float* conf, const int32_t* pred, int batch, int seq_len, int cand_lo, int cand_hi, int k,
                      int32_t* tokens, uint8_t* masked, int32_t* chosen_pos, int32_t* status, void* stream) {
  if (!conf || !pred || !tokens || !masked) return DKV_E_INVALID_ARG;
  if (batch < 1 || seq_len < 1 || k < 1 || cand_lo < 0 || cand_hi > seq_len || cand_lo > cand_hi) return DKV_E_SHAPE;
  launch_k(k_select_unmask, batch, 256, 0, static_cast<cudaStream_t>(stream), conf, pred, seq_len, cand_lo, cand_hi, k,
                                                                         nullptr, tokens, masked, chosen_pos, status);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

int dkv_step_host(dkv_cache* c, int32_t* tokens_host, uint8_t* masked_host, const int32_t* next_pos_host, int k,
                  int cand_lo, int cand_hi, int rows_bound, int32_t* chosen_host, void* stream) {
  if (!c || !tokens_host || !masked_host) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Arena& a = c->ar;
  const Dims& dm = c->dims;
  if (k < 1 || k > dm.kmax) return DKV_E_SHAPE;
  const size_t BL = static_cast<size_t>(dm.B) * dm.L;
  cudaMemcpyAsync(a.tok_stage, tokens_host, BL * 4, cudaMemcpyHostToDevice, st);
  cudaMemcpyAsync(a.mask_stage, masked_host, BL, cudaMemcpyHostToDevice, st);
  const int32_t* npos = nullptr;
  if (next_pos_host) {
    cudaMemcpyAsync(a.dpos_stage, next_pos_host, static_cast<size_t>(dm.B) * k * 4, cudaMemcpyHostToDevice, st);
    npos = a.dpos_stage;
  }
  int rc = do_step(c, a.tok_stage, a.mask_stage, npos, k, cand_lo, cand_hi, rows_bound, a.conf_i, a.pred_i, nullptr, st);
  if (rc) return rc;
  {
    Launch l(c, st, PC_SELECT, BL * 9.0, 0);
    launch_k(k_select_unmask, dm.B, 256, 0, st, a.conf_i, a.pred_i, dm.L, cand_lo, cand_hi, k, npos, a.tok_stage,
                                           a.mask_stage, a.chosen_stage, a.status);
  }
  cudaMemcpyAsync(tokens_host, a.tok_stage, BL * 4, cudaMemcpyDeviceToHost, st);
  cudaMemcpyAsync(masked_host, a.mask_stage, BL, cudaMemcpyDeviceToHost, st);
  if (chosen_host)
    cudaMemcpyAsync(chosen_host, a.chosen_stage, static_cast<size_t>(dm.B) * k * 4, cudaMemcpyDeviceToHost, st);
  if (cudaStreamSynchronize(st) != cudaSuccess) return DKV_E_CUDA;
  return DKV_OK;
}

int dkv_generate(dkv_cache* c, int32_t* tokens, uint8_t* masked, const int32_t* order_dev, int k, int block_len,
                 int n_steps, int32_t* chosen_dev, void* stream) {
  if (!c || !tokens || !masked) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  const Dims& dm = c->dims;
  Arena& a = c->ar;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (k < 1 || k > dm.kmax || dm.G % k) return DKV_E_SHAPE;
  if (block_len <= 0) block_len = dm.G;
  if (dm.G % block_len || block_len % k) return DKV_E_SHAPE;
  if (c->policy.kind == DKV_POLICY_GREEDY && !order_dev) return DKV_E_INVALID_ARG;
  const int T = dm.G / k;
  const int steps_per_block = block_len / k;
  const int first = c->step;   // continue where the handle stands
  const int last = n_steps > 0 ? std::min(T, first + n_steps) : T;
  for (int s = first; s < last; ++s) {
    const int blk = s / steps_per_block;
    const int lo = dm.P + blk * block_len, hi = lo + block_len;
    const int32_t* npos = order_dev ? order_dev + static_cast<size_t>(s) * dm.B * k : nullptr;
    int rc = do_step(c, tokens, masked, npos, k, lo, hi, dm.G - s * k, a.conf_i, a.pred_i, nullptr, st);
    if (rc) return rc;
    Launch l(c, st, PC_SELECT, dm.B * dm.L * 9.0, 0);
    launch_k(k_select_unmask, dm.B, 256, 0, st, a.conf_i, a.pred_i, dm.L, lo, hi, k, npos, tokens, masked,
                                           chosen_dev ? chosen_dev + static_cast<size_t>(s) * dm.B * k : nullptr,
                                           a.status);
  }
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

int dkv_get_stats(const dkv_cache* c, dkv_stats* out) {
  if (!c || !out) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  *out = c->stats;
  // the exact number of active rows is counted on the device by the compaction kernel
  unsigned long long act = 0;
  if (cudaStreamSynchronize(c->last_stream) != cudaSuccess) return DKV_E_CUDA;
  if (cudaMemcpy(&act, c->ar.status + 2, 8, cudaMemcpyDeviceToHost) != cudaSuccess) return DKV_E_CUDA;
  out->active_rows = static_cast<int64_t>(act);
  const_cast<dkv_cache*>(c)->stats.active_rows = out->active_rows;
  out->cache_ratio = c->stats.total_rows ? 1.0 - static_cast<double>(c->stats.active_rows) / c->stats.total_rows : 0.0;
  return DKV_OK;
}

int dkv_get_provenance(const dkv_cache* c, int32_t* written_step, void* stream) {
  if (!c || !written_step) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  cudaError_t e = cudaMemcpyAsync(written_step, c->ar.written_step, static_cast<size_t>(c->dims.B) * c->dims.L * 4,
                                  cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

int dkv_get_index_maps(const dkv_cache* c, int32_t* act_idx, int32_t* row_off, int32_t* inv, void* stream) {
  DKV_CHECK_CACHE(c);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t BL = static_cast<size_t>(c->dims.B) * c->dims.L;
  if (act_idx) cudaMemcpyAsync(act_idx, c->ar.act_idx, BL * 4, cudaMemcpyDeviceToDevice, st);
  if (row_off) cudaMemcpyAsync(row_off, c->ar.row_off, (c->dims.B + 1) * 4, cudaMemcpyDeviceToDevice, st);
  if (inv) cudaMemcpyAsync(inv, c->ar.inv, BL * 4, cudaMemcpyDeviceToDevice, st);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

int dkv_status(dkv_cache* c, int32_t* word) {
  DKV_CHECK_CACHE(c);
  int w = 0;
  if (cudaStreamSynchronize(c->last_stream) != cudaSuccess) return DKV_E_CUDA;
  if (cudaMemcpy(&w, c->ar.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return DKV_E_CUDA;
  if (word) *word = w;
  return w ? DKV_E_DEVICE : DKV_OK;
}

int dkv_cache_slots(const dkv_cache* c, int layer, void** k_slots, void** v_slots) {
  DKV_CHECK_CACHE(c);
  if (layer < 0 || layer >= c->model->desc.n_layers) return DKV_E_INVALID_ARG;
  const dkv_model_desc& md = c->model->desc;
  const size_t per = static_cast<size_t>(c->dims.B) * md.n_kv_heads * c->dims.L * md.head_dim * c->model->asize;
  if (k_slots) *k_slots = static_cast<uint8_t*>(c->ar.k_slots) + layer * per;
  if (v_slots) *v_slots = static_cast<uint8_t*>(c->ar.v_slots) + layer * per;
  return DKV_OK;
}

// ---------------------------------------------------- state export / import
namespace {

constexpr uint64_t STATE_MAGIC = 0x314554415453564bull;   // "KVSTATE1", little-endian
constexpr uint32_t STATE_VERSION = 1;

// Header of an exported state; the device sections follow in the order of state_sections().
struct StateHeader {
  uint64_t magic;
  uint32_t version, header_bytes;
  int64_t total_bytes;
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, dtype, act_dtype, elem_bytes;
  int32_t B, L, P, kmax;
  dkv_policy policy;
  int32_t step, last_refresh, pending_refresh, prev_rows_bound, have_dprev, prev_k;
  dkv_stats stats;
  uint64_t active_rows_dev;   // the device-side count of active rows
};

struct StateSection {
  void* dev;
  size_t bytes;
};

// What a later step reads from earlier ones: the K/V slots, both stored mask sets, both stored D
// sets and the provenance stamps.
int state_sections(const dkv_cache* c, StateSection* out /*[7]*/) {
  const Arena& a = c->ar;
  const dkv_model_desc& md = c->model->desc;
  const size_t BL = static_cast<size_t>(c->dims.B) * c->dims.L;
  const size_t slots = static_cast<size_t>(md.n_layers) * c->dims.B * md.n_kv_heads * c->dims.L * md.head_dim * c->model->asize;
  const size_t dset = static_cast<size_t>(c->dims.B) * c->dims.kmax * 4;
  out[0] = {a.k_slots, slots};
  out[1] = {a.v_slots, slots};
  out[2] = {a.mask_buf[0], BL};
  out[3] = {a.mask_buf[1], BL};
  out[4] = {a.d_buf[0], dset};
  out[5] = {a.d_buf[1], dset};
  out[6] = {a.written_step, BL * 4};
  return 7;
}

size_t state_total(const dkv_cache* c) {
  StateSection sec[7];
  const int n = state_sections(c, sec);
  size_t total = align_up(sizeof(StateHeader), 256);
  for (int i = 0; i < n; ++i) total += align_up(sec[i].bytes, 256);
  return total;
}

void state_fill_geometry(const dkv_cache* c, StateHeader* h) {
  const dkv_model_desc& md = c->model->desc;
  h->n_layers = md.n_layers;
  h->d_model = md.d_model;
  h->n_q_heads = md.n_q_heads;
  h->n_kv_heads = md.n_kv_heads;
  h->head_dim = md.head_dim;
  h->dtype = md.dtype;
  h->act_dtype = md.act_dtype;
  h->elem_bytes = static_cast<int32_t>(c->model->asize);
  h->B = c->dims.B;
  h->L = c->dims.L;
  h->P = c->dims.P;
  h->kmax = c->dims.kmax;
  h->policy = c->policy;
}

}  // namespace

size_t dkv_cache_state_bytes(const dkv_cache* c) {
  if (!c || !live_cache(c)) return 0;
  return state_total(c);
}

int dkv_cache_export(dkv_cache* c, void* state_host, size_t state_bytes, void* stream) {
  if (!c || !state_host) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  const size_t total = state_total(c);
  if (state_bytes < total) return DKV_E_NOMEM;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the steps so far may have run on another stream
  if (c->last_stream != st && cudaStreamSynchronize(c->last_stream) != cudaSuccess) return DKV_E_CUDA;
  uint8_t* dst = static_cast<uint8_t*>(state_host);
  StateHeader h;
  memset(&h, 0, sizeof(h));
  h.magic = STATE_MAGIC;
  h.version = STATE_VERSION;
  h.header_bytes = static_cast<uint32_t>(align_up(sizeof(StateHeader), 256));
  h.total_bytes = static_cast<int64_t>(total);
  state_fill_geometry(c, &h);
  h.step = c->step;
  h.last_refresh = c->last_refresh;
  h.pending_refresh = c->pending_refresh;
  h.prev_rows_bound = c->prev_rows_bound;
  h.have_dprev = c->have_dprev ? 1 : 0;
  h.prev_k = c->prev_k;
  h.stats = c->stats;
  StateSection sec[7];
  const int n = state_sections(c, sec);
  size_t off = h.header_bytes;
  for (int i = 0; i < n; ++i) {
    if (cudaMemcpyAsync(dst + off, sec[i].dev, sec[i].bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DKV_E_CUDA;
    off += align_up(sec[i].bytes, 256);
  }
  if (cudaMemcpyAsync(&h.active_rows_dev, c->ar.status + 2, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DKV_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DKV_E_CUDA;
  memset(dst, 0, h.header_bytes);
  memcpy(dst, &h, sizeof(h));
  return DKV_OK;
}

int dkv_cache_import(dkv_cache* c, const void* state_host, size_t state_bytes, void* stream) {
  if (!c || !state_host) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  if (state_bytes < sizeof(StateHeader)) return DKV_E_INVALID_ARG;
  StateHeader h;
  memcpy(&h, state_host, sizeof(h));
  if (h.magic != STATE_MAGIC || h.version != STATE_VERSION) return DKV_E_INVALID_ARG;
  StateHeader want;
  memset(&want, 0, sizeof(want));
  state_fill_geometry(c, &want);
  if (h.n_layers != want.n_layers || h.d_model != want.d_model || h.n_q_heads != want.n_q_heads ||
      h.n_kv_heads != want.n_kv_heads || h.head_dim != want.head_dim || h.dtype != want.dtype ||
      h.act_dtype != want.act_dtype || h.elem_bytes != want.elem_bytes || h.B != want.B || h.L != want.L ||
      h.P != want.P || h.kmax != want.kmax || memcmp(&h.policy, &want.policy, sizeof(dkv_policy)) != 0)
    return DKV_E_SHAPE;
  const size_t total = state_total(c);
  if (h.total_bytes != static_cast<int64_t>(total) || h.header_bytes != align_up(sizeof(StateHeader), 256) ||
      state_bytes < total)
    return DKV_E_SHAPE;
  if (h.step < 0 || h.last_refresh < 0 || h.pending_refresh < -1 || h.pending_refresh > DKV_REFRESH_DECODED_ONLY ||
      h.prev_rows_bound < 0 || h.prev_rows_bound > want.L || h.prev_k < 0 || h.prev_k > want.kmax)
    return DKV_E_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (c->last_stream != st && cudaStreamSynchronize(c->last_stream) != cudaSuccess) return DKV_E_CUDA;
  const uint8_t* src = static_cast<const uint8_t*>(state_host);
  StateSection sec[7];
  const int n = state_sections(c, sec);
  size_t off = h.header_bytes;
  for (int i = 0; i < n; ++i) {
    if (cudaMemcpyAsync(sec[i].dev, src + off, sec[i].bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return DKV_E_CUDA;
    off += align_up(sec[i].bytes, 256);
  }
  if (cudaMemcpyAsync(c->ar.status + 2, &h.active_rows_dev, 8, cudaMemcpyHostToDevice, st) != cudaSuccess) return DKV_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DKV_E_CUDA;
  c->step = h.step;
  c->last_refresh = h.last_refresh;
  c->pending_refresh = h.pending_refresh;
  c->prev_rows_bound = h.prev_rows_bound;
  c->have_dprev = h.have_dprev != 0;
  c->prev_k = h.prev_k;
  const int64_t launches = c->stats.kernel_launches;
  c->stats = h.stats;
  c->stats.kernel_launches = launches;   // launches are this handle's own
  c->last_stream = st;
  return DKV_OK;
}

int dkv_profile_enable(dkv_cache* c, int on) {
  DKV_CHECK_CACHE(c);
  if (!on && c->profiling) prof_flush(c);
  c->profiling = on != 0;
  return DKV_OK;
}

int dkv_profile_read(dkv_cache* c, dkv_profile_entry* out, int* n) {
  if (!c || !out || !n) return DKV_E_INVALID_ARG;
  DKV_CHECK_CACHE(c);
  prof_flush(c);
  const int cnt = std::min<int>(PC_COUNT, DKV_PROF_CLASSES);
  for (int i = 0; i < cnt; ++i) out[i] = c->prof[i];
  *n = cnt;
  for (int i = 0; i < PC_COUNT; ++i) {
    c->prof[i].launches = 0;
    c->prof[i].ms = c->prof[i].bytes = c->prof[i].flops = 0.0;
  }
  return DKV_OK;
}

int dkv_debug_tail_wait(dkv_cache* c, long long wait_cycles, int never_complete) {
  DKV_CHECK_CACHE(c);
  if (wait_cycles < 1000 || wait_cycles > GEMM_WAIT_CYCLES) return DKV_E_INVALID_ARG;
  c->tail_wait_cycles = wait_cycles;
  c->tail_extra = never_complete ? 1 : 0;
  return DKV_OK;
}

int dkv_trace_set(void* records, int capacity) {
  dkv::TraceRec* p = static_cast<dkv::TraceRec*>(records);
  unsigned int zero = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return DKV_E_CUDA;
  if (cudaMemcpyToSymbol(dkv::g_trace_n, &zero, sizeof(zero)) != cudaSuccess) return DKV_E_CUDA;
  if (cudaMemcpyToSymbol(dkv::g_trace_cap, &capacity, sizeof(capacity)) != cudaSuccess) return DKV_E_CUDA;
  if (cudaMemcpyToSymbol(dkv::g_trace_buf, &p, sizeof(p)) != cudaSuccess) return DKV_E_CUDA;
  return DKV_OK;
}

size_t dkv_gemm_workspace_bytes(int rows, int n) {
  if (rows < 1 || n < 1) return 0;
  return static_cast<size_t>(std::max(rows, 2048)) * n * 4 + 256;
}

int dkv_op_gemm(const void* x, const void* w, float* out, int rows, int n, int k, int dtype, int splits,
                void* workspace, size_t workspace_bytes, void* stream) {
  if (!x || !w) return DKV_E_INVALID_ARG;
  if (!out && dtype == DKV_F32) return DKV_E_INVALID_ARG;
  if (rows < 1 || n < 1 || k < 8 || k % 8) return DKV_E_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dtype == DKV_F32) return gemm_f32(static_cast<const float*>(x), static_cast<const float*>(w), n, k, rows, nullptr, out, st);
  if (dtype != DKV_BF16 && dtype != DKV_F16) return DKV_E_UNSUPPORTED;
  if (!workspace || workspace_bytes < dkv_gemm_workspace_bytes(rows, n)) return DKV_E_NOMEM;
  CUtensorMap tw, tx[N_BOX];
  int rc = make_tmap(&tw, w, n, k, GEMM_BM, dtype == DKV_F16);
  // above 256 rows the launch may pick narrower row tiles than the default: give it every box
  for (int i = (rows > 256 ? 0 : pick_box(rows)); i < (rows > 256 ? N_BOX : pick_box(rows) + 1) && !rc; ++i)
    rc = make_tmap(&tx[i], x, rows, k, box_rows(i), dtype == DKV_F16);
  if (rc) return rc;
  int s;
  long long stride;
  const long long part_rows = std::max(rows, 2048);
  GemmOpts o;
  o.forced_splits = splits;
  o.w_static = false;
  rc = gemm_tc(tw, tx, n, k, rows, nullptr, static_cast<float*>(workspace), part_rows, nullptr, dtype == DKV_BF16, st, &s,
               &stride, o);
  if (rc || !out) return rc;   // out == NULL: the split-K partials stay in the workspace
  const long long elems = static_cast<long long>(rows) * n;
  launch_k(k_reduce_partials, static_cast<int>(std::min<long long>(4 * NUM_SMS, (elems + 255) / 256)), 256, 0, st,
           static_cast<const float*>(workspace), s, stride, rows, nullptr, n, out);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

int dkv_op_attention(const void* q, const void* k_slots, const void* v_slots, void* o, const int32_t* row_off,
                     int batch, int rows_per_seq_bound, int seq_len, int n_q_heads, int n_kv_heads, int head_dim,
                     int dtype, void* stream) {
  if (!q || !k_slots || !v_slots || !o || !row_off) return DKV_E_INVALID_ARG;
  if (batch < 1 || rows_per_seq_bound < 1 || seq_len < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads) return DKV_E_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if ((dtype == DKV_BF16 || dtype == DKV_F16) && head_dim == ATC_DH && n_q_heads / n_kv_heads <= ATC_M) {
    // tensor maps for this call's buffers; the queries' row count is only known as a bound on the device,
    // so the map covers batch * bound rows (row_off never points past them)
    AttnMaps am;
    const long long q_rows = static_cast<long long>(batch) * rows_per_seq_bound;
    int rc = make_attn_maps(&am, q, q_rows, k_slots, v_slots, static_cast<long long>(batch) * n_kv_heads, seq_len,
                            seq_len, n_q_heads, n_kv_heads, dtype == DKV_F16);
    if (rc) return rc;
    return attention_tc(am, o, row_off, batch, rows_per_seq_bound, seq_len, n_q_heads, n_kv_heads, 0, dtype == DKV_BF16,
                        nullptr, st);
  }
  if (dtype == DKV_F32)
    return attention_simt<float>(static_cast<const float*>(q), static_cast<const float*>(k_slots),
                                 static_cast<const float*>(v_slots), static_cast<float*>(o), row_off, batch,
                                 rows_per_seq_bound, seq_len, n_q_heads, n_kv_heads, head_dim, st);
  if (dtype == DKV_BF16)
    return attention_16<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k_slots),
                                       static_cast<const __nv_bfloat16*>(v_slots), static_cast<__nv_bfloat16*>(o),
                                       row_off, batch, rows_per_seq_bound, seq_len, n_q_heads, n_kv_heads, head_dim, st);
  if (dtype == DKV_F16)
    return attention_16<__half>(static_cast<const __half*>(q), static_cast<const __half*>(k_slots),
                                static_cast<const __half*>(v_slots), static_cast<__half*>(o), row_off, batch,
                                rows_per_seq_bound, seq_len, n_q_heads, n_kv_heads, head_dim, st);
  return DKV_E_UNSUPPORTED;
}

// --------------------------------------------------------------------------
// dkv_op_gemm_static: the projection GEMM for callers that cannot allocate.
// The split-K partial sums go to a fixed array that is part of the library
// image instead of a caller-provided workspace.
// --------------------------------------------------------------------------
}  // extern "C"

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = static_cast<size_t>(DKV_STATIC_SCRATCH_BYTES);
constexpr int STATIC_MAX_DEVICES = 64;

// Device-resident scratch; one copy per GPU that loads the library, held until
// the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a pointer a kernel could use.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

// Per device: the device address of g_static_scratch, looked up once.
void* g_static_scratch_addr[STATIC_MAX_DEVICES] = {};

// Returns the device address of the scratch array on the current device.
int static_scratch_address(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return DKV_E_CUDA;
  if (!g_static_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DKV_E_CUDA;
    g_static_scratch_addr[dev] = ptr;
  }
  *out = static_cast<float*>(g_static_scratch_addr[dev]);
  return DKV_OK;
}

}  // namespace

extern "C" {

size_t dkv_static_scratch_bytes(void) { return STATIC_SCRATCH_BYTES; }

int dkv_op_gemm_static(const void* x, const void* w, float* out, int rows, int n, int k, int dtype, int splits,
                       void* stream) {
  if (!x || !w || !out) return DKV_E_INVALID_ARG;
  if (dtype != DKV_BF16 && dtype != DKV_F16) return DKV_E_UNSUPPORTED;
  if (rows < 1 || n < 1 || k < 8 || k % 8 || splits < 0) return DKV_E_SHAPE;
  // one [rows, n] fp32 slab per split must fit
  const size_t slab = static_cast<size_t>(rows) * static_cast<size_t>(n) * sizeof(float);
  if (slab > STATIC_SCRATCH_BYTES) return DKV_E_NOMEM;
  const long long max_slabs = static_cast<long long>(STATIC_SCRATCH_BYTES / slab);
  if (splits > max_slabs) return DKV_E_NOMEM;
  float* scratch = nullptr;
  int rc = static_scratch_address(&scratch);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CUtensorMap tw, tx[N_BOX];
  rc = make_tmap(&tw, w, n, k, GEMM_BM, dtype == DKV_F16);
  for (int i = (rows > 256 ? 0 : pick_box(rows)); i < (rows > 256 ? N_BOX : pick_box(rows) + 1) && !rc; ++i)
    rc = make_tmap(&tx[i], x, rows, k, box_rows(i), dtype == DKV_F16);
  if (rc) return rc;
  int s = 1;
  long long stride = 0;
  // part_rows bounds splits * rows, i.e. the number of [n]-float rows the scratch can hold
  const long long part_rows = max_slabs * rows;
  GemmOpts o;
  o.forced_splits = splits;
  o.w_static = false;
  rc = gemm_tc(tw, tx, n, k, rows, nullptr, scratch, part_rows, nullptr, dtype == DKV_BF16, st, &s, &stride, o);
  if (rc) return rc;
  // every float the reduction reads was written by the GEMM launch just above:
  // nothing in the shared scratch has to start at zero
  const long long elems = static_cast<long long>(rows) * n;
  launch_k(k_reduce_partials, static_cast<int>(std::min<long long>(4 * NUM_SMS, (elems + 255) / 256)), 256, 0, st,
           static_cast<const float*>(scratch), s, stride, rows, static_cast<const int*>(nullptr), n, out);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

int dkv_op_stream_probe(const void* streamed, long long streamed_bytes, const void* reread, long long reread_bytes,
                        int ctas, int chunk_bytes, int reread_chunk_bytes, int stages, int32_t* status, void* stream) {
  if (!streamed) return DKV_E_INVALID_ARG;
  if (ctas < 1 || ctas > 1024 || stages < 1 || stages > 32) return DKV_E_SHAPE;
  if (chunk_bytes < 16 || chunk_bytes % 16 || reread_chunk_bytes < 0 || reread_chunk_bytes % 16) return DKV_E_SHAPE;
  if (reread_chunk_bytes > 0 && (!reread || reread_bytes < reread_chunk_bytes)) return DKV_E_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(streamed) % 16 || reinterpret_cast<uintptr_t>(reread) % 16) return DKV_E_INVALID_ARG;
  const size_t smem = static_cast<size_t>(stages) * (chunk_bytes + reread_chunk_bytes) + 2 * stages * 8 + 16;
  if (smem > 227 * 1024) return DKV_E_NOMEM;
  StreamProbeParams p;
  p.a = static_cast<const uint8_t*>(streamed);
  p.b = static_cast<const uint8_t*>(reread);
  p.n_chunks = static_cast<int>(std::min<long long>(streamed_bytes / ctas / chunk_bytes, 1 << 30));
  if (p.n_chunks < 1) return DKV_E_SHAPE;
  p.a_per_cta = static_cast<long long>(p.n_chunks) * chunk_bytes;
  p.a_chunk = chunk_bytes;
  p.b_chunk = reread_chunk_bytes;
  p.b_span = reread_chunk_bytes > 0 ? reread_bytes / reread_chunk_bytes * reread_chunk_bytes : 0;
  p.stages = stages;
  p.wait_cycles = GEMM_WAIT_CYCLES;
  p.status = status;
  static PerDeviceOnce attr_once;
  if (attr_once.need() &&
      cudaFuncSetAttribute(k_stream_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
    return DKV_E_CUDA;
  k_stream_probe<<<ctas, 64, smem, static_cast<cudaStream_t>(stream)>>>(p);
  return cudaGetLastError() == cudaSuccess ? DKV_OK : DKV_E_CUDA;
}

}  // extern "C"
