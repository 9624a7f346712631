// C ABI of the library: handle, planner upload, kernel launches.  See include/libra.h.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "decode_kernel.cuh"
#include "kv_move_kernel.cuh"
#include "libra.h"
#include "merge_kernel.cuh"
#include "plan_kernel.cuh"
#include "plan_layout.hpp"
#include "planner.hpp"
#include "read_kernel.cuh"
#include "ring_kernel.cuh"

static_assert(LIBRA_ERR_WAIT_TIMEOUT == LIBRA_DEV_ERR_WAIT_TIMEOUT, "error bits");
static_assert(LIBRA_ERR_BAD_PAGE_ID == LIBRA_DEV_ERR_BAD_PAGE_ID, "error bits");
static_assert(LIBRA_ERR_SEQ_LEN_MISMATCH == LIBRA_DEV_ERR_SEQ_LEN_MISMATCH, "error bits");
static_assert(LIBRA_ERR_PLAN_OVERFLOW == LIBRA_DEV_ERR_PLAN_OVERFLOW, "error bits");

namespace {

using libra::DecodeParams;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

typedef void (*DecodeKernelFn)(const CUtensorMap, const CUtensorMap, const DecodeParams, const libra::ParamPlan);

struct Variant {
  int warps, stages;
  DecodeKernelFn fn[2][2];         // [D == 128][NT - 1]
  DecodeKernelFn fn_append[2][2];  // the same with the KV append compiled in
  int smem[2][2];                  // dynamic bytes
};


template <int NW, int ST>
Variant make_variant() {
  Variant v;
  v.warps = NW;
  v.stages = ST;
  v.fn[0][0] = libra::decode_kernel<64, 1, NW, ST>;
  v.fn[0][1] = libra::decode_kernel<64, 2, NW, ST>;
  v.fn[1][0] = libra::decode_kernel<128, 1, NW, ST>;
  v.fn[1][1] = libra::decode_kernel<128, 2, NW, ST>;
  v.fn_append[0][0] = libra::decode_kernel<64, 1, NW, ST, false, false, true>;
  v.fn_append[0][1] = libra::decode_kernel<64, 2, NW, ST, false, false, true>;
  v.fn_append[1][0] = libra::decode_kernel<128, 1, NW, ST, false, false, true>;
  v.fn_append[1][1] = libra::decode_kernel<128, 2, NW, ST, false, false, true>;
  v.smem[0][0] = v.smem[0][1] = libra::DecodeSmem<64, NW, ST>::kDynamicBytes;
  v.smem[1][0] = v.smem[1][1] = libra::DecodeSmem<128, NW, ST>::kDynamicBytes;
  return v;
}

// Block shapes that are compiled in.  Defaults: index 0 (8 warps x 3 stages) for one column tile; for two, on a plan
// with one slot per SM, index 1 (12 x 2): twice the tensor-core and softmax work per tile wants a third warp per
// scheduler to hide its latency (measured 2.5 - 4 % faster there than 8 x 3, 0.5 - 1 % slower with one tile); on a plan
// with two slots per SM (the default for two tiles) index 10, see below.
constexpr int kVariantOneTile = 0, kVariantTwoTiles = 1, kVariantShortUnits = 4, kVariantTinyUnits = 9, kVariantPair = 10;
// Two column tiles (9 - 16 score columns per KV head: more than 8 query heads per KV head, or several query tokens)
// double the work per tile and the per-unit merge; there two blocks of 6 warps x 2 stages per SM (96 KB and 168
// registers each, the kernel's launch bounds see to the registers), planned as two slots per SM, beat one block of
// 12 x 2: one block's start-up and merge overlap the other's streaming.  Same-run A/B, us per step, 12 x 2 -> 2 x (6 x 2):
// 16 query heads per KV head 64.3 -> 61.3 (lognormal_b64), 303 -> 286 (shift_b128), the two long workloads unchanged;
// 9 - 16 columns from several query tokens 68.1 -> 63.4 (lognormal_b64), 180.6 -> 175.8 (straggler_b8), 306 -> 290
// (shift_b128), 746 -> 749 (longtail_mix_b256).  With one column tile the two shapes are a wash.  Over an E4M3 cache:
// kFp8Pair.
constexpr int kTwoSlotCtas = 2;
// A block costs ~4 us of start-up and epilogue whatever its size and the default block is alone on its SM, so a batch
// of short sequences leaves the SMs waiting most of the time.  When no unit of a host plan is longer than this many
// tokens, 4 warps x 2 stages (64 KB: three blocks per SM, three units in flight) is used instead: the same bytes in
// flight per SM, measured 1.6x / 1.16x / 1.05x faster at 256 / 512 / 1024 tokens per sequence; and when none is longer
// than kTinyUnitTokens, 2 warps x 2 stages (32 KB, seven blocks per SM): 2.6x at 128 tokens.  A long unit on such a
// block would stream at a fraction of the SM's rate, hence only when there is none.
constexpr int kShortUnitTokens = 1024;
constexpr int kTinyUnitTokens = 256;
const std::vector<Variant>& variants() {
  static const std::vector<Variant> v = {
      make_variant<8, 3>(), make_variant<12, 2>(), make_variant<8, 2>(), make_variant<4, 3>(), make_variant<4, 2>(),
      make_variant<4, 4>(), make_variant<4, 6>(), make_variant<2, 6>(), make_variant<2, 4>(),
      make_variant<2, 2>(), make_variant<6, 2>(),
  };
  return v;
}

// Measurement build of the default block shape (copies only, no math); [D == 128][NT - 1]
constexpr int kLoadsOnlyWarps = 8, kLoadsOnlyStages = 3;
const DecodeKernelFn kLoadsOnlyFn[2][2] = {{libra::decode_kernel<64, 1, kLoadsOnlyWarps, kLoadsOnlyStages, true>,
                                            libra::decode_kernel<64, 2, kLoadsOnlyWarps, kLoadsOnlyStages, true>},
                                           {libra::decode_kernel<128, 1, kLoadsOnlyWarps, kLoadsOnlyStages, true>,
                                            libra::decode_kernel<128, 2, kLoadsOnlyWarps, kLoadsOnlyStages, true>}};
const int kLoadsOnlySmem[2] = {libra::DecodeSmem<64, kLoadsOnlyWarps, kLoadsOnlyStages>::kDynamicBytes,
                               libra::DecodeSmem<128, kLoadsOnlyWarps, kLoadsOnlyStages>::kDynamicBytes};

// 8-bit (E4M3) cache, head_dim 128: block shapes compiled in.  Half the bytes per tile leave half the time per tile,
// and two warps per scheduler cannot hide the conversion -> mma -> softmax chain in it, so 16 warps per SM are wanted:
// on a one-slot plan one block of 16 warps x 3 stages of 4 KB where the registers allow it (one column tile), 8 x 6
// otherwise; on a two-slot plan, the default, two blocks per SM (kFp8OnePair, kFp8Pair below).  Batches of short
// units get 4 x 2 or, up to kTinyUnitTokens, 2 x 4 (32 KB, seven blocks per SM: 1.4x / 1.9x / 2.6x / 3.5x faster than
// 16 x 3 at 1024 / 512 / 256 / 128 tokens per sequence).  fn[loads only][NT - 1]
// Two column tiles on a two-slot plan (the default for two tiles): two blocks of 6 x 4 per SM, as over bf16 pools
// (kVariantPair).  Same-run A/B against 8 x 6 on a one-slot plan, us per step: 16 query heads per KV head 50.2 -> 44.7
// (lognormal_b64), 124.7 -> 114.0 (straggler_b8), 225 -> 196 (shift_b128), 530 -> 512 (longtail_mix_b256); 16 columns
// from several query tokens 56.4 -> 48.6, 132.2 -> 121.0, 220.7 -> 195.9, 542 -> 530.
// One column tile on a two-slot plan (the default over E4M3 pools): two blocks of 8 x 3 per SM (the kernel's launch
// bounds hold them at 128 registers; at 130 only one was resident and the arrangement lost 5 - 20 %) against one block
// of 16 x 3 on a one-slot plan: 36.2 -> 31.5 us (lognormal_b64), 91.1 -> 91.1 (straggler_b8), 158.9 -> 142.0
// (shift_b128), 393 -> 351 (longtail_mix_b256; best regions 346.9 -> 334.7).
constexpr int kFp8OneTile = 2, kFp8TwoTiles = 1, kFp8ShortUnits = 5, kFp8TinyUnits = 6, kFp8Pair = 7, kFp8OnePair = 0;
struct Fp8Variant {
  int warps, stages;
  DecodeKernelFn fn[2][2][2];      // [D == 128][loads only][NT - 1]
  DecodeKernelFn fn_append[2][2];  // [D == 128][NT - 1], with the KV append compiled in
  int smem[2];                     // [D == 128]
};
template <int NW, int ST>
Fp8Variant make_fp8_variant() {
  Fp8Variant v;
  v.warps = NW;
  v.stages = ST;
  v.fn[0][0][0] = libra::decode_kernel<64, 1, NW, ST, false, true>;
  v.fn[0][0][1] = libra::decode_kernel<64, 2, NW, ST, false, true>;
  v.fn[0][1][0] = libra::decode_kernel<64, 1, NW, ST, true, true>;
  v.fn[0][1][1] = libra::decode_kernel<64, 2, NW, ST, true, true>;
  v.fn[1][0][0] = libra::decode_kernel<128, 1, NW, ST, false, true>;
  v.fn[1][0][1] = libra::decode_kernel<128, 2, NW, ST, false, true>;
  v.fn[1][1][0] = libra::decode_kernel<128, 1, NW, ST, true, true>;
  v.fn[1][1][1] = libra::decode_kernel<128, 2, NW, ST, true, true>;
  v.fn_append[0][0] = libra::decode_kernel<64, 1, NW, ST, false, true, true>;
  v.fn_append[0][1] = libra::decode_kernel<64, 2, NW, ST, false, true, true>;
  v.fn_append[1][0] = libra::decode_kernel<128, 1, NW, ST, false, true, true>;
  v.fn_append[1][1] = libra::decode_kernel<128, 2, NW, ST, false, true, true>;
  v.smem[0] = libra::DecodeSmem<64, NW, ST, 1>::kDynamicBytes;
  v.smem[1] = libra::DecodeSmem<128, NW, ST, 1>::kDynamicBytes;
  return v;
}
const std::vector<Fp8Variant>& fp8_variants() {
  static const std::vector<Fp8Variant> v = {make_fp8_variant<8, 3>(), make_fp8_variant<8, 6>(), make_fp8_variant<16, 3>(),
                                            make_fp8_variant<16, 2>(), make_fp8_variant<8, 4>(), make_fp8_variant<4, 2>(),
                                            make_fp8_variant<2, 4>(), make_fp8_variant<6, 4>()};
  return v;
}

constexpr int kMaxProfiledCalls = 4096;

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceGuard(int dev) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != dev) {
      err = cudaSetDevice(dev);
      switched = (err == cudaSuccess);
    }
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

struct libra_handle_s {
  libra_config_t cfg;
  libra::PlanParams params;          // the planner's parameters in force (defaults resolved)
  libra_plan_params_t params_in{};   // as given at creation (0 = default)
  int n_sm_dev = 0;
  bool two_slot_auto = false;        // the default of two slots per SM is in force (see kVariantPair)
  int group = 0;
  float scale_log2 = 0.f;
  int64_t stride_page = 0, stride_head = 0, stride_token = 0;
  int64_t pool_elems = 0;
  int last_cuda_error = 0;
  int variant = -1;         // -1: chosen by the number of column tiles
  int max_q_len = 1;        // query tokens per sequence the workspace is laid out for
  bool fp8 = false;         // the pools hold E4M3 codes; keys and values are code * k_scale / v_scale
  float k_scale = 1.f, v_scale = 1.f;
  int fp8_variant = -1;     // -1: chosen by the number of column tiles
  EncodeTiledFn encode = nullptr;

  // workspace layout: control words | arrival counters | partial LSE | partial O | oversized plans
  int64_t max_items = 0;
  size_t cnt_off = 0, cnt_bytes = 0, lse_off = 0, o_off = 0, plan_off = 0, plan_bytes = 0, workspace_bytes = 0;
  void* clean_workspace = nullptr;  // workspace whose control words and counters are known to be zero
  int combine_mode = 1;     // 0: separate kernel, 1: inside the decode kernel
  bool pdl = true;          // programmatic dependent launches (decode after its predecessor, combine after decode)
  float* lse_out = nullptr;     // optional second output of the step (libra_set_lse_output)
  bool early_prefetch = false;  // the caller's promise about the preceding kernel (libra_set_early_prefetch)
  bool l2_warmup = true;        // libra_set_cache_warmup

  // pinned staging for uploads of plans too large for the kernel parameters
  int32_t* staging[2] = {nullptr, nullptr};
  cudaEvent_t staging_done[2] = {nullptr, nullptr};
  bool staging_used[2] = {false, false};
  int next_staging = 0;

  // last plan
  bool planned = false;
  libra::HostPlan plan;
  std::vector<int32_t> items_flat;
  void* workspace = nullptr;
  int32_t num_items = 0;
  void* last_stream = nullptr;
  bool device_planned = false;  // the last plan was made by the device-side planner: counts live in the workspace
  int64_t decodes_on_plan = 0;  // decode launches enqueued since the last plan call
  int32_t length_hint = 0;      // libra_set_length_hint: the caller's bound on the lengths of device-planned batches (0 = none)
  int32_t dev_item_bound = 0;   // device-side plan: the most work items the planned batch can have (sizes the grids)
  int32_t planned_batch = 0;
  size_t dev_counts_off = 0, dev_per_seq_off = 0, dev_entries_off = 0, dev_fixes_off = 0;
  std::vector<int32_t> export_scratch;
  bool plan_in_params = true;   // the usual case: the plan travels with every launch
  libra::ParamPlan pp;          // work items, then one entry per empty sequence
  libra::ParamFix pf;           // merges for the combine kernel

  // tensor maps of the pools seen most recently (callers often rotate between a few pools)
  struct PoolMaps {
    const void* k_ptr = nullptr;
    const void* v_ptr = nullptr;
    CUtensorMap map_k, map_v;
  };
  static constexpr int kMapCache = 8;
  PoolMaps maps[kMapCache];
  int next_map = 0;
  int pos_head = 0, pos_page = 0, pos_token = 0;

  // profiling
  bool profiling = false;
  std::vector<cudaEvent_t> events;  // 3 per call
  int profiled_calls = 0;
  int64_t launches = 0;
};

namespace {

int fail_cuda(libra_handle_t h, cudaError_t e) {
  if (h) h->last_cuda_error = int(e);
  (void)cudaGetLastError();
  return LIBRA_CUDA_ERROR;
}

#define LIBRA_CUDA_TRY(h, expr)                       \
  do {                                                \
    cudaError_t e__ = (expr);                         \
    if (e__ != cudaSuccess) return fail_cuda(h, e__); \
  } while (0)

libra::PlanParams resolve_params(const libra_plan_params_t& in, int n_sm_device, bool two_slots = false) {
  libra::PlanParams p;
  if (two_slots) p.ctas_per_sm = kTwoSlotCtas;   // the default where two blocks per SM are resident (see kVariantPair)
  if (in.n_sm > 0) p.n_sm = in.n_sm;
  else if (n_sm_device > 0) p.n_sm = n_sm_device;
  if (in.ctas_per_sm > 0) p.ctas_per_sm = in.ctas_per_sm;
  if (in.items_per_slot > 0) p.items_per_slot = in.items_per_slot;
  if (in.chunk_align > 0) p.chunk_align = in.chunk_align;
  if (in.min_chunk > 0) p.min_chunk = in.min_chunk;
  if (in.max_splits > 0) p.max_splits = in.max_splits;
  if (in.refine < 0) p.refine = 0;   // -1 = never
  return p;
}

// Build the tiled tensor map of one pool: dimension 0 is head_dim (contiguous); the other three
// (token, head, page) are ordered by increasing stride.  Box = 64 elements x 16 tokens x 1 x 1 (a page of
// 32 or 64 tokens is read as 2 or 4 such boxes at token offsets 0, 16, ...).
int encode_pool_map(libra_handle_t h, const void* base, CUtensorMap* map, int* pos_head, int* pos_page, int* pos_token) {
  struct Dim {
    int64_t stride, size;
    uint32_t box;
    int kind;
  };
  Dim dims[3] = {{h->stride_token, h->cfg.page_size, 16u, 0},
                 {h->stride_head, h->cfg.num_kv_heads, 1u, 1},
                 {h->stride_page, h->cfg.num_pages, 1u, 2}};
  std::stable_sort(dims, dims + 3, [](const Dim& a, const Dim& b) { return a.stride < b.stride; });
  const int eb = h->fp8 ? 1 : 2;   // bytes per element; a box row is 128 bytes, or the whole 64-byte row of an 8-bit cache at head_dim 64
  const int row_bytes = std::min(128, h->cfg.head_dim * eb);
  cuuint64_t gdim[4] = {cuuint64_t(h->cfg.head_dim), 0, 0, 0};
  cuuint64_t gstride[3];
  cuuint32_t box[4] = {cuuint32_t(row_bytes / eb), 0, 0, 0};
  cuuint32_t estride[4] = {1, 1, 1, 1};
  for (int i = 0; i < 3; ++i) {
    gdim[i + 1] = cuuint64_t(dims[i].size);
    gstride[i] = cuuint64_t(dims[i].stride) * eb;
    box[i + 1] = dims[i].box;
    if (dims[i].kind == 0) *pos_token = i + 1;
    if (dims[i].kind == 1) *pos_head = i + 1;
    if (dims[i].kind == 2) *pos_page = i + 1;
  }
  CUresult r = h->encode(map, h->fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), gdim, gstride, box, estride,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    h->last_cuda_error = int(cudaErrorInvalidValue);
    return LIBRA_CUDA_ERROR;
  }
  return LIBRA_OK;
}

// Two slots per SM are the planner's default where a step has two column tiles (kVariantPair, kFp8Pair) and for every
// step over E4M3 pools (kFp8OnePair).
bool wants_two_slots(const libra_handle_s* h, bool whatever_the_pools) {
  return h->params_in.ctas_per_sm == 0 && (h->group * h->max_q_len > 8 || h->fp8 || whatever_the_pools);
}

// The parameters in force for the handle's present state; true if they changed (a plan made before is then void).
bool refresh_params(libra_handle_t h) {
  const bool two = wants_two_slots(h, false);
  const libra::PlanParams now = resolve_params(h->params_in, h->n_sm_dev, two);
  const bool changed = now.ctas_per_sm != h->params.ctas_per_sm;
  h->params = now;
  h->two_slot_auto = two;
  return changed;
}

// Workspace layout; the partial buffers hold max_q_len * num_q_heads rows per work item.  Sized for the larger of the
// planner's two defaults, so that switching the pools' type never asks for a larger workspace.
void compute_layout(libra_handle_t h) {
  const libra_config_t* cfg = &h->cfg;
  const size_t rows = size_t(h->max_q_len) * cfg->num_q_heads;
  h->max_items = libra::max_items(resolve_params(h->params_in, h->n_sm_dev, wants_two_slots(h, true)), cfg->num_kv_heads,
                                  cfg->max_batch);
  h->cnt_off = 256;  // the first 256 bytes hold the control words (the device error word)
  h->cnt_bytes = align_up(size_t(cfg->max_batch) * cfg->num_kv_heads * 4, 256);
  h->lse_off = h->cnt_off + h->cnt_bytes;
  h->o_off = h->lse_off + align_up(size_t(h->max_items) * rows * 4, 256);
  h->plan_off = h->o_off + align_up(size_t(h->max_items) * rows * cfg->head_dim * 4, 256);
  // plan region: counts | per-sequence arrays (device planner) | entries (items + empties) | merges
  h->dev_counts_off = h->plan_off;
  h->dev_per_seq_off = h->dev_counts_off + 256;
  h->dev_entries_off = h->dev_per_seq_off + align_up(size_t(4) * cfg->max_batch * sizeof(int32_t), 256);
  h->dev_fixes_off = h->dev_entries_off + align_up((size_t(h->max_items) + size_t(cfg->max_batch)) * sizeof(int4), 256);
  h->plan_bytes = h->dev_fixes_off + align_up(size_t(cfg->max_batch) * sizeof(int4), 256) - h->plan_off;
  h->workspace_bytes = h->plan_off + h->plan_bytes;
}

// ---- built-in scratch for libra_decode_attn_static --------------------------------------------
// A fixed region of device memory that is part of the loaded library image on every GPU, used as the
// workspace by callers that cannot provide one.  In host code `g_static_scratch` is only a handle
// for the symbol, not a device address: the address each device gives it is looked up once per
// device with cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[LIBRA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the built-in scratch on `device`, which must be the current device.
cudaError_t static_scratch_address(int device, void** ptr) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[device]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[device] = p;
  }
  *ptr = g_scratch_ptr[device];
  return cudaSuccess;
}

}  // namespace

extern "C" {

int libra_version(void) { return 100; }

const char* libra_status_string(int status) {
  switch (status) {
    case LIBRA_OK: return "ok";
    case LIBRA_INVALID_ARGUMENT: return "invalid argument";
    case LIBRA_UNSUPPORTED_SHAPE: return "unsupported shape";
    case LIBRA_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LIBRA_NOT_PLANNED: return "no plan has been made for this handle";
    case LIBRA_CUDA_ERROR: return "a CUDA call failed";
    case LIBRA_DEVICE_FLAGGED: return "a kernel recorded a problem in the device error word";
    default: return "unknown status";
  }
}

int libra_plan_host(const libra_plan_params_t* params, int32_t num_kv_heads, const int32_t* seq_lens, int32_t batch,
                    int32_t* chunk_target, int32_t* bucket, int32_t* num_splits, int32_t* chunk_len,
                    int32_t* item_offset, int32_t* items, int32_t items_capacity, int32_t* num_items,
                    int32_t* combine, int32_t* num_combine, int32_t* empty, int32_t* num_empty) {
  if (!params || batch < 0 || (batch > 0 && !seq_lens) || num_kv_heads <= 0 || items_capacity < 0) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (!chunk_target || !num_items || !num_combine || !num_empty) return LIBRA_INVALID_ARGUMENT;
  if (batch > 0 && (!bucket || !num_splits || !chunk_len || !item_offset || !combine || !empty)) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (params->n_sm <= 0) return LIBRA_INVALID_ARGUMENT;
  const libra::PlanParams p = resolve_params(*params, 0);
  libra::HostPlan pl;
  if (!libra::make_plan(p, num_kv_heads, seq_lens, batch, &pl)) return LIBRA_INVALID_ARGUMENT;
  *chunk_target = pl.chunk_target;
  *num_items = int32_t(pl.items.size());
  *num_combine = int32_t(pl.combine.size());
  *num_empty = int32_t(pl.empty.size());
  for (int32_t b = 0; b < batch; ++b) {
    bucket[b] = pl.bucket[b];
    num_splits[b] = pl.num_splits[b];
    chunk_len[b] = pl.chunk_len[b];
    item_offset[b] = pl.item_offset[b];
  }
  std::copy(pl.combine.begin(), pl.combine.end(), combine);
  std::copy(pl.empty.begin(), pl.empty.end(), empty);
  if (int64_t(pl.items.size()) > items_capacity) return LIBRA_WORKSPACE_TOO_SMALL;
  if (!pl.items.empty() && !items) return LIBRA_INVALID_ARGUMENT;
  for (size_t i = 0; i < pl.items.size(); ++i) {
    items[4 * i + 0] = pl.items[i].b;
    items[4 * i + 1] = pl.items[i].j;
    items[4 * i + 2] = pl.items[i].kv_begin;
    items[4 * i + 3] = pl.items[i].kv_end;
  }
  return LIBRA_OK;
}

int libra_create(libra_handle_t* handle, const libra_config_t* cfg) {
  if (!handle) return LIBRA_INVALID_ARGUMENT;
  *handle = nullptr;
  if (!cfg) return LIBRA_INVALID_ARGUMENT;
  if (cfg->num_q_heads <= 0 || cfg->num_kv_heads <= 0 || cfg->head_dim <= 0 || cfg->page_size <= 0 ||
      cfg->num_pages <= 0 || cfg->max_batch <= 0 || cfg->block_table_ld <= 0 || cfg->device < 0) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (cfg->num_q_heads % cfg->num_kv_heads != 0) return LIBRA_INVALID_ARGUMENT;
  if (!(cfg->sm_scale >= 0.f) || !std::isfinite(cfg->sm_scale)) return LIBRA_INVALID_ARGUMENT;
  const int group = cfg->num_q_heads / cfg->num_kv_heads;
  if (group > 16 || (cfg->head_dim != 64 && cfg->head_dim != 128)) return LIBRA_UNSUPPORTED_SHAPE;
  if (cfg->page_size != 16 && cfg->page_size != 32 && cfg->page_size != 64) return LIBRA_UNSUPPORTED_SHAPE;
  if (cfg->num_pages > (int64_t(1) << 31) - 1) return LIBRA_UNSUPPORTED_SHAPE;  // page ids are int32
  if (cfg->max_batch > libra::plan_layout::kMaxBatch) return LIBRA_UNSUPPORTED_SHAPE;

  int64_t sp = cfg->kv_stride_page, sh = cfg->kv_stride_head, st = cfg->kv_stride_token;
  if (sp == 0 && sh == 0 && st == 0) {  // HND
    st = cfg->head_dim;
    sh = int64_t(cfg->page_size) * cfg->head_dim;
    sp = sh * cfg->num_kv_heads;
  }
  if (sp <= 0 || sh <= 0 || st <= 0 || sp % 8 || sh % 8 || st % 8 || st < cfg->head_dim) return LIBRA_INVALID_ARGUMENT;
  if (sp * 2 >= (int64_t(1) << 40) || sh * 2 >= (int64_t(1) << 40) || st * 2 >= (int64_t(1) << 40)) {
    return LIBRA_UNSUPPORTED_SHAPE;
  }
  libra_plan_params_t pin = cfg->plan;
  if (pin.n_sm < 0 || pin.ctas_per_sm < 0 || pin.items_per_slot < 0 || pin.chunk_align < 0 || pin.min_chunk < 0 ||
      pin.max_splits < 0 || pin.refine < -1 || pin.refine > 1) {
    return LIBRA_INVALID_ARGUMENT;
  }

  libra_handle_s* h = new (std::nothrow) libra_handle_s();
  if (!h) return LIBRA_INVALID_ARGUMENT;
  h->cfg = *cfg;
  h->group = group;
  h->stride_page = sp;
  h->stride_head = sh;
  h->stride_token = st;
  const float scale = (cfg->sm_scale > 0.f) ? cfg->sm_scale : 1.0f / std::sqrt(float(cfg->head_dim));
  h->scale_log2 = scale * 1.4426950408889634f;

  int status = LIBRA_OK;
  do {
    int ndev = 0;
    cudaError_t e = cudaGetDeviceCount(&ndev);
    if (e != cudaSuccess || cfg->device >= ndev) {
      status = fail_cuda(h, e != cudaSuccess ? e : cudaErrorInvalidDevice);
      break;
    }
    DeviceGuard guard(cfg->device);
    if (guard.err != cudaSuccess) { status = fail_cuda(h, guard.err); break; }
    int n_sm = 0, cc_major = 0;
    if ((e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, cfg->device)) != cudaSuccess ||
        (e = cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, cfg->device)) != cudaSuccess) {
      status = fail_cuda(h, e);
      break;
    }
    if (cc_major != 10) {  // the kernels are built for sm_100a only
      status = fail_cuda(h, cudaErrorNoKernelImageForDevice);
      break;
    }
    h->params_in = pin;
    h->n_sm_dev = n_sm;
    refresh_params(h);
    if (!libra::valid_params(h->params) || h->params.chunk_align % cfg->page_size != 0) {
      status = LIBRA_INVALID_ARGUMENT;  // chunks must start on page boundaries
      break;
    }

    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
      status = fail_cuda(h, e != cudaSuccess ? e : cudaErrorSymbolNotFound);
      break;
    }
    h->encode = reinterpret_cast<EncodeTiledFn>(fn);

    for (const Variant& v : variants()) {
      for (int di = 0; di < 2 && status == LIBRA_OK; ++di) {
        for (int ni = 0; ni < 2; ++ni) {
          if (!v.fn[di][ni]) continue;
          e = cudaFuncSetAttribute(reinterpret_cast<const void*>(v.fn[di][ni]),
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, v.smem[di][ni]);
          if (e == cudaSuccess) {
            e = cudaFuncSetAttribute(reinterpret_cast<const void*>(v.fn_append[di][ni]),
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, v.smem[di][ni]);
          }
          if (e != cudaSuccess) { status = fail_cuda(h, e); break; }
        }
      }
    }
    if (status != LIBRA_OK) break;
    for (int di = 0; di < 4; ++di) {
      e = cudaFuncSetAttribute(reinterpret_cast<const void*>(kLoadsOnlyFn[di >> 1][di & 1]),
                               cudaFuncAttributeMaxDynamicSharedMemorySize, kLoadsOnlySmem[di >> 1]);
      if (e != cudaSuccess) break;
    }
    if (e != cudaSuccess) { status = fail_cuda(h, e); break; }
    for (const Fp8Variant& fv : fp8_variants()) {
      for (int i = 0; i < 8 && e == cudaSuccess; ++i) {
        e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fv.fn[i >> 2][(i >> 1) & 1][i & 1]),
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, fv.smem[i >> 2]);
      }
      for (int i = 0; i < 4 && e == cudaSuccess; ++i) {
        e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fv.fn_append[i >> 1][i & 1]),
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, fv.smem[i >> 1]);
      }
    }
    if (e != cudaSuccess) { status = fail_cuda(h, e); break; }
    e = cudaFuncSetAttribute(reinterpret_cast<const void*>(libra::plan_kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             int(libra::plan_kernel_smem_bytes(libra::kDevPlanThreads)));
    if (e != cudaSuccess) { status = fail_cuda(h, e); break; }

    compute_layout(h);

    for (int i = 0; i < 2; ++i) {
      if ((e = cudaHostAlloc(reinterpret_cast<void**>(&h->staging[i]), h->plan_bytes, cudaHostAllocDefault)) != cudaSuccess ||
          (e = cudaEventCreateWithFlags(&h->staging_done[i], cudaEventDisableTiming)) != cudaSuccess) {
        status = fail_cuda(h, e);
        break;
      }
    }
  } while (false);

  if (status != LIBRA_OK) {
    libra_destroy(h);
    return status;
  }
  *handle = h;
  return LIBRA_OK;
}

int libra_destroy(libra_handle_t h) {
  if (!h) return LIBRA_OK;
  {
    DeviceGuard guard(h->cfg.device);
    for (int i = 0; i < 2; ++i) {
      if (h->staging_done[i]) cudaEventDestroy(h->staging_done[i]);
      if (h->staging[i]) cudaFreeHost(h->staging[i]);
    }
    for (cudaEvent_t ev : h->events) cudaEventDestroy(ev);
    (void)cudaGetLastError();
  }
  delete h;
  return LIBRA_OK;
}

int libra_workspace_size(libra_handle_t h, size_t* bytes) {
  if (!h || !bytes) return LIBRA_INVALID_ARGUMENT;
  *bytes = h->workspace_bytes;
  return LIBRA_OK;
}

int libra_workspace_invalidate(libra_handle_t h) {
  if (!h) return LIBRA_INVALID_ARGUMENT;
  h->clean_workspace = nullptr;
  h->planned = false;
  return LIBRA_OK;
}

int libra_get_plan_params(libra_handle_t h, libra_plan_params_t* out) {
  if (!h || !out) return LIBRA_INVALID_ARGUMENT;
  out->n_sm = h->params.n_sm;
  out->ctas_per_sm = h->params.ctas_per_sm;
  out->items_per_slot = h->params.items_per_slot;
  out->chunk_align = h->params.chunk_align;
  out->min_chunk = h->params.min_chunk;
  out->max_splits = h->params.max_splits;
  out->refine = h->params.refine ? 1 : -1;
  return LIBRA_OK;
}

int libra_plan(libra_handle_t h, const int32_t* seq_lens_host, int32_t batch, void* workspace_dev, size_t workspace_bytes,
               void* stream) {
  if (!h || batch < 0 || batch > h->cfg.max_batch || (batch > 0 && !seq_lens_host) || !workspace_dev) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (reinterpret_cast<uintptr_t>(workspace_dev) % 256 != 0) return LIBRA_INVALID_ARGUMENT;
  if (workspace_bytes < h->workspace_bytes) return LIBRA_WORKSPACE_TOO_SMALL;
  const int64_t max_len = int64_t(h->cfg.block_table_ld) * h->cfg.page_size;
  for (int32_t b = 0; b < batch; ++b) {
    if (seq_lens_host[b] < 0 || seq_lens_host[b] > max_len) return LIBRA_INVALID_ARGUMENT;
  }
  h->planned = false;
  if (!libra::make_plan(h->params, h->cfg.num_kv_heads, seq_lens_host, batch, &h->plan)) return LIBRA_INVALID_ARGUMENT;
  const libra::HostPlan& pl = h->plan;
  if (int64_t(pl.items.size()) > h->max_items) return LIBRA_WORKSPACE_TOO_SMALL;  // cannot happen; see max_items()

  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  namespace L = libra::plan_layout;
  const int32_t n_items = int32_t(pl.items.size());
  const int32_t n_empty = int32_t(pl.empty.size());
  const int32_t n_combine = int32_t(pl.combine.size());
  h->plan_in_params = (n_items + n_empty <= L::kParamEntries) && (n_combine <= L::kParamFixEntries);

  // entries: work items (longest first), then one entry per empty sequence; merges separately
  int4* entries = h->pp.e;
  int4* fixes = h->pf.e;
  int k = 0;
  if (!h->plan_in_params) {
    k = h->next_staging;
    if (h->staging_used[k]) LIBRA_CUDA_TRY(h, cudaEventSynchronize(h->staging_done[k]));
    entries = reinterpret_cast<int4*>(h->staging[k]);
    fixes = entries + n_items + n_empty;
  }
  h->items_flat.resize(size_t(n_items) * 4);
  for (int32_t i = 0; i < n_items; ++i) {
    const libra::WorkItem& it = pl.items[i];
    entries[i] = make_int4(it.b | (it.j << L::kChunkShift) | (pl.num_splits[it.b] << L::kCountShift), it.kv_begin,
                           it.kv_end, (pl.num_splits[it.b] > 1) ? pl.item_offset[it.b] + it.j : -1);
    h->items_flat[4 * i + 0] = it.b;
    h->items_flat[4 * i + 1] = it.j;
    h->items_flat[4 * i + 2] = it.kv_begin;
    h->items_flat[4 * i + 3] = it.kv_end;
  }
  for (int32_t e = 0; e < n_empty; ++e) entries[n_items + e] = make_int4(pl.empty[e], 0, 0, 0);
  for (int32_t c = 0; c < n_combine; ++c) {
    const int32_t b = pl.combine[c];
    fixes[c] = make_int4(b, pl.item_offset[b], pl.num_splits[b], seq_lens_host[b]);
  }

  if (h->clean_workspace != workspace_dev) {  // control words and counters start at zero; the kernels keep the counters so
    h->clean_workspace = nullptr;
    LIBRA_CUDA_TRY(h, cudaMemsetAsync(workspace_dev, 0, h->cnt_off + h->cnt_bytes, st));
    h->clean_workspace = workspace_dev;
  }
  if (!h->plan_in_params) {
    const size_t bytes = size_t(n_items + n_empty + n_combine) * sizeof(int4);
    LIBRA_CUDA_TRY(h, cudaMemcpyAsync(static_cast<uint8_t*>(workspace_dev) + h->dev_entries_off, entries, bytes,
                                      cudaMemcpyHostToDevice, st));
    LIBRA_CUDA_TRY(h, cudaEventRecord(h->staging_done[k], st));
    h->staging_used[k] = true;
    h->next_staging = k ^ 1;
  }
  h->workspace = workspace_dev;
  h->num_items = n_items;
  h->last_stream = stream;
  h->planned = true;
  h->device_planned = false;
  h->decodes_on_plan = 0;
  h->planned_batch = batch;
  return LIBRA_OK;
}

int libra_plan_device(libra_handle_t h, const int32_t* seq_lens_dev, int32_t batch, void* workspace_dev,
                      size_t workspace_bytes, void* stream) {
  if (!h || batch < 0 || batch > h->cfg.max_batch || !seq_lens_dev || !workspace_dev) return LIBRA_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(workspace_dev) % 256 != 0) return LIBRA_INVALID_ARGUMENT;
  if (workspace_bytes < h->workspace_bytes) return LIBRA_WORKSPACE_TOO_SMALL;
  if (batch > libra::kDevPlanMax) return LIBRA_UNSUPPORTED_SHAPE;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace_dev);
  if (h->clean_workspace != workspace_dev) {
    h->clean_workspace = nullptr;
    LIBRA_CUDA_TRY(h, cudaMemsetAsync(workspace_dev, 0, h->cnt_off + h->cnt_bytes, st));
    h->clean_workspace = workspace_dev;
  }
  libra::PlanKernelParams p;
  p.seq_lens = seq_lens_dev;
  p.batch = batch;
  p.heads = h->cfg.num_kv_heads;
  p.slots = int64_t(h->params.n_sm) * h->params.ctas_per_sm * h->params.items_per_slot;
  p.chunk_align = h->params.chunk_align;
  p.min_chunk = h->params.min_chunk;
  p.max_splits = h->params.max_splits;
  p.wave_slots = int64_t(h->params.n_sm) * h->params.ctas_per_sm;
  p.refine = h->params.refine;
  const int64_t item_bound = std::min<int64_t>(libra::max_items(h->params, h->cfg.num_kv_heads, batch), h->max_items);
  p.max_items = int32_t(std::min<int64_t>(item_bound, libra::kDevPlanMax));
  const int threads = libra::plan_kernel_threads(batch, p.max_items);
  h->dev_item_bound = p.max_items;
  p.max_len = int32_t(std::min<int64_t>(int64_t(h->cfg.block_table_ld) * h->cfg.page_size, 0x7fffffff));
  p.counts = reinterpret_cast<int32_t*>(ws + h->dev_counts_off);
  p.per_seq = reinterpret_cast<int32_t*>(ws + h->dev_per_seq_off);
  p.entries = reinterpret_cast<int4*>(ws + h->dev_entries_off);
  p.fixes = reinterpret_cast<int4*>(ws + h->dev_fixes_off);
  p.error_word = reinterpret_cast<uint32_t*>(ws);
  {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(1);
    lc.blockDim = dim3(unsigned(threads));
    lc.dynamicSmemBytes = libra::plan_kernel_smem_bytes(threads);
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = h->pdl ? 1 : 0;   // a dependent of its predecessor: it waits inside before it reads or writes anything
    LIBRA_CUDA_TRY(h, cudaLaunchKernelEx(&lc, libra::plan_kernel, p));
  }
  ++h->launches;
  h->workspace = workspace_dev;
  h->last_stream = stream;
  h->planned = true;
  h->device_planned = true;
  h->decodes_on_plan = 0;
  h->plan_in_params = false;
  h->planned_batch = batch;
  return LIBRA_OK;
}

int libra_plan_export(libra_handle_t h, libra_plan_view_t* view) {
  if (!h || !view) return LIBRA_INVALID_ARGUMENT;
  if (!h->planned) return LIBRA_NOT_PLANNED;
  if (h->device_planned) {  // bring the device plan back (synchronises the stream of the plan call)
    DeviceGuard guard(h->cfg.device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(h->last_stream);
    const uint8_t* ws = static_cast<const uint8_t*>(h->workspace);
    int32_t counts[libra::plan_layout::kCountInts];
    LIBRA_CUDA_TRY(h, cudaMemcpyAsync(counts, ws + h->dev_counts_off, sizeof(counts), cudaMemcpyDeviceToHost, st));
    LIBRA_CUDA_TRY(h, cudaStreamSynchronize(st));
    namespace L = libra::plan_layout;
    const int32_t B = h->planned_batch, n_items = counts[L::kCntItems], n_cmb = counts[L::kCntCombine],
                  n_empty = counts[L::kCntEmpty];
    std::vector<int32_t> per_seq(size_t(4) * std::max(B, 1));
    std::vector<int4> entries(size_t(std::max(n_items + n_empty, 1)));
    std::vector<int4> fixes(size_t(std::max(n_cmb, 1)));
    LIBRA_CUDA_TRY(h, cudaMemcpyAsync(per_seq.data(), ws + h->dev_per_seq_off, size_t(4) * B * 4, cudaMemcpyDeviceToHost, st));
    LIBRA_CUDA_TRY(h, cudaMemcpyAsync(entries.data(), ws + h->dev_entries_off, size_t(n_items + n_empty) * 16,
                                      cudaMemcpyDeviceToHost, st));
    LIBRA_CUDA_TRY(h, cudaMemcpyAsync(fixes.data(), ws + h->dev_fixes_off, size_t(n_cmb) * 16, cudaMemcpyDeviceToHost, st));
    LIBRA_CUDA_TRY(h, cudaStreamSynchronize(st));
    libra::HostPlan& pl = h->plan;
    pl.batch = B;
    pl.chunk_target = counts[L::kCntChunkTarget];
    pl.bucket.assign(per_seq.begin(), per_seq.begin() + B);
    pl.num_splits.assign(per_seq.begin() + B, per_seq.begin() + 2 * B);
    pl.chunk_len.assign(per_seq.begin() + 2 * B, per_seq.begin() + 3 * B);
    pl.item_offset.assign(per_seq.begin() + 3 * B, per_seq.begin() + 4 * B);
    pl.items.resize(size_t(n_items));
    h->items_flat.resize(size_t(n_items) * 4);
    for (int32_t i = 0; i < n_items; ++i) {
      const int4 e = entries[size_t(i)];
      const int32_t b = e.x & (L::kMaxBatch - 1), j = (e.x >> L::kChunkShift) & 63;
      pl.items[size_t(i)] = libra::WorkItem{b, j, e.y, e.z};
      h->items_flat[4 * size_t(i) + 0] = b;
      h->items_flat[4 * size_t(i) + 1] = j;
      h->items_flat[4 * size_t(i) + 2] = e.y;
      h->items_flat[4 * size_t(i) + 3] = e.z;
    }
    pl.combine.resize(size_t(n_cmb));
    for (int32_t c = 0; c < n_cmb; ++c) pl.combine[size_t(c)] = fixes[size_t(c)].x;
    pl.empty.resize(size_t(n_empty));
    for (int32_t e = 0; e < n_empty; ++e) pl.empty[size_t(e)] = entries[size_t(n_items + e)].x;
    h->num_items = n_items;
  }
  const libra::HostPlan& pl = h->plan;
  view->batch = pl.batch;
  view->chunk_target = pl.chunk_target;
  view->num_items = int32_t(pl.items.size());
  view->num_combine = int32_t(pl.combine.size());
  view->num_empty = int32_t(pl.empty.size());
  view->bucket = pl.bucket.data();
  view->num_splits = pl.num_splits.data();
  view->chunk_len = pl.chunk_len.data();
  view->item_offset = pl.item_offset.data();
  view->items = h->items_flat.data();
  view->combine = pl.combine.data();
  view->empty = pl.empty.data();
  return LIBRA_OK;
}

int libra_set_combine_mode(libra_handle_t h, int32_t mode) {
  if (!h || mode < 0 || mode > 1) return LIBRA_INVALID_ARGUMENT;
  h->combine_mode = mode;
  return LIBRA_OK;
}

int libra_set_dependent_launch(libra_handle_t h, int32_t on) {
  if (!h || (on != 0 && on != 1)) return LIBRA_INVALID_ARGUMENT;
  h->pdl = (on == 1);
  return LIBRA_OK;
}

int libra_set_max_query_tokens(libra_handle_t h, int32_t max_q_len) {
  if (!h || max_q_len < 1) return LIBRA_INVALID_ARGUMENT;
  if (max_q_len * h->group > 16) return LIBRA_UNSUPPORTED_SHAPE;  // a unit's score tile has at most 16 columns
  if (max_q_len == h->max_q_len) return LIBRA_OK;
  h->max_q_len = max_q_len;
  refresh_params(h);
  compute_layout(h);
  h->planned = false;          // the workspace layout changed: plan again, into a workspace of the new size
  h->clean_workspace = nullptr;
  return LIBRA_OK;
}

int libra_set_kv_dtype(libra_handle_t h, int32_t dtype, float k_scale, float v_scale) {
  if (!h || (dtype != LIBRA_KV_BF16 && dtype != LIBRA_KV_E4M3)) return LIBRA_INVALID_ARGUMENT;
  if (dtype == LIBRA_KV_E4M3) {
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || !std::isfinite(k_scale) || !std::isfinite(v_scale)) return LIBRA_INVALID_ARGUMENT;
    // strides are in elements = bytes here: the tiled copies need 16-byte multiples
    if (h->stride_page % 16 || h->stride_head % 16 || h->stride_token % 16) return LIBRA_INVALID_ARGUMENT;
  }
  h->fp8 = (dtype == LIBRA_KV_E4M3);
  if (refresh_params(h)) h->planned = false;   // the planner's default slot count follows the pools' type: plan again
  h->fp8_variant = -1;
  h->k_scale = h->fp8 ? k_scale : 1.f;
  h->v_scale = h->fp8 ? v_scale : 1.f;
  for (int i = 0; i < libra_handle_s::kMapCache; ++i) h->maps[i].k_ptr = h->maps[i].v_ptr = nullptr;  // maps depend on the type
  return LIBRA_OK;
}

int libra_set_lse_output(libra_handle_t h, float* lse_dev) {
  if (!h || reinterpret_cast<uintptr_t>(lse_dev) % 4 != 0) return LIBRA_INVALID_ARGUMENT;
  h->lse_out = lse_dev;
  return LIBRA_OK;
}

int libra_set_early_prefetch(libra_handle_t h, int32_t on) {
  if (!h || (on != 0 && on != 1)) return LIBRA_INVALID_ARGUMENT;
  h->early_prefetch = (on == 1);
  return LIBRA_OK;
}

int libra_set_length_hint(libra_handle_t h, int32_t max_seq_len) {
  if (!h || max_seq_len < 0) return LIBRA_INVALID_ARGUMENT;
  h->length_hint = max_seq_len;
  return LIBRA_OK;
}

int libra_set_cache_warmup(libra_handle_t h, int32_t on) {
  if (!h || (on != 0 && on != 1)) return LIBRA_INVALID_ARGUMENT;
  h->l2_warmup = (on == 1);
  return LIBRA_OK;
}

int libra_set_variant(libra_handle_t h, int32_t warps, int32_t stages) {
  if (!h) return LIBRA_INVALID_ARGUMENT;
  if (h->fp8) {
    const std::vector<Fp8Variant>& fv = fp8_variants();
    for (size_t i = 0; i < fv.size(); ++i) {
      if (fv[i].warps == warps && fv[i].stages == stages) {
        h->fp8_variant = int(i);
        return LIBRA_OK;
      }
    }
    return LIBRA_UNSUPPORTED_SHAPE;
  }
  const std::vector<Variant>& vs = variants();
  const int di = (h->cfg.head_dim == 128) ? 1 : 0;
  const int ni = (h->group > 8) ? 1 : 0;
  for (size_t i = 0; i < vs.size(); ++i) {
    if (vs[i].warps == warps && vs[i].stages == stages && vs[i].fn[di][ni]) {
      h->variant = int(i);
      return LIBRA_OK;
    }
  }
  return LIBRA_UNSUPPORTED_SHAPE;
}

}  // extern "C"

namespace {

// Steps D and C; k_new / v_new non-null = append the current token's K and V rows on the way.
int decode_impl(libra_handle_t h, const void* q, const void* k_new, const void* v_new, const void* k_pages,
                const void* v_pages, const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream,
                bool loads_only = false, int32_t q_len = 1) {
  if (!h || !q || !k_pages || !v_pages || !block_table || !seq_lens || !out) return LIBRA_INVALID_ARGUMENT;
  if ((k_new == nullptr) != (v_new == nullptr)) return LIBRA_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(k_new) % 16 || reinterpret_cast<uintptr_t>(v_new) % 16) return LIBRA_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(k_pages) % 16 || reinterpret_cast<uintptr_t>(v_pages) % 16 ||
      reinterpret_cast<uintptr_t>(q) % 4 || reinterpret_cast<uintptr_t>(out) % 8) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (q_len < 1 || q_len > h->max_q_len) return LIBRA_INVALID_ARGUMENT;
  if (!h->planned) return LIBRA_NOT_PLANNED;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  libra_handle_s::PoolMaps* pm = nullptr;
  for (int i = 0; i < libra_handle_s::kMapCache; ++i) {
    if (h->maps[i].k_ptr == k_pages && h->maps[i].v_ptr == v_pages) pm = &h->maps[i];
  }
  if (!pm) {
    pm = &h->maps[h->next_map];
    h->next_map = (h->next_map + 1) % libra_handle_s::kMapCache;
    pm->k_ptr = pm->v_ptr = nullptr;
    int rc = encode_pool_map(h, k_pages, &pm->map_k, &h->pos_head, &h->pos_page, &h->pos_token);
    if (rc == LIBRA_OK) rc = encode_pool_map(h, v_pages, &pm->map_v, &h->pos_head, &h->pos_page, &h->pos_token);
    if (rc != LIBRA_OK) return rc;
    pm->k_ptr = k_pages;
    pm->v_ptr = v_pages;
  }

  uint8_t* ws = static_cast<uint8_t*>(h->workspace);
  uint32_t* err_dev = reinterpret_cast<uint32_t*>(ws);
  const int4* entries_dev = h->plan_in_params ? nullptr : reinterpret_cast<const int4*>(ws + h->dev_entries_off);
  const int32_t* dev_counts = h->device_planned ? reinterpret_cast<const int32_t*>(ws + h->dev_counts_off) : nullptr;

  cudaEvent_t* ev = nullptr;
  if (h->profiling && h->profiled_calls < kMaxProfiledCalls) {
    const size_t need = size_t(h->profiled_calls + 1) * 3;
    while (h->events.size() < need) {
      cudaEvent_t e;
      LIBRA_CUDA_TRY(h, cudaEventCreate(&e));
      h->events.push_back(e);
    }
    ev = &h->events[size_t(h->profiled_calls) * 3];
    LIBRA_CUDA_TRY(h, cudaEventRecord(ev[0], st));
  }

  const int di = (h->cfg.head_dim == 128) ? 1 : 0;
  const int ni = (h->group * q_len > 8) ? 1 : 0;
  // two column tiles: two blocks per SM where the plan was made for two slots; one column tile on such a plan
  // (a handle laid out for several query tokens that is given one): the same shape, so that the plan fits
  int auto_variant = ni ? (h->params.ctas_per_sm >= kTwoSlotCtas ? kVariantPair : kVariantTwoTiles)
                        : (h->two_slot_auto ? kVariantPair : kVariantOneTile);
  if (!ni && h->device_planned && h->length_hint > 0) {
    // the host has not seen the lengths; the caller's bound on them stands in for the longest unit
    if (h->length_hint <= kTinyUnitTokens) auto_variant = kVariantTinyUnits;
    else if (h->length_hint <= kShortUnitTokens) auto_variant = kVariantShortUnits;
  }
  if (!ni && !h->device_planned && !h->plan.items.empty()) {
    const int longest = h->plan.items.front().kv_end - h->plan.items.front().kv_begin;   // items are sorted longest first
    if (longest <= kTinyUnitTokens) auto_variant = kVariantTinyUnits;
    else if (longest <= kShortUnitTokens) auto_variant = kVariantShortUnits;
  }
  const Variant& v = variants()[h->variant >= 0 ? h->variant : auto_variant];
  const int32_t rows = q_len * h->cfg.num_q_heads;   // rows of q / out per sequence
  const bool fused = h->combine_mode == 1 || loads_only;
  // host plan: exact counts; device plan: upper bounds for the grids, the kernels read the counts themselves
  // (a device plan: one block at the end of the grid zeroes the rows of all empty sequences)
  const int32_t n_empty = h->device_planned ? 1 : int32_t(h->plan.empty.size());
  const int32_t n_combine = h->device_planned ? h->planned_batch : int32_t(h->plan.combine.size());
  const int32_t n_items_bound = h->device_planned ? h->dev_item_bound : h->num_items;
  const int32_t n_units = n_items_bound * h->cfg.num_kv_heads;
  if (n_units > 0 || n_empty > 0) {
    DecodeParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.block_table = block_table;
    p.seq_lens = seq_lens;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse_out = loads_only ? nullptr : h->lse_out;
    p.entries = entries_dev;
    p.dev_counts = dev_counts;
    p.partial_o = reinterpret_cast<float*>(ws + h->o_off);
    p.partial_lse = reinterpret_cast<float*>(ws + h->lse_off);
    p.error_word = err_dev;
    p.counters = reinterpret_cast<int32_t*>(ws + h->cnt_off);
    p.num_pages = h->cfg.num_pages;
    p.num_q_heads = rows;
    p.num_kv_heads = h->cfg.num_kv_heads;
    p.group = h->group;
    p.q_len = q_len;
    p.hq = h->cfg.num_q_heads;
    p.cols = q_len * h->group;
    p.block_table_ld = h->cfg.block_table_ld;
    p.scale_log2 = h->scale_log2 * h->k_scale;
    p.v_scale = h->fp8 ? h->v_scale : 1.f;
    p.pos_head = h->pos_head;
    p.pos_page = h->pos_page;
    p.pos_token = h->pos_token;
    p.tile_shift = (h->cfg.page_size == 16) ? 0 : (h->cfg.page_size == 32 ? 1 : 2);
    p.num_items = h->num_items;
    p.num_units = n_units;
    p.num_empty = n_empty;
    p.fused_combine = fused ? 1 : 0;
    p.early_prefetch = (h->early_prefetch && h->pdl) ? 1 : 0;
    // a plan in the workspace (device-made, or too large for the kernel parameters) may be read before the dependency
    // wait only once a decode launch has run on it: the kernel or copy that wrote it has then certainly finished
    p.l2_warmup = (h->l2_warmup && h->pdl && (h->plan_in_params || h->decodes_on_plan > 0)) ? 1 : 0;
    p.k_new = k_new;
    p.v_new = v_new;
    p.k_pool = const_cast<void*>(k_pages);
    p.v_pool = const_cast<void*>(v_pages);
    p.stride_page = h->stride_page;
    p.stride_head = h->stride_head;
    p.stride_token = h->stride_token;
    const unsigned grid = unsigned(n_units) + unsigned(n_empty);
    // launched as a programmatic dependent of whatever precedes it in the stream: its blocks may become
    // resident while that kernel drains; inside, they wait for it to finish before reading any input
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid);
    const bool full = k_new != nullptr || q_len > 1;   // the build with the append and several query tokens in it
    DecodeKernelFn fn = loads_only ? kLoadsOnlyFn[di][ni] : (full ? v.fn_append[di][ni] : v.fn[di][ni]);
    lc.blockDim = dim3(unsigned((loads_only ? kLoadsOnlyWarps : v.warps) * 32));
    lc.dynamicSmemBytes = size_t(loads_only ? kLoadsOnlySmem[di] : v.smem[di][ni]);
    if (h->fp8) {
      const bool two_slots = h->params.ctas_per_sm >= kTwoSlotCtas;
      int fp8_auto = ni ? (two_slots ? kFp8Pair : kFp8TwoTiles) : (two_slots ? kFp8OnePair : kFp8OneTile);
      if (!ni && !loads_only && auto_variant == kVariantShortUnits) fp8_auto = kFp8ShortUnits;
      if (!ni && !loads_only && auto_variant == kVariantTinyUnits) fp8_auto = kFp8TinyUnits;
      const Fp8Variant& fv = fp8_variants()[h->fp8_variant >= 0 ? h->fp8_variant : fp8_auto];
      fn = (full && !loads_only) ? fv.fn_append[di][ni] : fv.fn[di][loads_only ? 1 : 0][ni];
      lc.blockDim = dim3(unsigned(fv.warps * 32));
      lc.dynamicSmemBytes = size_t(fv.smem[di]);
    }
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = h->pdl ? 1 : 0;
    LIBRA_CUDA_TRY(h, cudaLaunchKernelEx(&lc, fn, pm->map_k, pm->map_v, p, h->pp));
    ++h->launches;
    ++h->decodes_on_plan;
  }
  if (ev) LIBRA_CUDA_TRY(h, cudaEventRecord(ev[1], st));
  if (!fused && n_combine > 0) {
    libra::CombineParams c;
    c.entries = h->plan_in_params ? nullptr
                                  : (h->device_planned ? reinterpret_cast<const int4*>(ws + h->dev_fixes_off)
                                                       : entries_dev + h->num_items + n_empty);
    c.dev_counts = dev_counts;
    c.partial_o = reinterpret_cast<const float*>(ws + h->o_off);
    c.partial_lse = reinterpret_cast<const float*>(ws + h->lse_off);
    c.seq_lens = seq_lens;
    c.out = static_cast<__nv_bfloat16*>(out);
    c.lse_out = h->lse_out;
    c.error_word = err_dev;
    c.num_q_heads = rows;
    // a programmatic dependent of the decode kernel: it may be scheduled while that kernel drains and
    // waits inside (griddepcontrol.wait) for it to finish
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(unsigned(n_combine), unsigned((rows + libra::kCombineWarps - 1) / libra::kCombineWarps));
    lc.blockDim = dim3(libra::kCombineWarps * 32);
    lc.dynamicSmemBytes = 0;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = (ev || !h->pdl) ? 0 : 1;  // with events around it, it is an ordinary launch
    if (h->cfg.head_dim == 128) LIBRA_CUDA_TRY(h, cudaLaunchKernelEx(&lc, libra::combine_kernel<128>, c, h->pf));
    else LIBRA_CUDA_TRY(h, cudaLaunchKernelEx(&lc, libra::combine_kernel<64>, c, h->pf));
    ++h->launches;
  }
  if (ev) {
    LIBRA_CUDA_TRY(h, cudaEventRecord(ev[2], st));
    ++h->profiled_calls;
  }
  h->last_stream = stream;
  return LIBRA_OK;
}

}  // namespace

extern "C" {

int libra_decode_attn(libra_handle_t h, const void* q, const void* k_pages, const void* v_pages,
                      const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream) {
  return decode_impl(h, q, nullptr, nullptr, k_pages, v_pages, block_table, seq_lens, out, stream);
}

int libra_decode_attn_append(libra_handle_t h, const void* q, const void* k_new, const void* v_new, void* k_pages,
                             void* v_pages, const int32_t* block_table, const int32_t* seq_lens, void* out,
                             void* stream) {
  if (!k_new || !v_new) return LIBRA_INVALID_ARGUMENT;
  return decode_impl(h, q, k_new, v_new, k_pages, v_pages, block_table, seq_lens, out, stream);
}

int libra_host_staging_size(libra_handle_t h, int32_t batch, size_t* bytes) {
  if (!h || !bytes || batch < 0 || batch > h->cfg.max_batch) return LIBRA_INVALID_ARGUMENT;
  const size_t qo = align_up(size_t(batch) * h->cfg.num_q_heads * h->cfg.head_dim * 2, 256);
  const size_t pool = align_up(size_t(h->cfg.num_pages) * size_t(h->stride_page) * 2, 256);
  const size_t bt = align_up(size_t(batch) * h->cfg.block_table_ld * 4, 256);
  const size_t sl = align_up(size_t(batch) * 4, 256);
  *bytes = 2 * qo + 2 * pool + bt + sl;
  return LIBRA_OK;
}

int libra_decode_attn_host(libra_handle_t h, const void* q_host, const void* k_pages_host, const void* v_pages_host,
                           const int32_t* block_table_host, const int32_t* seq_lens_host, int32_t batch, void* out_host,
                           void* staging_dev, size_t staging_bytes, void* workspace_dev, size_t workspace_bytes,
                           void* stream) {
  if (!h || !q_host || !k_pages_host || !v_pages_host || !block_table_host || !seq_lens_host || !out_host ||
      !staging_dev || batch <= 0) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (h->fp8) return LIBRA_UNSUPPORTED_SHAPE;   // the host-buffer path is sized for bf16 pools
  if (reinterpret_cast<uintptr_t>(staging_dev) % 256 != 0) return LIBRA_INVALID_ARGUMENT;
  size_t need = 0;
  int rc = libra_host_staging_size(h, batch, &need);
  if (rc != LIBRA_OK) return rc;
  if (staging_bytes < need) return LIBRA_WORKSPACE_TOO_SMALL;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const size_t q_bytes = size_t(batch) * h->cfg.num_q_heads * h->cfg.head_dim * 2;
  const size_t pool_bytes = size_t(h->cfg.num_pages) * size_t(h->stride_page) * 2;
  const size_t bt_bytes = size_t(batch) * h->cfg.block_table_ld * 4;
  const size_t sl_bytes = size_t(batch) * 4;
  uint8_t* base = static_cast<uint8_t*>(staging_dev);
  uint8_t* d_q = base;
  uint8_t* d_out = d_q + align_up(q_bytes, 256);
  uint8_t* d_k = d_out + align_up(q_bytes, 256);
  uint8_t* d_v = d_k + align_up(pool_bytes, 256);
  uint8_t* d_bt = d_v + align_up(pool_bytes, 256);
  uint8_t* d_sl = d_bt + align_up(bt_bytes, 256);

  // the plan needs only the host lengths, so it goes first and its upload overlaps the big copies
  rc = libra_plan(h, seq_lens_host, batch, workspace_dev, workspace_bytes, stream);
  if (rc != LIBRA_OK) return rc;
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_q, q_host, q_bytes, cudaMemcpyHostToDevice, st));
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_k, k_pages_host, pool_bytes, cudaMemcpyHostToDevice, st));
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_v, v_pages_host, pool_bytes, cudaMemcpyHostToDevice, st));
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_bt, block_table_host, bt_bytes, cudaMemcpyHostToDevice, st));
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_sl, seq_lens_host, sl_bytes, cudaMemcpyHostToDevice, st));
  rc = libra_decode_attn(h, d_q, d_k, d_v, reinterpret_cast<const int32_t*>(d_bt),
                         reinterpret_cast<const int32_t*>(d_sl), d_out, stream);
  if (rc != LIBRA_OK) return rc;
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(out_host, d_out, q_bytes, cudaMemcpyDeviceToHost, st));
  uint32_t word = 0;
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(&word, workspace_dev, 4, cudaMemcpyDeviceToHost, st));
  LIBRA_CUDA_TRY(h, cudaStreamSynchronize(st));
  if (word) LIBRA_CUDA_TRY(h, cudaMemsetAsync(workspace_dev, 0, 4, st));
  return word ? LIBRA_DEVICE_FLAGGED : LIBRA_OK;
}

int libra_host_io_staging_size(libra_handle_t h, int32_t batch, size_t* bytes) {
  if (!h || !bytes || batch < 0 || batch > h->cfg.max_batch) return LIBRA_INVALID_ARGUMENT;
  const size_t qo = align_up(size_t(batch) * h->cfg.num_q_heads * h->cfg.head_dim * 2, 256);
  const size_t bt = align_up(size_t(batch) * h->cfg.block_table_ld * 4, 256);
  const size_t sl = align_up(size_t(batch) * 4, 256);
  *bytes = 2 * qo + bt + sl;
  return LIBRA_OK;
}

int libra_decode_attn_host_io(libra_handle_t h, const void* q_host, const void* k_pages, const void* v_pages,
                              const int32_t* block_table_host, const int32_t* seq_lens_host, int32_t batch,
                              void* out_host, void* staging_dev, size_t staging_bytes, void* workspace_dev,
                              size_t workspace_bytes, void* stream) {
  if (!h || !q_host || !k_pages || !v_pages || !block_table_host || !seq_lens_host || !out_host || !staging_dev ||
      batch <= 0) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (reinterpret_cast<uintptr_t>(staging_dev) % 256 != 0) return LIBRA_INVALID_ARGUMENT;
  size_t need = 0;
  int rc = libra_host_io_staging_size(h, batch, &need);
  if (rc != LIBRA_OK) return rc;
  if (staging_bytes < need) return LIBRA_WORKSPACE_TOO_SMALL;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const size_t q_bytes = size_t(batch) * h->cfg.num_q_heads * h->cfg.head_dim * 2;
  const size_t bt_bytes = size_t(batch) * h->cfg.block_table_ld * 4;
  const size_t sl_bytes = size_t(batch) * 4;
  uint8_t* d_q = static_cast<uint8_t*>(staging_dev);
  uint8_t* d_out = d_q + align_up(q_bytes, 256);
  uint8_t* d_bt = d_out + align_up(q_bytes, 256);
  uint8_t* d_sl = d_bt + align_up(bt_bytes, 256);

  rc = libra_plan(h, seq_lens_host, batch, workspace_dev, workspace_bytes, stream);
  if (rc != LIBRA_OK) return rc;
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_q, q_host, q_bytes, cudaMemcpyHostToDevice, st));
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_bt, block_table_host, bt_bytes, cudaMemcpyHostToDevice, st));
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(d_sl, seq_lens_host, sl_bytes, cudaMemcpyHostToDevice, st));
  rc = libra_decode_attn(h, d_q, k_pages, v_pages, reinterpret_cast<const int32_t*>(d_bt),
                         reinterpret_cast<const int32_t*>(d_sl), d_out, stream);
  if (rc != LIBRA_OK) return rc;
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(out_host, d_out, q_bytes, cudaMemcpyDeviceToHost, st));
  uint32_t word = 0;
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(&word, workspace_dev, 4, cudaMemcpyDeviceToHost, st));
  LIBRA_CUDA_TRY(h, cudaStreamSynchronize(st));
  if (word) LIBRA_CUDA_TRY(h, cudaMemsetAsync(workspace_dev, 0, 4, st));
  return word ? LIBRA_DEVICE_FLAGGED : LIBRA_OK;
}

int libra_decode_attn_static(libra_handle_t h, const int32_t* seq_lens_host, int32_t batch, const void* q,
                             const void* k_pages, const void* v_pages, const int32_t* block_table,
                             const int32_t* seq_lens, void* out, void* stream) {
  if (!h) return LIBRA_INVALID_ARGUMENT;
  if (h->workspace_bytes > size_t(LIBRA_STATIC_SCRATCH_BYTES)) return LIBRA_WORKSPACE_TOO_SMALL;
  // everything libra_decode_attn would refuse is refused here, before the shared region or the handle's
  // plan is touched: a rejected call must not clear another call's error word or re-plan the handle
  if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !out) return LIBRA_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(k_pages) % 16 || reinterpret_cast<uintptr_t>(v_pages) % 16 ||
      reinterpret_cast<uintptr_t>(q) % 4 || reinterpret_cast<uintptr_t>(out) % 8) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (batch < 0 || batch > h->cfg.max_batch || (batch > 0 && !seq_lens_host)) return LIBRA_INVALID_ARGUMENT;
  {
    const int64_t max_len = int64_t(h->cfg.block_table_ld) * h->cfg.page_size;
    for (int32_t b = 0; b < batch; ++b) {
      if (seq_lens_host[b] < 0 || seq_lens_host[b] > max_len) return LIBRA_INVALID_ARGUMENT;
    }
  }
  void* scratch = nullptr;
  {
    DeviceGuard guard(h->cfg.device);  // the symbol's address is per device: look it up with that device current
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    const cudaError_t e = static_scratch_address(h->cfg.device, &scratch);
    if (e != cudaSuccess) return fail_cuda(h, e);
  }
  // the region keeps whatever the previous call (of any handle) left: have the plan step clear the
  // control words and arrival counters again, on `stream`, before the kernels run
  h->clean_workspace = nullptr;
  int rc = libra_plan(h, seq_lens_host, batch, scratch, size_t(LIBRA_STATIC_SCRATCH_BYTES), stream);
  if (rc != LIBRA_OK) return rc;
  return libra_decode_attn(h, q, k_pages, v_pages, block_table, seq_lens, out, stream);
}

int libra_last_cuda_error(libra_handle_t h) { return h ? h->last_cuda_error : 0; }

int libra_debug_error_word(libra_handle_t h, uint32_t* word) {
  if (!h || !word) return LIBRA_INVALID_ARGUMENT;
  if (!h->planned) return LIBRA_NOT_PLANNED;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  cudaStream_t st = static_cast<cudaStream_t>(h->last_stream);
  LIBRA_CUDA_TRY(h, cudaMemcpyAsync(word, h->workspace, 4, cudaMemcpyDeviceToHost, st));
  LIBRA_CUDA_TRY(h, cudaStreamSynchronize(st));
  if (*word) LIBRA_CUDA_TRY(h, cudaMemsetAsync(h->workspace, 0, 4, st));  // reading a set word clears it
  return LIBRA_OK;
}

}  // extern "C"

namespace {

int kv_move_impl(libra_handle_t h, bool gather, void* k_pages, void* v_pages, void* k_dense, void* v_dense,
                 const int32_t* block_table, const int32_t* seq_lens, const int64_t* token_offsets, int32_t batch,
                 int32_t max_seq_len, int32_t head_begin, int32_t head_count, void* error_word_dev, void* stream) {
  if (!h || !k_pages || !v_pages || !k_dense || !v_dense || !block_table || !seq_lens || !token_offsets ||
      !error_word_dev) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (batch < 0 || max_seq_len < 0 || head_begin < 0 || head_count <= 0 ||
      head_begin + head_count > h->cfg.num_kv_heads) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (int64_t(max_seq_len) > int64_t(h->cfg.block_table_ld) * h->cfg.page_size) return LIBRA_INVALID_ARGUMENT;
  if (reinterpret_cast<uintptr_t>(k_pages) % 16 || reinterpret_cast<uintptr_t>(v_pages) % 16 ||
      reinterpret_cast<uintptr_t>(k_dense) % 16 || reinterpret_cast<uintptr_t>(v_dense) % 16 ||
      reinterpret_cast<uintptr_t>(error_word_dev) % 4) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (batch == 0 || max_seq_len == 0) return LIBRA_OK;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  libra::KvMoveParams p;
  p.k_pool = static_cast<__nv_bfloat16*>(k_pages);
  p.v_pool = static_cast<__nv_bfloat16*>(v_pages);
  p.k_dense = static_cast<__nv_bfloat16*>(k_dense);
  p.v_dense = static_cast<__nv_bfloat16*>(v_dense);
  p.block_table = block_table;
  p.seq_lens = seq_lens;
  p.token_offsets = token_offsets;
  // an E4M3 row of 128 codes is moved as a row of 64 two-byte elements (strides are multiples of 16 bytes)
  const int64_t unit = h->fp8 ? 2 : 1;
  p.stride_page = h->stride_page / unit;
  p.stride_head = h->stride_head / unit;
  p.stride_token = h->stride_token / unit;
  p.num_pages = h->cfg.num_pages;
  p.block_table_ld = h->cfg.block_table_ld;
  p.head_begin = head_begin;
  p.head_count = head_count;
  p.page_size = h->cfg.page_size;
  p.error_word = static_cast<uint32_t*>(error_word_dev);
  const int pages = (max_seq_len + h->cfg.page_size - 1) / h->cfg.page_size;
  dim3 grid(unsigned((pages + libra::kMovePagesPerBlock - 1) / libra::kMovePagesPerBlock), unsigned(batch));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int row_units = h->cfg.head_dim / int(unit);   // two-byte elements per row: 128, 64, or 32 (8-bit, head_dim 64)
  if (row_units == 128) {
    if (gather) libra::kv_move_kernel<128, true><<<grid, libra::kMoveThreads, 0, st>>>(p);
    else libra::kv_move_kernel<128, false><<<grid, libra::kMoveThreads, 0, st>>>(p);
  } else if (row_units == 64) {
    if (gather) libra::kv_move_kernel<64, true><<<grid, libra::kMoveThreads, 0, st>>>(p);
    else libra::kv_move_kernel<64, false><<<grid, libra::kMoveThreads, 0, st>>>(p);
  } else {
    if (gather) libra::kv_move_kernel<32, true><<<grid, libra::kMoveThreads, 0, st>>>(p);
    else libra::kv_move_kernel<32, false><<<grid, libra::kMoveThreads, 0, st>>>(p);
  }
  LIBRA_CUDA_TRY(h, cudaGetLastError());
  ++h->launches;
  return LIBRA_OK;
}

}  // namespace

extern "C" {

int libra_kv_gather(libra_handle_t h, const void* k_pages, const void* v_pages, const int32_t* block_table,
                    const int32_t* seq_lens, const int64_t* token_offsets, int32_t batch, int32_t max_seq_len,
                    int32_t head_begin, int32_t head_count, void* k_dense, void* v_dense, void* error_word_dev,
                    void* stream) {
  return kv_move_impl(h, true, const_cast<void*>(k_pages), const_cast<void*>(v_pages), k_dense, v_dense, block_table,
                      seq_lens, token_offsets, batch, max_seq_len, head_begin, head_count, error_word_dev, stream);
}

int libra_kv_scatter(libra_handle_t h, const void* k_dense, const void* v_dense, const int32_t* block_table,
                     const int32_t* seq_lens, const int64_t* token_offsets, int32_t batch, int32_t max_seq_len,
                     int32_t head_begin, int32_t head_count, void* k_pages, void* v_pages, void* error_word_dev,
                     void* stream) {
  return kv_move_impl(h, false, k_pages, v_pages, const_cast<void*>(k_dense), const_cast<void*>(v_dense), block_table,
                      seq_lens, token_offsets, batch, max_seq_len, head_begin, head_count, error_word_dev, stream);
}

int libra_debug_wait_selftest(libra_handle_t h, void* stream) {
  if (!h) return LIBRA_INVALID_ARGUMENT;
  if (!h->planned) return LIBRA_NOT_PLANNED;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  libra::wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<uint32_t*>(h->workspace), 1024u);
  LIBRA_CUDA_TRY(h, cudaGetLastError());
  h->last_stream = stream;
  return LIBRA_OK;
}

int libra_decode_attn_multi(libra_handle_t h, const void* q, int32_t q_len, const void* k_pages, const void* v_pages,
                            const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream) {
  return decode_impl(h, q, nullptr, nullptr, k_pages, v_pages, block_table, seq_lens, out, stream, false, q_len);
}

int libra_decode_attn_multi_append(libra_handle_t h, const void* q, int32_t q_len, const void* k_new, const void* v_new,
                                   void* k_pages, void* v_pages, const int32_t* block_table, const int32_t* seq_lens,
                                   void* out, void* stream) {
  if (!k_new || !v_new) return LIBRA_INVALID_ARGUMENT;
  return decode_impl(h, q, k_new, v_new, k_pages, v_pages, block_table, seq_lens, out, stream, false, q_len);
}

int libra_debug_gather_read(libra_handle_t h, const void* q, const void* k_pages, const void* v_pages,
                            const int32_t* block_table, const int32_t* seq_lens, void* out, void* stream) {
  return decode_impl(h, q, nullptr, nullptr, k_pages, v_pages, block_table, seq_lens, out, stream, true);
}

int libra_debug_stream_read(libra_handle_t h, const void* buf_dev, size_t bytes, void* stream) {
  if (!h || !buf_dev || bytes < 16 || reinterpret_cast<uintptr_t>(buf_dev) % 16 != 0) return LIBRA_INVALID_ARGUMENT;
  if (!h->planned) return LIBRA_NOT_PLANNED;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  uint32_t* sink = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(h->workspace) + 128);  // an unused control word
  libra::stream_read_kernel<<<unsigned(h->params.n_sm * libra::kReadBlocksPerSm), libra::kReadThreads, 0,
                              static_cast<cudaStream_t>(stream)>>>(static_cast<const uint4*>(buf_dev), bytes / 16, sink);
  LIBRA_CUDA_TRY(h, cudaGetLastError());
  ++h->launches;
  h->last_stream = stream;
  return LIBRA_OK;
}

int libra_merge_parts(int32_t device, const void* parts_out, const float* parts_lse, int32_t n_parts, int64_t rows,
                      int32_t head_dim, void* out, float* lse_out, void* stream) {
  if (device < 0 || !parts_out || !parts_lse || !out || n_parts < 1 || n_parts > 64 || rows < 0) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (head_dim != 64 && head_dim != 128) return LIBRA_UNSUPPORTED_SHAPE;
  if (reinterpret_cast<uintptr_t>(parts_out) % 16 || reinterpret_cast<uintptr_t>(parts_lse) % 16 ||
      reinterpret_cast<uintptr_t>(out) % 16 || reinterpret_cast<uintptr_t>(lse_out) % 4) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (rows > (int64_t(1) << 31) * libra::kMergeWarps - 1) return LIBRA_INVALID_ARGUMENT;   // grid limit
  if (rows == 0) return LIBRA_OK;
  DeviceGuard guard(device);
  if (guard.err != cudaSuccess) return fail_cuda(nullptr, guard.err);
  libra::MergeParams p;
  p.parts_out = static_cast<const __nv_bfloat16*>(parts_out);
  p.parts_lse = parts_lse;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.lse_out = lse_out;
  p.rows = rows;
  p.n_parts = n_parts;
  const unsigned grid = unsigned((rows + libra::kMergeWarps - 1) / libra::kMergeWarps);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (head_dim == 128) libra::merge_parts_kernel<128><<<grid, libra::kMergeWarps * 32, 0, st>>>(p);
  else libra::merge_parts_kernel<64><<<grid, libra::kMergeWarps * 32, 0, st>>>(p);
  LIBRA_CUDA_TRY(nullptr, cudaGetLastError());
  return LIBRA_OK;
}

int libra_ring_step(int32_t device, void* dst, const void* own, const void* received, size_t bytes, int32_t dtype,
                    const uint32_t* ready_flag, uint32_t expected, uint32_t timeout_us, uint32_t* status_dev,
                    int32_t num_blocks, void* stream) {
  if (device < 0 || !dst || !received || !ready_flag || !status_dev) return LIBRA_INVALID_ARGUMENT;
  if (dtype != LIBRA_RING_F32 && dtype != LIBRA_RING_BF16) return LIBRA_INVALID_ARGUMENT;
  if (bytes % 16 != 0 || num_blocks < 0 || num_blocks > 64 || timeout_us == 0 || timeout_us > 10000000u) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (reinterpret_cast<uintptr_t>(dst) % 16 || reinterpret_cast<uintptr_t>(own) % 16 ||
      reinterpret_cast<uintptr_t>(received) % 16 || reinterpret_cast<uintptr_t>(ready_flag) % 4 ||
      reinterpret_cast<uintptr_t>(status_dev) % 4) {
    return LIBRA_INVALID_ARGUMENT;
  }
  DeviceGuard guard(device);
  if (guard.err != cudaSuccess) return fail_cuda(nullptr, guard.err);
  libra::RingStepParams p;
  p.dst = dst;
  p.own = own;
  p.received = received;
  p.n16 = bytes / 16;
  p.status = status_dev;
  p.bf16 = (dtype == LIBRA_RING_BF16) ? 1 : 0;
  libra::ring_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ready_flag, expected, timeout_us, status_dev);
  if (cudaGetLastError() != cudaSuccess) return LIBRA_CUDA_ERROR;
  libra::ring_step_kernel<<<unsigned(num_blocks == 0 ? 2 : num_blocks), libra::kRingThreads, 0,
                            static_cast<cudaStream_t>(stream)>>>(p);
  if (cudaGetLastError() != cudaSuccess) return LIBRA_CUDA_ERROR;
  return LIBRA_OK;
}

int libra_ring_all_reduce_local(int32_t device, void* const* bufs, int32_t n_members, size_t bytes, int32_t dtype,
                                size_t piece_bytes, const uint32_t* ready_flag, uint32_t expected, uint32_t timeout_us,
                                uint32_t* status_dev, int32_t num_blocks, void* stream) {
  if (!bufs || n_members < 1 || n_members > LIBRA_RING_MAX_MEMBERS || bytes % 16 != 0 || piece_bytes < 16 ||
      piece_bytes % 16 != 0) {
    return LIBRA_INVALID_ARGUMENT;
  }
  for (int32_t i = 0; i < n_members; ++i) {
    if (!bufs[i] || reinterpret_cast<uintptr_t>(bufs[i]) % 16 != 0) return LIBRA_INVALID_ARGUMENT;
  }
  libra_ring_t ring;
  int32_t ids[LIBRA_RING_MAX_MEMBERS];
  for (int32_t i = 0; i < n_members; ++i) ids[i] = i;
  int rc = libra_ring_init(&ring, ids, n_members);
  if (rc != LIBRA_OK) return rc;
  // every member's schedule; the receive records of one (phase, step) of all members form one round of launches
  std::vector<std::vector<libra_ring_op_t>> sched;
  sched.resize(size_t(n_members));
  for (int32_t i = 0; i < n_members; ++i) {
    int32_t need = 0;
    rc = libra_ring_schedule(&ring, i, int64_t(bytes), int64_t(piece_bytes), nullptr, 0, &need);
    if (rc != LIBRA_OK && rc != LIBRA_WORKSPACE_TOO_SMALL) return rc;
    sched[size_t(i)].resize(size_t(need));
    rc = libra_ring_schedule(&ring, i, int64_t(bytes), int64_t(piece_bytes), sched[size_t(i)].data(), need, &need);
    if (rc != LIBRA_OK) return rc;
  }
  std::vector<size_t> cursor;
  cursor.assign(size_t(n_members), 0);
  for (int32_t phase = 0; phase < 2; ++phase) {
    for (int32_t step = 0; step + 1 < n_members; ++step) {
      for (int32_t i = 0; i < n_members; ++i) {
        const std::vector<libra_ring_op_t>& ops = sched[size_t(i)];
        size_t& c = cursor[size_t(i)];
        for (; c < ops.size() && ops[c].phase == phase && ops[c].step == step; ++c) {
          const libra_ring_op_t& op = ops[c];
          if (op.kind == LIBRA_RING_OP_SEND) continue;   // on one device the receiver reads the sender's buffer in place
          uint8_t* mine = static_cast<uint8_t*>(bufs[i]) + op.offset;
          const uint8_t* theirs = static_cast<const uint8_t*>(bufs[op.peer]) + op.offset;
          rc = libra_ring_step(device, mine, op.kind == LIBRA_RING_OP_RECV_REDUCE ? mine : nullptr, theirs,
                               size_t(op.bytes), dtype, ready_flag, expected, timeout_us, status_dev, num_blocks, stream);
          if (rc != LIBRA_OK) return rc;
        }
      }
    }
  }
  return LIBRA_OK;
}

int libra_profile_begin(libra_handle_t h) {
  if (!h) return LIBRA_INVALID_ARGUMENT;
  h->profiling = true;
  h->profiled_calls = 0;
  return LIBRA_OK;
}

int libra_profile_end(libra_handle_t h, double* decode_ms, double* combine_ms, int32_t* calls) {
  if (!h) return LIBRA_INVALID_ARGUMENT;
  DeviceGuard guard(h->cfg.device);
  if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
  double d = 0.0, c = 0.0;
  for (int i = 0; i < h->profiled_calls; ++i) {
    cudaEvent_t* ev = &h->events[size_t(i) * 3];
    LIBRA_CUDA_TRY(h, cudaEventSynchronize(ev[2]));
    float a = 0.f, b = 0.f;
    LIBRA_CUDA_TRY(h, cudaEventElapsedTime(&a, ev[0], ev[1]));
    LIBRA_CUDA_TRY(h, cudaEventElapsedTime(&b, ev[1], ev[2]));
    d += a;
    c += b;
  }
  if (decode_ms) *decode_ms = d;
  if (combine_ms) *combine_ms = c;
  if (calls) *calls = h->profiled_calls;
  h->profiling = false;
  h->profiled_calls = 0;
  return LIBRA_OK;
}

int libra_launch_count(libra_handle_t h, int64_t* launches) {
  if (!h || !launches) return LIBRA_INVALID_ARGUMENT;
  *launches = h->launches;
  return LIBRA_OK;
}

}  // extern "C"
