// C-ABI entry points: plan creation, tensor-map encoding and the launch.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <new>

#include "../../include/exo_gemm.h"
#include "gemm_kernel.cuh"
#include "lean_kernel.cuh"
#include "lean_pair_kernel.cuh"
#include "repack.cuh"
#include "plan.h"
#ifdef EXO_GEMM_SHARE_PAIRS
#include "cluster4/share_pairs.cuh"
#endif

namespace exo {

using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const GemmParams);

template <int G, int BN, int KSUB>
static KernelFn pick_out(int out) {
  switch (out) {
    case EXO_GEMM_BF16: return exo_gemm_kernel<G, BN, kOutBf16, KSUB>;
    case EXO_GEMM_FP16: return exo_gemm_kernel<G, BN, kOutFp16, KSUB>;
    default:            return exo_gemm_kernel<G, BN, kOutFp32, KSUB>;
  }
}

template <int KSUB>
static KernelFn pick_shape(int cta_group, int bn, int out) {
  if (cta_group == 2) return bn == 256 ? pick_out<2, 256, KSUB>(out) : pick_out<2, 128, KSUB>(out);
  if (bn == 256) return pick_out<1, 256, KSUB>(out);
  if (bn == 128) return pick_out<1, 128, KSUB>(out);
  return pick_out<1, 64, KSUB>(out);
}

#ifdef EXO_GEMM_SHARE_PAIRS
constexpr bool kHaveSharePairs = true;
template <int KSUB>
static KernelFn pick_shared(int out) {
  switch (out) {
    case EXO_GEMM_BF16: return exo_gemm_kernel<2, 256, kOutBf16, KSUB, SharePairs>;
    case EXO_GEMM_FP16: return exo_gemm_kernel<2, 256, kOutFp16, KSUB, SharePairs>;
    default:            return exo_gemm_kernel<2, 256, kOutFp32, KSUB, SharePairs>;
  }
}
#else
constexpr bool kHaveSharePairs = false;
template <int KSUB>
static KernelFn pick_shared(int) { return nullptr; }
#endif

static KernelFn pick_tall(int out) {
  switch (out) {
    case EXO_GEMM_BF16: return exo_gemm_kernel<2, 256, kOutBf16, 1, NoShare, 2>;
    case EXO_GEMM_FP16: return exo_gemm_kernel<2, 256, kOutFp16, 1, NoShare, 2>;
    default:            return exo_gemm_kernel<2, 256, kOutFp32, 1, NoShare, 2>;
  }
}

// the instantiations that can add the parts of a cut tile onto C (fp32 C, plain tiles)
template <int KSUB>
static KernelFn pick_reduce(int cta_group, int bn) {
  if (cta_group == 2) return bn == 256 ? exo_gemm_kernel<2, 256, kOutFp32, KSUB, NoShare, 1, true>
                                       : exo_gemm_kernel<2, 128, kOutFp32, KSUB, NoShare, 1, true>;
  if (bn == 256) return exo_gemm_kernel<1, 256, kOutFp32, KSUB, NoShare, 1, true>;
  if (bn == 128) return exo_gemm_kernel<1, 128, kOutFp32, KSUB, NoShare, 1, true>;
  return exo_gemm_kernel<1, 64, kOutFp32, KSUB, NoShare, 1, true>;
}

static KernelFn pick_kernel(int cta_group, int bn, int ksub, int out, int pairs = 1, int mrep = 1, bool reduce = false) {
  if (reduce) return ksub == 2 ? pick_reduce<2>(cta_group, bn) : pick_reduce<1>(cta_group, bn);
  if (mrep == 2) return pick_tall(out);
  if (pairs == 2) return ksub == 2 ? pick_shared<2>(out) : pick_shared<1>(out);
  return ksub == 2 ? pick_shape<2>(cta_group, bn, out) : pick_shape<1>(cta_group, bn, out);
}

// the one-tile-per-CTA kernel: 128 x 64 or 128 x 128 tiles
template <int BN, int KSUB>
static KernelFn pick_lean_out(int out) {
  switch (out) {
    case EXO_GEMM_BF16: return exo_gemm_lean_kernel<BN, kOutBf16, KSUB>;
    case EXO_GEMM_FP16: return exo_gemm_lean_kernel<BN, kOutFp16, KSUB>;
    default:            return exo_gemm_lean_kernel<BN, kOutFp32, KSUB>;
  }
}
static KernelFn pick_lean(int bn, int ksub, int out) {
  if (bn == 128) return ksub == 2 ? pick_lean_out<128, 2>(out) : pick_lean_out<128, 1>(out);
  return ksub == 2 ? pick_lean_out<64, 2>(out) : pick_lean_out<64, 1>(out);
}

// ... and its form for a CTA pair per tile: 256 x 128 or 256 x 256
template <int BN, int KSUB>
static KernelFn pick_lean_pair_out(int out) {
  switch (out) {
    case EXO_GEMM_BF16: return exo_gemm_lean_pair_kernel<BN, kOutBf16, KSUB>;
    case EXO_GEMM_FP16: return exo_gemm_lean_pair_kernel<BN, kOutFp16, KSUB>;
    default:            return exo_gemm_lean_pair_kernel<BN, kOutFp32, KSUB>;
  }
}
static KernelFn pick_lean_pair(int bn, int ksub, int out) {
  if (bn == 256) return ksub == 2 ? pick_lean_pair_out<256, 2>(out) : pick_lean_pair_out<256, 1>(out);
  return ksub == 2 ? pick_lean_pair_out<128, 2>(out) : pick_lean_pair_out<128, 1>(out);
}

// kernel and dynamic shared memory of a plan's configuration
static KernelFn kernel_of(const TileConfig& cfg, int c_dtype, bool reduce) {
  if (cfg.lean && cfg.cta_group == 2) return pick_lean_pair(cfg.tile_n, cfg.ksub, c_dtype);
  if (cfg.lean) return pick_lean(cfg.tile_n, cfg.ksub, c_dtype);
  return pick_kernel(cfg.cta_group, cfg.tile_n, cfg.ksub, c_dtype, cfg.pairs, cfg.mrep, reduce);
}
static int smem_of(const TileConfig& cfg, int c_dtype) {
  if (cfg.lean && cfg.cta_group == 2) return lean_pair_smem_bytes(cfg.tile_n, cfg.ksub, cfg.stages, c_dtype == EXO_GEMM_FP32 ? 4 : 2);
  if (cfg.lean) return lean_smem_bytes(cfg.tile_n, cfg.ksub, cfg.stages, c_dtype == EXO_GEMM_FP32 ? 4 : 2, cfg.lean);
  return smem_bytes_for(cfg.cta_group, cfg.tile_n, cfg.ksub, cfg.stages, cfg.epi_bufs, cfg.mrep);
}

static thread_local int g_last_cuda_error = 0;

// K (in 16-bit-element units) from which a run that may store C straight from registers does so, for a
// 32-bit and for a 16-bit C.
constexpr int64_t kDirectMinK32 = 2048, kDirectMinK16 = 1024;

#ifdef EXO_GEMM_TRACE
constexpr size_t kStatusBytes = 32 + 3 * 4096 * 2 * 8;  // status block + clock stamps of CTA 0
#else
constexpr size_t kStatusBytes = 32;
#endif

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e == cudaSuccess && q == cudaDriverEntryPointSuccess) fn = (EncodeTiledFn)p;
    else g_last_cuda_error = (int)e;
  });
  return fn;
}

// 2-D tensor map over a matrix whose contiguous dimension has `inner` elements and
// whose other dimension has `outer` elements `ld` elements apart.
static CUresult encode_2d(CUtensorMap* map, int dtype, const void* base, uint64_t inner, uint64_t outer,
                          uint64_t ld, uint32_t box_inner, uint32_t box_outer, bool operand,
                          bool atom32 = false /* M/N-contiguous fp32 operand: 128-byte swizzle in 32-byte atoms */) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return CUDA_ERROR_NOT_FOUND;
  const CUtensorMapDataType dt = dtype == EXO_GEMM_FP32   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                 : dtype == EXO_GEMM_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                          : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * (uint64_t)elem_bytes(dtype)};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
            operand ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// The same with a third dimension: `batch` matrices `batch_stride` elements apart, boxes one matrix deep.
static CUresult encode_3d(CUtensorMap* map, int dtype, const void* base, uint64_t inner, uint64_t outer,
                          uint64_t ld, uint64_t batch, uint64_t batch_stride, uint32_t box_inner,
                          uint32_t box_outer, bool operand, bool atom32 = false) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return CUDA_ERROR_NOT_FOUND;
  const CUtensorMapDataType dt = dtype == EXO_GEMM_FP32   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                 : dtype == EXO_GEMM_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                          : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  const uint64_t es = (uint64_t)elem_bytes(dtype);
  // A repeated operand (stride 0) is described as a batch of one; the kernel then always asks for z = 0.
  cuuint64_t dims[3] = {inner, outer, batch_stride ? batch : 1};
  cuuint64_t strides[2] = {ld * es, batch_stride ? batch_stride * es : ld * es * (outer ? outer : 1)};
  cuuint32_t box[3] = {box_inner, box_outer, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
            operand ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

}  // namespace exo

struct exo_gemm_plan {
  exo_gemm_desc_t desc;                // as planned and launched: leading dimensions of repacked matrices rounded up
  exo_gemm_desc_t user_desc;           // as the caller gave it
  int repack;                          // 1 = A, 2 = B, 4 = C go through an aligned copy (rows not on 16-byte boundaries)
  void* d_pack[3];                     // the copies (NULL where not needed)
  exo::Canonical canon;
  exo::TileConfig cfg;
  exo::KernelFn kernel;
  int device;
  int sm_count;
  int smem_bytes;
  uint32_t* d_status;
  float* d_split_ws;                   // fp32 partials of the tail tiles' K-slices (NULL if none)
  uint32_t* d_split_flags;             // two counters per tail tile: arrivals of contributing warps, owner warps done
  exo::TailItem* d_tail_table;         // the workers' ranges of the tail tiles' k-blocks (4 entries per worker)
  std::atomic<int32_t> dbg_timeout_ms;
  std::atomic<int64_t> dbg_skip_k_block;
};

using namespace exo;

namespace {

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceGuard(int dev) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && dev >= 0 && dev != prev) {
      err = cudaSetDevice(dev);
      switched = err == cudaSuccess;
    }
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

exo_gemm_status_t cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  cudaGetLastError();  // clear the sticky-free error state of the runtime
  return EXO_GEMM_ERR_CUDA;
}

// How many clusters of `cluster` CTAs of kernel `probe` can be resident at once (GPC shapes may
// leave SMs that fit no further cluster).
// One kernel instantiation serves plans with different shared-memory sizes (ring and staging depth are
// run-time parameters), and the attribute belongs to the function, not to a launch: every kernel gets
// the same upper value, never a plan's own size, so plans that live side by side cannot lower it for
// one another.
cudaError_t allow_full_smem(KernelFn k) {
  return cudaFuncSetAttribute((const void*)k, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
}

cudaError_t max_active_clusters(KernelFn probe, int sms, int cluster, int* out) {
  const int smem = kSmemLimit - 1024;  // every plan's shared-memory request is close to the limit
  cudaError_t e = allow_full_smem(probe);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)(sms / cluster * cluster), 1, 1);
  lc.blockDim = dim3(kNumThreads, 1, 1);
  lc.dynamicSmemBytes = smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)cluster;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, (const void*)probe, &lc);
  if (e != cudaSuccess) return e;
  *out = n < sms / cluster ? n : sms / cluster;
  return cudaSuccess;
}

// Co-resident CTA pairs, and slots of two pairs (0 where the shared-operand variant is not built in
// or not wanted).  A slot runs as one 4-CTA cluster where the device finds four free SMs in a GPC
// and as two 2-CTA clusters elsewhere, so the pairs bound the slot count.
cudaError_t cluster_capacity(int sms, int c_dtype, const FlagOverrides& ov, int* max_pairs, int* max_quads) {
  *max_pairs = 0;
  *max_quads = 0;
  if (ov.cta_group == 1) return cudaSuccess;
  cudaError_t e = max_active_clusters(pick_kernel(2, 256, 2, c_dtype), sms, 2, max_pairs);
  if (e != cudaSuccess) return e;
  if (kHaveSharePairs && ov.share != 1) {
    int pairs_shared = 0;  // the variant kernel has its own resource footprint
    e = max_active_clusters(pick_kernel(2, 256, 2, c_dtype, 2), sms, 2, &pairs_shared);
    *max_quads = pairs_shared / 2 < sms / 4 ? pairs_shared / 2 : sms / 4;
  }
  return e;
}

// The descriptor with the leading dimension of every matrix in `mask` (1 = A, 2 = B, 4 = C) replaced by its
// contiguous extent rounded up to 64 elements: what the plan's aligned copy of that matrix looks like.
exo_gemm_desc_t aligned_desc(const exo_gemm_desc_t& d, int mask) {
  exo_gemm_desc_t e = d;
  int64_t outer, inner;
  if (mask & 1) { storage_shape(d.a_layout, d.M, d.K, &outer, &inner); e.lda = (inner + 63) / 64 * 64; }
  if (mask & 2) { storage_shape(d.b_layout, d.K, d.N, &outer, &inner); e.ldb = (inner + 63) / 64 * 64; }
  if (mask & 4) { storage_shape(d.c_layout, d.M, d.N, &outer, &inner); e.ldc = (inner + 63) / 64 * 64; }
  return e;
}

// rows, contiguous elements per row, leading dimension and element size of matrix m (0 = A, 1 = B, 2 = C)
void matrix_storage(const exo_gemm_desc_t& d, int m, int64_t* outer, int64_t* inner, int64_t* ld, int* bytes) {
  if (m == 0) { storage_shape(d.a_layout, d.M, d.K, outer, inner); *ld = d.lda; *bytes = elem_bytes(d.ab_dtype); }
  else if (m == 1) { storage_shape(d.b_layout, d.K, d.N, outer, inner); *ld = d.ldb; *bytes = elem_bytes(d.ab_dtype); }
  else { storage_shape(d.c_layout, d.M, d.N, outer, inner); *ld = d.ldc; *bytes = elem_bytes(d.c_dtype); }
}

int64_t pack_bytes(const exo_gemm_desc_t& aligned, int m) {
  int64_t outer, inner, ld; int bytes;
  matrix_storage(aligned, m, &outer, &inner, &ld, &bytes);
  return outer * ld * bytes;
}

void fill_info(const exo_gemm_plan* p, exo_gemm_info_t* info) {
  memset(info, 0, sizeof(*info));
  info->cta_group = p->cfg.cta_group;
  info->tile_m = 128 * p->cfg.cta_group * p->cfg.mrep;
  info->tile_n = p->cfg.tile_n;
  info->tile_k = sub_block_k(p->canon.ab_bytes) * p->cfg.ksub;
  info->stages = p->cfg.stages;
  info->grid = p->cfg.workers * p->cfg.cta_group * p->cfg.pairs * (p->cfg.lean ? p->cfg.lean : 1);
  info->cluster_size = p->cfg.lean ? p->cfg.lean * p->cfg.cta_group : p->cfg.cta_group * p->cfg.pairs;
  info->stages_direct = p->cfg.stages_direct;
  info->tail_workers = p->cfg.tail_workers;
  info->smem_bytes = p->smem_bytes;
  info->tmem_columns = p->cfg.lean ? p->cfg.tile_n : 2 * p->cfg.tile_n;
  info->lean_kernel = p->cfg.lean ? 1 : 0;
  info->tiles_m = p->cfg.tiles_m;
  info->tiles_n = p->cfg.tiles_n;
  info->raster_along_m = p->cfg.along_m;
  info->raster_band = p->cfg.band;
  info->swapped = p->canon.swapped;
  info->sm_count = p->sm_count;
  info->kernel_launches_per_run = (p->canon.M == 0 || p->canon.N == 0) ? 0 : 1;
  info->epilogue_buffers = p->cfg.epi_bufs;
  info->split_k = p->cfg.lean ? p->cfg.lean : p->cfg.split;
  info->tail_tiles = p->cfg.tail_tiles;
  info->batch_count = (int32_t)p->canon.batch;
  int64_t scratch = p->cfg.workspace_bytes;
  for (int m = 0; m < 3; ++m)
    if (p->repack & (1 << m)) scratch += pack_bytes(p->desc, m);
  info->workspace_bytes = (int32_t)(scratch > 2147483647LL ? 2147483647LL : scratch);
  info->repacked = p->repack;
}

}  // namespace

extern "C" {

exo_gemm_status_t exo_gemm_validate(const exo_gemm_desc_t* desc) { return validate_desc(desc); }

const char* exo_gemm_status_string(exo_gemm_status_t s) {
  switch (s) {
    case EXO_GEMM_OK: return "ok";
    case EXO_GEMM_ERR_NULL: return "null pointer argument";
    case EXO_GEMM_ERR_INVALID_ARG: return "invalid argument";
    case EXO_GEMM_ERR_UNSUPPORTED: return "unsupported configuration";
    case EXO_GEMM_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case EXO_GEMM_ERR_ARCH: return "device is not compute capability 10.x";
    case EXO_GEMM_ERR_CUDA: return "CUDA call failed";
    case EXO_GEMM_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

int exo_gemm_last_cuda_error(void) { return g_last_cuda_error; }

int64_t exo_gemm_schedule_enumerate(int32_t tiles_m, int32_t tiles_n, int32_t band, int32_t along_m,
                                    int32_t num_workers, int32_t worker, int32_t* out_m, int32_t* out_n,
                                    int64_t cap) {
  if (tiles_m < 0 || tiles_n < 0 || band < 1 || num_workers < 1 || worker < 0 || worker >= num_workers ||
      cap < 0 || (cap > 0 && (!out_m || !out_n)))
    return -1;
  const Raster r = make_raster(tiles_m, tiles_n, band, along_m ? 1 : 0);
  int64_t n = 0;
  for (int64_t t = worker; t < raster_total(r); t += num_workers, ++n) {
    if (n < cap) {
      const TileCoord c = raster_decode(r, t);
      out_m[n] = c.m;
      out_n[n] = c.n;
    }
  }
  return n;
}

int64_t exo_gemm_schedule_work(int64_t tiles, int32_t num_workers, int32_t tail_workers, int32_t num_k_blocks, int32_t snap,
                               int32_t owner_extra, int32_t worker, int64_t* out_tile, int32_t* out_slice, int32_t* out_slices,
                               int32_t* out_kb_begin, int32_t* out_kb_end, int64_t cap) {
  if (tiles < 0 || num_workers < 1 || tail_workers < 0 || tail_workers > num_workers || num_k_blocks < 0 || snap < 0 || owner_extra < 0 || worker < 0 ||
      worker >= num_workers || cap < 0 ||
      (cap > 0 && (!out_tile || !out_slice || !out_slices || !out_kb_begin || !out_kb_end)))
    return -1;
  WorkPlan w{};
  w.waves = (int32_t)(tiles / num_workers);
  w.full_tiles = (int64_t)w.waves * num_workers;
  w.tail_tiles = (int32_t)(tiles - w.full_tiles);
  w.tail_workers = tail_workers;
  TailItem* table = nullptr;
  if (tail_workers > 0) {
    // the plans the library makes: every range holds a k-block and no range is longer than a tile
    if (w.tail_tiles == 0 || tail_workers < w.tail_tiles || (int64_t)tail_workers > (int64_t)w.tail_tiles * num_k_blocks)
      return -1;
    table = new (std::nothrow) TailItem[4 * (size_t)num_workers];
    if (!table) return -1;
    w.slots = build_tail_table(w.tail_tiles, num_k_blocks, tail_workers, num_workers, table, snap, owner_extra);
    w.owner_extra = owner_extra;
    w.table = tail_workers % w.tail_tiles == 0 ? nullptr : table;   // whole slices are found by arithmetic, as on the device
  }
  int64_t n = 0;
  WorkItem wi;
  for (int64_t i = 0; work_item(w, worker, num_workers, i, num_k_blocks, &wi); ++i, ++n) {
    if (n < cap) {
      out_tile[n] = wi.tile;
      out_slice[n] = wi.slice;
      out_slices[n] = wi.slices;
      out_kb_begin[n] = wi.kb_begin;
      out_kb_end[n] = wi.kb_end;
    }
  }
  delete[] table;
  return n;
}

exo_gemm_status_t exo_gemm_plan_preview(const exo_gemm_desc_t* desc, int32_t sm_count, exo_gemm_info_t* info) {
  if (!info) return EXO_GEMM_ERR_NULL;
  exo_gemm_status_t st = validate_desc(desc);
  if (st != EXO_GEMM_OK) return st;
  if (sm_count < 1) return EXO_GEMM_ERR_INVALID_ARG;
  exo_gemm_plan p{};
  p.user_desc = *desc;
  p.repack = repack_mask(*desc);
  p.desc = aligned_desc(*desc, p.repack);
  p.canon = canonicalize(p.desc);
  p.sm_count = sm_count;
  const FlagOverrides ov = decode_flags(desc->flags, desc->flags2);
  if (ov.share >= 2 && !kHaveSharePairs) return EXO_GEMM_ERR_UNSUPPORTED;
  p.cfg = choose_config(p.canon, ov, sm_count, sm_count / 2, kHaveSharePairs ? sm_count / 4 : 0);
  p.cfg.workspace_bytes = ov.reduce_add ? 0 : split_workspace_bytes(p.cfg, desc->c_dtype);
  p.smem_bytes = smem_of(p.cfg, desc->c_dtype);
  fill_info(&p, info);
  return EXO_GEMM_OK;
}

exo_gemm_status_t exo_gemm_create_batched(exo_gemm_handle_t* out, const exo_gemm_desc_t* desc, int64_t batch_count,
                                          int64_t stride_a, int64_t stride_b, int64_t stride_c);

exo_gemm_status_t exo_gemm_create(exo_gemm_handle_t* out, const exo_gemm_desc_t* desc) {
  return exo_gemm_create_batched(out, desc, 1, 0, 0, 0);
}

exo_gemm_status_t exo_gemm_create_batched(exo_gemm_handle_t* out, const exo_gemm_desc_t* desc, int64_t batch_count,
                                          int64_t stride_a, int64_t stride_b, int64_t stride_c) {
  if (!out) return EXO_GEMM_ERR_NULL;
  exo_gemm_status_t st = validate_batch(desc, batch_count, stride_a, stride_b, stride_c);
  if (st != EXO_GEMM_OK) return st;

  int device = desc->device;
  cudaError_t e;
  if (device < 0) {
    e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  DeviceGuard guard(device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  int major = 0, sms = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
  if (e != cudaSuccess) return cuda_fail(e);
  if (major != 10) return EXO_GEMM_ERR_ARCH;  // no fallback path by design
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  if (e != cudaSuccess) return cuda_fail(e);
  if (!get_encode_fn()) return EXO_GEMM_ERR_CUDA;

  exo_gemm_plan* p = new (std::nothrow) exo_gemm_plan{};
  if (!p) return EXO_GEMM_ERR_CUDA;
  p->user_desc = *desc;
  p->repack = repack_mask(*desc);
  p->desc = aligned_desc(*desc, p->repack);
  p->canon = canonicalize(p->desc, batch_count, stride_a, stride_b, stride_c);
  p->device = device;
  p->sm_count = sms;
  p->dbg_timeout_ms = 0;
  p->dbg_skip_k_block = -1;
  const FlagOverrides ov = decode_flags(desc->flags, desc->flags2);

  if (ov.share >= 2 && !kHaveSharePairs) { delete p; return EXO_GEMM_ERR_UNSUPPORTED; }
  int max_pairs = 0, max_quads = 0;
  e = cluster_capacity(sms, desc->c_dtype, ov, &max_pairs, &max_quads);
  if (e != cudaSuccess) { delete p; return cuda_fail(e); }
  if (ov.share >= 2 && max_quads < 1) { delete p; return EXO_GEMM_ERR_UNSUPPORTED; }

  p->cfg = choose_config(p->canon, ov, sms, max_pairs, max_quads);
  p->cfg.workspace_bytes = ov.reduce_add ? 0 : split_workspace_bytes(p->cfg, desc->c_dtype);
  p->kernel = kernel_of(p->cfg, desc->c_dtype, ov.reduce_add);
  p->smem_bytes = smem_of(p->cfg, desc->c_dtype);
  e = allow_full_smem(p->kernel);
  if (e != cudaSuccess) { delete p; return cuda_fail(e); }
  e = cudaMalloc((void**)&p->d_status, kStatusBytes);
  if (e != cudaSuccess) { delete p; return cuda_fail(e); }
  e = cudaMemset(p->d_status, 0, kStatusBytes);
  for (int m = 0; m < 3 && e == cudaSuccess; ++m)   // aligned copies of the matrices whose rows TMA cannot address
    if (p->repack & (1 << m)) e = cudaMalloc(&p->d_pack[m], (size_t)pack_bytes(p->desc, m));
  if (e != cudaSuccess) {
    for (int m = 0; m < 3; ++m) cudaFree(p->d_pack[m]);
    cudaFree(p->d_status);
    delete p;
    return cuda_fail(e);
  }
  if (p->cfg.tail_workers > 0) {  // scratch for the K-slices of the tail tiles, and who computes which
    const size_t flag_bytes = 2 * sizeof(uint32_t) * (size_t)p->cfg.tail_tiles * (size_t)p->cfg.pairs;
    if (ov.reduce_add) {   // the parts meet in C itself: no workspace, no counters
      p->cfg.workspace_bytes = 0;
    } else {
      e = cudaMalloc((void**)&p->d_split_ws, (size_t)p->cfg.workspace_bytes);
      if (e == cudaSuccess) e = cudaMalloc((void**)&p->d_split_flags, flag_bytes);
      if (e == cudaSuccess) e = cudaMemset(p->d_split_flags, 0, flag_bytes);
    }
    const size_t table_entries = 4 * (size_t)p->cfg.workers;
    TailItem* table = new (std::nothrow) TailItem[table_entries];
    if (e == cudaSuccess && !table) e = cudaErrorMemoryAllocation;
    if (e == cudaSuccess) {
      const int64_t k_scaled = p->canon.K * (p->canon.ab_bytes / 2);
      const int32_t nkb = (int32_t)((k_scaled + kBlockK * p->cfg.ksub - 1) / (kBlockK * p->cfg.ksub));
      build_tail_table(p->cfg.tail_tiles, nkb, p->cfg.tail_workers, p->cfg.workers, table, p->cfg.snap, p->cfg.owner_extra);
      e = cudaMalloc((void**)&p->d_tail_table, table_entries * sizeof(TailItem));
    }
    if (e == cudaSuccess) e = cudaMemcpy(p->d_tail_table, table, table_entries * sizeof(TailItem), cudaMemcpyHostToDevice);
    delete[] table;
    if (e != cudaSuccess) {
      cudaFree(p->d_split_ws);
      cudaFree(p->d_split_flags);
      cudaFree(p->d_tail_table);
      cudaFree(p->d_status);
      for (int m = 0; m < 3; ++m) cudaFree(p->d_pack[m]);
      delete p;
      return cuda_fail(e);
    }
  }
  *out = p;
  return EXO_GEMM_OK;
}

exo_gemm_status_t exo_gemm_get_info(exo_gemm_handle_t plan, exo_gemm_info_t* info) {
  if (!plan || !info) return EXO_GEMM_ERR_NULL;
  fill_info(plan, info);
  return EXO_GEMM_OK;
}

int32_t exo_gemm_has_shared_operand_clusters(void) { return kHaveSharePairs ? 1 : 0; }

// one-shot test settings of the plan-less entry point (exo_gemm_debug_set with a NULL plan)
static std::atomic<int32_t> g_static_dbg_timeout_ms{0};
static std::atomic<int64_t> g_static_dbg_skip_k_block{-1};

exo_gemm_status_t exo_gemm_debug_set(exo_gemm_handle_t plan, int32_t timeout_ms, int64_t skip_k_block) {
  if (timeout_ms < 0 || timeout_ms > 10000) return EXO_GEMM_ERR_INVALID_ARG;
  if (!plan) {
    g_static_dbg_timeout_ms = timeout_ms;
    g_static_dbg_skip_k_block = skip_k_block;
    return EXO_GEMM_OK;
  }
  plan->dbg_timeout_ms = timeout_ms;
  plan->dbg_skip_k_block = skip_k_block;
  return EXO_GEMM_OK;
}

}  // extern "C"

namespace {

// The argument checks of a run.  *launch is false for an empty problem (nothing to enqueue).
exo_gemm_status_t check_run_args(const exo_gemm_plan* plan, const void* A, const void* B, const void* C, float alpha,
                                 bool* launch) {
  *launch = false;
  const Canonical& cn = plan->canon;
  if (cn.M == 0 || cn.N == 0) return EXO_GEMM_OK;
  const bool read_ab = alpha != 0.f && cn.K > 0;
  if (!C || (read_ab && (!A || !B))) return EXO_GEMM_ERR_NULL;
  // 16 bytes for a matrix that TMA addresses in place; its element size for one that is copied first
  const uintptr_t ab_mask = (uintptr_t)cn.ab_bytes - 1, c_mask = (uintptr_t)cn.c_bytes - 1;
  if ((uintptr_t)C & ((plan->repack & 4) ? c_mask : 15u)) return EXO_GEMM_ERR_ALIGNMENT;
  if (read_ab && (((uintptr_t)A & ((plan->repack & 1) ? ab_mask : 15u)) || ((uintptr_t)B & ((plan->repack & 2) ? ab_mask : 15u))))
    return EXO_GEMM_ERR_ALIGNMENT;
  *launch = true;
  return EXO_GEMM_OK;
}

// Tensor maps and the launch, for arguments that passed check_run_args.
exo_gemm_status_t launch_plan(exo_gemm_plan* plan, const void* A, const void* B, void* C, float alpha, float beta,
                              void* cuda_stream) {
  const Canonical& cn = plan->canon;
  const bool read_ab = alpha != 0.f && cn.K > 0;
  const exo_gemm_desc_t& d = plan->desc;
  const TileConfig& cfg = plan->cfg;
  const void* opA = cn.swapped ? B : A;
  const void* opB = cn.swapped ? A : B;

  GemmParams prm{};
  prm.M = (int32_t)cn.M;
  prm.N = (int32_t)cn.N;
  prm.K = (int32_t)cn.K;
  const int sub_k = sub_block_k(cn.ab_bytes);
  const int stage_k = sub_k * cfg.ksub;
  prm.num_k_blocks = read_ab ? (int32_t)((cn.K + stage_k - 1) / stage_k) : 0;
  prm.raster = make_raster(cfg.tiles_m, cfg.tiles_n, cfg.band, cfg.along_m);
  prm.batch = (uint32_t)cn.batch;
  prm.tiles_per_batch = (uint32_t)cfg.tiles_m * (uint32_t)cfg.tiles_n;
  prm.by_tiles_per_batch = make_fast_div(prm.tiles_per_batch);
  prm.a_z_mask = cn.stride_a ? 0xFFFFFFFFu : 0u;
  prm.b_z_mask = cn.stride_b ? 0xFFFFFFFFu : 0u;
  // Where nothing has to be read back from C and every row of C starts and ends on a 32-byte boundary,
  // the epilogue can store from registers (one full sector per lane) and the staging buffers' shared
  // memory goes to the operand ring.  That pays where the main loop bounds a tile (a seventh stage.  fp32 C:
  // +0.8 % at 4096^3, +1.6 % at 6144 x 6144 x 2048; bf16 C: +6 % at 4096 x 4096 x 1024, +3 % at 8192 x 8192 x
  // 1024 and 4096 x 4096 x 1536); where the epilogue does, a row per lane is the slower way to store (32
  // lines per instruction.  fp32 C: -8 to -13 % at K = 512, -2 to -4 % at K = 1000; bf16 C: -3 to -5 % at
  // K = 512), so short K loops keep the staged path.  So does a request for a staging depth
  // (EXO_GEMM_FLAG_EPI_BUFFERS).
  // (An fp32 C is twice the bytes: the last tile's drain, which nothing hides, takes the row-per-lane stores
  // 9.7 k clocks against 6 k staged, so there the path also wants six or more tiles per worker to pay:
  // 2048^3 and 4096 x 4096 x 2048 -4 %, 2048 x 2048 x 4096 -2 %, 6144 x 6144 x 2048 +1.8 %.)
  // (Problems of less than one wave whose tiles are all cut along K are the exception: +1 to +5 % with the
  // registers-to-global path, whose owner adds the partial sums in registers anyway.)
  const bool long_enough = cn.c_bytes == 2 ? cn.K * (cn.ab_bytes / 2) >= kDirectMinK16
                                           : (cn.K * (cn.ab_bytes / 2) >= kDirectMinK32 &&
                                              (cfg.full_tiles >= 6 * (int64_t)cfg.workers || (cfg.full_tiles == 0 && cfg.tail_workers > 0)));
  const bool direct = !cfg.lean && cfg.stages_direct > 0 && long_enough && beta == 0.f && ((uintptr_t)C & 31u) == 0 &&
                      (cn.ldc * cn.c_bytes) % 32 == 0 && (cn.N * cn.c_bytes) % 32 == 0 &&
                      (cn.batch <= 1 || (cn.stride_c * cn.c_bytes) % 32 == 0);
  prm.stages = direct ? cfg.stages_direct : cfg.stages;
  prm.epi_bufs = direct ? 0 : cfg.epi_bufs;
  // An output much larger than L2 behind a short K loop pushes the operand panels out of L2 between the
  // tiles that share them (12288 x 12288 x 512, fp32 C: L2 hit rate 52 %, DRAM reads 3.2x the operands'
  // size); stored with the evict-first priority it does not: +4.3 % there, +3.1 % at 6144 x 6144 x 512,
  // +0.4 % at K = 1024, -0.3 % at K = 2048, 0 at 4096^3.
  prm.c_evict_first = (cn.M * cn.N * cn.c_bytes * cn.batch >= (64ll << 20) && cn.K * (cn.ab_bytes / 2) <= 1024) ? 1u : 0u;
  prm.c_ptr = C;
  prm.ldc_bytes = cn.ldc * cn.c_bytes;
  prm.c_batch_bytes = cn.stride_c * cn.c_bytes;
  // the tail tiles are cut along K only when there is a K loop to cut and scratch to reduce through
  const bool split_now = cfg.tail_workers > 0 && read_ab && plan->d_tail_table != nullptr;   // (the table exists for every cutting plan)
  const bool reduce_add = split_now && (d.flags & (1u << 11)) != 0;
  // the reduce-add form needs C to hold beta * C_in before the launch: it can for beta == 1 (as it is) and
  // beta == 0 (cleared below)
  if (reduce_add && beta != 0.f && beta != 1.f) return EXO_GEMM_ERR_UNSUPPORTED;
  prm.reduce_add = reduce_add ? 1u : 0u;
  const bool whole_slices = cfg.tail_workers > 0 && cfg.tail_workers % cfg.tail_tiles == 0;
  prm.work = WorkPlan{cfg.full_tiles, (int32_t)(cfg.full_tiles / cfg.workers), cfg.tail_tiles, split_now ? cfg.tail_workers : 0,
                      cfg.slots, cfg.owner_extra, whole_slices ? nullptr : plan->d_tail_table};
  prm.split_ws = plan->d_split_ws;
  prm.split_flags = plan->d_split_flags;
  prm.split_arrivals = (uint32_t)(kEpiWarps * cfg.cta_group * cfg.mrep);
  prm.alpha = read_ab ? alpha : 0.f;
  prm.beta = beta;
  prm.idesc = make_idesc(d.ab_dtype, cn.a_mn_major, cn.b_mn_major, 128 * cfg.cta_group, cfg.tile_n);
  prm.a = make_staging(cn.a_mn_major, kBlockM * cfg.mrep, cfg.ksub, cn.ab_bytes);
  prm.b = make_staging(cn.b_mn_major, cfg.tile_n / cfg.cta_group, cfg.ksub, cn.ab_bytes);
  prm.sub_k = (uint32_t)sub_k;
  prm.umma_k = (uint32_t)sub_k / 4;
  prm.tf32 = d.ab_dtype == EXO_GEMM_FP32 ? 1u : 0u;
  prm.status = plan->d_status;
  const int32_t dbg_ms = plan->dbg_timeout_ms.exchange(0);
  // SM clocks, converted at 2 GHz (an upper bound of the SM clock, so the real limit is not shorter)
  prm.timeout_cycles = (uint64_t)(dbg_ms > 0 ? dbg_ms : 4000) * 2000000ull;
  prm.debug_skip_k_block = plan->dbg_skip_k_block.exchange(-1);

  CUtensorMap tm_a, tm_b, tm_c;
  memset(&tm_a, 0, sizeof tm_a);
  memset(&tm_b, 0, sizeof tm_b);
  CUresult r;
  const int b_rows = cfg.tile_n / cfg.cta_group;
  const int a_rows = kBlockM * cfg.mrep / cfg.pairs;  // pairs that share A fetch half of a CTA's rows each
  const uint32_t c_box = d.c_dtype == EXO_GEMM_FP32 ? 32 : 64;
  const bool atom32 = d.ab_dtype == EXO_GEMM_FP32;   // only read for M/N-contiguous operands
  if (cn.batch <= 1) {
    if (read_ab) {
      r = cn.a_mn_major ? encode_2d(&tm_a, d.ab_dtype, opA, cn.M, cn.K, cn.lda, sub_k, stage_k, true, atom32)
                        : encode_2d(&tm_a, d.ab_dtype, opA, cn.K, cn.M, cn.lda, sub_k, a_rows, true);
      if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return EXO_GEMM_ERR_CUDA; }
      r = cn.b_mn_major ? encode_2d(&tm_b, d.ab_dtype, opB, cn.N, cn.K, cn.ldb, sub_k, stage_k, true, atom32)
                        : encode_2d(&tm_b, d.ab_dtype, opB, cn.K, cn.N, cn.ldb, sub_k, b_rows, true);
      if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return EXO_GEMM_ERR_CUDA; }
    }
    r = encode_2d(&tm_c, d.c_dtype, C, cn.N, cn.M, cn.ldc, c_box, 32, false);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return EXO_GEMM_ERR_CUDA; }
  } else {  // strided batch: the matrix index is the third tensor-map coordinate
    if (read_ab) {
      r = cn.a_mn_major
              ? encode_3d(&tm_a, d.ab_dtype, opA, cn.M, cn.K, cn.lda, cn.batch, cn.stride_a, sub_k, stage_k, true, atom32)
              : encode_3d(&tm_a, d.ab_dtype, opA, cn.K, cn.M, cn.lda, cn.batch, cn.stride_a, sub_k, a_rows, true);
      if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return EXO_GEMM_ERR_CUDA; }
      r = cn.b_mn_major
              ? encode_3d(&tm_b, d.ab_dtype, opB, cn.N, cn.K, cn.ldb, cn.batch, cn.stride_b, sub_k, stage_k, true, atom32)
              : encode_3d(&tm_b, d.ab_dtype, opB, cn.K, cn.N, cn.ldb, cn.batch, cn.stride_b, sub_k, b_rows, true);
      if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return EXO_GEMM_ERR_CUDA; }
    }
    r = encode_3d(&tm_c, d.c_dtype, C, cn.N, cn.M, cn.ldc, cn.batch, cn.stride_c, c_box, 32, false);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return EXO_GEMM_ERR_CUDA; }
  }
  if (!read_ab) { tm_a = tm_c; tm_b = tm_c; }  // never dereferenced for data; keeps the prefetch valid

  DeviceGuard guard(plan->device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3((unsigned)((int64_t)cfg.workers * cfg.cta_group * cfg.pairs * (cfg.lean ? cfg.lean : 1)), 1, 1);
  lc.blockDim = dim3(!cfg.lean ? (unsigned)kNumThreads
                               : (cfg.cta_group == 2 ? (unsigned)kLeanPairThreads : (unsigned)lean_threads(cfg.tile_n, (int)cn.c_bytes)), 1, 1);
  lc.dynamicSmemBytes = direct ? smem_bytes_for(cfg.cta_group, cfg.tile_n, cfg.ksub, cfg.stages_direct, 0, cfg.mrep)
                               : plan->smem_bytes;
  lc.stream = (cudaStream_t)cuda_stream;
  cudaLaunchAttribute at[3];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)(cfg.lean ? cfg.lean * cfg.cta_group : cfg.cta_group);
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  // Programmatic dependent launch: this kernel's CTAs may start (barrier set-up, TMEM allocation)
  // while the previous kernel in the stream drains; the kernel waits for that kernel before it
  // touches global memory, so stream order is kept for data.
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 2;
  if (cfg.pairs == 2 && (d.flags2 & 3u) != 3u) {
    // Slots of four CTAs: 4-CTA clusters wherever four SMs of a GPC are free, else two regular pairs.
    at[2].id = cudaLaunchAttributePreferredClusterDimension;
    at[2].val.preferredClusterDim.x = 4;
    at[2].val.preferredClusterDim.y = 1;
    at[2].val.preferredClusterDim.z = 1;
    lc.numAttrs = 3;
  }
  cudaError_t e;
  if (reduce_add && beta == 0.f) {   // every part adds onto zeros
    for (int64_t b = 0; b < cn.batch; ++b) {
      e = cudaMemset2DAsync(static_cast<char*>(C) + b * cn.stride_c * cn.c_bytes, (size_t)(cn.ldc * cn.c_bytes), 0,
                            (size_t)(cn.N * cn.c_bytes), (size_t)cn.M, (cudaStream_t)cuda_stream);
      if (e != cudaSuccess) return cuda_fail(e);
    }
  }
  // (The arrival counters of a K-slicing plan need nothing from the host per run: which run this is follows
  // from a second counter on the device, so the same parameters can be replayed from a CUDA graph.)
  e = cudaLaunchKernelEx(&lc, plan->kernel, tm_a, tm_b, tm_c, prm);
  if (e != cudaSuccess) return cuda_fail(e);
  return EXO_GEMM_OK;
}

// One pass of repack.cuh's kernel over matrix m (0 = A, 1 = B, 2 = C) between the caller's layout and the plan's
// aligned copy, in the direction given.
exo_gemm_status_t copy_matrix(const exo_gemm_plan* plan, int m, void* dst, const void* src, bool into_aligned, void* cuda_stream) {
  int64_t outer, inner, ld_user, ld_aligned; int bytes;
  matrix_storage(plan->user_desc, m, &outer, &inner, &ld_user, &bytes);
  matrix_storage(plan->desc, m, &outer, &inner, &ld_aligned, &bytes);
  uint32_t seg = 0, blocks = 0;
  if (!repack_grid(inner, outer, &seg, &blocks)) return EXO_GEMM_ERR_UNSUPPORTED;
  const int64_t dst_ld = into_aligned ? ld_aligned : ld_user, src_ld = into_aligned ? ld_user : ld_aligned;
  if (bytes == 2)
    exo_repack_kernel<uint16_t><<<blocks, kRepackThreads, 0, (cudaStream_t)cuda_stream>>>((uint16_t*)dst, dst_ld, (const uint16_t*)src, src_ld, inner, seg);
  else
    exo_repack_kernel<uint32_t><<<blocks, kRepackThreads, 0, (cudaStream_t)cuda_stream>>>((uint32_t*)dst, dst_ld, (const uint32_t*)src, src_ld, inner, seg);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? EXO_GEMM_OK : cuda_fail(e);
}

}  // namespace

extern "C" {

exo_gemm_status_t exo_gemm_run(exo_gemm_handle_t plan, const void* A, const void* B, void* C, float alpha,
                               float beta, void* cuda_stream) {
  if (!plan) return EXO_GEMM_ERR_NULL;
  bool launch = false;
  exo_gemm_status_t st = check_run_args(plan, A, B, C, alpha, &launch);
  if (st != EXO_GEMM_OK || !launch) return st;
  if (!plan->repack) return launch_plan(plan, A, B, C, alpha, beta, cuda_stream);
  // Matrices whose rows TMA cannot address travel through the plan's aligned copies: operands in before the
  // GEMM, C in as well if it is read, C out after it (only its M x N elements: the caller's padding is untouched).
  DeviceGuard guard(plan->device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  const bool read_ab = alpha != 0.f && plan->canon.K > 0;
  const void* user[3] = {A, B, C};
  const void* eff[3] = {A, B, C};
  for (int m = 0; m < 3; ++m) {
    if (!(plan->repack & (1 << m))) continue;
    eff[m] = plan->d_pack[m];
    if (m < 2 ? !read_ab : beta == 0.f) continue;   // never read: nothing to copy in
    st = copy_matrix(plan, m, plan->d_pack[m], user[m], /*into_aligned=*/true, cuda_stream);
    if (st != EXO_GEMM_OK) return st;
  }
  st = launch_plan(plan, eff[0], eff[1], const_cast<void*>(eff[2]), alpha, beta, cuda_stream);
  if (st != EXO_GEMM_OK || !(plan->repack & 4)) return st;
  return copy_matrix(plan, 2, C, plan->d_pack[2], /*into_aligned=*/false, cuda_stream);
}

exo_gemm_status_t exo_gemm_check(exo_gemm_handle_t plan, uint32_t* detail) {
  if (!plan) return EXO_GEMM_ERR_NULL;
  DeviceGuard guard(plan->device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  uint32_t h[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  cudaError_t e = cudaMemcpy(h, plan->d_status, 32, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  if (detail) memcpy(detail, h, 32);
  if (h[0] == kStatusOk) return EXO_GEMM_OK;
  e = cudaMemset(plan->d_status, 0, 32);
  if (e != cudaSuccess) return cuda_fail(e);
  if (plan->d_split_flags) {  // an abandoned run may have left the counters of the tail tiles out of step
    e = cudaMemset(plan->d_split_flags, 0, 2 * sizeof(uint32_t) * (size_t)plan->cfg.tail_tiles * (size_t)plan->cfg.pairs);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return EXO_GEMM_ERR_DEVICE_TIMEOUT;
}

// ---------------------------------------------------------------------------------------
// Allocation-free entry point.  The only global memory the kernel needs beyond A, B and C
// is its status block; here that block lives in a file-scope device array instead of a
// cudaMalloc'ed one.  In host code the array's name is only a host-side stand-in for the
// device object: its device address comes from cudaGetSymbolAddress, once per device.
constexpr size_t kStaticScratchBytes = 256;  // stated maximum; the status block needs kStatusBytes
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
uint32_t* g_static_ptr[kMaxDevices] = {};  // device address of g_static_scratch, per device

// Set-up, once per device, with that device current.
cudaError_t static_scratch_for_current_device(int device, uint32_t** out) {
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[device]) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[device] = static_cast<uint32_t*>(ptr);
  }
  *out = g_static_ptr[device];
  return cudaSuccess;
}
}  // namespace

exo_gemm_status_t exo_gemm_run_static(const exo_gemm_desc_t* desc, const void* A, const void* B, void* C,
                                      float alpha, float beta, void* cuda_stream, uint32_t* detail) {
  exo_gemm_status_t st = validate_desc(desc);
  if (st != EXO_GEMM_OK) return st;
  if (kStatusBytes > kStaticScratchBytes) return EXO_GEMM_ERR_UNSUPPORTED;  // scratch need beyond the static array

  int device = desc->device;
  cudaError_t e;
  if (device < 0) {
    e = cudaGetDevice(&device);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (device >= kMaxDevices) return EXO_GEMM_ERR_UNSUPPORTED;
  DeviceGuard guard(device);
  if (guard.err != cudaSuccess) return cuda_fail(guard.err);
  int major = 0, sms = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
  if (e != cudaSuccess) return cuda_fail(e);
  if (major != 10) return EXO_GEMM_ERR_ARCH;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  if (e != cudaSuccess) return cuda_fail(e);
  if (!get_encode_fn()) return EXO_GEMM_ERR_CUDA;

  // a plan on the stack: same choices as exo_gemm_create, nothing allocated
  exo_gemm_plan plan{};
  if (repack_mask(*desc)) return EXO_GEMM_ERR_UNSUPPORTED;   // an aligned copy would be scratch, which this entry point does not own
  plan.desc = *desc;
  plan.user_desc = *desc;
  plan.canon = canonicalize(*desc);
  plan.device = device;
  plan.sm_count = sms;
  FlagOverrides ov = decode_flags(desc->flags, desc->flags2);
  ov.no_workspace = true;  // K-slicing of the tail tiles needs device scratch this entry point may not allocate
  if (ov.share >= 2 && !kHaveSharePairs) return EXO_GEMM_ERR_UNSUPPORTED;
  int max_pairs = 0, max_quads = 0;
  e = cluster_capacity(sms, desc->c_dtype, ov, &max_pairs, &max_quads);
  if (e != cudaSuccess) return cuda_fail(e);
  if (ov.share >= 2 && max_quads < 1) return EXO_GEMM_ERR_UNSUPPORTED;
  plan.cfg = choose_config(plan.canon, ov, sms, max_pairs, max_quads);
  plan.kernel = kernel_of(plan.cfg, desc->c_dtype, false);
  plan.smem_bytes = smem_of(plan.cfg, desc->c_dtype);
  e = allow_full_smem(plan.kernel);
  if (e != cudaSuccess) return cuda_fail(e);

  // every argument check comes before anything is enqueued, as in exo_gemm_run
  bool launch = false;
  st = check_run_args(&plan, A, B, C, alpha, &launch);
  if (st != EXO_GEMM_OK) return st;
  if (!launch) {  // empty problem: nothing runs, nothing to report
    if (detail) memset(detail, 0, 32);
    return EXO_GEMM_OK;
  }
  e = static_scratch_for_current_device(device, &plan.d_status);
  if (e != cudaSuccess) return cuda_fail(e);
  // the array keeps the last call's contents: the status words must start at zero
  e = cudaMemsetAsync(plan.d_status, 0, kStatusBytes, (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e);
  plan.dbg_timeout_ms = g_static_dbg_timeout_ms.exchange(0);
  plan.dbg_skip_k_block = g_static_dbg_skip_k_block.exchange(-1);

  st = launch_plan(&plan, A, B, C, alpha, beta, cuda_stream);
  if (st != EXO_GEMM_OK || !detail) return st;

  // blocking mode: wait for the kernel and report what it recorded
  e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e);
  uint32_t h[8];
  e = cudaMemcpy(h, plan.d_status, 32, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e);
  memcpy(detail, h, 32);
  return h[0] == kStatusOk ? EXO_GEMM_OK : EXO_GEMM_ERR_DEVICE_TIMEOUT;
}

#ifdef EXO_GEMM_TRACE
// Development aid: copies the clock stamps of CTA 0 (3 roles x 4096 x 2 int64) to the host.
exo_gemm_status_t exo_gemm_debug_read_trace(exo_gemm_handle_t plan, long long* out) {
  if (!plan || !out) return EXO_GEMM_ERR_NULL;
  cudaError_t e = cudaMemcpy(out, plan->d_status + 8, kStatusBytes - 32, cudaMemcpyDeviceToHost);
  return e == cudaSuccess ? EXO_GEMM_OK : cuda_fail(e);
}
#endif

exo_gemm_status_t exo_gemm_destroy(exo_gemm_handle_t plan) {
  if (!plan) return EXO_GEMM_OK;
  exo_gemm_status_t st = EXO_GEMM_OK;
  {
    DeviceGuard guard(plan->device);
    if (plan->d_status) {
      cudaError_t e = cudaFree(plan->d_status);
      if (e != cudaSuccess) st = cuda_fail(e);
    }
    if (plan->d_split_ws) cudaFree(plan->d_split_ws);
    if (plan->d_split_flags) cudaFree(plan->d_split_flags);
    if (plan->d_tail_table) cudaFree(plan->d_tail_table);
    for (int m = 0; m < 3; ++m)
      if (plan->d_pack[m]) cudaFree(plan->d_pack[m]);
  }
  delete plan;
  return st;
}

}  // extern "C"
