// C ABI of the fold decode library: argument checks, tensor-map creation, workspace
// carving and kernel launches.  Nothing here allocates device memory or synchronises.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "fold_common.cuh"
#include "fold_estimate.cuh"
#include "fold_merge.cuh"
#include "fold_planes.cuh"
#include "fold_probe.cuh"
#include "fold_scan.cuh"
#include "fold_scan_umma.cuh"
#include "fold_scan_decode.cuh"

using namespace fold;

namespace {

constexpr size_t kHeaderBytes = 256;
constexpr int kSmemPerSm = 233472;       // 228 KB per SM
constexpr int kSmemPerCtaMax = 232448;   // 227 KB opt-in per CTA
constexpr int kSmemCtaReserve = 1024;
constexpr long long kMaxStackedRows = 4096;   // query rows stacked on one (sequence, kv head)

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline int ilog2(int v) { int s = 0; while ((1 << s) < v) ++s; return s; }

struct Geometry {
  int B, Hq, Hkv, G, D, stack, R, num_seqs, max_slots;
  long long slot_stride;
  size_t slot_bytes;
  bool planes;            // two-plane INT8 keys
  size_t q_off, ws_bytes; // workspace: where the split query rows start (planes), and the total
};

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
// bytes after the slots for the split query rows: codes [rows][2][D], then one eta per row
inline size_t qplane_bytes(long long rows, int D) { return round_up((size_t)rows * 2 * D, 256) + round_up((size_t)rows * 4, 256); }

int check_kv(const fold_kv &kv, int D, int Hkv) {
  const bool planes = kv.k_plane_a != nullptr, vplanes = kv.v_plane_1 != nullptr;
  if ((!kv.k && !planes) || (!kv.v && !vplanes) || !kv.seqlens) return FOLD_EINVAL;
  if (vplanes) {
    if (!planes) return FOLD_EUNSUPPORTED;                   // the E4M3 value planes go with the two-plane keys
    if (!kv.v_plane_2 || !aligned(kv.v_plane_1, 16) || !aligned(kv.v_plane_2, 16)) return FOLD_EINVAL;
    if (kv.v_scale_log2 < -100 || kv.v_scale_log2 > 100) return FOLD_EINVAL;
  }
  if (!aligned(kv.k, 16) || !aligned(kv.v, 16)) return FOLD_EINVAL;
  if (planes) {
    if (!kv.k_plane_b || !kv.k_scale) return FOLD_EINVAL;
    if (!aligned(kv.k_plane_a, 16) || !aligned(kv.k_plane_b, 16) || !aligned(kv.k_scale, 16)) return FOLD_EINVAL;
    if (kv.plane_stride_tok < D || kv.plane_stride_head < 0 || kv.plane_stride_seq < 0) return FOLD_EINVAL;
    if (kv.plane_stride_tok % 16 || kv.plane_stride_head % 16 || kv.plane_stride_seq % 16) return FOLD_EINVAL;
    if (kv.scale_stride_seq < 0 || kv.scale_stride_head < 0 || kv.scale_stride_seq % 8 || kv.scale_stride_head % 8)
      return FOLD_EINVAL;
  }
  if (kv.num_seqs < 1 || kv.max_seqlen < 0) return FOLD_EINVAL;
  if (kv.stride_tok < D || kv.stride_head < 0 || kv.stride_seq < 0) return FOLD_EINVAL;
  if (kv.stride_tok % 8 || kv.stride_head % 8 || kv.stride_seq % 8) return FOLD_EINVAL;
  // an axis with more than one entry needs a stride that spans a row: a broadcast (zero) stride would make the tensor
  // maps and the plain loads disagree about where rows lie
  if (Hkv > 1 && kv.stride_head < D) return FOLD_EINVAL;
  if ((kv.page_table ? kv.num_pages : kv.num_seqs) > 1 && kv.stride_seq < D) return FOLD_EINVAL;
  if (planes) {
    if (Hkv > 1 && kv.plane_stride_head < D) return FOLD_EINVAL;
    if ((kv.page_table ? kv.num_pages : kv.num_seqs) > 1 && kv.plane_stride_seq < D) return FOLD_EINVAL;
  }
  if (kv.v_block_mean && Hkv > 1 && kv.mean_stride_head < D) return FOLD_EINVAL;
  if (kv.page_table) {
    if (kv.page_size < 16 || (kv.page_size & (kv.page_size - 1))) return FOLD_EUNSUPPORTED;
    if (kv.num_pages < 1 || kv.max_pages_per_seq < 1) return FOLD_EINVAL;
    if ((long long)kv.max_pages_per_seq * kv.page_size < kv.max_seqlen) return FOLD_EINVAL;
  } else {
    if (kv.capacity < kv.max_seqlen || kv.capacity < 1) return FOLD_EINVAL;
  }
  if (kv.v_block_mean) {
    if (!aligned(kv.v_block_mean, 16)) return FOLD_EINVAL;
    if (kv.mean_stride_seq < 0 || kv.mean_stride_block < D || kv.mean_stride_head < 0) return FOLD_EINVAL;
    if (kv.mean_stride_seq % 8 || kv.mean_stride_block % 8 || kv.mean_stride_head % 8) return FOLD_EINVAL;
  }
  return FOLD_OK;
}

int check_args(const fold_args *a, Geometry *g, bool need_out) {
  if (!a) return FOLD_EINVAL;
  if (a->head_dim != 64 && a->head_dim != 128) return FOLD_EUNSUPPORTED;
  if (a->batch < 1 || a->num_q_heads < 1 || a->num_kv_heads < 1 || a->stack < 1) return FOLD_EINVAL;
  if (a->num_q_heads % a->num_kv_heads) return FOLD_EINVAL;
  if (a->batch % a->stack || a->batch / a->stack != a->kv.num_seqs) return FOLD_EINVAL;
  if (a->batch > 65535) return FOLD_EUNSUPPORTED;           // requests and sequences index a grid's y / z dimension
  if (!a->q || !aligned(a->q, 16) || a->q_stride_b % 8 || a->q_stride_h % 8) return FOLD_EINVAL;
  if (a->q_stride_h < a->head_dim && a->num_q_heads > 1) return FOLD_EINVAL;
  if (int rc = check_kv(a->kv, a->head_dim, a->num_kv_heads)) return rc;
  if (!(a->softmax_scale > 0.f) || isinf(a->softmax_scale)) return FOLD_EINVAL;
  if (a->z_mode < FOLD_Z_ESTIMATE || a->z_mode > FOLD_Z_ZERO) return FOLD_EINVAL;
  if (!a->z || !aligned(a->z, 4)) return FOLD_EINVAL;
  if (isnan(a->depth_T) || a->depth_T < 0.f) return FOLD_EINVAL;
  if (a->num_splits < 0) return FOLD_EINVAL;
  if (need_out && (!a->out || !aligned(a->out, 2))) return FOLD_EINVAL;
  if (a->draft_len < 0 || a->draft_len > 32) return FOLD_EINVAL;
  if (a->draft_len > 0 && (!a->draft_mask || !aligned(a->draft_mask, 4))) return FOLD_EINVAL;
  const int G = a->num_q_heads / a->num_kv_heads;
  const long long R = (long long)a->stack * G;
  if (G > kMaxRows || R > kMaxStackedRows) return FOLD_EUNSUPPORTED;
  g->B = a->batch; g->Hq = a->num_q_heads; g->Hkv = a->num_kv_heads; g->G = G; g->D = a->head_dim;
  g->stack = a->stack; g->R = (int)R; g->num_seqs = a->kv.num_seqs;
  g->max_slots = max_chunks_upto(a->kv.max_seqlen);
  if (g->max_slots < 1) g->max_slots = 1;
  g->slot_stride = (long long)g->R * g->D + ((g->R + 3) / 4) * 4;
  g->slot_bytes = (size_t)g->num_seqs * g->Hkv * g->max_slots * g->slot_stride * sizeof(float);
  g->planes = a->kv.k_plane_a != nullptr;
  g->q_off = round_up(kHeaderBytes + g->slot_bytes, 256);
  g->ws_bytes = g->planes ? g->q_off + qplane_bytes((long long)g->B * g->Hq, g->D) : kHeaderBytes + g->slot_bytes;
  if (g->planes) {
    if (isnan(a->refine_tau)) return FOLD_EINVAL;
    // the two-plane scan: blocks of up to 16 rows (a block's verdicts are ORed over its rows), no exact-maximum pass;
    // draft rows share their sequence's verdicts, so they stay within one block
    if ((R > kMaxRows && a->draft_len > 0) || a->z_mode == FOLD_Z_EXACT_MAX) return FOLD_EUNSUPPORTED;
    if (a->kv.v_plane_1 && isnan(a->refine_tau_v)) return FOLD_EINVAL;
  }
  return FOLD_OK;
}

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// 4-D view of a cache tensor: axis 0 is the channel, the token / head / sequence-or-page axes
// follow in order of increasing stride (MapAxes returns where each landed).  Box = box_ch channels
// x box_tok tokens, swizzled, out-of-range elements read as zero.
struct MapAxes { int pos_tok, pos_head, pos_seq; };

// `elem` bytes per element (2: BF16 rows, 1: INT8 plane rows), strides in elements; the box spans `box_ch` channels.
int make_map_of(CUtensorMap *map, MapAxes *axes, const void *ptr, const fold_kv &kv, int D, int Hkv, int box_tok, int elem,
                long long stride_tok, long long stride_head, long long stride_seq, int box_ch, CUtensorMapSwizzle swizzle,
                CUtensorMapL2promotion promo) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FOLD_ECUDA;
  const bool paged = kv.page_table != nullptr;
  struct Axis { cuuint64_t extent, stride; cuuint32_t box; int id; };
  Axis ax[3] = {{(cuuint64_t)(paged ? kv.page_size : kv.capacity), (cuuint64_t)stride_tok * elem, (cuuint32_t)box_tok, 0},
                {(cuuint64_t)Hkv, (cuuint64_t)stride_head * elem, 1u, 1},
                {(cuuint64_t)(paged ? kv.num_pages : kv.num_seqs), (cuuint64_t)stride_seq * elem, 1u, 2}};
  // extent-1 axes carry no information: sort them last, the rest by stride
  for (int i = 0; i < 3; ++i)
    for (int j = i + 1; j < 3; ++j) {
      const bool i_one = ax[i].extent == 1, j_one = ax[j].extent == 1;
      if ((i_one && !j_one) || (i_one == j_one && ax[j].stride < ax[i].stride)) { Axis t = ax[i]; ax[i] = ax[j]; ax[j] = t; }
    }
  cuuint64_t prev_stride = (cuuint64_t)D * elem, prev_extent = 1;
  for (int i = 0; i < 3; ++i) {
    if (ax[i].extent == 1 || ax[i].stride == 0) ax[i].stride = prev_stride * prev_extent;
    prev_stride = ax[i].stride; prev_extent = ax[i].extent;
  }
  cuuint64_t dims[4] = {(cuuint64_t)D, ax[0].extent, ax[1].extent, ax[2].extent};
  cuuint64_t strides[3] = {ax[0].stride, ax[1].stride, ax[2].stride};
  cuuint32_t box[4] = {(cuuint32_t)box_ch, ax[0].box, ax[1].box, ax[2].box};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  for (int i = 0; i < 3; ++i) {
    if (ax[i].id == 0) axes->pos_tok = i + 1;
    if (ax[i].id == 1) axes->pos_head = i + 1;
    if (ax[i].id == 2) axes->pos_seq = i + 1;
  }
  CUresult rc = fn(map, elem == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 4,
                   const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, promo,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? FOLD_OK : FOLD_ECUDA;
}

// BF16 key / value rows: a box of 64 channels x box_tok tokens, 128-byte swizzle.
int make_map(CUtensorMap *map, MapAxes *axes, const void *ptr, const fold_kv &kv, int D, int Hkv, int box_tok) {
  return make_map_of(map, axes, ptr, kv, D, Hkv, box_tok, 2, kv.stride_tok, kv.stride_head, kv.stride_seq, 64,
                     CU_TENSOR_MAP_SWIZZLE_128B,
                     D == 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// Key plane A (INT8): one box spans the whole D-byte row; 128-byte swizzle for 128-byte rows, 64-byte for 64-byte rows.
int make_plane_map(CUtensorMap *map, MapAxes *axes, const fold_kv &kv, int D, int Hkv, int box_tok) {
  return make_map_of(map, axes, kv.k_plane_a, kv, D, Hkv, box_tok, 1, kv.plane_stride_tok, kv.plane_stride_head,
                     kv.plane_stride_seq, D, D == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// ------------------------------------------------------------------ launches
// Launch with programmatic stream serialization: the kernel may begin (its prologue, up to its
// griddepcontrol.wait) while the kernel before it in the stream drains.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// The first kernel of a call reads the caller's inputs (q, the newest cache rows, seqlens, the page table) before its
// dependency wait.  Behind a kernel of the library that is safe; behind the CALLER's kernel it is only safe if those
// inputs were complete before that kernel started, which the caller says with FOLD_INPUTS_SETTLED.  Otherwise the
// kernel is launched in plain stream order.
template <typename... KArgs, typename... Args>
cudaError_t launch_first(bool early, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  if (early) return launch_pdl(kernel, grid, block, smem, st, args...);
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

KvLevel kv_level(const fold_kv &kv, int stack) {
  KvLevel L;
  L.k = static_cast<const __nv_bfloat16 *>(kv.k);
  L.stride_seq = kv.stride_seq; L.stride_tok = kv.stride_tok; L.stride_head = kv.stride_head;
  L.page_table = kv.page_table;
  L.seqlens = kv.seqlens;
  L.paged = kv.page_table != nullptr;
  L.page_shift = L.paged ? ilog2(kv.page_size) : 0;
  L.max_pages = kv.max_pages_per_seq;
  L.num_pages = kv.num_pages > 0 ? kv.num_pages : 1;
  L.stack = stack;
  L.max_seqlen = kv.max_seqlen;
  return L;
}

EstParams est_params(const fold_args *a, const Geometry &g) {
  EstParams p;
  memset(&p, 0, sizeof(p));
  p.q = static_cast<const __nv_bfloat16 *>(a->q);
  p.q_stride_b = a->q_stride_b; p.q_stride_h = a->q_stride_h;
  p.z = a->z;
  p.Hq = g.Hq; p.Hkv = g.Hkv; p.G = g.G;
  p.scale_log2 = (float)((double)a->softmax_scale * 1.4426950408889634);
  p.draft_mask = a->draft_len > 0 ? a->draft_mask : nullptr;
  p.draft_len = a->draft_len;
  return p;
}

PlaneView plane_view(const fold_kv &kv) {
  PlaneView v;
  v.a = kv.k_plane_a; v.b = kv.k_plane_b;
  v.stride_seq = kv.plane_stride_seq; v.stride_tok = kv.plane_stride_tok; v.stride_head = kv.plane_stride_head;
  v.scale = static_cast<const __nv_bfloat16 *>(kv.k_scale);
  v.sc_stride_seq = kv.scale_stride_seq; v.sc_stride_head = kv.scale_stride_head;
  v.page_table = kv.page_table; v.seqlens = kv.seqlens;
  v.paged = kv.page_table != nullptr;
  v.page_shift = v.paged ? ilog2(kv.page_size) : 0;
  v.max_pages = kv.max_pages_per_seq;
  v.num_pages = kv.num_pages > 0 ? kv.num_pages : 1;
  v.max_seqlen = kv.max_seqlen;
  v.v1 = kv.v_plane_1; v.v2 = kv.v_plane_2;
  v.v_scale = ldexpf(1.f, kv.v_scale_log2);
  return v;
}

// Two-plane keys: the front kernel splits the query rows into the workspace whatever the reference mode, and
// forms the estimate when asked to.
// The two-plane front kernel over the levels of a cascade (one level: a plain decode).  Every level's workspace gets
// the split query rows; the reference is estimated over the levels' keys in order when levels[0] asks for it.  The
// levels share q, z, batch and head counts (checked by the callers); gs[l] is level l's geometry.
int launch_planes_front_levels(const fold_args *const *levels, const Geometry *gs, int n_levels, cudaStream_t st,
                               bool zero_header) {
  const fold_args *a = levels[0];
  const Geometry &g = gs[0];
  FrontParams p;
  memset(&p, 0, sizeof(p));
  p.q = static_cast<const __nv_bfloat16 *>(a->q);
  p.q_stride_b = a->q_stride_b; p.q_stride_h = a->q_stride_h;
  p.n_levels = n_levels;
  for (int l = 0; l < n_levels; ++l) {
    uint8_t *ws = static_cast<uint8_t *>(levels[l]->workspace);
    p.lv[l].qplanes = reinterpret_cast<int8_t *>(ws + gs[l].q_off);
    p.lv[l].qeta = reinterpret_cast<float *>(ws + gs[l].q_off + round_up((size_t)g.B * g.Hq * 2 * g.D, 256));
    p.lv[l].kv = plane_view(levels[l]->kv);
    p.lv[l].stack = gs[l].stack;
    p.lv[l].hdr = zero_header ? static_cast<fold_ws_header *>(levels[l]->workspace) : nullptr;
  }
  p.z = a->z;
  p.write_z = a->z_mode == FOLD_Z_ESTIMATE;
  p.Hq = g.Hq; p.Hkv = g.Hkv; p.G = g.G;
  p.scale_log2 = (float)((double)a->softmax_scale * 1.4426950408889634);
  {                                                          // drafts sit at the end of the last level
    const fold_args *al = levels[n_levels - 1];
    p.draft_mask = al->draft_len > 0 ? al->draft_mask : nullptr;
    p.draft_len = al->draft_len;
  }
  if (a->z_mode == FOLD_Z_ZERO) {
    const int rows = g.B * g.Hq;
    fold_fill_kernel<<<(rows + 255) / 256, 256, 0, st>>>(a->z, rows, 0.f);
  }
  const dim3 grid(g.Hkv, g.B);
  const bool early = (a->flags & FOLD_INPUTS_SETTLED) != 0;
  const cudaError_t rc = g.D == 128 ? launch_first(early, fold_planes_front_kernel<128>, grid, dim3(kFrontThreads), 0, st, p)
                                    : launch_first(early, fold_planes_front_kernel<64>, grid, dim3(kFrontThreads), 0, st, p);
  if (rc != cudaSuccess) return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

int launch_planes_front(const fold_args *a, const Geometry &g, cudaStream_t st, bool zero_header = false) {
  return launch_planes_front_levels(&a, &g, 1, st, zero_header);
}

// zero_header: the kernel launched here also zeroes the first 64 bytes of a->workspace; header_zeroed_by_reference()
// says whether this call's mode launches such a kernel
bool header_zeroed_by_reference(const fold_args *a, const Geometry &g) { return g.planes || a->z_mode == FOLD_Z_ESTIMATE; }
int launch_reference(const fold_args *a, const Geometry &g, cudaStream_t st, bool zero_header = false) {
  if (g.planes) return launch_planes_front(a, g, st, zero_header);
  if (a->z_mode == FOLD_Z_GIVEN) return FOLD_OK;
  const int rows = g.B * g.Hq;
  if (a->z_mode == FOLD_Z_ZERO) {
    fold_fill_kernel<<<(rows + 255) / 256, 256, 0, st>>>(a->z, rows, 0.f);
  } else {
    if (g.G > kMaxRows) return FOLD_EUNSUPPORTED;
    EstParams p = est_params(a, g);
    p.n_levels = 1;
    p.lv[0] = kv_level(a->kv, a->stack);
    p.hdr[0] = (zero_header && a->z_mode == FOLD_Z_ESTIMATE) ? static_cast<fold_ws_header *>(a->workspace) : nullptr;
    const dim3 grid(g.Hkv, g.B);
    if (a->z_mode == FOLD_Z_ESTIMATE) {
      const bool early = (a->flags & FOLD_INPUTS_SETTLED) != 0;
      const cudaError_t rc = g.D == 128 ? launch_first(early, fold_estimate_kernel<128>, grid, dim3(kEstSampleThreads), 0, st, p)
                                        : launch_first(early, fold_estimate_kernel<64>, grid, dim3(kEstSampleThreads), 0, st, p);
      if (rc != cudaSuccess) return FOLD_ECUDA;
    } else {
      if (g.D == 128) fold_exact_max_kernel<128><<<grid, kEstThreads, 0, st>>>(p);
      else fold_exact_max_kernel<64><<<grid, kEstThreads, 0, st>>>(p);
    }
  }
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

// The opt-in to large dynamic shared memory is a per-device attribute of the kernel: set at the kernel's first launch on
// a device and remembered in an atomic flag (two host threads racing on a first launch both set it; that is harmless).
// These flags and the address of the static scratch array are the only state the library keeps: no device resources.
typedef std::atomic<int> SmemFlags[64];
template <typename Kernel>
int opt_in_smem(Kernel k, SmemFlags &configured) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FOLD_ECUDA;
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerCtaMax) != cudaSuccess)
      return FOLD_ECUDA;
    if (dev >= 0 && dev < 64) configured[dev].store(1, std::memory_order_release);
  }
  return FOLD_OK;
}

// Ring depths: two CTAs per SM when a useful ring fits, else one CTA with a deeper ring.
template <int D>
int launch_dense_n(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, dim3 grid, cudaStream_t st) {
  using LO = DenseLayout<D, narrow_tile_keys<D>()>;
  const int per_cta2 = kSmemPerSm / 2 - kSmemCtaReserve;
  int stages = (per_cta2 - LO::total(0, p.R)) / (LO::kStage + 16);
  if (stages < 3) stages = (kSmemPerCtaMax - LO::total(0, p.R)) / (LO::kStage + 16);
  if (stages > 8) stages = 8;
  if (stages < 2) return FOLD_EUNSUPPORTED;
  p.stages = stages;
  p.vr = 0;
  static SmemFlags configured;
  if (int rc = opt_in_smem(fold_scan_dense_kernel<D>, configured)) return rc;
  if (launch_pdl(fold_scan_dense_kernel<D>, grid, dim3(kDenseThreads), LO::total(stages, p.R), st, mk, mv, p) != cudaSuccess)
    return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

// 9..16 rows: rows on N in two 8-row tiles per warp.
template <int D>
int launch_dense_nt2(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, dim3 grid, cudaStream_t st) {
  using LO = DenseWideLayout<D>;
  const int per_cta2 = kSmemPerSm / 2 - kSmemCtaReserve;
  int stages = (per_cta2 - LO::total(0)) / (LO::kStage + 16);
  if (stages > 8) stages = 8;
  if (stages < 2) return FOLD_EUNSUPPORTED;
  p.stages = stages;
  p.vr = 0;
  static SmemFlags configured;
  if (int rc = opt_in_smem(fold_scan_dense_nt2_kernel<D>, configured)) return rc;
  if (launch_pdl(fold_scan_dense_nt2_kernel<D>, grid, dim3(kDenseThreads), LO::total(stages), st, mk, mv, p) != cudaSuccess)
    return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}
template <int D>
int launch_dense(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, dim3 grid, cudaStream_t st) {
  // rows on N (half the MMAs and accumulators of rows on M), 16 KB key tiles at either head dimension
  return p.R <= kNarrowRows ? launch_dense_n<D>(mk, mv, p, grid, st) : launch_dense_nt2<D>(mk, mv, p, grid, st);
}

// Stacked rows: the dense ring without reduction buffers; one CTA per (split, 64-row group).  With the block tail
// every stage also carries the tile's block-mean row (1 KB more per stage).
template <int D, bool GATED, bool TAIL>
int launch_stacked_as(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, dim3 grid, cudaStream_t st) {
  using LO = DenseLayout<D>;
  constexpr int kStageBytes = LO::kStage + (TAIL ? 1024 : 0);
  const int per_cta2 = kSmemPerSm / 2 - kSmemCtaReserve;
  int stages = (per_cta2 - LO::total(0, 0)) / (kStageBytes + 16);
  if (stages > 8) stages = 8;
  if (stages < 2) return FOLD_EUNSUPPORTED;
  p.stages = stages;
  p.vr = 0;
  grid.x *= (p.R + 63) / 64;
  static SmemFlags configured;
  if (int e = opt_in_smem(fold_scan_stacked_kernel<D, GATED, TAIL>, configured)) return e;
  if (launch_pdl(fold_scan_stacked_kernel<D, GATED, TAIL>, grid, dim3(kDenseThreads),
                 LO::total(stages, 0) + stages * (kStageBytes - LO::kStage), st, mk, mv, p) != cudaSuccess)
    return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}
template <int D>
int launch_stacked(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, dim3 grid, bool gated, cudaStream_t st) {
  if (!gated) return launch_stacked_as<D, false, false>(mk, mv, p, grid, st);
  return p.vmean ? launch_stacked_as<D, true, true>(mk, mv, p, grid, st) : launch_stacked_as<D, true, false>(mk, mv, p, grid, st);
}

// Stacked rows on tcgen05 (head_dim 128, at least 64 stacked rows): one CTA per (split, 128-row tile).
int launch_stacked_umma(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, dim3 grid, bool gated, bool tail,
                        cudaStream_t st) {
  p.stages = kUmmaStages;
  p.vr = 0;
  grid.x *= (p.R + kUmmaRows - 1) / kUmmaRows;
  static SmemFlags configured_g, configured_d, configured_t;
  cudaError_t rc;
  if (gated && tail) {
    if (int e = opt_in_smem(fold_scan_stacked_umma_kernel<true, true>, configured_t)) return e;
    rc = launch_pdl(fold_scan_stacked_umma_kernel<true, true>, grid, dim3(kUmmaThreads), UmmaLayout::kTotal, st, mk, mv, p);
  } else if (gated) {
    if (int e = opt_in_smem(fold_scan_stacked_umma_kernel<true, false>, configured_g)) return e;
    rc = launch_pdl(fold_scan_stacked_umma_kernel<true, false>, grid, dim3(kUmmaThreads), UmmaLayout::kTotal, st, mk, mv, p);
  } else {
    if (int e = opt_in_smem(fold_scan_stacked_umma_kernel<false, false>, configured_d)) return e;
    rc = launch_pdl(fold_scan_stacked_umma_kernel<false, false>, grid, dim3(kUmmaThreads), UmmaLayout::kTotal, st, mk, mv, p);
  }
  if (rc != cudaSuccess) return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

// More than 128 stacked rows: one CTA per (split, pair of 128-row tiles); the two tiles alternate on the tensor pipe.
int launch_stacked_pair(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, dim3 grid, bool gated,
                        cudaStream_t st) {
  p.stages = kPairStages;
  p.vr = 0;
  grid.x *= (p.R + kPairRows - 1) / kPairRows;
  static SmemFlags configured_g, configured_d;
  cudaError_t rc;
  if (gated) {
    if (int e = opt_in_smem(fold_scan_stacked_pair_kernel<true>, configured_g)) return e;
    rc = launch_pdl(fold_scan_stacked_pair_kernel<true>, grid, dim3(kPairThreads), PairLayout::kTotal, st, mk, mv, p);
  } else {
    if (int e = opt_in_smem(fold_scan_stacked_pair_kernel<false>, configured_d)) return e;
    rc = launch_pdl(fold_scan_stacked_pair_kernel<false>, grid, dim3(kPairThreads), PairLayout::kTotal, st, mk, mv, p);
  }
  if (rc != cudaSuccess) return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

// Row blocks of up to 16 rows at head_dim 128 on tcgen05: a persistent grid of at most one CTA per SM, two workers each.
int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
    return 148;
  return n;
}
bool cooperative_launch_supported() {
  int dev = 0, v = 0;
  return cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && v != 0;
}
// f.mode != 0: the whole decode in this launch, which is then a cooperative one (its CTAs meet at a grid-wide barrier
// between the scan and the partial add; the grid is one CTA per SM at most, so all of them are resident).
template <bool GATED, int NC, bool TAIL, int KEYS>
int launch_decode_as(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, const FusedParams &f, int ctas, cudaStream_t st) {
  static SmemFlags configured;
  if (int rc = opt_in_smem(fold_scan_decode_kernel<GATED, NC, TAIL, KEYS>, configured)) return rc;
  cudaError_t rc;
  if (f.mode) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(ctas); cfg.blockDim = dim3(kDecThreads); cfg.dynamicSmemBytes = DecLayout::kTotal; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    rc = cudaLaunchKernelEx(&cfg, fold_scan_decode_kernel<GATED, NC, TAIL, KEYS>, mk, mv, p, f);
  } else {
    rc = launch_pdl(fold_scan_decode_kernel<GATED, NC, TAIL, KEYS>, dim3(ctas), dim3(kDecThreads), DecLayout::kTotal, st, mk, mv, p, f);
  }
  if (rc != cudaSuccess) return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}
template <bool GATED, bool TAIL, int KEYS>
int launch_decode_rows(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, const FusedParams &f, int ctas, cudaStream_t st) {
  if (p.R == 1) return launch_decode_as<GATED, 1, TAIL, KEYS>(mk, mv, p, f, ctas, st);
  if (p.R <= 4) return launch_decode_as<GATED, 4, TAIL, KEYS>(mk, mv, p, f, ctas, st);
  if (p.R <= 8) return launch_decode_as<GATED, 8, TAIL, KEYS>(mk, mv, p, f, ctas, st);
  return FOLD_EUNSUPPORTED;                                  // more rows stay on the mma.sync kernels
}
// keys: the key ring's depth for a depth-gated scan (2, 3 or 4 of the six stages; scheduling only); dense decode runs 2.
template <bool GATED, bool TAIL>
int launch_decode(const CUtensorMap &mk, const CUtensorMap &mv, ScanParams &p, const FusedParams &f, int ctas, int keys,
                  cudaStream_t st) {
  if (!GATED) return launch_decode_rows<GATED, TAIL, 2>(mk, mv, p, f, ctas, st);
  if (keys == 2) return launch_decode_rows<GATED, TAIL, 2>(mk, mv, p, f, ctas, st);
  if (keys == 4) return launch_decode_rows<GATED, TAIL, 4>(mk, mv, p, f, ctas, st);
  return launch_decode_rows<GATED, TAIL, 3>(mk, mv, p, f, ctas, st);
}

// Narrow row blocks (rows on N): unpadded value slices; three K stages (measured: a fourth buys nothing and costs L1).
template <int D, bool TAIL, int NT>
int launch_gated_narrow(const CUtensorMap &mk, const CUtensorMap &mvs, ScanParams &p, dim3 grid, cudaStream_t st) {
  using LN = GatedNarrowLayout<D, TAIL, NT>;
  const int per_cta2 = kSmemPerSm / 2 - kSmemCtaReserve;
  int nvr = 2;
  int nstages = (per_cta2 - LN::total(0, nvr)) / (LN::kKStage + 16);
  if (nstages > 3) nstages = 3;
  if (nstages < 2 || nvr < 1 || LN::total(nstages, nvr) > kSmemPerCtaMax) return FOLD_EUNSUPPORTED;
  p.stages = nstages;
  p.vr = nvr;
  static SmemFlags configured;
  if (int rc = opt_in_smem(fold_scan_gated_narrow_kernel<D, TAIL, NT>, configured)) return rc;
  if (launch_pdl(fold_scan_gated_narrow_kernel<D, TAIL, NT>, grid, dim3(kGatedThreads), LN::total(nstages, nvr), st, mk, mvs, p) !=
      cudaSuccess)
    return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

// Gated scan: value slots hold rows whose requests can only be issued after scoring, so shared
// memory is split between the key ring and the value slots of each slice.
template <int D>
int launch_gated(const CUtensorMap &mk, const CUtensorMap &mvs, ScanParams &p, dim3 grid, cudaStream_t st) {
  if (p.R <= kNarrowRows)                                    // rows on N; with or without the block tail
    return p.vmean ? launch_gated_narrow<D, true, 1>(mk, mvs, p, grid, st) : launch_gated_narrow<D, false, 1>(mk, mvs, p, grid, st);
  // 9..16 rows: two 8-row N tiles per warp
  return p.vmean ? launch_gated_narrow<D, true, 2>(mk, mvs, p, grid, st) : launch_gated_narrow<D, false, 2>(mk, mvs, p, grid, st);
}

// Rows per (sequence, kv head) up to which the row-block kernels run (in 16-row groups, each its own CTA sharing the
// kv head's tiles through L2); beyond, the stacked-row kernels.
int row_block_rows() {
  return 2 * kMaxRows;
}

// CTAs per (sequence, kv head).  A CTA pays a few microseconds to start (barriers, first loads), so it should
// walk at least ~32 tiles; below about one and a half waves of CTAs the machine is not filled, so short
// batches are cut finer instead.  Only scheduling: the result does not depend on the choice.
int choose_splits(const fold_args *a, const Geometry &g, int tile_keys) {
  const int n = a->kv.max_seqlen;
  int max_chunks = num_chunks_of(n) > 0 ? num_chunks_of(n) : 1;
  if (max_chunks > 65535) max_chunks = 65535;               // splits index a grid dimension (a split walks several chunks)
  if (a->num_splits > 0) return a->num_splits < max_chunks ? a->num_splits : max_chunks;
  const long long units = (long long)g.num_seqs * g.Hkv *
                          (g.planes ? (g.R + kMaxRows - 1) / kMaxRows :
                           g.R > 128 ? (g.R + 255) / 256 : (g.R <= row_block_rows() ? (g.R + kMaxRows - 1) / kMaxRows : 1));   // CTAs per split
  const int tiles_unit = max_chunks * (chunk_keys_of(n) / tile_keys);
  int s = tiles_unit / 32;
  s = s < 1 ? 1 : (s > max_chunks ? max_chunks : s);
  while (units * s < 444 && s < max_chunks) ++s;
  // even shares: every CTA of the longest sequence gets the same whole number of chunks (14 splits of 16 chunks
  // would finish no sooner than 8)
  const int per = max_chunks / s > 1 ? max_chunks / s : 1;
  return (max_chunks + per - 1) / per;
}

// As many plane-A stages as fit beside the gather buffers with kPlaneCtasPerSm CTAs on an SM.
template <int D, bool DRAFTS, bool TAIL, bool VFP8, int NT>
int launch_planes_nt(const CUtensorMap &ma, const CUtensorMap &mv, PlaneScanParams &pp, dim3 grid, cudaStream_t st) {
  using LO = PlaneLayout<D, TAIL>;
  const int per_cta = kSmemPerSm / kPlaneCtasPerSm - kSmemCtaReserve;
  int stages = (per_cta - LO::total(0)) / (LO::kStage + 16);
  if (stages > LO::kMaxStages) stages = LO::kMaxStages;
  if (stages < 2) return FOLD_EUNSUPPORTED;
  pp.s.stages = stages;
  static SmemFlags configured;
  if (int rc = opt_in_smem(fold_scan_planes_kernel<D, DRAFTS, TAIL, VFP8, NT>, configured)) return rc;
  if (launch_pdl(fold_scan_planes_kernel<D, DRAFTS, TAIL, VFP8, NT>, grid, dim3(kDenseThreads), LO::total(stages), st, ma, mv, pp) !=
      cudaSuccess)
    return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}
// up to 8 rows per (sequence, kv head): one 8-row tile; 9 to 16: two
template <int D, bool DRAFTS, bool TAIL, bool VFP8 = false>
int launch_planes_as(const CUtensorMap &ma, const CUtensorMap &mv, PlaneScanParams &pp, dim3 grid, cudaStream_t st) {
  return pp.s.R <= kNarrowRows ? launch_planes_nt<D, DRAFTS, TAIL, VFP8, 1>(ma, mv, pp, grid, st)
                               : launch_planes_nt<D, DRAFTS, TAIL, VFP8, 2>(ma, mv, pp, grid, st);
}
template <int D>
int launch_planes_kernel(const CUtensorMap &ma, const CUtensorMap &mv, PlaneScanParams &pp, dim3 grid, cudaStream_t st) {
  const bool drafts = pp.s.draft_len > 0, tail = pp.s.vmean != nullptr;      // (separate instantiations: registers)
  if (pp.kv.v1)                                              // E4M3 values: their cut model is applied at the chunk's end
    return drafts ? launch_planes_as<D, true, false, true>(ma, mv, pp, grid, st) : launch_planes_as<D, false, false, true>(ma, mv, pp, grid, st);
  if (drafts) return tail ? launch_planes_as<D, true, true>(ma, mv, pp, grid, st) : launch_planes_as<D, true, false>(ma, mv, pp, grid, st);
  return tail ? launch_planes_as<D, false, true>(ma, mv, pp, grid, st) : launch_planes_as<D, false, false>(ma, mv, pp, grid, st);
}

// Two-plane keys: one kernel for dense and finite depth (the depth gate is a comparison against -T = -inf).
int launch_scan_planes(const fold_args *a, const Geometry &g, cudaStream_t st) {
  const fold_kv &kv = a->kv;
  const bool paged = kv.page_table != nullptr;
  const int tile_keys = kPlaneTileKeys;
  const int box_tok = paged ? (kv.page_size < tile_keys ? kv.page_size : tile_keys) : tile_keys;
  CUtensorMap ma;
  MapAxes axes;
  if (int rc = make_plane_map(&ma, &axes, kv, g.D, g.Hkv, box_tok)) return rc;
  CUtensorMap mv = ma;                                       // value rows of one 16-key sub-slice as a box (BF16 values)
  MapAxes vaxes = axes;
  if (!kv.v_plane_1)
    if (int rc = make_map(&mv, &vaxes, kv.v, kv, g.D, g.Hkv, 16)) return rc;
  PlaneScanParams pp;
  memset(&pp, 0, sizeof(pp));
  pp.vpos_tok = vaxes.pos_tok; pp.vpos_head = vaxes.pos_head; pp.vpos_seq = vaxes.pos_seq;
  pp.box_min = 13;
  ScanParams &p = pp.s;
  p.z = a->z;
  p.seqlens = kv.seqlens;
  p.page_table = kv.page_table;
  p.v = static_cast<const __nv_bfloat16 *>(kv.v);
  p.v_stride_seq = kv.stride_seq; p.v_stride_tok = kv.stride_tok; p.v_stride_head = kv.stride_head;
  p.slots = reinterpret_cast<float *>(static_cast<uint8_t *>(a->workspace) + kHeaderBytes);
  p.slot_stride = g.slot_stride;
  p.hdr = static_cast<fold_ws_header *>(a->workspace);
  p.max_slots = g.max_slots; p.max_seqlen = kv.max_seqlen;
  p.Hq = g.Hq; p.Hkv = g.Hkv; p.G = g.G; p.stack = g.stack; p.R = g.R;
  p.paged = paged; p.page_shift = paged ? ilog2(kv.page_size) : 0;
  p.max_pages = kv.max_pages_per_seq; p.num_pages = kv.num_pages > 0 ? kv.num_pages : 1;
  p.box_tok = box_tok;
  p.pos_tok = axes.pos_tok; p.pos_head = axes.pos_head; p.pos_seq = axes.pos_seq;
  p.num_splits = choose_splits(a, g, tile_keys);
  p.scale_log2 = (float)((double)a->softmax_scale * 1.4426950408889634);
  p.neg_T = isinf(a->depth_T) ? -INFINITY : -a->depth_T;
  p.row_groups = (g.R + kMaxRows - 1) / kMaxRows;            // blocks of 16 rows, each its own CTA (a cascade's shared level)
  p.draft_mask = a->draft_len > 0 ? a->draft_mask : nullptr;
  p.draft_len = a->draft_len;
  if (!isinf(a->depth_T) && kv.v_plane_1) {                  // 8-bit values: the table holds the sequences' mean rows (block 0)
    pp.vrun = static_cast<const __nv_bfloat16 *>(kv.v_block_mean);
    pp.vrun_stride_seq = kv.mean_stride_seq; pp.vrun_stride_head = kv.mean_stride_head;
  } else if (!isinf(a->depth_T)) {                           // block tail: nothing is cut in dense decode
    p.vmean = static_cast<const __nv_bfloat16 *>(kv.v_block_mean);
    p.vm_stride_seq = kv.mean_stride_seq; p.vm_stride_block = kv.mean_stride_block; p.vm_stride_head = kv.mean_stride_head;
  }
  pp.kv = plane_view(kv);
  uint8_t *ws = static_cast<uint8_t *>(a->workspace);
  pp.qplanes = reinterpret_cast<const int8_t *>(ws + g.q_off);
  pp.qeta = reinterpret_cast<const float *>(ws + g.q_off + round_up((size_t)g.B * g.Hq * 2 * g.D, 256));
  pp.auto_tau_v = a->refine_tau_v == 0.f;
  pp.neg_tau_v = a->refine_tau_v < 0.f ? INFINITY : -a->refine_tau_v;
  pp.auto_tau = a->refine_tau == 0.f;
  pp.neg_tau = a->refine_tau < 0.f ? INFINITY : -a->refine_tau;      // tau = inf -> -inf: every live key
  const dim3 grid(g.Hkv * p.row_groups, p.num_splits, g.num_seqs);
  return g.D == 128 ? launch_planes_kernel<128>(ma, mv, pp, grid, st) : launch_planes_kernel<64>(ma, mv, pp, grid, st);
}

// Does the whole decode fit one launch of the tcgen05 row-block kernel?  Head_dim 128, up to 8 rows per (sequence, kv
// head), one request per sequence, the reference estimated or given, and one wave: at most one canonical chunk per
// worker (two workers per CTA, one CTA per SM).  The result's bits are those of the separate launches.
bool one_launch_decode(const fold_args *a, const Geometry &g) {
  if (g.planes || g.D != 128 || g.R > kDecMaxRows || g.stack != 1) return false;
  if (a->flags & FOLD_SEPARATE_LAUNCHES) return false;
  if (a->z_mode != FOLD_Z_ESTIMATE && a->z_mode != FOLD_Z_GIVEN) return false;
  // measured on a B200 (8 heads x 4096 keys, calls back to back): given reference 16.5 us in one launch against 18.6 in
  // two; estimated reference 19.8 against 19.0 in three -- so the estimate keeps its own kernel unless asked
  if (a->z_mode == FOLD_Z_ESTIMATE && !(a->flags & FOLD_ONE_LAUNCH)) return false;
  const long long entries = (long long)g.num_seqs * g.Hkv * ((g.max_slots + 1) & ~1);   // chunk-major list, even per unit
  if (entries > 2LL * sm_count()) return false;
  if (a->num_splits > 0 && a->num_splits < g.max_slots) return false;   // a split hint that bounds the grid: honour it
  return cooperative_launch_supported();
}

int launch_scan(const fold_args *a, const Geometry &g, cudaStream_t st, const FusedParams *fused = nullptr) {
  if (g.planes) return launch_scan_planes(a, g, st);
  const fold_kv &kv = a->kv;
  const bool paged = kv.page_table != nullptr;
  // narrow row blocks walk 16 KB key tiles: 128 keys at D = 64
  // (row blocks of 9..16 rows run the same kernels with two N tiles per warp)
  const bool narrow_tiles = g.R <= row_block_rows();
  const bool gated = !isinf(a->depth_T);
  // head_dim 128, up to 8 rows: the tcgen05 row-block kernel (keys on M, 128-key tiles)
  // Which kernel runs may depend on the head dimension, the rows per (sequence, kv head) and the depth being finite
  // only -- never on the batch or on lengths: a slot's bits must not depend on what else is decoded.
  const bool decode_umma = g.D == 128 && g.R <= kDecMaxRows;
  const int tile_keys = decode_umma ? kDecKeys : (narrow_tiles && g.D == 64) ? narrow_tile_keys<64>() : kTileKeys;
  const int box_tok = paged ? (kv.page_size < tile_keys ? kv.page_size : tile_keys) : tile_keys;
  CUtensorMap mk, mv;
  MapAxes axes;
  if (int rc = make_map(&mk, &axes, kv.k, kv, g.D, g.Hkv, box_tok)) return rc;
  const bool stacked = g.R > row_block_rows();
  // dense and stacked: value tiles like key tiles; gated: a box of one 16-key slice
  // (the tcgen05 row-block kernel: groups of 32 keys, or of a page if pages are shorter)
  const int vbox = decode_umma ? (paged && kv.page_size < 32 ? kv.page_size : 32) : 16;
  if (int rc = make_map(&mv, &axes, kv.v, kv, g.D, g.Hkv, (gated && !stacked) ? vbox : box_tok)) return rc;

  ScanParams p;
  memset(&p, 0, sizeof(p));
  p.q = static_cast<const __nv_bfloat16 *>(a->q);
  p.q_stride_b = a->q_stride_b; p.q_stride_h = a->q_stride_h;
  p.z = a->z;
  p.seqlens = kv.seqlens;
  p.page_table = kv.page_table;
  p.v = static_cast<const __nv_bfloat16 *>(kv.v);
  p.k = static_cast<const __nv_bfloat16 *>(kv.k);
  p.v_stride_seq = kv.stride_seq; p.v_stride_tok = kv.stride_tok; p.v_stride_head = kv.stride_head;
  p.draft_mask = a->draft_len > 0 ? a->draft_mask : nullptr;
  p.draft_len = a->draft_len;
  p.vmean = static_cast<const __nv_bfloat16 *>(kv.v_block_mean);
  p.vm_stride_seq = kv.mean_stride_seq; p.vm_stride_block = kv.mean_stride_block; p.vm_stride_head = kv.mean_stride_head;
  p.slots = reinterpret_cast<float *>(static_cast<uint8_t *>(a->workspace) + kHeaderBytes);
  p.slot_stride = g.slot_stride;
  p.hdr = static_cast<fold_ws_header *>(a->workspace);
  p.max_slots = g.max_slots; p.max_seqlen = kv.max_seqlen;
  p.Hq = g.Hq; p.Hkv = g.Hkv; p.G = g.G; p.stack = g.stack; p.R = g.R;
  p.num_seqs = g.num_seqs;
  p.paged = paged; p.page_shift = paged ? ilog2(kv.page_size) : 0;
  p.max_pages = kv.max_pages_per_seq; p.num_pages = kv.num_pages > 0 ? kv.num_pages : 1;
  p.box_tok = box_tok;
  p.pos_tok = axes.pos_tok; p.pos_head = axes.pos_head; p.pos_seq = axes.pos_seq;
  p.scale_log2 = (float)((double)a->softmax_scale * 1.4426950408889634);
  p.neg_T = isinf(a->depth_T) ? -INFINITY : -a->depth_T;
  if (decode_umma) {
    // one CTA per SM at most, two workers each; the split hint only bounds the grid (never a bit of the result)
    const long long units = (long long)g.num_seqs * g.Hkv;
    long long ctas = (units * g.max_slots + 1) / 2;
    if (a->num_splits > 0 && (units * a->num_splits + 1) / 2 < ctas) ctas = (units * a->num_splits + 1) / 2;
    const int sms = sm_count();
    if (ctas > sms) ctas = sms;
    p.vr = vbox;                                             // tokens per value box
    p.box_min = vbox * 13 / 16;                              // fetch a group whole from this many live rows on
    p.num_splits = 1;
    p.stages = 8;                                            // tiles the L2 requests run ahead of the ring
    FusedParams f;
    memset(&f, 0, sizeof(f));
    if (fused) {
      f = *fused;
      p.chunk_major = 1;
      ctas = units * ((g.max_slots + 1) / 2);                // one chunk per worker at most
    }
    // The caller's expectation of the live fraction picks the ring's split.  Measured on a B200 (us, splits 2+4 / 3+3 /
    // 4+2): all live, group 4 -- 321.6 / 332.5 / 320.1; 90 % live, MHA, 8192-key sequences -- 1265 / 1251 / 1286; half
    // live, paged -- 278.5 / 272.8 / 300.6; 16 % live -- 1786 / 1532 / 1738; nothing live, 1024-key chunks -- 1504 / 1297 /
    // 1240 and 239.7 / 192.2 / 183.2; nothing live, 256-key chunks -- 978 / 858 / 912.  So: 95 % and more live -> two key
    // and four value stages (dense decode's split); under 2 % with 1024-key chunks -> four and two; else three and three.
    const float lh = a->live_hint;
    const int keys = !(lh > 0.f) ? 3 : (lh >= 0.95f ? 2 : (lh < 0.02f && kv.max_seqlen > 8192 ? 4 : 3));
    if (!gated) return launch_decode<false, false>(mk, mv, p, f, (int)ctas, 2, st);
    return p.vmean ? launch_decode<true, true>(mk, mv, p, f, (int)ctas, keys, st) : launch_decode<true, false>(mk, mv, p, f, (int)ctas, keys, st);
  }
  p.num_splits = choose_splits(a, g, tile_keys);

  // row-block kernels: kv heads on x (fastest), splits on y; stacked kernels: (row group, split) on x, heads on y
  p.row_groups = stacked || g.R <= kMaxRows ? 1 : (g.R + kMaxRows - 1) / kMaxRows;
  const dim3 grid = stacked ? dim3(p.num_splits, g.Hkv, g.num_seqs) : dim3(g.Hkv * p.row_groups, p.num_splits, g.num_seqs);
  p.box_min = 13;
  if (stacked) {
    // with a table of block means the single-tile tcgen05 kernel serves every row count from 64 up (a CTA per 128 rows:
    // the pair kernel's tensor memory has no room for the cut-mass operand)
    const bool tail = gated && p.vmean != nullptr;
    if (g.D == 128 && g.R > kUmmaRows && !tail) return launch_stacked_pair(mk, mv, p, grid, gated, st);
    if (g.D == 128 && g.R >= 64) return launch_stacked_umma(mk, mv, p, grid, gated, tail, st);
    return g.D == 128 ? launch_stacked<128>(mk, mv, p, grid, gated, st) : launch_stacked<64>(mk, mv, p, grid, gated, st);
  }
  if (g.D == 128) return gated ? launch_gated<128>(mk, mv, p, grid, st) : launch_dense<128>(mk, mv, p, grid, st);
  return gated ? launch_gated<64>(mk, mv, p, grid, st) : launch_dense<64>(mk, mv, p, grid, st);
}

void fill_partials(const fold_args *a, const Geometry &g, fold_partials *dst) {
  dst->slots = reinterpret_cast<float *>(static_cast<uint8_t *>(a->workspace) + kHeaderBytes);
  dst->seqlens = a->kv.seqlens;
  dst->z = a->z;
  dst->batch = g.B; dst->num_q_heads = g.Hq; dst->num_kv_heads = g.Hkv; dst->head_dim = g.D; dst->stack = g.stack;
  dst->num_seqs = g.num_seqs; dst->max_slots = g.max_slots; dst->rows = g.R;
  dst->slot_stride = g.slot_stride;
  dst->max_seqlen = a->kv.max_seqlen;
}

}  // namespace

extern "C" {

int32_t fold_chunk_keys(int32_t n) { return chunk_keys_of(n); }
int32_t fold_num_chunks(int32_t n) { return n <= 0 ? 0 : num_chunks_of(n); }

size_t fold_workspace_bytes(const fold_args *args) {
  Geometry g;
  fold_args tmp;
  if (!args) return 0;
  tmp = *args;
  // sizing must not depend on pointers the caller has not allocated yet
  if (tmp.head_dim != 64 && tmp.head_dim != 128) return 0;
  if (tmp.batch < 1 || tmp.num_q_heads < 1 || tmp.num_kv_heads < 1 || tmp.stack < 1) return 0;
  if (tmp.num_q_heads % tmp.num_kv_heads || tmp.batch % tmp.stack) return 0;
  const int G = tmp.num_q_heads / tmp.num_kv_heads;
  const long long R = (long long)tmp.stack * G;
  if (G > kMaxRows || R > kMaxStackedRows || tmp.kv.max_seqlen < 0) return 0;
  g.max_slots = max_chunks_upto(tmp.kv.max_seqlen);
  if (g.max_slots < 1) g.max_slots = 1;
  g.slot_stride = R * tmp.head_dim + ((R + 3) / 4) * 4;
  const size_t base = kHeaderBytes + (size_t)(tmp.batch / tmp.stack) * tmp.num_kv_heads * g.max_slots * g.slot_stride * sizeof(float);
  if (!tmp.kv.k_plane_a) return base;
  return round_up(base, 256) + qplane_bytes((long long)tmp.batch * tmp.num_q_heads, tmp.head_dim);
}

}  // extern "C"

namespace {
// zero_headers: the estimate kernel also zeroes every level's workspace header (the cascade's scans then need no memset)
int estimate_levels(const fold_args *const *levels, int n_levels, fold_stream stream, bool zero_headers) {
  if (!levels || n_levels < 1 || n_levels > kMaxLevels) return FOLD_EINVAL;
  const fold_args *a0 = levels[0];
  if (!a0) return FOLD_EINVAL;
  for (int l = 1; l < n_levels; ++l)                         // a cascade keeps to one key format
    if (!levels[l] || (levels[l]->kv.k_plane_a != nullptr) != (a0->kv.k_plane_a != nullptr)) return FOLD_EUNSUPPORTED;
  if (a0->kv.k_plane_a) {                                    // two-plane keys: the split rows go to every level's workspace
    Geometry gs[kMaxLevels];
    fold_args tmp[kMaxLevels];
    const fold_args *tp[kMaxLevels];
    for (int l = 0; l < n_levels; ++l) {
      const fold_args *a = levels[l];
      if (a->q != a0->q || a->z != a0->z || a->batch != a0->batch || a->num_q_heads != a0->num_q_heads ||
          a->num_kv_heads != a0->num_kv_heads || a->head_dim != a0->head_dim || a->softmax_scale != a0->softmax_scale)
        return FOLD_EINVAL;
      tmp[l] = *a;
      tmp[l].z_mode = FOLD_Z_ESTIMATE;
      tp[l] = &tmp[l];
      if (int rc = check_args(&tmp[l], &gs[l], false)) return rc;
      if (l + 1 < n_levels && tmp[l].draft_len > 0) return FOLD_EINVAL;      // drafts end the last level
      if (!tmp[l].workspace || !aligned(tmp[l].workspace, 256)) return FOLD_EINVAL;
      if (tmp[l].workspace_bytes < gs[l].ws_bytes) return FOLD_EWORKSPACE;
    }
    return launch_planes_front_levels(tp, gs, n_levels, static_cast<cudaStream_t>(stream), zero_headers);
  }
  if (a0->head_dim != 64 && a0->head_dim != 128) return FOLD_EUNSUPPORTED;
  if (a0->batch < 1 || a0->num_q_heads < 1 || a0->num_kv_heads < 1 || a0->num_q_heads % a0->num_kv_heads)
    return FOLD_EINVAL;
  if (!a0->q || !a0->z || !aligned(a0->q, 16) || a0->q_stride_b % 8 || a0->q_stride_h % 8) return FOLD_EINVAL;
  if (!(a0->softmax_scale > 0.f) || isinf(a0->softmax_scale)) return FOLD_EINVAL;
  const int G = a0->num_q_heads / a0->num_kv_heads;
  if (G > kMaxRows) return FOLD_EUNSUPPORTED;
  Geometry g;
  g.B = a0->batch; g.Hq = a0->num_q_heads; g.Hkv = a0->num_kv_heads; g.G = G; g.D = a0->head_dim;
  EstParams p = est_params(a0, g);
  p.n_levels = n_levels;
  {                                                          // drafts sit at the end of the last level
    const fold_args *al = levels[n_levels - 1];
    if (!al || al->draft_len < 0 || al->draft_len > 32) return FOLD_EINVAL;
    if (al->draft_len > 0 && (!al->draft_mask || !aligned(al->draft_mask, 4))) return FOLD_EINVAL;
    p.draft_mask = al->draft_len > 0 ? al->draft_mask : nullptr;
    p.draft_len = al->draft_len;
  }
  for (int l = 0; l < n_levels; ++l) {
    const fold_args *a = levels[l];
    if (!a || a->head_dim != a0->head_dim || a->num_kv_heads != a0->num_kv_heads || a->batch != a0->batch)
      return FOLD_EINVAL;
    if (a->stack < 1 || a->batch % a->stack || a->batch / a->stack != a->kv.num_seqs) return FOLD_EINVAL;
    if (int rc = check_kv(a->kv, a->head_dim, a->num_kv_heads)) return rc;
    p.lv[l] = kv_level(a->kv, a->stack);
    if (zero_headers) {
      if (!a->workspace || !aligned(a->workspace, 256)) return FOLD_EINVAL;
      if (a->workspace_bytes < kHeaderBytes) return FOLD_EWORKSPACE;
      p.hdr[l] = static_cast<fold_ws_header *>(a->workspace);
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid(g.Hkv, g.B);
  const bool early = (a0->flags & FOLD_INPUTS_SETTLED) != 0;
  const cudaError_t rc = g.D == 128 ? launch_first(early, fold_estimate_kernel<128>, grid, dim3(kEstSampleThreads), 0, st, p)
                                    : launch_first(early, fold_estimate_kernel<64>, grid, dim3(kEstSampleThreads), 0, st, p);
  if (rc != cudaSuccess) return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

// header_done: the workspace header has been zeroed by a kernel already in the stream
// reference_done: the level's reference kernel (a cascade's two-plane front kernel over all levels) is already in the stream
int decode_split_impl(const fold_args *args, fold_partials *dst, fold_stream stream, bool header_done,
                      bool reference_done = false) {
  Geometry g;
  if (int rc = check_args(args, &g, false)) return rc;
  if (!dst) return FOLD_EINVAL;
  if (!args->workspace || !aligned(args->workspace, 256)) return FOLD_EINVAL;
  if (args->workspace_bytes < g.ws_bytes) return FOLD_EWORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the header is zeroed by the reference kernel where one runs (estimate, or the two-plane front kernel), else by a
  // memset issued first, so that reference -> scan -> partial add stay adjacent kernels in the stream
  const bool by_kernel = !reference_done && header_zeroed_by_reference(args, g);
  if (!by_kernel && !header_done && cudaMemsetAsync(args->workspace, 0, 64, st) != cudaSuccess) return FOLD_ECUDA;
  if (!reference_done)
    if (int rc = launch_reference(args, g, st, by_kernel)) return rc;
  if (int rc = launch_scan(args, g, st)) return rc;
  fill_partials(args, g, dst);
  return FOLD_OK;
}
}  // namespace

extern "C" {

int fold_estimate_z(const fold_args *const *levels, int n_levels, fold_stream stream) {
  return estimate_levels(levels, n_levels, stream, false);
}

int fold_decode_split(const fold_args *args, fold_partials *dst, fold_stream stream) {
  return decode_split_impl(args, dst, stream, false);
}

int fold_cascade_merge(const fold_partials *const *levels, int n_levels, void *out, float *lse, int32_t *row_status,
                       fold_stream stream) {
  if (!levels || n_levels < 1 || n_levels > kMaxLevels || !out) return FOLD_EINVAL;
  const fold_partials *p0 = levels[0];
  if (!p0) return FOLD_EINVAL;
  if (p0->head_dim != 64 && p0->head_dim != 128) return FOLD_EUNSUPPORTED;
  MergeParams p;
  memset(&p, 0, sizeof(p));
  for (int l = 0; l < n_levels; ++l) {
    const fold_partials *q = levels[l];
    if (!q || !q->slots || !q->seqlens || !q->z) return FOLD_EINVAL;
    if (q->batch != p0->batch || q->num_q_heads != p0->num_q_heads || q->num_kv_heads != p0->num_kv_heads ||
        q->head_dim != p0->head_dim || q->z != p0->z)
      return FOLD_EINVAL;
    if (q->stack < 1 || q->batch % q->stack || q->num_seqs != q->batch / q->stack) return FOLD_EINVAL;
    if (q->rows != q->stack * (q->num_q_heads / q->num_kv_heads) || q->max_slots < 1) return FOLD_EINVAL;
    p.lv[l].slots = q->slots; p.lv[l].seqlens = q->seqlens; p.lv[l].slot_stride = q->slot_stride;
    p.lv[l].stack = q->stack; p.lv[l].max_slots = q->max_slots; p.lv[l].rows = q->rows;
    p.lv[l].max_seqlen = q->max_seqlen;
  }
  p.z = p0->z;
  p.out = static_cast<__nv_bfloat16 *>(out);
  p.lse = lse; p.row_status = row_status;
  p.n_levels = n_levels; p.Hq = p0->num_q_heads; p.Hkv = p0->num_kv_heads;
  p.G = p0->num_q_heads / p0->num_kv_heads; p.D = p0->head_dim;
  // warps per row (a power of two up to 16): about 8 slots per warp.  One level whose slots then fit a warp's
  // registers is merged in one load pass; otherwise two passes, and fewer warps when the rows alone fill the machine.
  int total_slots = 0;
  for (int l = 0; l < n_levels; ++l) total_slots += max_chunks_upto(levels[l]->max_seqlen);
  const long long n_rows = (long long)p0->batch * p.Hq;
  int warps = 1;
  while (warps < kMergeMaxWarps && warps * 8 < total_slots) warps <<= 1;
  const bool resident = n_levels == 1 && (total_slots + warps - 1) / warps <= kMergeResident;
  if (!resident)
    while (warps > 1 && n_rows * warps > 4096) warps >>= 1;
  const int cta_warps = warps < 4 ? 4 : warps;
  const long long rows_per_cta = cta_warps / warps;
  const dim3 grid((unsigned)((n_rows + rows_per_cta - 1) / rows_per_cta)), block(32 * cta_warps);
  const cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool res = resident && (total_slots + warps - 1) / warps <= kMergeResident;
  cudaError_t rc;
  if (p.D == 128)
    rc = res ? launch_pdl(fold_merge_kernel<4, true>, grid, block, 0, st, p, warps, n_rows)
             : launch_pdl(fold_merge_kernel<4, false>, grid, block, 0, st, p, warps, n_rows);
  else
    rc = res ? launch_pdl(fold_merge_kernel<2, true>, grid, block, 0, st, p, warps, n_rows)
             : launch_pdl(fold_merge_kernel<2, false>, grid, block, 0, st, p, warps, n_rows);
  if (rc != cudaSuccess) return FOLD_ECUDA;
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

int fold_block_means(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, fold_stream stream) {
  if (!kv || num_kv_heads < 1) return FOLD_EINVAL;
  if (head_dim != 64 && head_dim != 128) return FOLD_EUNSUPPORTED;
  if (!kv->v_block_mean) return FOLD_EINVAL;
  if (int rc = check_kv(*kv, head_dim, num_kv_heads)) return rc;
  const int max_blocks = (kv->max_seqlen + 63) / 64;
  if (max_blocks == 0) return FOLD_OK;
  MeanParams p;
  p.v = static_cast<const __nv_bfloat16 *>(kv->v);
  p.v_stride_seq = kv->stride_seq; p.v_stride_tok = kv->stride_tok; p.v_stride_head = kv->stride_head;
  p.mean = static_cast<__nv_bfloat16 *>(const_cast<void *>(kv->v_block_mean));
  p.m_stride_seq = kv->mean_stride_seq; p.m_stride_block = kv->mean_stride_block; p.m_stride_head = kv->mean_stride_head;
  p.seqlens = kv->seqlens; p.page_table = kv->page_table;
  p.max_seqlen = kv->max_seqlen;
  p.page_shift = kv->page_table ? ilog2(kv->page_size) : 0;
  p.max_pages = kv->max_pages_per_seq; p.num_pages = kv->num_pages > 0 ? kv->num_pages : 1;
  p.Hkv = num_kv_heads;
  const dim3 grid((max_blocks + 3) / 4, num_kv_heads, kv->num_seqs), block(32, 4);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (head_dim == 128) fold_block_mean_kernel<128><<<grid, block, 0, st>>>(p);
  else fold_block_mean_kernel<64><<<grid, block, 0, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

int fold_running_means(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, fold_stream stream) {
  if (!kv || num_kv_heads < 1) return FOLD_EINVAL;
  if (head_dim != 64 && head_dim != 128) return FOLD_EUNSUPPORTED;
  if (!kv->v_block_mean || !kv->v) return FOLD_EINVAL;
  if (int rc = check_kv(*kv, head_dim, num_kv_heads)) return rc;
  MeanParams p;
  p.v = static_cast<const __nv_bfloat16 *>(kv->v);
  p.v_stride_seq = kv->stride_seq; p.v_stride_tok = kv->stride_tok; p.v_stride_head = kv->stride_head;
  p.mean = static_cast<__nv_bfloat16 *>(const_cast<void *>(kv->v_block_mean));
  p.m_stride_seq = kv->mean_stride_seq; p.m_stride_block = kv->mean_stride_block; p.m_stride_head = kv->mean_stride_head;
  p.seqlens = kv->seqlens; p.page_table = kv->page_table;
  p.max_seqlen = kv->max_seqlen;
  p.page_shift = kv->page_table ? ilog2(kv->page_size) : 0;
  p.max_pages = kv->max_pages_per_seq; p.num_pages = kv->num_pages > 0 ? kv->num_pages : 1;
  p.Hkv = num_kv_heads;
  const dim3 grid(num_kv_heads, kv->num_seqs), block(32, kRunMeanWarps);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (head_dim == 128) fold_running_mean_kernel<128><<<grid, block, 0, st>>>(p);
  else fold_running_mean_kernel<64><<<grid, block, 0, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

int fold_quantize_keys(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, const int32_t *first_token,
                       fold_stream stream) {
  if (!kv || num_kv_heads < 1) return FOLD_EINVAL;
  if (head_dim != 64 && head_dim != 128) return FOLD_EUNSUPPORTED;
  if (!kv->k || !kv->k_plane_a) return FOLD_EINVAL;
  if (int rc = check_kv(*kv, head_dim, num_kv_heads)) return rc;
  if (kv->max_seqlen == 0) return FOLD_OK;
  QuantParams p;
  memset(&p, 0, sizeof(p));
  p.k = static_cast<const __nv_bfloat16 *>(kv->k);
  p.k_stride_seq = kv->stride_seq; p.k_stride_tok = kv->stride_tok; p.k_stride_head = kv->stride_head;
  p.kv = plane_view(*kv);
  p.first_token = first_token;
  const dim3 grid((kv->max_seqlen + kQuantRowsPerCta - 1) / kQuantRowsPerCta, num_kv_heads, kv->num_seqs);
  const dim3 block(32, kQuantWarps);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (head_dim == 128) fold_quantize_keys_kernel<128><<<grid, block, 0, st>>>(p);
  else fold_quantize_keys_kernel<64><<<grid, block, 0, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

int fold_quantize_values(const fold_kv *kv, int32_t num_kv_heads, int32_t head_dim, const int32_t *first_token,
                         fold_stream stream) {
  if (!kv || num_kv_heads < 1) return FOLD_EINVAL;
  if (head_dim != 64 && head_dim != 128) return FOLD_EUNSUPPORTED;
  if (!kv->v || !kv->v_plane_1) return FOLD_EINVAL;
  if (int rc = check_kv(*kv, head_dim, num_kv_heads)) return rc;
  if (kv->max_seqlen == 0) return FOLD_OK;
  QuantValueParams p;
  memset(&p, 0, sizeof(p));
  p.v = static_cast<const __nv_bfloat16 *>(kv->v);
  p.v_stride_seq = kv->stride_seq; p.v_stride_tok = kv->stride_tok; p.v_stride_head = kv->stride_head;
  p.kv = plane_view(*kv);
  p.first_token = first_token;
  p.inv_scale = ldexpf(1.f, -kv->v_scale_log2);
  const dim3 grid((kv->max_seqlen + kQuantRowsPerCta - 1) / kQuantRowsPerCta, num_kv_heads, kv->num_seqs);
  const dim3 block(32, kQuantWarps);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (head_dim == 128) fold_quantize_values_kernel<128><<<grid, block, 0, st>>>(p);
  else fold_quantize_values_kernel<64><<<grid, block, 0, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

int fold_decode(const fold_args *args, fold_stream stream) {
  Geometry g;
  if (int rc = check_args(args, &g, true)) return rc;
  if (one_launch_decode(args, g)) {
    if (!args->workspace || !aligned(args->workspace, 256)) return FOLD_EINVAL;
    if (args->workspace_bytes < g.ws_bytes) return FOLD_EWORKSPACE;
    FusedParams f;
    memset(&f, 0, sizeof(f));
    f.mode = args->z_mode == FOLD_Z_ESTIMATE ? 1 : 2;
    f.est = est_params(args, g);
    f.est.n_levels = 1;
    f.est.lv[0] = kv_level(args->kv, args->stack);
    fold_partials part;
    fill_partials(args, g, &part);
    MergeLevel &lv = f.mrg.lv[0];
    lv.slots = part.slots; lv.seqlens = part.seqlens; lv.slot_stride = part.slot_stride;
    lv.stack = part.stack; lv.max_slots = part.max_slots; lv.rows = part.rows; lv.max_seqlen = part.max_seqlen;
    f.mrg.z = args->z;
    f.mrg.out = static_cast<__nv_bfloat16 *>(args->out);
    f.mrg.lse = args->lse; f.mrg.row_status = args->row_status;
    f.mrg.n_levels = 1; f.mrg.Hq = g.Hq; f.mrg.Hkv = g.Hkv; f.mrg.G = g.G; f.mrg.D = g.D;
    return launch_scan(args, g, static_cast<cudaStream_t>(stream), &f);
  }
  fold_partials part;
  if (int rc = fold_decode_split(args, &part, stream)) return rc;
  const fold_partials *lv[1] = {&part};
  return fold_cascade_merge(lv, 1, args->out, args->lse, args->row_status, stream);
}

int32_t fold_decode_launches(const fold_args *args) {
  Geometry g;
  if (check_args(args, &g, true)) return 0;
  if (one_launch_decode(args, g)) return 1;
  int n = 2;                                                 // scan, partial add
  if (g.planes || args->z_mode != FOLD_Z_GIVEN) ++n;         // reference (or the two-plane front kernel)
  if (g.planes && args->z_mode == FOLD_Z_ZERO) ++n;
  return n;
}

int fold_decode_cascade(const fold_args *const *levels, int n_levels, fold_stream stream) {
  if (!levels || n_levels < 1 || n_levels > kMaxLevels || !levels[0]) return FOLD_EINVAL;
  const fold_args *a0 = levels[0];
  if (a0->z_mode != FOLD_Z_ESTIMATE && a0->z_mode != FOLD_Z_GIVEN) return FOLD_EINVAL;
  const bool planes = a0->kv.k_plane_a != nullptr;           // two-plane keys: every level, or none
  for (int l = 0; l < n_levels; ++l)
    if (levels[l] && (levels[l]->kv.k_plane_a != nullptr) != planes) return FOLD_EUNSUPPORTED;
  fold_args lv[kMaxLevels];
  for (int l = 0; l < n_levels; ++l) {
    const fold_args *a = levels[l];
    if (!a || a->q != a0->q || a->z != a0->z || a->batch != a0->batch || a->num_q_heads != a0->num_q_heads ||
        a->num_kv_heads != a0->num_kv_heads || a->head_dim != a0->head_dim || a->depth_T != a0->depth_T ||
        a->softmax_scale != a0->softmax_scale)
      return FOLD_EINVAL;
    Geometry g;
    lv[l] = *a;
    lv[l].z_mode = FOLD_Z_GIVEN;
    if (int rc = check_args(&lv[l], &g, l == 0)) return rc;
  }
  const bool est = a0->z_mode == FOLD_Z_ESTIMATE;            // the estimate kernel then zeroes every level's header too
  if (planes) {
    // one front kernel for the whole cascade: the split query rows into every level's workspace, the headers cleared,
    // the reference over the levels' keys in order if it is to be estimated
    if (est) {
      if (int rc = estimate_levels(levels, n_levels, stream, true)) return rc;
    } else {
      Geometry gs[kMaxLevels];
      const fold_args *tp[kMaxLevels];
      for (int l = 0; l < n_levels; ++l) {
        tp[l] = &lv[l];
        if (int rc = check_args(&lv[l], &gs[l], false)) return rc;
        if (!lv[l].workspace || !aligned(lv[l].workspace, 256)) return FOLD_EINVAL;
        if (lv[l].workspace_bytes < gs[l].ws_bytes) return FOLD_EWORKSPACE;
      }
      if (int rc = launch_planes_front_levels(tp, gs, n_levels, static_cast<cudaStream_t>(stream), true)) return rc;
    }
  } else if (est) {
    if (int rc = estimate_levels(levels, n_levels, stream, true)) return rc;
  }
  const bool hdr_done = est || planes;
  fold_partials parts[kMaxLevels];
  const fold_partials *pp[kMaxLevels];
  for (int l = 0; l < n_levels; ++l) pp[l] = &parts[l];
  // Once the reference is fixed the levels are independent: with a side stream and two events from the caller the first
  // level (the shared prefix: a tensor-bound kernel on fewer CTAs than SMs) is scanned there while the others are
  // scanned on `stream`, forked and joined with the events, so the caller still sees one ordered call on `stream`.
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n_levels >= 2 && a0->side_stream && a0->side_fork_event && a0->side_join_event) {
    cudaStream_t side = static_cast<cudaStream_t>(a0->side_stream);
    cudaEvent_t fork = static_cast<cudaEvent_t>(a0->side_fork_event), join = static_cast<cudaEvent_t>(a0->side_join_event);
    if (side == st) return FOLD_EINVAL;
    if (cudaEventRecord(fork, st) != cudaSuccess || cudaStreamWaitEvent(side, fork, 0) != cudaSuccess) return FOLD_ECUDA;
    int rc = decode_split_impl(&lv[0], &parts[0], a0->side_stream, hdr_done, planes);
    const bool recorded = cudaEventRecord(join, side) == cudaSuccess;
    for (int l = 1; l < n_levels && rc == FOLD_OK; ++l) rc = decode_split_impl(&lv[l], &parts[l], stream, hdr_done, planes);
    // join in every case, so that the side stream never holds work the caller's stream does not wait for
    if (!recorded || cudaStreamWaitEvent(st, join, 0) != cudaSuccess) return FOLD_ECUDA;
    if (rc) return rc;
    return fold_cascade_merge(pp, n_levels, a0->out, a0->lse, a0->row_status, stream);
  }
  for (int l = 0; l < n_levels; ++l)
    if (int rc = decode_split_impl(&lv[l], &parts[l], stream, hdr_done, planes)) return rc;
  return fold_cascade_merge(pp, n_levels, a0->out, a0->lse, a0->row_status, stream);
}

// ------------------------------------------------------------------ host-buffer variant
namespace {
struct HostPlan {
  size_t q, k, v, table, lens, z, out, lse, status, ws, total;
  size_t q_bytes, kv_bytes, table_bytes, lens_bytes, rows;
  // two-plane keys (and E4M3 value planes): the planes' spans and the scales' span
  size_t pa, pb, sc, v1, v2, plane_bytes, scale_bytes;
};
size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
bool plan_host(const fold_args *a, HostPlan *h) {
  const fold_kv &kv = a->kv;
  const bool paged = kv.page_table != nullptr;
  const long long outer = paged ? kv.num_pages : kv.num_seqs;
  const long long toks = paged ? kv.page_size : kv.capacity;
  if (outer < 1 || toks < 1) return false;
  const long long span = (outer - 1) * kv.stride_seq + (toks - 1) * kv.stride_tok +
                         (long long)(a->num_kv_heads - 1) * kv.stride_head + a->head_dim;
  h->rows = (size_t)a->batch * a->num_q_heads;
  h->q_bytes = ((size_t)(a->batch - 1) * a->q_stride_b + (size_t)(a->num_q_heads - 1) * a->q_stride_h + a->head_dim) * 2;
  h->kv_bytes = (size_t)span * 2;
  h->table_bytes = paged ? (size_t)kv.num_seqs * kv.max_pages_per_seq * 4 : 0;
  h->lens_bytes = (size_t)kv.num_seqs * 4;
  h->plane_bytes = h->scale_bytes = 0;
  if (kv.k_plane_a) {                                        // one byte per code; a scale row is readable up to the next 8 tokens
    h->plane_bytes = (size_t)((outer - 1) * kv.plane_stride_seq + (toks - 1) * kv.plane_stride_tok +
                              (long long)(a->num_kv_heads - 1) * kv.plane_stride_head + a->head_dim);
    h->scale_bytes = (size_t)((outer - 1) * kv.scale_stride_seq + (long long)(a->num_kv_heads - 1) * kv.scale_stride_head +
                              ((toks + 7) & ~7LL)) * 2;
  }
  size_t o = 0;
  h->q = o; o += up256(h->q_bytes);
  h->k = o; o += kv.k ? up256(h->kv_bytes) : 0;              // (with two-plane keys the BF16 keys may be absent,
  h->v = o; o += kv.v ? up256(h->kv_bytes) : 0;              //  with E4M3 value planes the BF16 values)
  h->pa = o; o += up256(h->plane_bytes);
  h->pb = o; o += up256(h->plane_bytes);
  h->sc = o; o += up256(h->scale_bytes);
  h->v1 = o; o += kv.v_plane_1 ? up256(h->plane_bytes) : 0;
  h->v2 = o; o += kv.v_plane_1 ? up256(h->plane_bytes) : 0;
  h->table = o; o += up256(h->table_bytes);
  h->lens = o; o += up256(h->lens_bytes);
  h->z = o; o += up256(h->rows * 4);
  h->out = o; o += up256(h->rows * a->head_dim * 2);
  h->lse = o; o += up256(h->rows * 4);
  h->status = o; o += up256(h->rows * 4);
  h->ws = o; o += up256(fold_workspace_bytes(a));
  h->total = o;
  return true;
}
}  // namespace

size_t fold_host_staging_bytes(const fold_args *host_args) {
  HostPlan h;
  if (!host_args || fold_workspace_bytes(host_args) == 0 || !plan_host(host_args, &h)) return 0;
  return h.total;
}

int fold_decode_host(const fold_args *ha, void *staging, size_t staging_bytes, fold_stream stream) {
  if (!ha || !staging || !aligned(staging, 256)) return FOLD_EINVAL;
  const bool planes = ha->kv.k_plane_a != nullptr, vplanes = ha->kv.v_plane_1 != nullptr;
  if (!ha->q || !ha->kv.seqlens || !ha->out) return FOLD_EINVAL;
  if ((!ha->kv.k && !planes) || (!ha->kv.v && !vplanes)) return FOLD_EINVAL;
  if (planes && (!ha->kv.k_plane_b || !ha->kv.k_scale)) return FOLD_EINVAL;
  if (vplanes && (!planes || !ha->kv.v_plane_2)) return planes ? FOLD_EINVAL : FOLD_EUNSUPPORTED;
  if (ha->z_mode == FOLD_Z_GIVEN && !ha->z) return FOLD_EINVAL;
  if (ha->kv.v_block_mean) return FOLD_EUNSUPPORTED;        // the block tail is not offered for host buffers
  if (ha->draft_len != 0) return FOLD_EUNSUPPORTED;         // nor are draft masks
  HostPlan h;
  if (fold_workspace_bytes(ha) == 0 || !plan_host(ha, &h)) return FOLD_EINVAL;
  if (staging_bytes < h.total) return FOLD_EWORKSPACE;
  uint8_t *d = static_cast<uint8_t *>(staging);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  fold_args da = *ha;
  da.q = d + h.q;
  da.kv.k = ha->kv.k ? d + h.k : nullptr;
  da.kv.v = ha->kv.v ? d + h.v : nullptr;
  if (planes) {
    da.kv.k_plane_a = reinterpret_cast<const int8_t *>(d + h.pa);
    da.kv.k_plane_b = reinterpret_cast<const int8_t *>(d + h.pb);
    da.kv.k_scale = d + h.sc;
  }
  if (vplanes) { da.kv.v_plane_1 = d + h.v1; da.kv.v_plane_2 = d + h.v2; }
  da.kv.page_table = ha->kv.page_table ? reinterpret_cast<const int32_t *>(d + h.table) : nullptr;
  da.kv.seqlens = reinterpret_cast<const int32_t *>(d + h.lens);
  da.z = reinterpret_cast<float *>(d + h.z);
  da.out = d + h.out;
  da.lse = reinterpret_cast<float *>(d + h.lse);
  da.row_status = reinterpret_cast<int32_t *>(d + h.status);
  da.workspace = d + h.ws;
  da.workspace_bytes = fold_workspace_bytes(ha);
  Geometry g;
  if (int rc = check_args(&da, &g, true)) return rc;
  bool ok = true;
  ok &= cudaMemcpyAsync(d + h.q, ha->q, h.q_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (ha->kv.k) ok &= cudaMemcpyAsync(d + h.k, ha->kv.k, h.kv_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (ha->kv.v) ok &= cudaMemcpyAsync(d + h.v, ha->kv.v, h.kv_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (planes) {
    ok &= cudaMemcpyAsync(d + h.pa, ha->kv.k_plane_a, h.plane_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + h.pb, ha->kv.k_plane_b, h.plane_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + h.sc, ha->kv.k_scale, h.scale_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  }
  if (vplanes) {
    ok &= cudaMemcpyAsync(d + h.v1, ha->kv.v_plane_1, h.plane_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok &= cudaMemcpyAsync(d + h.v2, ha->kv.v_plane_2, h.plane_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  }
  if (h.table_bytes)
    ok &= cudaMemcpyAsync(d + h.table, ha->kv.page_table, h.table_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok &= cudaMemcpyAsync(d + h.lens, ha->kv.seqlens, h.lens_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (ha->z_mode == FOLD_Z_GIVEN)
    ok &= cudaMemcpyAsync(d + h.z, ha->z, h.rows * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) return FOLD_ECUDA;
  if (int rc = fold_decode(&da, stream)) return rc;
  ok &= cudaMemcpyAsync(ha->out, d + h.out, h.rows * ha->head_dim * 2, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (ha->lse) ok &= cudaMemcpyAsync(ha->lse, d + h.lse, h.rows * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (ha->row_status)
    ok &= cudaMemcpyAsync(ha->row_status, d + h.status, h.rows * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (ha->z && ha->z_mode != FOLD_Z_GIVEN)
    ok &= cudaMemcpyAsync(ha->z, d + h.z, h.rows * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  return ok ? FOLD_OK : FOLD_ECUDA;
}

// ------------------------------------------------------------------ decode without a caller workspace
// Scratch for callers that may not allocate: the header and (A, L) slots of one decode call live in
// this array, which every device that loads the library holds until exit.  In host code the name
// below is only a handle for cudaGetSymbolAddress, never a device address: kernels are given the
// address that call returns (looked up once per device, with that device current).
static __device__ __align__(256) unsigned char g_fold_static_scratch[FOLD_STATIC_SCRATCH_BYTES];

namespace {
std::atomic<void *> g_static_scratch_addr[64];   // device address of the array, per device ordinal (first call: looked up, stored)

int static_scratch_address(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FOLD_ECUDA;
  if (dev < 0 || dev >= 64) return FOLD_EUNSUPPORTED;
  void *addr = g_static_scratch_addr[dev].load(std::memory_order_acquire);
  if (!addr) {                                 // first call on this device: resolve the symbol here (threads racing on
    //                                            it look up the same address and store the same value)
    if (cudaGetSymbolAddress(&addr, g_fold_static_scratch) != cudaSuccess || !addr) return FOLD_ECUDA;
    g_static_scratch_addr[dev].store(addr, std::memory_order_release);
  }
  *out = addr;
  return FOLD_OK;
}
}  // namespace

int fold_decode_static(const fold_args *args, fold_stream stream) {
  if (!args) return FOLD_EINVAL;
  const size_t need = fold_workspace_bytes(args);
  if (need == 0) return FOLD_EINVAL;
  if (need > (size_t)FOLD_STATIC_SCRATCH_BYTES) return FOLD_ETOOLARGE;
  void *scratch = nullptr;
  if (int rc = static_scratch_address(&scratch)) return rc;
  fold_args a = *args;
  a.workspace = scratch;                       // the header is re-zeroed by the scan's own memset; slots are
  a.workspace_bytes = FOLD_STATIC_SCRATCH_BYTES;   // written before they are read, so nothing else needs clearing
  return fold_decode(&a, stream);
}

int fold_probe_read(const void *buffer, size_t bytes, uint64_t *sink, fold_stream stream) {
  if (!buffer || !aligned(buffer, 16) || bytes < 16) return FOLD_EINVAL;
  const int ctas = 4 * sm_count();
  fold_probe_read_kernel<<<ctas, kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4 *>(buffer), bytes / 16, reinterpret_cast<unsigned long long *>(sink));
  return cudaGetLastError() == cudaSuccess ? FOLD_OK : FOLD_ECUDA;
}

const char *fold_status_string(int status) {
  switch (status) {
    case FOLD_OK: return "ok";
    case FOLD_EINVAL: return "invalid argument";
    case FOLD_EUNSUPPORTED: return "unsupported shape or layout";
    case FOLD_EWORKSPACE: return "workspace too small";
    case FOLD_ECUDA: return "CUDA call failed";
    case FOLD_ETOOLARGE: return "call needs more scratch than the library's built-in array holds";
    default: return "unknown status";
  }
}

int fold_version(void) { return 102; }   // 101: flags, side stream, fold_probe_read; 102: fold_decode_launches, live_hint


}  // extern "C"
