// Host side of the C ABI declared in include/osdp.h: argument checks, the slice table, the
// workspace plan, TMA descriptor encoding and kernel launches.  No allocation, no stream
// synchronisation (except osdp_read_device_status), no CPU fallback: if the CUDA path cannot
// run, the call returns an error.
#include "../../include/osdp.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <string.h>

#include <atomic>
#include <cmath>
#include <mutex>

#include "osdp_aux.cuh"
#include "osdp_gemm.cuh"

using namespace osdp;

namespace {

thread_local int g_last_cuda_error = 0;

// One lock for the rare first-use set-up paths (driver entry point, per-device attributes); the hot
// path only reads an atomic flag.
std::mutex g_setup_mutex;

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return OSDP_ERR_CUDA;
}
int cu_fail(CUresult r) {
  g_last_cuda_error = 100000 + (int)r;   // driver-API codes are reported offset by 100000
  return OSDP_ERR_CUDA;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

int get_encode_fn(EncodeTiledFn *out) {
  static std::atomic<EncodeTiledFn> fn{nullptr};
  EncodeTiledFn f = fn.load(std::memory_order_acquire);
  if (!f) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess) return cuda_fail(e);
    if (q != cudaDriverEntryPointSuccess || !p) return cuda_fail(cudaErrorNotSupported);
    f = (EncodeTiledFn)p;
    fn.store(f, std::memory_order_release);
  }
  *out = f;
  return OSDP_OK;
}

std::atomic<int> g_dev_sms[64];

int device_sms(int *sms) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return cuda_fail(cudaErrorInvalidDevice);
  int n = g_dev_sms[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    g_dev_sms[dev].store(n, std::memory_order_relaxed);
  }
  *sms = n;
  return OSDP_OK;
}

// Two internal streams and three events per device, created at the first call that wants them: small
// independent launches of one call (the weight-gradient GEMMs of an MLP slice next to its dX GEMM) are
// forked onto them from the caller's stream and joined back into it, so that they fill the SMs together.
// The fork / join is plain event record + wait, which a stream capture follows into the side streams.
struct SideStreams {
  cudaStream_t s[2];
  cudaEvent_t fork, join[2];
  cudaEvent_t ring[3][2];   // "this stream (0: the caller's, 1, 2: internal) is done with slice s", by the parity of s
};
SideStreams g_side[64];
std::atomic<bool> g_side_ready[64];
std::mutex g_side_mutex;   // one call at a time enqueues a fork / join section (the events are shared)

int side_streams(SideStreams **out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return cuda_fail(cudaErrorInvalidDevice);
  if (!g_side_ready[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_side_ready[dev].load(std::memory_order_relaxed)) {
      SideStreams &S = g_side[dev];
      for (int i = 0; i < 2; ++i) {
        e = cudaStreamCreateWithFlags(&S.s[i], cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(e);
        e = cudaEventCreateWithFlags(&S.join[i], cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail(e);
      }
      for (int i = 0; i < 6; ++i) {
        e = cudaEventCreateWithFlags(&S.ring[i / 2][i % 2], cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail(e);
      }
      e = cudaEventCreateWithFlags(&S.fork, cudaEventDisableTiming);
      if (e != cudaSuccess) return cuda_fail(e);
      g_side_ready[dev].store(true, std::memory_order_release);
    }
  }
  *out = &g_side[dev];
  return OSDP_OK;
}

// One fork / join section: launches that may run next to the caller's stream go to the internal streams
// between begin() and end().  end() always runs (the destructor calls it on an early return), so the caller's
// stream is joined with whatever was queued on the internal streams even when a launch in between failed.
// If the internal streams are in use by a stream capture other than the caller's own (a capture that pulled
// them in and has not ended yet), the section does not fork: everything goes to the caller's stream.
struct ForkJoin {
  SideStreams *side = nullptr;
  std::unique_lock<std::mutex> lock;
  cudaStream_t main = nullptr;
  int n = 0;
  bool open = false;

  static bool foreign_capture(cudaStream_t caller, cudaStream_t internal) {
    cudaStreamCaptureStatus si = cudaStreamCaptureStatusNone, sc = cudaStreamCaptureStatusNone;
    unsigned long long idi = 0, idc = 0;
    if (cudaStreamGetCaptureInfo(internal, &si, &idi) != cudaSuccess) { cudaGetLastError(); return true; }
    if (si == cudaStreamCaptureStatusNone) return false;
    if (cudaStreamGetCaptureInfo(caller, &sc, &idc) != cudaSuccess) { cudaGetLastError(); return true; }
    return !(sc == cudaStreamCaptureStatusActive && si == cudaStreamCaptureStatusActive && idc == idi);
  }
  // acquire the internal streams (first use creates them); no GPU work is queued yet
  int acquire(cudaStream_t caller, int n_streams) {
    int rc = side_streams(&side);
    if (rc) return rc;
    lock = std::unique_lock<std::mutex>(g_side_mutex);
    main = caller;
    n = n_streams;
    for (int i = 0; i < n; ++i)
      if (foreign_capture(caller, side->s[i])) { n = 0; break; }
    return OSDP_OK;
  }
  int begin() {
    if (!side || n == 0) return OSDP_OK;
    cudaError_t e = cudaEventRecord(side->fork, main);
    for (int i = 0; i < n && e == cudaSuccess; ++i) e = cudaStreamWaitEvent(side->s[i], side->fork, 0);
    if (e != cudaSuccess) return cuda_fail(e);
    open = true;
    return OSDP_OK;
  }
  cudaStream_t stream(int i) const { return (open && i < n) ? side->s[i] : main; }
  // Edges inside a section whose work is pipelined over slices: mark(q, b) records "stream q (0: the caller's,
  // 1, 2: internal) has got this far" under parity b; after(q, b, t) makes stream t wait for the latest such mark.
  // Without a fork everything is on the caller's stream and both do nothing: program order holds.
  cudaStream_t lane(int q) const { return q == 0 ? main : stream(q - 1); }
  int mark(int q, int b) {
    if (!open) return OSDP_OK;
    cudaError_t e = cudaEventRecord(side->ring[q][b], lane(q));
    return e == cudaSuccess ? OSDP_OK : cuda_fail(e);
  }
  int after(int q, int b, int t) {
    if (!open || lane(q) == lane(t)) return OSDP_OK;
    cudaError_t e = cudaStreamWaitEvent(lane(t), side->ring[q][b], 0);
    return e == cudaSuccess ? OSDP_OK : cuda_fail(e);
  }
  int end() {
    if (!open) return OSDP_OK;
    open = false;
    cudaError_t first = cudaSuccess;
    for (int i = 0; i < n; ++i) {
      cudaError_t e = cudaEventRecord(side->join[i], side->s[i]);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(main, side->join[i], 0);
      if (e != cudaSuccess && first == cudaSuccess) first = e;
    }
    return first == cudaSuccess ? OSDP_OK : cuda_fail(first);
  }
  ~ForkJoin() { end(); }
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ------------------------------------------------------------------------------------------------
// Slice table (Section 3.3, step 1)

int slice_len(int64_t D, int k, int64_t *L) {
  if (k < 0 || k > OSDP_MAX_SPLIT) return OSDP_ERR_BAD_SPLIT;
  if (k == 0) k = 1;
  if (D <= 0) return OSDP_ERR_BAD_SHAPE;
  int64_t l = (D + k - 1) / k;
  l = (l + 7) / 8 * 8;
  if ((int64_t)(k - 1) * l >= D) return OSDP_ERR_BAD_SPLIT;
  *L = l;
  return OSDP_OK;
}

// ------------------------------------------------------------------------------------------------
// Workspace plan.  Region 0 is always the 256-byte status block.

struct WsPlan {
  size_t carry_off, carry_bytes;      // fp32 running sum of the summed output
  size_t stage0_off, stage0_bytes;    // bf16 slice staging (G_s, A_s)
  size_t stage1_off, stage1_bytes;    // second bf16 slice staging (dZ_s)
  size_t stage2_off, stage2_bytes;    // third bf16 slice staging (recomputed Z1_s)
  size_t part_off, part_bytes;        // column-sum partials
  size_t stage_stride;                // distance between the two sets of slice staging buffers (0: one set)
  size_t total;
};

// The backward of an MLP block whose slices are small (each GEMM of a slice at most one wave of 256 x 256 tiles on
// 74 CTA pairs) is bound by the latency of its chain of small kernels.  An all-slices call then keeps two sets of
// slice staging buffers, so that a slice's weight-gradient GEMMs run beside the next slice's first GEMM.
inline bool mlp_bwd_pipelined(int64_t M, int64_t L, int k) { return k > 2 && cdiv(M, 256) * cdiv(L, 256) <= 74; }

// fp32 running sum of a P x Q output, kept as boxes of 32 x 32 (both extents padded to whole boxes)
inline size_t carry_bytes(int64_t P, int64_t Q) { return (size_t)(cdiv(P, 32) * 32) * (size_t)(cdiv(Q, 32) * 32) * 4; }

int plan_workspace(int64_t M, int64_t N, int64_t K, int k, int split_dim, int act, int op, int flags, WsPlan *w) {
  const bool fp32_carry = !(flags & OSDP_FLAG_CARRY_BF16);
  // The linear ops carry a running sum through memory only when the operator is swept once per slice: the
  // *_slice entry points and all-slices calls in slice-major order (both ask with OSDP_FLAG_SLICE_MAJOR), paired
  // slices, and the backward with an activation (its G_s is staged slice by slice).  Otherwise an all-slices
  // call keeps every tile's sum in tensor memory across the slices.
  const bool swept = (flags & (OSDP_FLAG_SLICE_MAJOR | OSDP_FLAG_PAIR_SLICES)) != 0;
  memset(w, 0, sizeof(*w));
  if (M <= 0 || N <= 0 || K <= 0) return OSDP_ERR_BAD_SHAPE;
  if (k == 0) k = 1;
  size_t off = 256;
  auto take = [&](size_t bytes, size_t *o, size_t *b) {
    *o = off;
    *b = bytes;
    off = align_up(off + bytes, 256);
  };
  const size_t chunks = (size_t)((M + COLSUM_ROWS_PER_CHUNK - 1) / COLSUM_ROWS_PER_CHUNK);
  int64_t L = 0;
  int rc;
  switch (op) {
    case OSDP_OP_LINEAR_FWD:
      if (split_dim != OSDP_SPLIT_OUT && split_dim != OSDP_SPLIT_RED) return OSDP_ERR_BAD_SPLIT;
      rc = slice_len(split_dim == OSDP_SPLIT_OUT ? N : K, k, &L);
      if (rc) return rc;
      if (split_dim == OSDP_SPLIT_RED && k > 1 && fp32_carry && swept)
        take(carry_bytes(M, N), &w->carry_off, &w->carry_bytes);
      break;
    case OSDP_OP_LINEAR_BWD:
      if (split_dim != OSDP_SPLIT_OUT && split_dim != OSDP_SPLIT_RED) return OSDP_ERR_BAD_SPLIT;
      rc = slice_len(split_dim == OSDP_SPLIT_OUT ? N : K, k, &L);
      if (rc) return rc;
      if (split_dim == OSDP_SPLIT_OUT && k > 1 && fp32_carry && (swept || act != OSDP_ACT_NONE))
        take(carry_bytes(M, K), &w->carry_off, &w->carry_bytes);
      if (act != OSDP_ACT_NONE)
        take((size_t)M * (split_dim == OSDP_SPLIT_OUT ? L : N) * 2, &w->stage0_off, &w->stage0_bytes);
      take(chunks * (size_t)N * 4, &w->part_off, &w->part_bytes);
      break;
    case OSDP_OP_MLP_FWD:   // N = ffn, K = hidden
      rc = slice_len(N, k, &L);
      if (rc) return rc;
      if (k > 1 && fp32_carry) take(carry_bytes(M, K), &w->carry_off, &w->carry_bytes);
      take((size_t)M * L * 2, &w->stage0_off, &w->stage0_bytes);
      break;
    case OSDP_OP_MLP_BWD:
      rc = slice_len(N, k, &L);
      if (rc) return rc;
      if (k > 1 && fp32_carry) take(carry_bytes(M, K), &w->carry_off, &w->carry_bytes);
      w->stage_stride = mlp_bwd_pipelined(M, L, k) ? align_up((size_t)M * L * 2, 256) : 0;
      take(w->stage_stride + (size_t)M * L * 2, &w->stage0_off, &w->stage0_bytes);
      take(w->stage_stride + (size_t)M * L * 2, &w->stage1_off, &w->stage1_bytes);
      if (flags & OSDP_FLAG_RECOMPUTE) take(w->stage_stride + (size_t)M * L * 2, &w->stage2_off, &w->stage2_bytes);
      // db1's slice (one set of partial sums per set of staging buffers) and db2 side by side
      take(chunks * (size_t)((w->stage_stride ? 2 : 1) * L + K) * 4, &w->part_off, &w->part_bytes);
      break;
    default:
      return OSDP_ERR_UNSUPPORTED;
  }
  w->total = off;
  return OSDP_OK;
}

// ------------------------------------------------------------------------------------------------
// GEMM launch

// A row-major bf16 matrix view used as a GEMM operand.  `inner` is the contiguous extent.
// K-major: inner is the reduction dimension; MN-major: inner is the output dimension.
struct Operand {
  const void *base;
  int64_t inner, outer, ld;
  bool mn_major;
  bool whole;   // true: the view is the whole operator and the launch's slices cut it;
                // false: the view is already one slice (or is not cut at all)
};

struct GemmCall {
  Operand a, b;
  int64_t P, Q, R;
  int mode;
  int64_t L;
  int k_total, s_begin, s_end;
  int64_t bn_P, bn_Q;   // extents that choose the tile width (the unsplit operator's, so k never changes it)
  Epilogue epi;
  int carry_bf16;   // MODE_RED: running sum in `out` (bf16) instead of the fp32 carry buffer
  int pair_slices;  // MODE_RED: accumulate two adjacent slices per pass
  int slice_major;  // MODE_RED, all slices in the launch: sweep slice by slice with the carry (else: slices inside a tile)
  int out_is_slice; // MODE_ROWS / MODE_COLS: `epi.out` is the slice's own compact matrix, not the whole output
  int fp8;          // operands are fp8 e4m3 (1 byte per element) instead of bf16
  int compact;      // the launch runs next to another GEMM of the call: CTA pairs on 256-wide tiles even when few
  int n_peers;      // > 0: the output slice is reduce-added row block by row block into peer_out[0..n_peers)
  void *peer_out[8];
  int *status;
};

int encode3d(CUtensorMap *m, CUtensorMapDataType dt, const void *base, const cuuint64_t dims[3],
             const cuuint64_t strides_bytes[2], const cuuint32_t box[3], bool swizzle = true) {
  EncodeTiledFn fn;
  int rc = get_encode_fn(&fn);
  if (rc) return rc;
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, dt, 3, const_cast<void *>(base), dims, strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cu_fail(r);
  return OSDP_OK;
}

// A row-major matrix view [outer][inner] (leading dimension ld, elements of elem_bytes) as the
// two 3-D maps the kernel uses.  The slice index is a tensor coordinate: for slices 0..k-2 the map
// has a dimension of extent k-1 and stride L (in the cut dimension's units); the last slice, which
// may be shorter, gets a map of its own so that out-of-range elements are zero-filled on loads and
// dropped on stores instead of running into the neighbouring slice.
//   mid : the slice coordinate is dimension 1 (the slices cut the contiguous dimension), else 2
//   cut : the view is the whole matrix and is cut into k slices of length L; otherwise both maps
//         describe the view as it is (slice extent 1)
struct ViewSpec {
  const void *base;
  int elem_bytes;
  CUtensorMapDataType dt;
  int64_t inner, outer, ld;
  bool mid, cut;
  int64_t L;
  int k;
  cuuint32_t box_inner, box_outer;
};

int make_sliced_maps(const ViewSpec &v, CUtensorMap *main_map, CUtensorMap *tail_map) {
  const char *base = static_cast<const char *>(v.base);
  const cuuint64_t es = (cuuint64_t)v.elem_bytes;
  const cuuint64_t ldb = (cuuint64_t)v.ld * es;
  int rc;
  if (!v.cut) {
    if (v.mid) {
      const cuuint64_t dims[3] = {(cuuint64_t)v.inner, 1, (cuuint64_t)v.outer};
      const cuuint64_t str[2] = {(cuuint64_t)v.inner * es, ldb};
      const cuuint32_t box[3] = {v.box_inner, 1, v.box_outer};
      rc = encode3d(tail_map, v.dt, base, dims, str, box);
    } else {
      const cuuint64_t dims[3] = {(cuuint64_t)v.inner, (cuuint64_t)v.outer, 1};
      const cuuint64_t str[2] = {ldb, ldb * (cuuint64_t)v.outer};
      const cuuint32_t box[3] = {v.box_inner, v.box_outer, 1};
      rc = encode3d(tail_map, v.dt, base, dims, str, box);
    }
    if (rc) return rc;
    *main_map = *tail_map;
    return OSDP_OK;
  }
  const int64_t k1 = v.k - 1;
  if (v.mid) {   // the slices cut the contiguous dimension
    const cuuint64_t str[2] = {(cuuint64_t)v.L * es, ldb};
    const cuuint32_t box[3] = {v.box_inner, 1, v.box_outer};
    const cuuint64_t dims_main[3] = {(cuuint64_t)v.L, (cuuint64_t)k1, (cuuint64_t)v.outer};
    rc = encode3d(main_map, v.dt, base, dims_main, str, box);
    if (rc) return rc;
    const cuuint64_t dims_tail[3] = {(cuuint64_t)(v.inner - k1 * v.L), 1, (cuuint64_t)v.outer};
    return encode3d(tail_map, v.dt, base + k1 * v.L * (int64_t)es, dims_tail, str, box);
  }
  // the slices cut the strided dimension
  const cuuint64_t str[2] = {ldb, ldb * (cuuint64_t)v.L};
  const cuuint32_t box[3] = {v.box_inner, v.box_outer, 1};
  const cuuint64_t dims_main[3] = {(cuuint64_t)v.inner, (cuuint64_t)v.L, (cuuint64_t)k1};
  rc = encode3d(main_map, v.dt, base, dims_main, str, box);
  if (rc) return rc;
  const cuuint64_t dims_tail[3] = {(cuuint64_t)v.inner, (cuuint64_t)(v.outer - k1 * v.L), 1};
  return encode3d(tail_map, v.dt, base + k1 * v.L * (int64_t)ldb, dims_tail, str, box);
}

int make_operand_maps(const Operand &op, bool is_a, int mode, int64_t L, int k, int tile_rows, CUtensorMap *main_map,
                      CUtensorMap *tail_map, int *sc_mul, int eb = 2) {
  ViewSpec v;
  v.base = op.base; v.elem_bytes = eb;
  v.dt = (eb == 1) ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  v.inner = op.inner; v.outer = op.outer; v.ld = op.ld;
  v.mid = op.mn_major ? (mode == (is_a ? MODE_ROWS : MODE_COLS)) : (mode == MODE_RED);
  const bool role_sliced = is_a ? (mode == MODE_ROWS || mode == MODE_RED) : (mode == MODE_COLS || mode == MODE_RED);
  v.cut = role_sliced && op.whole && k > 1;
  v.L = L; v.k = k;
  v.box_inner = (cuuint32_t)(128 / eb);                                   // 128 bytes of the contiguous dimension
  v.box_outer = op.mn_major ? (cuuint32_t)(128 / eb) : (cuuint32_t)tile_rows;   // MN-major: one k-block of rows
  *sc_mul = v.cut ? 1 : 0;
  return make_sliced_maps(v, main_map, tail_map);
}

// Output-side maps: boxes of 32 rows x 128 bytes written by one epilogue warp.
int make_output_maps(void *base, bool fp32, int64_t P, int64_t Q, int64_t ld, int mode, int64_t L, int k,
                     CUtensorMap *main_map, CUtensorMap *tail_map, int *sc_mul, bool whole = true) {
  ViewSpec v;
  v.base = base; v.elem_bytes = fp32 ? 4 : 2;
  v.dt = fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
  v.inner = Q; v.outer = P; v.ld = ld;   // whole == false: P x Q are the slice's own extents
  v.mid = (mode == MODE_COLS);
  v.cut = (mode == MODE_COLS || mode == MODE_ROWS) && k > 1 && whole;
  v.L = L; v.k = k;
  v.box_inner = fp32 ? 32 : 64;
  v.box_outer = 32;
  if (sc_mul) *sc_mul = v.cut ? 1 : 0;
  return make_sliced_maps(v, main_map, tail_map);
}

// One kernel variant: sets its attributes once per device, sizes the grid and launches.
// `units` = work items of the launch (tiles, summed over slices for concatenated outputs).
template <int BN, bool A_MN, bool B_MN, bool CTA2, bool HEAVY = false, int EB = 2>
int launch_variant(const GemmParams &p, int64_t units, int sms, cudaStream_t stream) {
  static std::atomic<bool> attr_done[64];
  static std::atomic<int> max_clusters[64];
  using SL = SmemLayout<BN, CTA2, HEAVY>;
  auto kernel = gemm_kernel<BN, A_MN, B_MN, CTA2, HEAVY, EB>;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  dev &= 63;
  if (!attr_done[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::TOTAL);
    if (e != cudaSuccess) return cuda_fail(e);
    if (CTA2) {
      cudaLaunchConfig_t q = {};
      q.gridDim = dim3(2 * sms, 1, 1);
      q.blockDim = dim3(SL::THREADS, 1, 1);
      q.dynamicSmemBytes = SL::TOTAL;
      cudaLaunchAttribute qa[1];
      qa[0].id = cudaLaunchAttributeClusterDimension;
      qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
      q.attrs = qa; q.numAttrs = 1;
      int n = 0;
      e = cudaOccupancyMaxActiveClusters(&n, kernel, &q);
      if (e != cudaSuccess) return cuda_fail(e);
      if (n < 1) return cuda_fail(cudaErrorLaunchOutOfResources);
      max_clusters[dev].store(n, std::memory_order_relaxed);
    }
    attr_done[dev].store(true, std::memory_order_release);
  }
  const int64_t cap = CTA2 ? max_clusters[dev].load(std::memory_order_relaxed) : sms;
  const int n_units = (int)(units < cap ? units : cap);
  if (n_units <= 0) return OSDP_OK;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(CTA2 ? 2 * n_units : n_units, 1, 1);
  cfg.blockDim = dim3(SL::THREADS, 1, 1);
  cfg.dynamicSmemBytes = SL::TOTAL;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTA2 ? 2 : 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  // the kernel's prologue may overlap the tail of the previous kernel on the stream (it waits with
  // griddepcontrol.wait before touching global memory)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  e = cudaLaunchKernelEx(&cfg, kernel, p);
  if (e != cudaSuccess) return cuda_fail(e);
  return OSDP_OK;
}

template <int BN, bool CTA2>
int launch_bn(const GemmParams &p, bool a_mn, bool b_mn, bool heavy, int64_t units, int sms, cudaStream_t stream) {
  if (p.bk == 128) {   // fp8 operands: tiles from 128 columns up (an MN-major chunk is 128 wide)
    if constexpr (BN >= 128) {
      if (!a_mn && !b_mn) return launch_variant<BN, false, false, CTA2, false, 1>(p, units, sms, stream);
      if (!a_mn && b_mn) return launch_variant<BN, false, true, CTA2, false, 1>(p, units, sms, stream);
      if (a_mn && b_mn) return launch_variant<BN, true, true, CTA2, false, 1>(p, units, sms, stream);
    }
    return OSDP_ERR_UNSUPPORTED;
  }
  if constexpr (BN == 128 || BN == 256) {
    // eight epilogue warps for epilogues with a transcendental per element (forward with activation,
    // activation backward): only the operand layouts those launches use
    if (heavy && !a_mn && !b_mn) return launch_variant<BN, false, false, CTA2, true>(p, units, sms, stream);
    if (heavy && !a_mn && b_mn) return launch_variant<BN, false, true, CTA2, true>(p, units, sms, stream);
  }
  if (!a_mn && !b_mn) return launch_variant<BN, false, false, CTA2>(p, units, sms, stream);
  if (!a_mn && b_mn) return launch_variant<BN, false, true, CTA2>(p, units, sms, stream);
  if (a_mn && b_mn) return launch_variant<BN, true, true, CTA2>(p, units, sms, stream);
  return OSDP_ERR_UNSUPPORTED;
}

// Work items (tiles, summed over the launch's slices for concatenated outputs) for a tile shape.
int64_t count_items(const GemmCall &c, int tm, int bn) {
  if (c.mode == MODE_RED) return cdiv(c.P, tm) * cdiv(c.Q, bn);
  const int64_t rows_full = (c.mode == MODE_ROWS) ? c.L : c.P;
  const int64_t cols_full = (c.mode == MODE_COLS) ? c.L : c.Q;
  const int nsl = c.s_end - c.s_begin;
  const int last = c.s_end - 1;
  const int64_t rows_last = (c.mode == MODE_ROWS) ? ((c.P - last * c.L) < c.L ? (c.P - last * c.L) : c.L) : c.P;
  const int64_t cols_last = (c.mode == MODE_COLS) ? ((c.Q - last * c.L) < c.L ? (c.Q - last * c.L) : c.L) : c.Q;
  return (int64_t)(nsl - 1) * cdiv(rows_full, tm) * cdiv(cols_full, bn) + cdiv(rows_last, tm) * cdiv(cols_last, bn);
}

// ---- prepared launches, remembered per host thread
struct PreparedKey {
  uint64_t w[64];
  uint64_t hash;
};
struct Prepared {
  bool valid = false;
  PreparedKey key;
  GemmParams p;
  bool pair, heavy;
  int bn;
  int64_t items;
};
constexpr int PREPARED_SLOTS = 128;
thread_local Prepared g_prepared[PREPARED_SLOTS];

// Every field of the call, one by one (struct padding never enters the key), plus the current device.
void make_key(const GemmCall &c, PreparedKey *k) {
  memset(k, 0, sizeof(*k));
  int n = 0;
  auto put = [&](uint64_t v) { k->w[n++] = v; };
  auto putp = [&](const void *ptr) { put((uint64_t)reinterpret_cast<uintptr_t>(ptr)); };
  auto putf = [&](float f) { uint32_t u; memcpy(&u, &f, 4); put(u); };
  int dev = 0;
  cudaGetDevice(&dev);
  put((uint64_t)dev);
  for (const Operand *o : {&c.a, &c.b}) {
    putp(o->base); put((uint64_t)o->inner); put((uint64_t)o->outer); put((uint64_t)o->ld);
    put((o->mn_major ? 1u : 0u) | (o->whole ? 2u : 0u));
  }
  put((uint64_t)c.P); put((uint64_t)c.Q); put((uint64_t)c.R); put((uint64_t)c.L);
  put((uint64_t)c.bn_P); put((uint64_t)c.bn_Q);
  put(((uint64_t)(uint32_t)c.mode) | ((uint64_t)(uint32_t)c.k_total << 32));
  put(((uint64_t)(uint32_t)c.s_begin) | ((uint64_t)(uint32_t)c.s_end << 32));
  const Epilogue &e = c.epi;
  putp(e.out); put((uint64_t)e.ld_out); putp(e.carry); put((uint64_t)e.ld_carry); putp(e.bias);
  putp(e.z_save); put((uint64_t)e.ld_z); putp(e.gz); put((uint64_t)e.ld_gz); putp(e.act_out); put((uint64_t)e.ld_act_out);
  put(((uint64_t)(uint32_t)e.out_fp32) | ((uint64_t)(uint32_t)e.accumulate << 8) | ((uint64_t)(uint32_t)e.act << 16) |
      ((uint64_t)(uint32_t)e.gz_act << 24));
  putf(e.scale);
  put(((uint64_t)(uint32_t)c.carry_bf16) | ((uint64_t)(uint32_t)c.pair_slices << 8) | ((uint64_t)(uint32_t)c.slice_major << 16) |
      ((uint64_t)(uint32_t)c.out_is_slice << 24) | ((uint64_t)(uint32_t)c.fp8 << 32) | ((uint64_t)(uint32_t)c.n_peers << 40) |
      ((uint64_t)(uint32_t)c.compact << 48));
  for (int q = 0; q < 8; ++q) putp(q < c.n_peers ? c.peer_out[q] : nullptr);
  putp(c.status);
  uint64_t h = 1469598103934665603ull;
  for (int i = 0; i < n; ++i) { h ^= k->w[i]; h *= 1099511628211ull; h ^= h >> 29; }
  k->hash = h;
}

int launch_prepared(const Prepared &s, bool a_mn, bool b_mn, int sms, cudaStream_t stream) {
  if (s.pair && s.bn == 512) return launch_bn<512, true>(s.p, a_mn, b_mn, false, s.items, sms, stream);
  if (s.pair) return launch_bn<256, true>(s.p, a_mn, b_mn, s.heavy, s.items, sms, stream);
  switch (s.bn) {
    case 256: return launch_bn<256, false>(s.p, a_mn, b_mn, s.heavy, s.items, sms, stream);
    case 128: return launch_bn<128, false>(s.p, a_mn, b_mn, s.heavy, s.items, sms, stream);
    default: return launch_bn<64, false>(s.p, a_mn, b_mn, s.heavy, s.items, sms, stream);
  }
}

int launch_gemm(const GemmCall &c, cudaStream_t stream) {
  int sms = 0;
  int rc = device_sms(&sms);
  if (rc) return rc;
  // Summed output with the exact carry, short slices (reduction length <= 512 per slice) and many tiles
  // per CTA pair (16 or more): one launch per slice.  The main loop of such a slice is shorter than its
  // epilogue's carry traffic, and measured on B200 a launch boundary between slices is then faster than
  // letting the CTAs drift across slices inside one launch (16384 x 8192 x 8192: k = 16 4.5 -> 3.9 ms,
  // k = 32 7.8 -> 7.1 ms; no gain at k <= 8, a loss with the bf16 running sum, and a loss of 20 % on
  // operators with only a few tiles per pair such as 8192 x 2048 x 2048).  Same arithmetic, same bits.
  // Summed output, every slice in this launch, no option that concerns the carry: a tile walks the slices'
  // k-blocks in order with its accumulator kept in tensor memory; nothing is carried through memory.
  const bool in_tmem = c.mode == MODE_RED && c.k_total > 1 && c.s_begin == 0 && c.s_end == c.k_total &&
                       !c.slice_major && !c.pair_slices && !c.carry_bf16;
  if (c.mode == MODE_RED && !in_tmem && c.s_end - c.s_begin > 1 && !c.pair_slices && !c.carry_bf16 && c.L <= 512 &&
      cdiv(c.P, 2 * BM) * cdiv(c.Q, 256) >= (int64_t)16 * (sms / 2)) {
    for (int s = c.s_begin; s < c.s_end; ++s) {
      GemmCall one = c;
      one.s_begin = s;
      one.s_end = s + 1;
      rc = launch_gemm(one, stream);
      if (rc) return rc;
    }
    return OSDP_OK;
  }
  // A training loop issues the same launches step after step: the prepared kernel parameters (about twenty
  // encoded tensor maps and the tile choice) are kept per host thread, keyed by every field of the call.
  PreparedKey key;
  make_key(c, &key);
  Prepared &slot = g_prepared[key.hash % PREPARED_SLOTS];
  if (slot.valid && memcmp(&slot.key, &key, sizeof(key)) == 0)
    return launch_prepared(slot, c.a.mn_major, c.b.mn_major, sms, stream);
  slot.valid = false;   // (re)built below; stays invalid if anything fails on the way
  slot.key = key;
  // Tile shape from the unsplit operator's extents only: the same for every k, so that concatenated
  // outputs are computed by exactly the same instruction sequence whatever the split.
  // Large operators: CTA pairs on 256 x 256 tiles.  Smaller ones: single CTAs, narrower tiles, so
  // that there are enough tiles to occupy the SMs.  The pair tile is taken from a third of the SMs' worth of
  // tiles on (49 pairs of 74): measured on B200, operators with 64 pair tiles (4096 x 1024 and 2048 x 2048
  // outputs) run 8-11 % faster on 64 CTA pairs than on 128 single CTAs, with 32 pair tiles there is no
  // difference, with 16 the narrower single-CTA tiles win.
  // A GEMM that the call runs next to another one (a weight-gradient GEMM forked beside dX) takes pair tiles from 8
  // tiles on: the same latency on a quarter of the SMs (a 1024 x 512 slice gradient over 4096 tokens: 28 us on 16
  // SMs instead of 26 us on 64), which leaves the SMs to its neighbour.  Measured on B200, backward of the MLP
  // block: 4096 tokens, hidden 1024, ffn 4096 k = 2 0.26 -> 0.21 ms, k = 4 0.41 -> 0.32 ms (k = 8 unchanged);
  // 8192 tokens, hidden 2048, ffn 8192 k = 8 1.60 -> 1.28 ms; linear layers of 1024 to 2048 outputs -1 to -7 %.
  const int64_t pair_tiles = cdiv(c.bn_P, 2 * BM) * cdiv(c.bn_Q, 256);
  const bool pair = pair_tiles >= (int64_t)sms / 3 || (c.compact && pair_tiles >= 8 && !c.fp8);
  int bn = 64;
  const int64_t want = (int64_t)sms * 4 / 5;
  if (pair || cdiv(c.bn_P, BM) * cdiv(c.bn_Q, 256) >= want) bn = 256;
  else if (cdiv(c.bn_P, BM) * cdiv(c.bn_Q, 128) >= want) bn = 128;
  const int eb = c.fp8 ? 1 : 2;
  if (c.fp8 && bn < 128) bn = 128;
  const int tm = pair ? 2 * BM : BM;
  // Widest tile, 256 x 512 per CTA pair: eight MMAs per k-block instead of four for the same barrier traffic of
  // the thread that issues them (which paces the main loop) and 25 % fewer operand bytes per flop, but the
  // accumulators fill the tensor memory, so the epilogue no longer
  // overlaps the next tile's main loop.  It pays off for long reductions and when it does not leave
  // a ragged last wave.  Measured model, per tile and CTA pair: 256-wide 6.5 ns per reduction
  // element (epilogue hidden), 512-wide 11.5 ns per element plus 5 us of exposed epilogue; time =
  // rounds of the persistent schedule x tile time.  Both tiles produce the same bits per element
  // (same k-block order), so the choice may differ between launches.  Summed outputs that carry their
  // running sum through memory keep 256 (the carry traffic needs the overlapped epilogue).
  // So does the GEMM whose epilogue reads a second tensor element-wise (direct stores, slower: better hidden).
  if (pair && (c.mode != MODE_RED || in_tmem) && c.epi.gz == nullptr) {
    const int64_t units = sms / 2;
    const double red_len = (double)c.R * (c.fp8 ? 0.5 : 1.0);   // an fp8 k-step covers twice the elements
    // (With both operands K-major the 256-wide tile is 2-6 % faster than this model says when the GPU runs at burst
    // clocks, 16384 x 8192 x 8192 forward 1414 against 1439 us, but 3-4 % slower in the power-capped state that a
    // training loop runs in, 1.739 against 1.670 ms: it moves more bytes per flop through shared memory, L2 and
    // DRAM.  The model follows the sustained state.)
    const double t_n = (double)cdiv(count_items(c, 2 * BM, 256), units) * (6.5e-3 * red_len) + 5.0;
    const double t_w = (double)cdiv(count_items(c, 2 * BM, 512), units) * (11.5e-3 * red_len + 5.0);
    if (t_w < 0.97 * t_n) bn = 512;
  }

  GemmParams &p = slot.p;
  memset(&p, 0, sizeof(p));
  rc = make_operand_maps(c.a, true, c.mode, c.L, c.k_total, BM, &p.a_main, &p.a_tail, &p.a_sc_mul, eb);
  if (rc) return rc;
  rc = make_operand_maps(c.b, false, c.mode, c.L, c.k_total, pair ? 128 : bn, &p.b_main, &p.b_tail, &p.b_sc_mul, eb);
  if (rc) return rc;
  p.bk = 128 / eb;
  p.P = (int)c.P; p.Q = (int)c.Q; p.R = (int)c.R;
  p.mode = c.mode; p.L = (int)c.L; p.k_total = c.k_total; p.s_begin = c.s_begin; p.s_end = c.s_end;
  p.epi = c.epi;
  if (p.epi.scale == 0.0f) p.epi.scale = 1.0f;   // callers that zero-fill the call leave it unset
  p.status = c.status;
  p.carry_bf16 = (c.mode == MODE_RED && c.k_total > 1) ? c.carry_bf16 : 0;
  p.red_group = in_tmem ? c.k_total : ((c.mode == MODE_RED && c.pair_slices && c.s_end - c.s_begin > 1) ? 2 : 1);
  // Two k-blocks per barrier round of the operand ring, except where the epilogue carries a running sum through memory.
  p.round_kblocks = (c.mode == MODE_RED && c.k_total > 1 && !in_tmem) ? 1 : 2;
  // Outputs leave through TMA.  The epilogue that reads a second tensor element-wise (gz) does too
  // (its input arrives by TMA as well) when the launch is unsliced and writes bf16, which is how the MLP
  // backward uses it; otherwise that epilogue falls back to direct stores from registers.
  const bool gz_tma = c.epi.gz && c.mode == MODE_NONE && !c.epi.out_fp32 && !c.epi.accumulate && !c.epi.bias &&
                      !c.epi.z_save && c.epi.act == ACT_NONE;
  p.tma_epilogue = (c.epi.gz == nullptr || gz_tma) ? 1 : 0;
  if (gz_tma) {
    const cuuint64_t dims[3] = {(cuuint64_t)c.Q, (cuuint64_t)c.P, 1};
    const cuuint32_t box32[3] = {32, 32, 1};
    const cuuint64_t sg[2] = {(cuuint64_t)c.epi.ld_gz * 2, (cuuint64_t)c.epi.ld_gz * 2 * (cuuint64_t)c.P};
    rc = encode3d(&p.gz32_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, c.epi.gz, dims, sg, box32, false);
    if (rc) return rc;
    const cuuint32_t boxpf[3] = {(cuuint32_t)bn, 32, 1};
    rc = encode3d(&p.gz_pf_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, c.epi.gz, dims, sg, boxpf, false);
    if (rc) return rc;
    const cuuint64_t so[2] = {(cuuint64_t)c.epi.ld_out * 2, (cuuint64_t)c.epi.ld_out * 2 * (cuuint64_t)c.P};
    rc = encode3d(&p.out32_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, c.epi.out, dims, so, box32, false);
    if (rc) return rc;
    if (c.epi.act_out) {
      const cuuint64_t sa[2] = {(cuuint64_t)c.epi.ld_act_out * 2, (cuuint64_t)c.epi.ld_act_out * 2 * (cuuint64_t)c.P};
      rc = encode3d(&p.z32_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, c.epi.act_out, dims, sa, box32, false);
      if (rc) return rc;
    }
  }
  if (p.tma_epilogue && !gz_tma) {
    if (c.out_is_slice && c.k_total > 1 && (c.mode == MODE_ROWS || c.mode == MODE_COLS)) {
      // the launch covers one slice and writes it as a compact matrix of the slice's extents
      if (c.s_end - c.s_begin != 1 || c.epi.z_save) return OSDP_ERR_UNSUPPORTED;
      const int64_t full = (c.mode == MODE_ROWS) ? c.P : c.Q;
      const int64_t ls = (full - c.s_begin * c.L < c.L) ? full - c.s_begin * c.L : c.L;
      rc = make_output_maps(c.epi.out, c.epi.out_fp32 != 0, c.mode == MODE_ROWS ? ls : c.P,
                            c.mode == MODE_COLS ? ls : c.Q, c.epi.ld_out, c.mode, c.L, c.k_total, &p.out_main,
                            &p.out_tail, &p.out_sc_mul, false);
    } else {
      rc = make_output_maps(c.epi.out, c.epi.out_fp32 != 0, c.P, c.Q, c.epi.ld_out, c.mode, c.L, c.k_total,
                            &p.out_main, &p.out_tail, &p.out_sc_mul);
    }
    if (rc) return rc;
    if (c.epi.z_save) {
      rc = make_output_maps(c.epi.z_save, false, c.P, c.Q, c.epi.ld_z, c.mode, c.L, c.k_total, &p.z_main, &p.z_tail,
                            nullptr);
      if (rc) return rc;
    }
    if (c.mode == MODE_RED && c.k_total > 1 && !p.carry_bf16 && !in_tmem) {
      // the carry, box by box (see GemmParams): [boxes * 32 rows, 32 columns], 128 bytes per row
      const int64_t cb = cdiv(c.Q, 32), boxes = cdiv(c.P, 32) * cb;
      p.carry_cb = (int)cb;
      const cuuint64_t cdims[3] = {32, (cuuint64_t)boxes * 32, 1};
      const cuuint64_t cstr[2] = {128, (cuuint64_t)boxes * 32 * 128};
      const cuuint32_t cbox[3] = {32, 32, 1};
      rc = encode3d(&p.carry_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, c.epi.carry, cdims, cstr, cbox, true);
      if (rc) return rc;
      const cuuint32_t pbox[3] = {32, (cuuint32_t)(bn > 256 ? 256 : bn), 1};   // the bn / 32 boxes of a warp's tile rows
      rc = encode3d(&p.carry_pf_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, c.epi.carry, cdims, cstr, pbox, false);
      if (rc) return rc;
      const cuuint64_t dims[3] = {(cuuint64_t)c.Q, (cuuint64_t)c.P, 1};
      if (!c.epi.out_fp32) {
        // the last slice's bf16 results leave as unswizzled boxes of 32 rows x 32 columns
        const cuuint32_t box32[3] = {32, 32, 1};
        const cuuint64_t so[2] = {(cuuint64_t)c.epi.ld_out * 2, (cuuint64_t)c.epi.ld_out * 2 * (cuuint64_t)c.P};
        rc = encode3d(&p.out32_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, c.epi.out, dims, so, box32, false);
        if (rc) return rc;
        if (c.epi.z_save) {
          const cuuint64_t sz[2] = {(cuuint64_t)c.epi.ld_z * 2, (cuuint64_t)c.epi.ld_z * 2 * (cuuint64_t)c.P};
          rc = encode3d(&p.z32_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, c.epi.z_save, dims, sz, box32, false);
          if (rc) return rc;
        }
      }

    }
  }

  if (c.n_peers > 0) {
    // The epilogue scatters the (compact) output over the ranks' buffers, always as reduce-adds.
    if (!p.tma_epilogue || c.mode == MODE_RED || c.n_peers > 8 || c.epi.gz || c.epi.z_save || c.epi.bias ||
        c.epi.act != ACT_NONE || (c.k_total > 1 && (!c.out_is_slice || c.s_end - c.s_begin != 1)))
      return OSDP_ERR_UNSUPPORTED;
    const int64_t full_r = c.P, full_c = c.Q;
    const int64_t ls = (c.k_total > 1) ? (((c.mode == MODE_ROWS ? full_r : full_c) - c.s_begin * c.L < c.L)
                                              ? (c.mode == MODE_ROWS ? full_r : full_c) - c.s_begin * c.L : c.L) : 0;
    const int64_t rows = (c.k_total > 1 && c.mode == MODE_ROWS) ? ls : full_r;
    const int64_t cols = (c.k_total > 1 && c.mode == MODE_COLS) ? ls : full_c;
    if (rows % c.n_peers || (rows / c.n_peers) % 32) return OSDP_ERR_UNSUPPORTED;
    p.n_peers = c.n_peers;
    p.rows_per_peer = (int)(rows / c.n_peers);
    for (int q = 0; q < c.n_peers; ++q) {
      if (!c.peer_out[q] || !aligned16(c.peer_out[q])) return c.peer_out[q] ? OSDP_ERR_ALIGNMENT : OSDP_ERR_NULL_POINTER;
      CUtensorMap unused;
      rc = make_output_maps(c.peer_out[q], c.epi.out_fp32 != 0, p.rows_per_peer, cols, cols, c.mode, c.L, c.k_total,
                            &unused, &p.peer_out[q], nullptr, false);
      if (rc) return rc;
    }
  }

  // Work items of this launch (one per scheduling unit and tile).
  slot.pair = pair;
  slot.bn = bn;
  slot.items = count_items(c, tm, bn);
  slot.heavy = (c.epi.act != ACT_NONE || gz_tma) && c.mode != MODE_RED && p.tma_epilogue && !c.fp8;
  // A launch that gives every scheduling unit at most one tile has its whole epilogue exposed (nothing follows
  // to overlap it with): eight epilogue warps, each draining half of the tile's columns, halve that time.
  if (slot.items <= (pair ? sms / 2 : sms) && p.tma_epilogue && !c.fp8 && (bn == 128 || bn == 256) &&
      (c.mode == MODE_NONE || c.mode == MODE_COLS || c.mode == MODE_ROWS))
    slot.heavy = true;
  slot.valid = true;
  return launch_prepared(slot, c.a.mn_major, c.b.mn_major, sms, stream);
}

Epilogue plain_epilogue(void *out, int64_t ld, int fp32) {
  Epilogue e;
  memset(&e, 0, sizeof(e));
  e.out = out;
  e.ld_out = ld;
  e.out_fp32 = fp32;
  return e;
}

// Launch of a helper kernel that takes part in programmatic dependent launch like the GEMMs.
template <typename... KArgs, typename... Args>
int launch_aux(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
  if (e != cudaSuccess) return cuda_fail(e);
  return OSDP_OK;
}

int launch_colsum(const void *g, int64_t ld, int64_t M, int c0, int ncols, float *partial, float *out,
                  cudaStream_t stream) {
  const int chunks = (int)cdiv(M, COLSUM_ROWS_PER_CHUNK);
  dim3 grid((unsigned)cdiv(ncols, 64), (unsigned)chunks);
  if (chunks == 1)   // one chunk of rows: its sums are the result (same summation order as the two-pass form)
    return launch_aux(colsum_partial_kernel, grid, dim3(256), stream, (const __nv_bfloat16 *)g, (long long)ld,
                      (long long)M, c0, ncols, out + c0, ncols);
  int rc = launch_aux(colsum_partial_kernel, grid, dim3(256), stream, (const __nv_bfloat16 *)g, (long long)ld,
                      (long long)M, c0, ncols, partial, ncols);
  if (rc) return rc;
  return launch_aux(colsum_final_kernel, dim3((unsigned)cdiv(ncols, 256)), dim3(256), stream,
                    (const float *)partial, ncols, chunks, ncols, out + c0);
}

int launch_act_backward(const void *dy, int64_t ld_dy, const void *z, int64_t ld_z, void *g, int64_t ld_g, int64_t M,
                        int c0, int ncols, int act, cudaStream_t stream) {
  int sms = 0;
  int rc = device_sms(&sms);
  if (rc) return rc;
  const int64_t total = M * (ncols / 8);
  int64_t blocks = cdiv(total, 256);
  if (blocks > (int64_t)sms * 16) blocks = (int64_t)sms * 16;
  return launch_aux(act_backward_kernel, dim3((unsigned)blocks), dim3(256), stream, (const __nv_bfloat16 *)dy,
                    (long long)ld_dy, (const __nv_bfloat16 *)z, (long long)ld_z, (__nv_bfloat16 *)g, (long long)ld_g,
                    (long long)M, c0, ncols, act);
}

// ------------------------------------------------------------------------------------------------
// Argument checks shared by the linear entry points

int check_common(int64_t M, int64_t N, int64_t K, int k, int split_dim, int act, int64_t *L) {
  if (M <= 0 || N <= 0 || K <= 0) return OSDP_ERR_BAD_SHAPE;
  const int64_t lim = (int64_t)1 << 30;
  if (M > lim || N > lim || K > lim) return OSDP_ERR_BAD_SHAPE;
  if ((N & 7) || (K & 7)) return OSDP_ERR_ALIGNMENT;
  if (split_dim != OSDP_SPLIT_OUT && split_dim != OSDP_SPLIT_RED) return OSDP_ERR_BAD_SPLIT;
  if (act != OSDP_ACT_NONE && act != OSDP_ACT_GELU_TANH && act != OSDP_ACT_GELU_ERF) return OSDP_ERR_UNSUPPORTED;
  return slice_len(split_dim == OSDP_SPLIT_OUT ? N : K, k, L);
}

int check_ws(const void *ws, size_t ws_bytes, const WsPlan &plan) {
  if (!ws) return OSDP_ERR_NULL_POINTER;
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return OSDP_ERR_ALIGNMENT;
  if (ws_bytes < plan.total) return OSDP_ERR_WORKSPACE_TOO_SMALL;
  return OSDP_OK;
}

int check_flags(int flags, int allowed, int act, const void *z_save) {
  if (flags & ~allowed) return OSDP_ERR_UNSUPPORTED;
  if ((flags & OSDP_FLAG_PAIR_SLICES) && (flags & OSDP_FLAG_CARRY_BF16)) return OSDP_ERR_UNSUPPORTED;
  if ((flags & OSDP_FLAG_CARRY_BF16) && (act != OSDP_ACT_NONE || z_save)) return OSDP_ERR_UNSUPPORTED;
  return OSDP_OK;
}

// `ld_w_slice` > 0: `w_flat` + `w_offset` is not the whole operator but slice `s_begin` of it, gathered into
// a compact matrix with that leading dimension ([slice rows, K] under OUT, [N, slice columns] under RED).
int fwd_impl(const void *x, const void *w_flat, int64_t w_offset, const float *bias, int64_t M, int64_t N, int64_t K,
             int k, int split_dim, int act, int flags, int s_begin, int s_end, bool single, void *out, void *z_save,
             void *ws, size_t ws_bytes, void *stream, int64_t ld_w_slice = 0, int fp8 = 0, float scale = 1.0f) {
  // fp8: x and W are e4m3 bytes (16 elements per 16 bytes: extents, offset and slice length multiples of 16)
  if (!x || !w_flat || !out) return OSDP_ERR_NULL_POINTER;
  {
    const int frc = check_flags(flags, OSDP_FLAG_CARRY_BF16 | OSDP_FLAG_SLICE_MAJOR | (single ? 0 : OSDP_FLAG_PAIR_SLICES),
                                act, z_save);
    if (frc) return frc;
  }
  if (single) flags |= OSDP_FLAG_SLICE_MAJOR;   // one slice per call is slice-major by construction
  int64_t L = 0;
  int rc = check_common(M, N, K, k, split_dim, act, &L);
  if (rc) return rc;
  if (k == 0) k = 1;
  if (single) {
    if (s_begin < 0 || s_begin >= k) return OSDP_ERR_BAD_SPLIT;
    s_end = s_begin + 1;
  } else {
    s_begin = 0;
    s_end = k;
  }
  if (w_offset < 0 || (w_offset & 7)) return OSDP_ERR_ALIGNMENT;
  if (fp8 && ((N & 15) || (K & 15) || (w_offset & 15) || (k > 1 && (L & 15)) || !std::isfinite(scale) || ld_w_slice > 0))
    return (ld_w_slice > 0 || !std::isfinite(scale)) ? OSDP_ERR_UNSUPPORTED : OSDP_ERR_ALIGNMENT;
  if (!aligned16(x) || !aligned16(w_flat) || !aligned16(out) || !aligned16(z_save) || !aligned16(bias))
    return OSDP_ERR_ALIGNMENT;
  WsPlan plan;
  rc = plan_workspace(M, N, K, k, split_dim, act, OSDP_OP_LINEAR_FWD, flags, &plan);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes, plan);
  if (rc) return rc;

  const void *w = static_cast<const char *>(w_flat) + w_offset * (fp8 ? 1 : 2);
  GemmCall c;
  memset(&c, 0, sizeof(c));
  c.fp8 = fp8;
  c.a = Operand{x, K, M, K, false, true};
  c.b = Operand{w, K, N, K, false, true};
  if (ld_w_slice > 0) {
    if (!single) return OSDP_ERR_UNSUPPORTED;
    if (ld_w_slice & 7) return OSDP_ERR_ALIGNMENT;
    const int64_t D = (split_dim == OSDP_SPLIT_OUT) ? N : K;
    const int64_t ls = (D - s_begin * L < L) ? D - s_begin * L : L;
    if (ld_w_slice < (split_dim == OSDP_SPLIT_OUT ? K : ls)) return OSDP_ERR_BAD_SHAPE;
    c.b = (split_dim == OSDP_SPLIT_OUT) ? Operand{w, K, ls, ld_w_slice, false, false}
                                        : Operand{w, ls, N, ld_w_slice, false, false};
  }
  c.P = M; c.Q = N; c.R = K;
  c.bn_P = M; c.bn_Q = N;
  c.mode = (k == 1) ? MODE_NONE : (split_dim == OSDP_SPLIT_OUT ? MODE_COLS : MODE_RED);
  c.L = L; c.k_total = k; c.s_begin = s_begin; c.s_end = s_end;
  c.epi = plain_epilogue(out, N, 0);
  c.epi.scale = scale;
  c.epi.bias = bias;
  c.epi.z_save = static_cast<__nv_bfloat16 *>(z_save);
  c.epi.ld_z = N;
  c.epi.act = act;
  c.epi.carry = reinterpret_cast<float *>(static_cast<char *>(ws) + plan.carry_off);
  c.epi.ld_carry = N;
  c.carry_bf16 = (flags & OSDP_FLAG_CARRY_BF16) ? 1 : 0;
  c.pair_slices = (flags & OSDP_FLAG_PAIR_SLICES) ? 1 : 0;
  c.slice_major = (flags & OSDP_FLAG_SLICE_MAJOR) ? 1 : 0;
  c.status = static_cast<int *>(ws);
  return launch_gemm(c, static_cast<cudaStream_t>(stream));
}

int bwd_impl(const void *dy, const void *x, const void *w_flat, int64_t w_offset, const void *z_saved, int64_t M,
             int64_t N, int64_t K, int k, int split_dim, int act, int s_begin, int s_end, bool single, void *dx,
             void *dw_flat, int64_t dw_offset, int dw_dtype, int flags, float *dbias, void *ws, size_t ws_bytes,
             void *stream_, int64_t ld_w_slice = 0, int64_t ld_dw_slice = 0, int fp8 = 0, float scale_dx = 1.0f,
             float scale_dw = 1.0f, void *const *dw_peers = nullptr, int n_peers = 0) {
  // dw_peers: the slice's weight gradient is not written to dw_flat but reduce-added, row block by row block,
  // into the n_peers ranks' buffers (the reduce-scatter of the slice done by the GEMM's epilogue)
  // fp8: dy, x and W are e4m3 bytes; no activation, no bias gradient (G = dY must itself be an fp8 operand)
  // ld_w_slice > 0: W is slice `s_begin` gathered into a compact matrix (see fwd_impl);
  // ld_dw_slice > 0: dW of the slice is written as a compact matrix of the same shape.
  if (!dy || !x || !w_flat) return OSDP_ERR_NULL_POINTER;
  // the bf16 running sum concerns dX only, which has neither bias nor activation of its own
  if (flags & ~(OSDP_FLAG_ACCUMULATE_DW | OSDP_FLAG_CARRY_BF16 | OSDP_FLAG_SLICE_MAJOR |
                (single ? 0 : OSDP_FLAG_PAIR_SLICES)))
    return OSDP_ERR_UNSUPPORTED;
  if (single) flags |= OSDP_FLAG_SLICE_MAJOR;   // one slice per call is slice-major by construction
  if ((flags & OSDP_FLAG_PAIR_SLICES) && ((flags & OSDP_FLAG_CARRY_BF16) || act != OSDP_ACT_NONE))
    return OSDP_ERR_UNSUPPORTED;   // with an activation the backward runs slice by slice (staged G_s)
  const int accumulate = (flags & OSDP_FLAG_ACCUMULATE_DW) ? 1 : 0;
  int64_t L = 0;
  int rc = check_common(M, N, K, k, split_dim, act, &L);
  if (rc) return rc;
  if (k == 0) k = 1;
  if (single) {
    if (s_begin < 0 || s_begin >= k) return OSDP_ERR_BAD_SPLIT;
    s_end = s_begin + 1;
  } else {
    s_begin = 0;
    s_end = k;
  }
  if (act != OSDP_ACT_NONE && !z_saved) return OSDP_ERR_NULL_POINTER;
  if (dbias && cdiv(M, COLSUM_ROWS_PER_CHUNK) > 65535) return OSDP_ERR_BAD_SHAPE;   // the column sum's grid limit
  if (fp8) {
    if (act != OSDP_ACT_NONE || dbias || ld_w_slice > 0 || ld_dw_slice > 0 || !std::isfinite(scale_dx) ||
        !std::isfinite(scale_dw))
      return OSDP_ERR_UNSUPPORTED;
    if ((N & 15) || (K & 15) || (w_offset & 15) || (k > 1 && (L & 15))) return OSDP_ERR_ALIGNMENT;
  }
  if (dw_dtype != OSDP_DTYPE_BF16 && dw_dtype != OSDP_DTYPE_FP32) return OSDP_ERR_UNSUPPORTED;
  if (w_offset < 0 || (w_offset & 7) || dw_offset < 0 || (dw_offset & 7)) return OSDP_ERR_ALIGNMENT;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(w_flat) || !aligned16(z_saved) || !aligned16(dx) ||
      !aligned16(dw_flat) || !aligned16(dbias))
    return OSDP_ERR_ALIGNMENT;
  WsPlan plan;
  rc = plan_workspace(M, N, K, k, split_dim, act, OSDP_OP_LINEAR_BWD, flags, &plan);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes, plan);
  if (rc) return rc;

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  char *wsb = static_cast<char *>(ws);
  const void *w = static_cast<const char *>(w_flat) + w_offset * (fp8 ? 1 : 2);
  float *partial = reinterpret_cast<float *>(wsb + plan.part_off);
  float *carry = reinterpret_cast<float *>(wsb + plan.carry_off);
  __nv_bfloat16 *stage = reinterpret_cast<__nv_bfloat16 *>(wsb + plan.stage0_off);
  int *status = static_cast<int *>(ws);
  void *dw = nullptr;
  if (dw_flat)
    dw = (dw_dtype == OSDP_DTYPE_FP32) ? (void *)(static_cast<float *>(dw_flat) + dw_offset)
                                       : (void *)(static_cast<__nv_bfloat16 *>(dw_flat) + dw_offset);
  const bool out_split = (split_dim == OSDP_SPLIT_OUT);
  const int64_t D = out_split ? N : K;
  const int64_t ls0 = (D - s_begin * L < L) ? D - s_begin * L : L;   // extent of slice s_begin
  if (ld_w_slice > 0 || ld_dw_slice > 0) {
    if (!single) return OSDP_ERR_UNSUPPORTED;
    if ((ld_w_slice & 7) || (ld_dw_slice & 7)) return OSDP_ERR_ALIGNMENT;
    if (ld_w_slice > 0 && ld_w_slice < (out_split ? K : ls0)) return OSDP_ERR_BAD_SHAPE;
    if (ld_dw_slice > 0 && ld_dw_slice < (out_split ? K : ls0)) return OSDP_ERR_BAD_SHAPE;
  }

  auto dx_call = [&](const Operand &g, int sb, int se) {
    GemmCall c;
    memset(&c, 0, sizeof(c));
    c.fp8 = fp8;
    c.a = g;                                        // G [M,N], reduction N contiguous
    c.b = Operand{w, K, N, K, true, true};          // W [N,K]: output dim K contiguous
    if (ld_w_slice > 0)
      c.b = out_split ? Operand{w, K, ls0, ld_w_slice, true, false} : Operand{w, ls0, N, ld_w_slice, true, false};
    c.P = M; c.Q = K; c.R = N; c.bn_P = M; c.bn_Q = K;
    c.mode = (k == 1) ? MODE_NONE : (out_split ? MODE_RED : MODE_COLS);
    c.L = L; c.k_total = k; c.s_begin = sb; c.s_end = se;
    c.epi = plain_epilogue(dx, K, 0);
    c.epi.scale = scale_dx;
    c.epi.carry = carry;
    c.epi.ld_carry = K;
    c.carry_bf16 = (flags & OSDP_FLAG_CARRY_BF16) ? 1 : 0;
    c.pair_slices = (flags & OSDP_FLAG_PAIR_SLICES) ? 1 : 0;
    c.slice_major = (flags & OSDP_FLAG_SLICE_MAJOR) ? 1 : 0;
    c.status = status;
    return launch_gemm(c, stream);
  };
  auto dw_call = [&](const Operand &gt, int sb, int se) {
    GemmCall c;
    memset(&c, 0, sizeof(c));
    c.fp8 = fp8;
    c.a = gt;                                       // G^T: output dim N contiguous in G
    c.b = Operand{x, K, M, K, true, true};          // X [M,K]: output dim K contiguous
    c.P = N; c.Q = K; c.R = M; c.bn_P = N; c.bn_Q = K;
    c.mode = (k == 1) ? MODE_NONE : (out_split ? MODE_ROWS : MODE_COLS);
    c.L = L; c.k_total = k; c.s_begin = sb; c.s_end = se;
    c.epi = plain_epilogue(dw, ld_dw_slice > 0 ? ld_dw_slice : K, dw_dtype == OSDP_DTYPE_FP32);
    c.epi.scale = scale_dw;
    c.epi.accumulate = accumulate;
    c.out_is_slice = (ld_dw_slice > 0 && k > 1) ? 1 : 0;
    c.compact = (dx && dw) ? 1 : 0;   // runs next to the dX GEMM
    if (n_peers > 0) {
      c.n_peers = n_peers;
      for (int q = 0; q < n_peers && q < 8; ++q) c.peer_out[q] = dw_peers[q];
    }
    c.status = status;
    return launch_gemm(c, stream);
  };

  if (act == OSDP_ACT_NONE) {
    // dX, dW and db do not depend on one another: when both GEMMs are wanted, dW and db run on an internal
    // stream next to dX (fork from and join into `stream`), so that each fills the SMs that the other's last,
    // partly filled wave of tiles leaves idle.  Measured on B200, backward only: 256 x 2048 x 512 42 -> 34 us;
    // 8192 x 2048 x 2048 +8 %, 4096 x 4096 x 1024 +7 %, 8192 x 2048 x 8192 +5 %, 32768 x 4096 x 4096 +3 %,
    // 16384 x 8192 x 8192 +0.3 % (k = 8: +1 %); one shape tried lost (8192 x 6144 x 2048, -1.5 %).
    ForkJoin fj;
    cudaStream_t s_main = stream;
    if (dx && dw) {
      rc = fj.acquire(stream, 1);
      if (rc) return rc;
      rc = fj.begin();
      if (rc) return rc;
    }
    cudaStream_t s_side = fj.stream(0);
    stream = s_main;
    if (dx) { rc = dx_call(Operand{dy, N, M, N, false, true}, s_begin, s_end); if (rc) return rc; }
    stream = s_side;
    if (dw) { rc = dw_call(Operand{dy, N, M, N, true, true}, s_begin, s_end); if (rc) return rc; }
    // The short column sum goes behind the shorter of the two GEMM chains: dX reduces over N, dW over the M
    // tokens, and with equal flops the longer reduction has the fewer tiles and takes longer.
    if (dx && M >= N) stream = s_main;
    if (dbias) {
      if (out_split) {
        const int64_t c0 = (int64_t)s_begin * L;
        const int64_t c1 = ((int64_t)s_end * L < N) ? (int64_t)s_end * L : N;
        rc = launch_colsum(dy, N, M, (int)c0, (int)(c1 - c0), partial, dbias, stream);
      } else if (s_begin == 0) {
        rc = launch_colsum(dy, N, M, 0, (int)N, partial, dbias, stream);
      }
      if (rc) return rc;
    }
    stream = s_main;
    return fj.end();
  }

  // With an activation the GEMMs read G = dY (.) act'(Z) from staging.  As above, when both are wanted dW (and
  // db) run on the internal stream next to dX; they join before the staging is written again.
  ForkJoin fj;
  if (dx && dw) {
    rc = fj.acquire(stream, 1);
    if (rc) return rc;
  }
  cudaStream_t s_main = stream;
  auto fork = [&]() -> int {
    int r = fj.begin();
    if (r) return r;
    stream = fj.stream(0);
    return OSDP_OK;
  };
  auto join = [&]() -> int {
    stream = s_main;
    return fj.end();
  };

  if (out_split) {
    // Slice by slice: G_s = dY[:,R_s] (.) act'(Z[:,R_s]) into slice-sized staging, then the slice's GEMMs.
    for (int s = s_begin; s < s_end; ++s) {
      const int64_t c0 = (int64_t)s * L;
      const int64_t ls = (c0 + L < N ? c0 + L : N) - c0;
      rc = launch_act_backward(dy, N, z_saved, N, stage, L, M, (int)c0, (int)ls, act, stream);
      if (rc) return rc;
      rc = fork();                                     // from here on `stream` is the internal one, if any
      if (rc) return rc;
      if (dw) { rc = dw_call(Operand{stage, ls, M, L, true, false}, s, s + 1); if (rc) return rc; }
      if (dbias) { rc = launch_colsum(stage, L, M, 0, (int)ls, partial, dbias + c0, stream); if (rc) return rc; }
      stream = s_main;
      if (dx) { rc = dx_call(Operand{stage, ls, M, L, false, false}, s, s + 1); if (rc) return rc; }
      rc = join();
      if (rc) return rc;
    }
    return OSDP_OK;
  }
  // RED split: G is needed whole by every slice.
  if (s_begin == 0) {
    rc = launch_act_backward(dy, N, z_saved, N, stage, N, M, 0, (int)N, act, stream);
    if (rc) return rc;
  }
  rc = fork();
  if (rc) return rc;
  if (s_begin == 0 && dbias) { rc = launch_colsum(stage, N, M, 0, (int)N, partial, dbias, stream); if (rc) return rc; }
  if (dw) { rc = dw_call(Operand{stage, N, M, N, true, true}, s_begin, s_end); if (rc) return rc; }
  stream = s_main;
  if (dx) { rc = dx_call(Operand{stage, N, M, N, false, true}, s_begin, s_end); if (rc) return rc; }
  return join();
}

}  // namespace

// ================================================================================================
// C ABI

extern "C" {

int osdp_version(void) { return OSDP_VERSION; }

const char *osdp_status_string(int status) {
  switch (status) {
    case OSDP_OK: return "ok";
    case OSDP_ERR_NULL_POINTER: return "null pointer";
    case OSDP_ERR_BAD_SHAPE: return "bad shape";
    case OSDP_ERR_BAD_SPLIT: return "bad split";
    case OSDP_ERR_ALIGNMENT: return "alignment";
    case OSDP_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case OSDP_ERR_UNSUPPORTED: return "unsupported";
    case OSDP_ERR_CUDA: return "CUDA error";
    case OSDP_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case OSDP_ERR_EXCEEDS_STATIC_SCRATCH: return "problem larger than the library's built-in scratch";
    case OSDP_ERR_SEARCH_LIMIT: return "plan search stopped at its node budget";
    default: return "unknown status";
  }
}

int osdp_last_cuda_error(void) { return g_last_cuda_error; }

int osdp_slice_range(int64_t D, int k_split, int slice_idx, int64_t *begin, int64_t *end) {
  if (!begin || !end) return OSDP_ERR_NULL_POINTER;
  int64_t L = 0;
  int rc = slice_len(D, k_split, &L);
  if (rc) return rc;
  const int k = k_split == 0 ? 1 : k_split;
  if (slice_idx < 0 || slice_idx >= k) return OSDP_ERR_BAD_SPLIT;
  *begin = (int64_t)slice_idx * L;
  *end = (*begin + L < D) ? *begin + L : D;
  return OSDP_OK;
}

int osdp_split_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int k_split, int split_dim, int act, int op,
                                      int flags, size_t *bytes) {
  if (!bytes) return OSDP_ERR_NULL_POINTER;
  if (act != OSDP_ACT_NONE && act != OSDP_ACT_GELU_TANH && act != OSDP_ACT_GELU_ERF) return OSDP_ERR_UNSUPPORTED;
  if (flags & ~(OSDP_FLAG_ACCUMULATE_DW | OSDP_FLAG_CARRY_BF16 | OSDP_FLAG_RECOMPUTE | OSDP_FLAG_PAIR_SLICES |
                OSDP_FLAG_SLICE_MAJOR))
    return OSDP_ERR_UNSUPPORTED;
  if ((flags & OSDP_FLAG_RECOMPUTE) && op != OSDP_OP_MLP_BWD) return OSDP_ERR_UNSUPPORTED;
  if ((flags & (OSDP_FLAG_PAIR_SLICES | OSDP_FLAG_SLICE_MAJOR)) && op != OSDP_OP_LINEAR_FWD && op != OSDP_OP_LINEAR_BWD)
    return OSDP_ERR_UNSUPPORTED;
  WsPlan plan;
  int rc = plan_workspace(M, N, K, k_split, split_dim, act, op, flags, &plan);
  if (rc) return rc;
  *bytes = plan.total;
  return OSDP_OK;
}

int osdp_suggest_granularity(int64_t M, int64_t N, int64_t K, int split_dim, int act, int op, int flags,
                             size_t budget_bytes, int max_k, int *k_split) {
  if (!k_split) return OSDP_ERR_NULL_POINTER;
  if (max_k < 1 || max_k > OSDP_MAX_SPLIT) return OSDP_ERR_BAD_SPLIT;
  size_t bytes = 0;
  int rc = osdp_split_linear_workspace_bytes(M, N, K, 1, split_dim, act, op, flags, &bytes);
  if (rc) return rc;   // bad shape / op / flags: the same verdict as the call itself would give
  for (int k = 1; k <= max_k; ++k) {
    rc = osdp_split_linear_workspace_bytes(M, N, K, k, split_dim, act, op, flags, &bytes);
    if (rc == OSDP_ERR_BAD_SPLIT) continue;   // this k would leave an empty slice
    if (rc) return rc;
    if (bytes <= budget_bytes) {
      *k_split = k;
      return OSDP_OK;
    }
  }
  return OSDP_ERR_WORKSPACE_TOO_SMALL;
}

int osdp_split_linear_fwd(const void *x, const void *w_flat, int64_t w_offset, const float *bias, int64_t M,
                          int64_t N, int64_t K, int k_split, int split_dim, int act, int flags, void *out,
                          void *z_save, void *ws, size_t ws_bytes, void *stream) {
  return fwd_impl(x, w_flat, w_offset, bias, M, N, K, k_split, split_dim, act, flags, 0, 0, false, out, z_save, ws,
                  ws_bytes, stream);
}

int osdp_split_linear_fwd_slice(const void *x, const void *w_flat, int64_t w_offset, const float *bias, int64_t M,
                                int64_t N, int64_t K, int k_split, int split_dim, int act, int flags, int slice_idx,
                                void *out, void *z_save, void *ws, size_t ws_bytes, void *stream) {
  return fwd_impl(x, w_flat, w_offset, bias, M, N, K, k_split, split_dim, act, flags, slice_idx, 0, true, out, z_save,
                  ws, ws_bytes, stream);
}

int osdp_split_linear_bwd(const void *dy, const void *x, const void *w_flat, int64_t w_offset, const void *z_saved,
                          int64_t M, int64_t N, int64_t K, int k_split, int split_dim, int act, void *dx,
                          void *dw_flat, int64_t dw_offset, int dw_dtype, int flags, float *dbias, void *ws,
                          size_t ws_bytes, void *stream) {
  return bwd_impl(dy, x, w_flat, w_offset, z_saved, M, N, K, k_split, split_dim, act, 0, 0, false, dx, dw_flat,
                  dw_offset, dw_dtype, flags, dbias, ws, ws_bytes, stream);
}

int osdp_split_linear_bwd_slice(const void *dy, const void *x, const void *w_flat, int64_t w_offset,
                                const void *z_saved, int64_t M, int64_t N, int64_t K, int k_split, int split_dim,
                                int act, int slice_idx, void *dx, void *dw_flat, int64_t dw_offset, int dw_dtype,
                                int flags, float *dbias, void *ws, size_t ws_bytes, void *stream) {
  return bwd_impl(dy, x, w_flat, w_offset, z_saved, M, N, K, k_split, split_dim, act, slice_idx, 0, true, dx, dw_flat,
                  dw_offset, dw_dtype, flags, dbias, ws, ws_bytes, stream);
}

int osdp_split_linear_fwd_f8(const void *x8, const void *w8_flat, int64_t w_offset, float scale, const float *bias,
                             int64_t M, int64_t N, int64_t K, int k_split, int split_dim, int act, int flags,
                             void *out, void *z_save, void *ws, size_t ws_bytes, void *stream) {
  return fwd_impl(x8, w8_flat, w_offset, bias, M, N, K, k_split, split_dim, act, flags, 0, 0, false, out, z_save, ws,
                  ws_bytes, stream, 0, 1, scale);
}

int osdp_split_linear_bwd_f8(const void *dy8, const void *x8, const void *w8_flat, int64_t w_offset, float scale_dx,
                             float scale_dw, int64_t M, int64_t N, int64_t K, int k_split, int split_dim, void *dx,
                             void *dw_flat, int64_t dw_offset, int dw_dtype, int flags, void *ws, size_t ws_bytes,
                             void *stream) {
  return bwd_impl(dy8, x8, w8_flat, w_offset, nullptr, M, N, K, k_split, split_dim, OSDP_ACT_NONE, 0, 0, false, dx,
                  dw_flat, dw_offset, dw_dtype, flags, nullptr, ws, ws_bytes, stream, 0, 0, 1, scale_dx, scale_dw);
}

int osdp_zdp_shard_layout(int64_t N, int64_t K, int k_split, int split_dim, int world, int slice_idx,
                          int64_t *slice_elems, int64_t *shard_elems, int64_t *shard_offset, int64_t *ld) {
  if (N <= 0 || K <= 0) return OSDP_ERR_BAD_SHAPE;
  if ((N & 7) || (K & 7)) return OSDP_ERR_ALIGNMENT;
  if (split_dim != OSDP_SPLIT_OUT && split_dim != OSDP_SPLIT_RED) return OSDP_ERR_BAD_SPLIT;
  if (world < 1 || world > 65536) return OSDP_ERR_BAD_SHAPE;
  const bool out_split = (split_dim == OSDP_SPLIT_OUT);
  const int64_t D = out_split ? N : K;
  const int64_t other = out_split ? K : N;
  int64_t L = 0;
  int rc = slice_len(D, k_split, &L);
  if (rc) return rc;
  const int k = k_split == 0 ? 1 : k_split;
  if (slice_idx < 0 || slice_idx > k) return OSDP_ERR_BAD_SPLIT;
  int64_t off = 0, ls = 0, elems = 0, shard = 0;
  for (int s = 0; s <= slice_idx; ++s) {
    off += shard;
    if (s == k) { ls = 0; elems = 0; shard = 0; break; }
    ls = (D - s * L < L) ? D - s * L : L;
    elems = ls * other;
    shard = (elems + (int64_t)world * 8 - 1) / ((int64_t)world * 8) * 8;
  }
  if (slice_elems) *slice_elems = elems;
  if (shard_elems) *shard_elems = shard;
  if (shard_offset) *shard_offset = off;
  if (ld) *ld = out_split ? K : ls;
  return OSDP_OK;
}

int osdp_zdp_linear_fwd_slice(const void *x, const void *w_slice, int64_t ld_w, const float *bias, int64_t M,
                              int64_t N, int64_t K, int k_split, int split_dim, int act, int flags, int slice_idx,
                              void *out, void *z_save, void *ws, size_t ws_bytes, void *stream) {
  if (ld_w <= 0) return OSDP_ERR_BAD_SHAPE;
  return fwd_impl(x, w_slice, 0, bias, M, N, K, k_split, split_dim, act, flags, slice_idx, 0, true, out, z_save, ws,
                  ws_bytes, stream, ld_w);
}

int osdp_zdp_linear_bwd_slice(const void *dy, const void *x, const void *w_slice, int64_t ld_w, const void *z_saved,
                              int64_t M, int64_t N, int64_t K, int k_split, int split_dim, int act, int slice_idx,
                              void *dx, void *dw_slice, int64_t ld_dw, int dw_dtype, int flags, float *dbias,
                              void *ws, size_t ws_bytes, void *stream) {
  if (ld_w <= 0 || (dw_slice && ld_dw <= 0)) return OSDP_ERR_BAD_SHAPE;
  return bwd_impl(dy, x, w_slice, 0, z_saved, M, N, K, k_split, split_dim, act, slice_idx, 0, true, dx, dw_slice, 0,
                  dw_dtype, flags, dbias, ws, ws_bytes, stream, ld_w, dw_slice ? ld_dw : 0);
}

int osdp_zdp_linear_bwd_slice_scatter(const void *dy, const void *x, const void *w_slice, int64_t ld_w,
                                      const void *z_saved, int64_t M, int64_t N, int64_t K, int k_split, int split_dim,
                                      int act, int slice_idx, void *dx, void *const *dw_peers, int world, int dw_dtype,
                                      int flags, float *dbias, void *ws, size_t ws_bytes, void *stream) {
  if (ld_w <= 0) return OSDP_ERR_BAD_SHAPE;
  if (!dw_peers) return OSDP_ERR_NULL_POINTER;
  if (world < 1 || world > 8) return OSDP_ERR_UNSUPPORTED;
  if (flags & OSDP_FLAG_ACCUMULATE_DW) return OSDP_ERR_UNSUPPORTED;   // the scatter always adds
  int64_t ld = 0;
  int rc = osdp_zdp_shard_layout(N, K, k_split, split_dim, world, slice_idx, nullptr, nullptr, nullptr, &ld);
  if (rc) return rc;
  return bwd_impl(dy, x, w_slice, 0, z_saved, M, N, K, k_split, split_dim, act, slice_idx, 0, true, dx, dw_peers[0], 0,
                  dw_dtype, flags, dbias, ws, ws_bytes, stream, ld_w, ld, 0, 1.0f, 1.0f, dw_peers, world);
}

// One slice of a sharded MLP block given as gathered compact matrices (and where its weight gradients go).
struct MlpSlice {
  int idx;                    // the slice; the call covers this slice only
  const void *w1, *w2;        // W1[F_s,:] as [len F_s, hidden] (contiguous rows), W2[:,F_s] as [hidden, len F_s]
  int64_t ld_w2;
  void *dw1, *dw2;            // same shapes, dw_dtype; or the ranks' buffers for the epilogue's reduce-scatter
  int64_t ld_dw2;
  void *const *dw1_peers, *const *dw2_peers;
  int world;
};

static int mlp_fwd_impl(const void *x, const void *w_flat, int64_t off_w1, const float *b1, int64_t off_w2,
                        const float *b2, int64_t M, int64_t hidden, int64_t ffn, int k_split, int act, int flags,
                        void *out, void *z1_save, void *ws, size_t ws_bytes, void *stream_, const MlpSlice *cs) {
  if (!x || !w_flat || !out) return OSDP_ERR_NULL_POINTER;
  if (flags & ~OSDP_FLAG_CARRY_BF16) return OSDP_ERR_UNSUPPORTED;   // the second layer has no activation: allowed
  int64_t L = 0;
  int rc = check_common(M, ffn, hidden, k_split, OSDP_SPLIT_OUT, act, &L);
  if (rc) return rc;
  const int k = k_split == 0 ? 1 : k_split;
  if (off_w1 < 0 || off_w2 < 0 || (off_w1 & 7) || (off_w2 & 7)) return OSDP_ERR_ALIGNMENT;
  if (!aligned16(x) || !aligned16(w_flat) || !aligned16(out) || !aligned16(z1_save) || !aligned16(b1) ||
      !aligned16(b2))
    return OSDP_ERR_ALIGNMENT;
  WsPlan plan;
  rc = plan_workspace(M, ffn, hidden, k, OSDP_SPLIT_OUT, act, OSDP_OP_MLP_FWD, flags, &plan);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes, plan);
  if (rc) return rc;

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  char *wsb = static_cast<char *>(ws);
  const __nv_bfloat16 *w1 = static_cast<const __nv_bfloat16 *>(w_flat) + off_w1;   // [ffn, hidden]
  const __nv_bfloat16 *w2 = static_cast<const __nv_bfloat16 *>(w_flat) + off_w2;   // [hidden, ffn]
  __nv_bfloat16 *a_s = reinterpret_cast<__nv_bfloat16 *>(wsb + plan.stage0_off);   // A_s [M, ls], ld L
  float *carry = reinterpret_cast<float *>(wsb + plan.carry_off);
  int *status = static_cast<int *>(ws);

  if (cs && (cs->idx < 0 || cs->idx >= k)) return OSDP_ERR_BAD_SPLIT;
  for (int s = cs ? cs->idx : 0; s < (cs ? cs->idx + 1 : k); ++s) {
    const int64_t lo = (int64_t)s * L;
    const int64_t ls = (lo + L < ffn ? lo + L : ffn) - lo;
    // A_s = act(X W1[F_s,:]^T + b1[F_s])
    GemmCall c;
    memset(&c, 0, sizeof(c));
    c.a = Operand{x, hidden, M, hidden, false, false};
    c.b = Operand{cs ? static_cast<const __nv_bfloat16 *>(cs->w1) : w1 + lo * hidden, hidden, ls, hidden, false, false};
    c.P = M; c.Q = ls; c.R = hidden; c.bn_P = M; c.bn_Q = L;
    c.mode = MODE_NONE; c.L = ls; c.k_total = 1; c.s_begin = 0; c.s_end = 1;
    c.epi = plain_epilogue(a_s, L, 0);
    c.epi.bias = b1 ? b1 + lo : nullptr;
    c.epi.z_save = z1_save ? static_cast<__nv_bfloat16 *>(z1_save) + lo : nullptr;
    c.epi.ld_z = ffn;
    c.epi.act = act;
    c.status = status;
    rc = launch_gemm(c, stream);
    if (rc) return rc;
    // Y (+)= A_s W2[:,F_s]^T ; + b2 after the last slice
    memset(&c, 0, sizeof(c));
    c.a = Operand{a_s, ls, M, L, false, false};
    c.b = cs ? Operand{cs->w2, ls, hidden, cs->ld_w2, false, false} : Operand{w2, ffn, hidden, ffn, false, true};
    c.P = M; c.Q = hidden; c.R = ffn; c.bn_P = M; c.bn_Q = hidden;
    c.mode = (k == 1) ? MODE_NONE : MODE_RED;
    c.L = L; c.k_total = k; c.s_begin = s; c.s_end = s + 1;
    c.epi = plain_epilogue(out, hidden, 0);
    c.epi.bias = b2;
    c.epi.carry = carry;
    c.epi.ld_carry = hidden;
    c.carry_bf16 = (flags & OSDP_FLAG_CARRY_BF16) ? 1 : 0;
    c.status = status;
    rc = launch_gemm(c, stream);
    if (rc) return rc;
  }
  return OSDP_OK;
}

static int mlp_bwd_impl(const void *dy, const void *x, const void *w_flat, int64_t off_w1, const float *b1,
                        int64_t off_w2, const void *z1_saved, int64_t M, int64_t hidden, int64_t ffn, int k_split,
                        int act, void *dx, void *dw_flat, int64_t dw_off_w1, int64_t dw_off_w2, int dw_dtype,
                        int flags, float *db1, float *db2, void *ws, size_t ws_bytes, void *stream_,
                        const MlpSlice *cs) {
  if (flags & ~(OSDP_FLAG_ACCUMULATE_DW | OSDP_FLAG_CARRY_BF16 | OSDP_FLAG_RECOMPUTE)) return OSDP_ERR_UNSUPPORTED;
  const bool recompute = (flags & OSDP_FLAG_RECOMPUTE) != 0;
  if (!dy || !x || !w_flat || (!recompute && !z1_saved)) return OSDP_ERR_NULL_POINTER;
  if (!aligned16(b1)) return OSDP_ERR_ALIGNMENT;
  const int accumulate = (flags & OSDP_FLAG_ACCUMULATE_DW) ? 1 : 0;
  int64_t L = 0;
  int rc = check_common(M, ffn, hidden, k_split, OSDP_SPLIT_OUT, act, &L);
  if (rc) return rc;
  const int k = k_split == 0 ? 1 : k_split;
  if (dw_dtype != OSDP_DTYPE_BF16 && dw_dtype != OSDP_DTYPE_FP32) return OSDP_ERR_UNSUPPORTED;
  if (off_w1 < 0 || off_w2 < 0 || (off_w1 & 7) || (off_w2 & 7) || dw_off_w1 < 0 || dw_off_w2 < 0 ||
      (dw_off_w1 & 7) || (dw_off_w2 & 7))
    return OSDP_ERR_ALIGNMENT;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(w_flat) || !aligned16(z1_saved) || !aligned16(dx) ||
      !aligned16(dw_flat) || !aligned16(db1) || !aligned16(db2))
    return OSDP_ERR_ALIGNMENT;
  WsPlan plan;
  rc = plan_workspace(M, ffn, hidden, k, OSDP_SPLIT_OUT, act, OSDP_OP_MLP_BWD, flags, &plan);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes, plan);
  if (rc) return rc;

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  char *wsb = static_cast<char *>(ws);
  const __nv_bfloat16 *w1 = static_cast<const __nv_bfloat16 *>(w_flat) + off_w1;
  const __nv_bfloat16 *w2 = static_cast<const __nv_bfloat16 *>(w_flat) + off_w2;
  const __nv_bfloat16 *z1 = static_cast<const __nv_bfloat16 *>(z1_saved);
  __nv_bfloat16 *a_s = reinterpret_cast<__nv_bfloat16 *>(wsb + plan.stage0_off);
  __nv_bfloat16 *dz_s = reinterpret_cast<__nv_bfloat16 *>(wsb + plan.stage1_off);
  __nv_bfloat16 *z1_s = reinterpret_cast<__nv_bfloat16 *>(wsb + plan.stage2_off);
  float *carry = reinterpret_cast<float *>(wsb + plan.carry_off);
  float *partial = reinterpret_cast<float *>(wsb + plan.part_off);
  const size_t part_set = ((size_t)((M + COLSUM_ROWS_PER_CHUNK - 1) / COLSUM_ROWS_PER_CHUNK)) * (size_t)L;
  float *partial2 = partial + (plan.stage_stride ? 2 : 1) * part_set;   // db2's
  int *status = static_cast<int *>(ws);
  const int fp32 = dw_dtype == OSDP_DTYPE_FP32;
  auto dw_ptr = [&](int64_t off) -> void * {
    if (!dw_flat) return nullptr;
    return fp32 ? (void *)(static_cast<float *>(dw_flat) + off) : (void *)(static_cast<__nv_bfloat16 *>(dw_flat) + off);
  };

  if (cs && (cs->idx < 0 || cs->idx >= k)) return OSDP_ERR_BAD_SPLIT;
  // db2 = column sums of dY: independent of everything else; it runs next to the first slice's GEMMs (below)
  bool db2_pending = db2 && (!cs || cs->idx == 0);
  // The slice's weight-gradient GEMMs are forked onto the internal streams next to its dX GEMM.  Measured on
  // B200: hidden 1024 / ffn 4096 / 4096 tokens at k = 8 1.06 -> 0.84 ms; hidden 2048 / ffn 8192 at k = 4 +7.5 %;
  // hidden 4096 / ffn 16384 / 8192 tokens +1.5 %; hidden 8192 / ffn 32768 at k = 8 +0.5 %.
  const bool concurrent = dw_flat != nullptr;
  // Small slices, all of them in this call: two sets of staging buffers, used in turn.  The slice's weight-gradient
  // GEMMs then need not finish before the next slice's first GEMM writes its buffers, only before the slice after
  // that does; the caller's stream carries dZ_s -> dX -> db1 slice after slice without waiting for them.
  // Measured on B200 (backward, 4096 tokens, hidden 1024, ffn 4096): k = 4 0.32 -> 0.29 ms, k = 8 0.52 -> 0.40 ms;
  // 8192 tokens: k = 8 0.83 -> 0.64 ms.
  const bool piped = !cs && concurrent && plan.stage_stride != 0;
  ForkJoin pipe;
  if (piped) {
    rc = pipe.acquire(stream, 2);
    if (rc) return rc;
    rc = pipe.begin();
    if (rc) return rc;
  }
  __nv_bfloat16 *const a_s0 = a_s, *const dz_s0 = dz_s, *const z1_s0 = z1_s;
  float *const partial0 = partial;
  for (int s = cs ? cs->idx : 0; s < (cs ? cs->idx + 1 : k); ++s) {
    const int64_t lo = (int64_t)s * L;
    const int64_t ls = (lo + L < ffn ? lo + L : ffn) - lo;
    const int par = s & 1;
    if (piped) {
      const size_t shift = (size_t)par * plan.stage_stride;
      a_s = reinterpret_cast<__nv_bfloat16 *>(reinterpret_cast<char *>(a_s0) + shift);
      dz_s = reinterpret_cast<__nv_bfloat16 *>(reinterpret_cast<char *>(dz_s0) + shift);
      z1_s = reinterpret_cast<__nv_bfloat16 *>(reinterpret_cast<char *>(z1_s0) + shift);
      partial = partial0 + (size_t)par * part_set;
      if (s >= 2) {   // slice s - 2's weight-gradient GEMMs have read this set of buffers
        rc = pipe.after(1, par, 0);
        if (rc) return rc;
        rc = pipe.after(2, par, 0);
        if (rc) return rc;
      }
    }
    const __nv_bfloat16 *w1s = cs ? static_cast<const __nv_bfloat16 *>(cs->w1) : w1 + lo * hidden;   // [ls, hidden]
    const __nv_bfloat16 *w2s = cs ? static_cast<const __nv_bfloat16 *>(cs->w2) : w2 + lo;            // [hidden, ls]
    const int64_t ld_w2s = cs ? cs->ld_w2 : ffn;
    GemmCall c;
    if (recompute) {
      // Z1_s = X W1[F_s,:]^T + b1[F_s] (the forward's first GEMM again, same bits), A_s = act(Z1_s)
      memset(&c, 0, sizeof(c));
      c.a = Operand{x, hidden, M, hidden, false, false};
      c.b = Operand{w1s, hidden, ls, hidden, false, false};
      c.P = M; c.Q = ls; c.R = hidden; c.bn_P = M; c.bn_Q = L;
      c.mode = MODE_NONE; c.L = ls; c.k_total = 1; c.s_begin = 0; c.s_end = 1;
      c.epi = plain_epilogue(a_s, L, 0);
      c.epi.bias = b1 ? b1 + lo : nullptr;
      c.epi.z_save = z1_s;
      c.epi.ld_z = L;
      c.epi.act = act;
      c.status = status;
      rc = launch_gemm(c, stream);
      if (rc) return rc;
    }
    // dZ_s = (dY W2[:,F_s]) (.) act'(Z1_s);  A_s = act(Z1_s) unless it was just recomputed
    memset(&c, 0, sizeof(c));
    c.a = Operand{dy, hidden, M, hidden, false, false};
    c.b = Operand{w2s, ls, hidden, ld_w2s, true, false};
    c.P = M; c.Q = ls; c.R = hidden; c.bn_P = M; c.bn_Q = L;
    c.mode = MODE_NONE; c.L = ls; c.k_total = 1; c.s_begin = 0; c.s_end = 1;
    c.epi = plain_epilogue(dz_s, L, 0);
    c.epi.gz = recompute ? z1_s : z1 + lo;
    c.epi.ld_gz = recompute ? L : ffn;
    c.epi.gz_act = act;
    c.epi.act_out = recompute ? nullptr : a_s;
    c.epi.ld_act_out = L;
    c.status = status;
    c.compact = piped ? 1 : 0;   // the previous slice's weight-gradient GEMMs are still running beside it
    rc = launch_gemm(c, stream);
    if (rc) return rc;
    // The slice's three remaining GEMMs and its column sum depend only on what has been launched so far.
    // They are forked onto the internal streams so that they share the SMs (each fills the others' partly
    // filled last wave of tiles).
    ForkJoin fj;
    if (piped) {
      rc = pipe.mark(0, par);
      if (rc) return rc;
      rc = pipe.after(0, par, 1);
      if (rc) return rc;
      rc = pipe.after(0, par, 2);
      if (rc) return rc;
    } else if (concurrent) {
      rc = fj.acquire(stream, 2);
      if (rc) return rc;
      rc = fj.begin();
      if (rc) return rc;
    }
    cudaStream_t s_dw2 = piped ? pipe.stream(0) : fj.stream(0), s_dw1 = piped ? pipe.stream(1) : fj.stream(1);
    if (db2_pending) {
      // its partial sums use the part of the scratch past the slice's own (db1's) columns
      rc = launch_colsum(dy, hidden, M, 0, (int)hidden, partial2, db2, s_dw2);
      if (rc) return rc;
      db2_pending = false;
    }
    if (dw_flat) {
      // dW2[:,F_s] = dY^T A_s
      memset(&c, 0, sizeof(c));
      c.a = Operand{dy, hidden, M, hidden, true, false};
      c.b = Operand{a_s, ls, M, L, true, false};
      c.P = hidden; c.Q = ls; c.R = M; c.bn_P = hidden; c.bn_Q = L;
      c.mode = MODE_NONE; c.L = ls; c.k_total = 1; c.s_begin = 0; c.s_end = 1;
      c.epi = cs ? plain_epilogue(cs->dw2_peers ? cs->dw2_peers[0] : cs->dw2, cs->ld_dw2, fp32)
                 : plain_epilogue(dw_ptr(dw_off_w2 + lo), ffn, fp32);
      c.epi.accumulate = accumulate;
      c.compact = concurrent ? 1 : 0;
      if (cs && cs->dw2_peers) {
        c.n_peers = cs->world;
        for (int q = 0; q < cs->world && q < 8; ++q) c.peer_out[q] = cs->dw2_peers[q];
      }
      c.status = status;
      rc = launch_gemm(c, s_dw2);
      if (rc) return rc;
      // dW1[F_s,:] = dZ_s^T X
      memset(&c, 0, sizeof(c));
      c.a = Operand{dz_s, ls, M, L, true, false};
      c.b = Operand{x, hidden, M, hidden, true, false};
      c.P = ls; c.Q = hidden; c.R = M; c.bn_P = L; c.bn_Q = hidden;
      c.mode = MODE_NONE; c.L = ls; c.k_total = 1; c.s_begin = 0; c.s_end = 1;
      c.epi = cs ? plain_epilogue(cs->dw1_peers ? cs->dw1_peers[0] : cs->dw1, hidden, fp32)
                 : plain_epilogue(dw_ptr(dw_off_w1 + lo * hidden), hidden, fp32);
      c.epi.accumulate = accumulate;
      c.compact = concurrent ? 1 : 0;
      if (cs && cs->dw1_peers) {
        c.n_peers = cs->world;
        for (int q = 0; q < cs->world && q < 8; ++q) c.peer_out[q] = cs->dw1_peers[q];
      }
      c.status = status;
      rc = launch_gemm(c, s_dw1);
      if (rc) return rc;
    }
    // db1[F_s]: a short kernel; it goes behind the short dX GEMM on the caller's stream rather than behind a
    // long weight-gradient GEMM (4096 tokens, hidden 1024, k = 8: 10 us less per slice)
    if (db1 && !dx) { rc = launch_colsum(dz_s, L, M, 0, (int)ls, partial, db1 + lo, s_dw1); if (rc) return rc; }
    if (dx) {
      // dX (+)= dZ_s W1[F_s,:]
      memset(&c, 0, sizeof(c));
      c.a = Operand{dz_s, ls, M, L, false, false};
      c.b = cs ? Operand{w1s, hidden, ls, hidden, true, false} : Operand{w1, hidden, ffn, hidden, true, true};
      c.P = M; c.Q = hidden; c.R = ffn; c.bn_P = M; c.bn_Q = hidden;
      c.mode = (k == 1) ? MODE_NONE : MODE_RED;
      c.L = L; c.k_total = k; c.s_begin = s; c.s_end = s + 1;
      c.epi = plain_epilogue(dx, hidden, 0);
      c.epi.carry = carry;
      c.epi.ld_carry = hidden;
      c.carry_bf16 = (flags & OSDP_FLAG_CARRY_BF16) ? 1 : 0;
      c.status = status;
      rc = launch_gemm(c, stream);
      if (rc) return rc;
      if (db1) { rc = launch_colsum(dz_s, L, M, 0, (int)ls, partial, db1 + lo, stream); if (rc) return rc; }
    }
    if (piped) {
      rc = pipe.mark(1, par);
      if (rc) return rc;
      rc = pipe.mark(2, par);
      if (rc) return rc;
    }
    // join: the next slice reuses the staging buffers these launches read
    rc = fj.end();
    if (rc) return rc;
  }
  return pipe.end();
}

int osdp_split_mlp_fwd(const void *x, const void *w_flat, int64_t off_w1, const float *b1, int64_t off_w2,
                       const float *b2, int64_t M, int64_t hidden, int64_t ffn, int k_split, int act, int flags,
                       void *out, void *z1_save, void *ws, size_t ws_bytes, void *stream) {
  return mlp_fwd_impl(x, w_flat, off_w1, b1, off_w2, b2, M, hidden, ffn, k_split, act, flags, out, z1_save, ws,
                      ws_bytes, stream, nullptr);
}

int osdp_split_mlp_bwd(const void *dy, const void *x, const void *w_flat, int64_t off_w1, const float *b1,
                       int64_t off_w2, const void *z1_saved, int64_t M, int64_t hidden, int64_t ffn, int k_split,
                       int act, void *dx, void *dw_flat, int64_t dw_off_w1, int64_t dw_off_w2, int dw_dtype,
                       int flags, float *db1, float *db2, void *ws, size_t ws_bytes, void *stream) {
  return mlp_bwd_impl(dy, x, w_flat, off_w1, b1, off_w2, z1_saved, M, hidden, ffn, k_split, act, dx, dw_flat,
                      dw_off_w1, dw_off_w2, dw_dtype, flags, db1, db2, ws, ws_bytes, stream, nullptr);
}

int osdp_zdp_mlp_fwd_slice(const void *x, const void *w1_slice, const void *w2_slice, int64_t ld_w2, const float *b1,
                           const float *b2, int64_t M, int64_t hidden, int64_t ffn, int k_split, int act, int flags,
                           int slice_idx, void *out, void *z1_save, void *ws, size_t ws_bytes, void *stream) {
  if (!w1_slice || !w2_slice) return OSDP_ERR_NULL_POINTER;
  if (ld_w2 <= 0 || (ld_w2 & 7)) return ld_w2 <= 0 ? OSDP_ERR_BAD_SHAPE : OSDP_ERR_ALIGNMENT;
  if (!aligned16(w1_slice) || !aligned16(w2_slice)) return OSDP_ERR_ALIGNMENT;
  MlpSlice cs;
  memset(&cs, 0, sizeof(cs));
  cs.idx = slice_idx; cs.w1 = w1_slice; cs.w2 = w2_slice; cs.ld_w2 = ld_w2;
  return mlp_fwd_impl(x, w1_slice, 0, b1, 0, b2, M, hidden, ffn, k_split, act, flags, out, z1_save, ws, ws_bytes,
                      stream, &cs);
}

int osdp_zdp_mlp_bwd_slice(const void *dy, const void *x, const void *w1_slice, const void *w2_slice, int64_t ld_w2,
                           const float *b1, const void *z1_saved, int64_t M, int64_t hidden, int64_t ffn,
                           int k_split, int act, int slice_idx, void *dx, void *dw1_slice, void *dw2_slice,
                           int64_t ld_dw2, void *const *dw1_peers, void *const *dw2_peers, int world, int dw_dtype,
                           int flags, float *db1, float *db2, void *ws, size_t ws_bytes, void *stream) {
  if (!w1_slice || !w2_slice) return OSDP_ERR_NULL_POINTER;
  if (ld_w2 <= 0 || (ld_w2 & 7)) return ld_w2 <= 0 ? OSDP_ERR_BAD_SHAPE : OSDP_ERR_ALIGNMENT;
  if (!aligned16(w1_slice) || !aligned16(w2_slice) || !aligned16(dw1_slice) || !aligned16(dw2_slice))
    return OSDP_ERR_ALIGNMENT;
  const bool scatter = dw1_peers || dw2_peers;
  if (scatter && (!dw1_peers || !dw2_peers)) return OSDP_ERR_NULL_POINTER;
  if (scatter && (world < 1 || world > 8 || (flags & OSDP_FLAG_ACCUMULATE_DW))) return OSDP_ERR_UNSUPPORTED;
  const bool want_dw = scatter || (dw1_slice && dw2_slice);
  if (!scatter && ((dw1_slice != nullptr) != (dw2_slice != nullptr))) return OSDP_ERR_NULL_POINTER;
  if (want_dw && !scatter && (ld_dw2 <= 0 || (ld_dw2 & 7))) return ld_dw2 <= 0 ? OSDP_ERR_BAD_SHAPE : OSDP_ERR_ALIGNMENT;
  MlpSlice cs;
  memset(&cs, 0, sizeof(cs));
  cs.idx = slice_idx; cs.w1 = w1_slice; cs.w2 = w2_slice; cs.ld_w2 = ld_w2;
  cs.dw1 = dw1_slice; cs.dw2 = dw2_slice; cs.ld_dw2 = ld_dw2;
  cs.dw1_peers = dw1_peers; cs.dw2_peers = dw2_peers; cs.world = world;
  if (scatter) {   // the compact dW2_s is [hidden, len F_s]: its leading dimension is the slice length
    int64_t b = 0, e = 0;
    int rc = osdp_slice_range(ffn, k_split, slice_idx, &b, &e);
    if (rc) return rc;
    cs.ld_dw2 = e - b;
  }
  // dw_flat only says whether weight gradients are wanted; the slice's own matrices are in `cs`
  return mlp_bwd_impl(dy, x, w1_slice, 0, b1, 0, z1_saved, M, hidden, ffn, k_split, act, dx,
                      want_dw ? const_cast<void *>(w1_slice) : nullptr, 0, 0, dw_dtype, flags, db1, db2, ws, ws_bytes,
                      stream, &cs);
}

int osdp_debug_wait_probe(void *ws, int64_t limit_us, void *stream_) {
  if (!ws) return OSDP_ERR_NULL_POINTER;
  if (limit_us < 1 || limit_us > 1000000) return OSDP_ERR_BAD_SHAPE;
  wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream_)>>>(static_cast<int *>(ws),
                                                                    (unsigned long long)limit_us * 1000ull);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  return OSDP_OK;
}

int osdp_read_device_status(void *ws, int *status, void *stream_) {
  if (!ws || !status) return OSDP_ERR_NULL_POINTER;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(e);
  if (word != 0) {
    e = cudaMemsetAsync(ws, 0, sizeof(int), stream);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  *status = (word == 0) ? OSDP_OK : OSDP_ERR_DEVICE_TIMEOUT;
  return OSDP_OK;
}

}  // extern "C"


// ================================================================================================
// Bias gradient without any allocation.
//
// Some callers cannot hand this library a workspace because they cannot allocate device memory
// at the point of the call: code running inside a memory-pool or allocator callback, a plug-in
// whose host framework owns every byte of the device and forbids cudaMalloc after start-up, or a
// real-time loop that must not take the allocator's lock.  For them this entry point computes the
// bias gradient db[n] = sum_m dY[m,n] with the partial sums kept in an array that is part of the
// library image itself.

namespace {

// Scratch for the two-pass column sum: ceil(M/1024) x N fp32 partials.  4 MiB, reserved on every
// GPU that loads this library for as long as the process lives.
__device__ __align__(256) float g_noalloc_partials[OSDP_NOALLOC_MAX_PARTIALS];

// In host code `g_noalloc_partials` is only a handle for the runtime, not a device address:
// the address a kernel may use is looked up per device, once, with that device current.
std::atomic<float *> g_noalloc_ptr[64];

int noalloc_scratch(float **ptr) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return cuda_fail(cudaErrorInvalidDevice);
  float *dp = g_noalloc_ptr[dev].load(std::memory_order_acquire);
  if (!dp) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_partials);   // with device `dev` current
    if (e != cudaSuccess) return cuda_fail(e);
    if (!p) return cuda_fail(cudaErrorInvalidSymbol);
    dp = static_cast<float *>(p);
    g_noalloc_ptr[dev].store(dp, std::memory_order_release);
  }
  *ptr = dp;
  return OSDP_OK;
}

}  // namespace

extern "C" int osdp_bias_grad_noalloc(const void *dy, int64_t M, int64_t N, float *dbias, void *stream) {
  if (!dy || !dbias) return OSDP_ERR_NULL_POINTER;
  if (M <= 0 || N <= 0 || M > ((int64_t)1 << 30) || N > ((int64_t)1 << 30)) return OSDP_ERR_BAD_SHAPE;
  if (N & 7) return OSDP_ERR_ALIGNMENT;
  if (!aligned16(dy) || !aligned16(dbias)) return OSDP_ERR_ALIGNMENT;
  const int64_t chunks = cdiv(M, COLSUM_ROWS_PER_CHUNK);
  // the chunk count is also a grid dimension of the first pass (at most 65535)
  if (chunks > 65535 || chunks * N > (int64_t)OSDP_NOALLOC_MAX_PARTIALS) return OSDP_ERR_EXCEEDS_STATIC_SCRATCH;
  float *partials = nullptr;
  int rc = noalloc_scratch(&partials);   // first call on a device: looks the address up
  if (rc) return rc;
  // Every partial that the second pass reads is written by the first pass of the same call, so
  // nothing left in the array by an earlier call can reach the result and nothing needs clearing.
  return launch_colsum(dy, N, M, 0, (int)N, partials, dbias, static_cast<cudaStream_t>(stream));
}
