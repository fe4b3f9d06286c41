// Persistent, warp-specialised bf16 GEMM for sm_100a: TMA -> shared-memory ring -> tcgen05.mma
// with fp32 accumulators in tensor memory -> fused epilogue.  One CTA per SM.
//
// It computes, for a range of slices of the operator (Section 3.3 of the paper: partition,
// process the slices one after another, combine), tiles of  OUT[P,Q] = A[P,R] * B[Q,R]^T  where
// the slice cuts either the output columns, the output rows, or the reduction dimension R:
//   MODE_COLS / MODE_ROWS : slices write disjoint parts of OUT (concatenation); the tile list is
//                           walked in slice-major order, no dependence between slices.
//   MODE_RED              : every slice contributes to every tile (sum over slices); each CTA owns
//                           a fixed set of tiles and walks slices in the outer loop, carrying the
//                           fp32 partial sum of a tile through global memory between slices.  The
//                           same thread writes and later re-reads a carry element, so no
//                           cross-CTA synchronisation exists anywhere in this kernel.
// Both operands may be K-major (reduction contiguous) or MN-major (output dim contiguous); the three
// GEMMs of a linear layer need (K,K) forward, (K,MN) dX and (MN,MN) dW.
//
// Warp roles (256 threads): warp 0 TMA producer, warp 1 MMA issuer, warp 2 TMEM allocator,
// warps 4-7 epilogue (warp w reads TMEM lanes 32*(w%4) ...).  Two TMEM accumulators so that the
// epilogue of tile i overlaps the main loop of tile i+1.
// Every mbarrier wait is bounded in time; on expiry the CTA records a status code and unwinds.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace osdp {

constexpr int BM = 128;       // tile rows  (UMMA M, cta_group::1)
constexpr int BK = 64;        // reduction elements per pipeline stage (one 128-byte swizzle span)
constexpr int UMMA_K = 16;    // reduction elements per tcgen05.mma (bf16)
constexpr int NUM_THREADS = 256;
constexpr int GROUP_M = 16;   // tile rasterisation: tiles of 16 tile-rows share operand tiles in L2
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s per wait

enum : int { MODE_NONE = 0, MODE_COLS = 1, MODE_ROWS = 2, MODE_RED = 3 };
enum : int { ACT_NONE = 0, ACT_GELU_TANH = 1, ACT_GELU_ERF = 2 };
enum : int { STATUS_TIMEOUT_PRODUCER = 101, STATUS_TIMEOUT_MMA = 102, STATUS_TIMEOUT_EPILOGUE = 103 };

struct Epilogue {
  void *out;                 // [P,Q] final output (bf16 or fp32)
  long long ld_out;
  int out_fp32;
  int accumulate;            // out += instead of out =
  float *carry;              // [P,Q] fp32 running sum for MODE_RED (unused otherwise)
  long long ld_carry;
  const float *bias;         // [Q] or null; added when the tile is finalised
  __nv_bfloat16 *z_save;     // [P,Q] or null; pre-activation written when finalised
  long long ld_z;
  int act;                   // activation applied when finalised
  const __nv_bfloat16 *gz;   // [P,Q] or null: multiply the result by act'(gz) (activation backward)
  long long ld_gz;
  int gz_act;
  __nv_bfloat16 *act_out;    // [P,Q] or null: also write act(gz) here
  long long ld_act_out;
  float scale;               // the accumulator is multiplied by this before anything else (fp8 operands' scales)
};

struct GemmParams {
  CUtensorMap a_main, a_tail, b_main, b_tail;   // 3-D maps: slices 0..k-2 / the last slice
  int P, Q, R;               // output rows, output cols, reduction extent (whole operator)
  int mode;                  // which dimension the slices cut
  int L;                     // slice length in that dimension
  int k_total;               // number of slices of the operator
  int s_begin, s_end;        // slices processed by this launch
  int a_sc_mul, b_sc_mul;    // 1: the operand map has a slice coordinate; 0: the operand is one slice already
  // Output-side maps (3-D, same slice-coordinate scheme): final output, saved pre-activation, fp32 carry.
  CUtensorMap out_main, out_tail, z_main, z_tail, carry_map;
  // The fp32 carry of a summed output belongs to this kernel alone (written by slice s, read by slice s + 1 of the
  // same tile), so it is not kept as an [P, Q] matrix but box by box: box (rb, cb) = rows 32 rb .., columns 32 cb ..
  // is one contiguous 4 KB block at index rb * carry_cb + cb, and a warp's boxes of a tile are adjacent (whole
  // DRAM pages instead of 128-byte row segments 4 Q bytes apart).  carry_map: a [boxes * 32, 32] matrix, box 32 x 32.
  CUtensorMap carry_pf_map;  // the same memory, box of (tile width / 32) * 32 rows: a warp's boxes of a tile, for L2 prefetch
  CUtensorMap out32_map, z32_map;   // bf16 out / second bf16 output (z_save, act_out) as unswizzled boxes of 32 x 32:
                                    // the last slice of a summed output and the epilogue that reads gz
  CUtensorMap gz32_map;             // the element-wise second input gz, same boxes
  CUtensorMap gz_pf_map;            // gz as boxes of 32 rows x BN columns, for L2 prefetch
  // Output scattered over the ranks of a data-parallel group (a weight-gradient slice reduce-scattered by the
  // epilogue itself): rank q owns rows [q * rows_per_peer, (q + 1) * rows_per_peer) of the slice's compact
  // matrix; peer_out[q] maps that block in rank q's memory (its own, or a peer-mapped address) and every box
  // is reduce-added there.  n_peers = 0: not used.
  CUtensorMap peer_out[8];
  int n_peers, rows_per_peer;
  int out_sc_mul;
  int red_group;             // MODE_RED: slices whose products a tile accumulates in one pass (1, or 2 = adjacent pairs)
  int round_kblocks;         // k-blocks per barrier round of the operand ring that the launch asks for (1 or 2)
  int carry_cb;              // fp32 carry: boxes of 32 columns per row block (the carry is stored box by box, see carry_map)
  int carry_bf16;            // MODE_RED: the running sum is kept in `out` itself, in bf16 (no fp32 carry buffer)
  int tma_epilogue;          // 1: outputs leave through shared-memory staging + TMA; 0: direct stores
  int bk;                    // reduction elements per k-block: 128 / (bytes per operand element)
  Epilogue epi;
  int *status;               // device status word or null
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the CTA is unwinding (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          int *status, int code, unsigned long long limit_ns = WAIT_LIMIT_NS) {
  if (mbar_try_wait(bar, parity)) return true;
  uint32_t polls = 0;
  unsigned long long t0 = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++polls & 255u) == 0u) {
      if (*abort_flag) return false;
      unsigned long long now = globaltimer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit_ns) {
        *abort_flag = 1;
        if (status) atomicCAS(status, 0, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap *m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// Shared -> global tensor store / reduce-add; completion is tracked in bulk async-groups of the issuing thread.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
// Asks the memory system to bring a box of a tensor into L2 (no shared-memory destination, no completion).
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap *map, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float4 ld_shared_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
// ---- CTA-pair (cluster of 2) forms.  The pair shares one MMA: the even CTA (rank 0) issues it.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// Both CTAs of the pair load into their own shared memory; the bytes are counted on the
// barrier of the even CTA (the barrier address with the pair bit cleared).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0,
                                                 int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar & 0xFEFFFFFFu), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t cta_rank) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
      "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}"
      ::"r"(bar), "r"(cta_rank)
      : "memory");
}
template <bool CTA2>
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  if (CTA2)
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
  else
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
}
template <bool CTA2>
__device__ __forceinline__ void tmem_relinquish() {
  if (CTA2) asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  else asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
template <bool CTA2>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  if (CTA2) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
  else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
template <bool CTA2>
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                        uint32_t accumulate) {
  if (CTA2)
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// COLL: use of the tensor core's collector buffer for the A operand.  0: none.  1: this MMA leaves its A operand in
// the buffer (fill); 2: this MMA takes A from the buffer, for the last time (lastuse).  The 256 x 512 tile issues two
// MMAs per k-step that share A (one per 256-column group): the second does not read A from shared memory again.
// Same bits; measured on B200 in the power-capped state: -0.1 ... -0.3 % per step at the benchmark shape.
template <bool CTA2, int COLL = 0>
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  if (CTA2 && COLL == 1)
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16.collector::a::fill [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  else if (CTA2 && COLL == 2)
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16.collector::a::lastuse [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  else if (CTA2)
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// mbarrier arrives once every tcgen05.mma issued so far by this thread has completed; in the
// pair form the arrival is delivered to the same barrier in both CTAs.
template <bool CTA2>
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  if (CTA2) {
    const uint16_t mask = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(mask)
        : "memory");
  } else {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
  }
}
__device__ __forceinline__ void tmem_ld_x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// Accumulator values times the product of the operands' scales (1 for bf16 operands: exact, skipped).
__device__ __forceinline__ void scale_acc(uint32_t (&v)[32], float scale) {
  if (scale != 1.0f) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * scale);
  }
}

// ------------------------------------------------------------------------------------------------
// Descriptors

// Shared-memory matrix descriptor, 128-byte swizzle, version 1 (sm_100).
//  K-major tile  [rows][64 bf16]: rows are 128 B apart, groups of 8 rows 1024 B apart (SBO).
//  MN-major tile [chunks of 64 MN][64 k-rows of 128 B]: 8 k-rows = 1024 B (SBO), MN chunks
//  8192 B apart (LBO).
// EB = bytes per operand element (2: bf16, 1: fp8 e4m3).  A stage always holds 128 bytes of the
// contiguous dimension per row, i.e. 128 / EB elements: 64 bf16 or 128 fp8 of the reduction for a K-major
// tile (one k-block), 64 or 128 output rows/columns per chunk for an MN-major one; a k-block is
// 128 / EB reduction elements, one tcgen05.mma covers 32 / EB of them (32 bytes of a K-major row).
template <bool MN_MAJOR, int EB = 2>
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  constexpr uint64_t lbo = MN_MAJOR ? (uint64_t)(((128 / EB) * 128) >> 4) : 1ull;
  constexpr uint64_t sbo = 1024 >> 4;
  uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= lbo << 16;
  d |= sbo << 32;
  d |= 1ull << 46;   // descriptor version
  d |= 2ull << 61;   // SWIZZLE_128B
  return d;
}
// Bytes the start address moves per UMMA_K step inside a stage.
template <bool MN_MAJOR, int EB = 2>
__device__ __forceinline__ constexpr uint32_t desc_k_advance() {
  return MN_MAJOR ? ((32 / EB) * 128) : 32;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = BN.
// (operand format field: 1 = bf16 under kind::f16, 0 = e4m3 under kind::f8f6f4; accumulator fp32)
template <int UM, int BN, bool A_MN, bool B_MN, int EB = 2>
__device__ __forceinline__ constexpr uint32_t make_idesc() {
  return (1u << 4) | ((EB == 2 ? 1u : 0u) << 7) | ((EB == 2 ? 1u : 0u) << 10) | ((A_MN ? 1u : 0u) << 15) |
         ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(UM >> 4) << 24);
}

template <int BN, bool CTA2, bool HEAVY = false>
struct SmemLayout {
  static constexpr int BNL = CTA2 ? BN / 2 : BN;   // B rows held by one CTA (a pair splits B between its CTAs)
  // A pair's tile is made of NG column groups of 256 (one tcgen05.mma each per k-step, sharing A);
  // of each group a CTA holds GB_ROWS rows of B.
  static constexpr int NG = (CTA2 && BN > 256) ? BN / 256 : 1;
  static constexpr int GB_ROWS = CTA2 ? BNL / NG : BN;
  static constexpr int UMMA_N = BN / NG;
  // Accumulator sets in tensor memory (512 columns in all): two, so that the epilogue of a tile
  // overlaps the next tile's main loop, unless one tile already needs all 512 columns.
  static constexpr int NBUF = (BN > 256) ? 1 : 2;
  // With a single accumulator set the epilogue is exposed: eight warps drain it (two per TMEM lane
  // quarter, half of the columns each) instead of four.  HEAVY: the same eight warps for epilogues
  // with a transcendental per element (activation, activation backward), which four warps, one per
  // scheduler, cannot finish within a short main loop.
  static constexpr int EPI_WARPS = (BN > 256 || HEAVY) ? 8 : 4;
  static constexpr int THREADS = 128 + 32 * EPI_WARPS;
  static constexpr int A_BYTES = BM * 128;    // 128 bytes of the contiguous dimension per row, whatever the type
  static constexpr int B_BYTES = BNL * 128;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  // Epilogue staging: STG_BUFS boxes of 4 KB per epilogue warp (boxes in flight to/from global memory).
  static constexpr int STG_BUFS = (BN > 256 || HEAVY) ? 1 : 2;
  static constexpr int STG_BYTES = EPI_WARPS * STG_BUFS * 4096;
  static constexpr int RING_BYTES = 229376 - STG_BYTES;
  static constexpr int STAGES = (RING_BYTES / STAGE_BYTES) > 8 ? 8 : (RING_BYTES / STAGE_BYTES);
  // Stages are handed from the producer to the MMA thread, and back, UNIT at a time (one barrier round per UNIT
  // k-blocks).  The thread that issues the tcgen05.mma instructions is the pace-setter of the main loop: an
  // instruction occupies it for about as long as the tensor pipe works on it, so every other instruction it
  // executes per round (barrier poll, fence, commit: about 100 cycles that cannot be hidden behind the last MMA)
  // is time the pipe idles.  Measured on B200 with time stamps in the MMA thread: a k-block of the 256 x 256 pair
  // tile takes 512 cycles of tensor work; 546-566 with no barrier traffic at all, 630-675 with one round per
  // k-block, 570-610 with one round per two k-blocks.  With six or more stages two k-blocks share a round (the ring still has three or four rounds in
  // flight); the rings with four stages keep one k-block per round (two rounds in flight would not cover the
  // latency of the copies).
  // Launches whose epilogue moves a running sum through the same path to the L2 keep one k-block per round
  // (finer refill of the ring: measured +5 % with two), so the launch chooses; UNIT is the most a variant allows.
  static constexpr int UNIT = (STAGES >= 6) ? 2 : 1;
  static constexpr int STG_OFFSET = STAGES * STAGE_BYTES;
  static constexpr int BAR_OFFSET = STG_OFFSET + STG_BYTES;
  static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;   // barriers + alignment slack
  static constexpr int TMEM_COLS = NBUF * BN;
};

// ------------------------------------------------------------------------------------------------
// Tile schedule (identical in every warp role)

struct Work {
  int s;                     // slice (MODE_RED with pairing: the first slice of the pair)
  int s_count;               // slices accumulated in this pass (1, or 2 under MODE_RED pairing)
  int row0, row_end;         // output rows of the tile, clipped extent of the slice
  int col0, col_end;
  int kblocks;               // reduction blocks of this slice
  int a_row, b_col;          // TMA coordinates (slice-relative where that dimension is sliced)
  int carry_in, carry_out;
  int first_of_slice;        // MODE_RED: this CTA's first tile of slice s
};

__device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// TM x BN is the tile of one scheduling unit (a CTA, or a CTA pair); bid / G are the unit's index
// and the number of units in the grid.
template <int TM, int BN>
__device__ __forceinline__ bool get_work(const GemmParams &p, int i, int bid, int G, Work &w) {
  const int nsl = p.s_end - p.s_begin;
  int s, t, rows, cols;
  if (p.mode == MODE_RED) {
    const int tiles = ceil_div(p.P, TM) * ceil_div(p.Q, BN);
    if (bid >= tiles) return false;
    const int n_my = (tiles - bid + G - 1) / G;
    const int grp = p.red_group > 1 ? p.red_group : 1;
    const int srel = i / n_my;
    if (srel >= ceil_div(nsl, grp)) return false;
    s = p.s_begin + srel * grp;
    w.s_count = min(grp, p.s_end - s);
    t = bid + (i - srel * n_my) * G;
    rows = p.P;
    cols = p.Q;
    w.first_of_slice = (i == srel * n_my);
  } else {
    w.first_of_slice = 0;
    w.s_count = 1;
    const int rows_full = (p.mode == MODE_ROWS) ? p.L : p.P;
    const int cols_full = (p.mode == MODE_COLS) ? p.L : p.Q;
    const int t_full = ceil_div(rows_full, TM) * ceil_div(cols_full, BN);
    const long long widx = (long long)bid + (long long)i * G;
    long long srel = widx / t_full;
    if (srel > nsl - 1) srel = nsl - 1;
    s = p.s_begin + (int)srel;
    const long long tl = widx - srel * t_full;
    rows = (p.mode == MODE_ROWS) ? min(p.L, p.P - s * p.L) : p.P;
    cols = (p.mode == MODE_COLS) ? min(p.L, p.Q - s * p.L) : p.Q;
    if (tl >= (long long)ceil_div(rows, TM) * ceil_div(cols, BN)) return false;
    t = (int)tl;
  }
  const int tiles_m = ceil_div(rows, TM), tiles_n = ceil_div(cols, BN);
  constexpr int GM = GROUP_M * BM / TM;   // same number of rows per group whatever the unit
  const int group = GM * tiles_n;
  const int g = t / group;
  const int first_m = g * GM;
  const int gm = min(GM, tiles_m - first_m);
  const int tm = first_m + (t - g * group) % gm;
  const int tn = (t - g * group) / gm;
  const int row_base = (p.mode == MODE_ROWS) ? s * p.L : 0;
  const int col_base = (p.mode == MODE_COLS) ? s * p.L : 0;
  w.s = s;
  w.a_row = tm * TM;
  w.b_col = tn * BN;
  w.row0 = row_base + w.a_row;
  w.col0 = col_base + w.b_col;
  w.row_end = row_base + rows;
  w.col_end = col_base + cols;
  if (p.mode == MODE_RED) {
    w.kblocks = 0;
    for (int ss = s; ss < s + w.s_count; ++ss) w.kblocks += ceil_div(min(p.L, p.R - ss * p.L), p.bk);
  } else {
    w.kblocks = ceil_div(p.R, p.bk);
  }
  w.carry_in = (p.mode == MODE_RED) && !p.carry_bf16 && (s > 0);
  w.carry_out = (p.mode == MODE_RED) && !p.carry_bf16 && (s + w.s_count - 1 < p.k_total - 1);
  return true;
}

// ------------------------------------------------------------------------------------------------
// Epilogue arithmetic on 8 consecutive columns of one row

// tanh on the special-function unit (tanh.approx.f32: about 2^-11 relative error, far inside the bf16
// rounding of everything that is computed from it here); the library call costs tens of instructions.
__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float gelu_f(float x, int act) {
  if (act == ACT_GELU_TANH) {
    const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
    return 0.5f * x * (1.0f + tanh_fast(u));
  }
  if (act == ACT_GELU_ERF) return 0.5f * x * (1.0f + erff(x * 0.7071067811865476f));
  return x;
}
__device__ __forceinline__ float gelu_grad_f(float x, int act) {
  if (act == ACT_GELU_TANH) {
    const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
    const float t = tanh_fast(u);
    const float du = 0.7978845608028654f * (1.0f + 0.134145f * x * x);
    return 0.5f * (1.0f + t) + 0.5f * x * (1.0f - t * t) * du;
  }
  if (act == ACT_GELU_ERF) {
    const float Phi = 0.5f * (1.0f + erff(x * 0.7071067811865476f));
    const float phi = 0.3989422804014327f * __expf(-0.5f * x * x);
    return Phi + x * phi;
  }
  return 1.0f;
}
// act'(x) and act(x) together (they share the transcendental)
__device__ __forceinline__ void gelu_grad_and_value_f(float x, int act, float &grad, float &value) {
  if (act == ACT_GELU_TANH) {
    const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
    const float t = tanh_fast(u);
    const float du = 0.7978845608028654f * (1.0f + 0.134145f * x * x);
    const float h = 0.5f * (1.0f + t);
    grad = h + 0.5f * x * (1.0f - t * t) * du;
    value = x * h;
    return;
  }
  if (act == ACT_GELU_ERF) {
    const float Phi = 0.5f * (1.0f + erff(x * 0.7071067811865476f));
    const float phi = 0.3989422804014327f * __expf(-0.5f * x * x);
    grad = Phi + x * phi;
    value = x * Phi;
    return;
  }
  grad = 1.0f;
  value = x;
}
// The same over small arrays, with the choice of the activation outside the element loop: the loop body is
// then straight-line code whose N independent chains the compiler interleaves (with the choice inside, every
// element was a branchy sequence executed one after another: about 180 cycles per element).
template <int N>
__device__ __forceinline__ void gelu_array(float (&f)[N], int act) {
  if (act == ACT_GELU_TANH) {
#pragma unroll
    for (int j = 0; j < N; ++j) f[j] = gelu_f(f[j], ACT_GELU_TANH);
  } else if (act == ACT_GELU_ERF) {
#pragma unroll
    for (int j = 0; j < N; ++j) f[j] = gelu_f(f[j], ACT_GELU_ERF);
  }
}
template <int N>
__device__ __forceinline__ void gelu_grad_array(const float (&x)[N], float (&grad)[N], int act) {
  if (act == ACT_GELU_TANH) {
#pragma unroll
    for (int j = 0; j < N; ++j) grad[j] = gelu_grad_f(x[j], ACT_GELU_TANH);
  } else if (act == ACT_GELU_ERF) {
#pragma unroll
    for (int j = 0; j < N; ++j) grad[j] = gelu_grad_f(x[j], ACT_GELU_ERF);
  } else {
#pragma unroll
    for (int j = 0; j < N; ++j) grad[j] = 1.0f;
  }
}
template <int N>
__device__ __forceinline__ void gelu_grad_and_value_array(float (&x)[N], float (&grad)[N], int act) {   // x <- act(x)
  if (act == ACT_GELU_TANH) {
#pragma unroll
    for (int j = 0; j < N; ++j) gelu_grad_and_value_f(x[j], ACT_GELU_TANH, grad[j], x[j]);
  } else if (act == ACT_GELU_ERF) {
#pragma unroll
    for (int j = 0; j < N; ++j) gelu_grad_and_value_f(x[j], ACT_GELU_ERF, grad[j], x[j]);
  } else {
#pragma unroll
    for (int j = 0; j < N; ++j) grad[j] = 1.0f;
  }
}
__device__ __forceinline__ void unpack_bf16x8(const uint4 &u, float (&f)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    f[2 * j] = __uint_as_float(w[j] << 16);
    f[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint4 pack_bf16x8(const float (&f)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * j], f[2 * j + 1]);
    w[j] = *reinterpret_cast<uint32_t *>(&h);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void epilogue8(const Epilogue &e, long long row, int col, float (&f)[8],
                                          int carry_in, int carry_out) {
  if (carry_in) {
    const float4 *c = reinterpret_cast<const float4 *>(e.carry + row * e.ld_carry + col);
    const float4 c0 = c[0], c1 = c[1];
    f[0] += c0.x; f[1] += c0.y; f[2] += c0.z; f[3] += c0.w;
    f[4] += c1.x; f[5] += c1.y; f[6] += c1.z; f[7] += c1.w;
  }
  if (carry_out) {
    float4 *c = reinterpret_cast<float4 *>(e.carry + row * e.ld_carry + col);
    c[0] = make_float4(f[0], f[1], f[2], f[3]);
    c[1] = make_float4(f[4], f[5], f[6], f[7]);
    return;
  }
  if (e.bias) {
    const float4 b0 = *reinterpret_cast<const float4 *>(e.bias + col);
    const float4 b1 = *reinterpret_cast<const float4 *>(e.bias + col + 4);
    f[0] += b0.x; f[1] += b0.y; f[2] += b0.z; f[3] += b0.w;
    f[4] += b1.x; f[5] += b1.y; f[6] += b1.z; f[7] += b1.w;
  }
  if (e.z_save) *reinterpret_cast<uint4 *>(e.z_save + row * e.ld_z + col) = pack_bf16x8(f);
  gelu_array(f, e.act);
  if (e.gz) {
    float z[8];
    unpack_bf16x8(*reinterpret_cast<const uint4 *>(e.gz + row * e.ld_gz + col), z);
    float grad[8];
    gelu_grad_and_value_array(z, grad, e.gz_act);
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] *= grad[j];
    if (e.act_out) *reinterpret_cast<uint4 *>(e.act_out + row * e.ld_act_out + col) = pack_bf16x8(z);
  }
  if (e.out_fp32) {
    float4 *o = reinterpret_cast<float4 *>(reinterpret_cast<float *>(e.out) + row * e.ld_out + col);
    if (e.accumulate) {
      const float4 o0 = o[0], o1 = o[1];
      f[0] += o0.x; f[1] += o0.y; f[2] += o0.z; f[3] += o0.w;
      f[4] += o1.x; f[5] += o1.y; f[6] += o1.z; f[7] += o1.w;
    }
    o[0] = make_float4(f[0], f[1], f[2], f[3]);
    o[1] = make_float4(f[4], f[5], f[6], f[7]);
  } else {
    uint4 *o = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(e.out) + row * e.ld_out + col);
    if (e.accumulate) {
      float old[8];
      unpack_bf16x8(*o, old);
#pragma unroll
      for (int j = 0; j < 8; ++j) f[j] += old[j];
    }
    *o = pack_bf16x8(f);
  }
}

// ------------------------------------------------------------------------------------------------
// The kernel

// CTA2 = true: the scheduling unit is a cluster of two CTAs working on a 256 x BN tile with one
// tcgen05.mma.cta_group::2 issued by the even CTA.  Each CTA loads its own 128 rows of A and half
// of the B tile (BN/2 rows), holds the accumulator of its 128 rows in its own tensor memory and
// runs its own epilogue.  Per CTA a stage is 32 KB instead of 48 KB (6 stages instead of 4) and
// half as many B bytes cross from L2 to shared memory per flop.
template <int BN, bool A_MN, bool B_MN, bool CTA2, bool HEAVY = false, int EB = 2>
__global__ void __launch_bounds__((BN > 256 || HEAVY) ? 384 : 256, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
  using SL = SmemLayout<BN, CTA2, HEAVY>;
  constexpr int BKE = 128 / EB;   // reduction elements per k-block
  constexpr int CW = 128 / EB;    // output rows / columns per 128-byte chunk of an MN-major operand
  constexpr int TM = CTA2 ? 2 * BM : BM;
  constexpr int BNL = SL::BNL;
  const uint32_t rank = CTA2 ? cluster_ctarank() : 0u;
  const int bid = CTA2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int G = CTA2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

  const uint32_t bar_base = smem_base + SL::BAR_OFFSET;
  auto full_bar = [&](int st) { return bar_base + 8u * st; };
  auto empty_bar = [&](int st) { return bar_base + 8u * (SL::STAGES + st); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * SL::STAGES + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * SL::STAGES + 2 + b); };
  uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(smem_gen + SL::BAR_OFFSET + 8 * (2 * SL::STAGES + 4));
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int unit = (SL::UNIT > 1 && p.round_kblocks > 1) ? SL::UNIT : 1;   // k-blocks per barrier round
  const int groups = SL::STAGES / unit;                                     // rounds in the ring

  // Programmatic dependent launch: the next kernel on the stream may be scheduled as soon as this
  // grid's CTAs retire and may run its own prologue; it touches global memory only after its
  // griddepcontrol.wait (below), which returns once this grid has completed and flushed.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (threadIdx.x == 0) {
    for (int g = 0; g < SL::STAGES; ++g) {   // a launch uses the first STAGES / unit of them
      mbar_init(full_bar(g), 1);
      mbar_init(empty_bar(g), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), SL::EPI_WARPS * (CTA2 ? 2 : 1));
    }
    for (int b = 0; b < SL::EPI_WARPS * SL::STG_BUFS; ++b) mbar_init(bar_base + 8u * (2 * SL::STAGES + 5 + b), 1);   // carry prefetch
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&p.a_main);
    prefetch_tmap(&p.a_tail);
    prefetch_tmap(&p.b_main);
    prefetch_tmap(&p.b_tail);
    if (p.tma_epilogue) {
      prefetch_tmap(&p.out_main);
      prefetch_tmap(&p.out_tail);
      prefetch_tmap(&p.carry_map);
    }
  }
  if (warp == 2) {
    tmem_alloc<CTA2>(smem_u32(tmem_holder), SL::TMEM_COLS);
    tmem_relinquish<CTA2>();
  }
  tc_fence_before();
  __syncthreads();
  if (CTA2) cluster_sync_all();   // the peer's barriers exist before anything is signalled across the pair
  tc_fence_after();
  // Everything above touched only shared and tensor memory.  From here on the kernel reads and
  // writes global memory that an earlier kernel on the stream may have produced or may still read.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t tmem_base = *tmem_holder;

  // Which operand dimension the slice coordinate belongs to (fixed by mode and operand major).
  const bool a_sliced = (p.mode == MODE_ROWS) || (p.mode == MODE_RED);
  const bool b_sliced = (p.mode == MODE_COLS) || (p.mode == MODE_RED);
  const bool a_mid = A_MN ? (p.mode == MODE_ROWS) : (p.mode == MODE_RED);   // slice cuts A's contiguous dim
  const bool b_mid = B_MN ? (p.mode == MODE_COLS) : (p.mode == MODE_RED);

  // With both operands MN-major a stage takes four to six copies; two warps then walk the ring in
  // lock step (warp 0 arms the stage's barrier and loads A, warp 3 loads B) so that two threads issue
  // them in parallel.  Otherwise warp 0 does it all (measured: the split costs 1-2 % there).
  constexpr bool SPLIT_PRODUCER = A_MN && B_MN;
  if (warp == 0 || (SPLIT_PRODUCER && warp == 3)) {
    // ------------------------------------------------------------------ TMA producer(s)
    const bool load_a = (warp == 0);
    const bool load_b = SPLIT_PRODUCER ? (warp == 3) : true;
    int grp = 0, sub = 0, n_sub = 0;       // round of the ring being filled, k-block inside it, k-blocks it will hold
    uint32_t phase = 0;
    uint32_t armed = 0, armed_phase = 0;   // per-round bookkeeping for the unwind path
    bool ok = true;
    Work w;
    for (int i = 0; ok && get_work<TM, BN>(p, i, bid, G, w); ++i) {
      w.a_row += (int)rank * BM;            // this CTA's rows of the pair's tile
      w.b_col += (int)rank * SL::GB_ROWS * (CTA2 ? 1 : 0);   // ... and its half of each 256-column group of B
      int tile_left = w.kblocks;            // k-blocks of this tile still to load (a round never spans two tiles)
      for (int sl = 0; sl < w.s_count && ok; ++sl) {
      const int ss = w.s + sl;               // the slice whose operand boxes are loaded now
      const bool tail = (ss == p.k_total - 1);
      const CUtensorMap *amap = (a_sliced && !tail) ? &p.a_main : &p.a_tail;
      const CUtensorMap *bmap = (b_sliced && !tail) ? &p.b_main : &p.b_tail;
      const int a_sc = (a_sliced && !tail) ? ss * p.a_sc_mul : 0;
      const int b_sc = (b_sliced && !tail) ? ss * p.b_sc_mul : 0;
      const int nkb = (p.mode == MODE_RED) ? ceil_div(min(p.L, p.R - ss * p.L), BKE) : w.kblocks;
      for (int kb = 0; kb < nkb; ++kb) {
        if (sub == 0) {
          ok = mbar_wait(empty_bar(grp), phase ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_PRODUCER);
          if (!ok) break;
          n_sub = min(unit, tile_left);
          if (lane == 0 && load_a && (!CTA2 || rank == 0))
            mbar_expect_tx(full_bar(grp), (uint32_t)n_sub * SL::STAGE_BYTES * (CTA2 ? 2 : 1));
          armed |= 1u << grp;
          armed_phase = (armed_phase & ~(1u << grp)) | (phase << grp);
        }
        if (lane == 0) {
          const uint32_t sa = smem_base + (uint32_t)(grp * unit + sub) * SL::STAGE_BYTES;
          const uint32_t sb = sa + SL::A_BYTES;
          const uint32_t fb = full_bar(grp);
          const int kc = kb * BKE;
          auto tma_load = [&](uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2) {
            if (CTA2) tma_load_3d_pair(dst, map, fb, c0, c1, c2);
            else tma_load_3d(dst, map, fb, c0, c1, c2);
          };
          if (!load_a) {
          } else if (A_MN) {
#pragma unroll
            for (int j = 0; j < BM / CW; ++j) {
              const int in = w.a_row + j * CW;
              if (a_mid) tma_load(sa + j * (BKE * 128), amap, in, a_sc, kc);
              else tma_load(sa + j * (BKE * 128), amap, in, kc, a_sc);
            }
          } else {
            if (a_mid) tma_load(sa, amap, kc, a_sc, w.a_row);
            else tma_load(sa, amap, kc, w.a_row, a_sc);
          }
          if (!load_b) {
          } else if (B_MN) {
#pragma unroll
            for (int j = 0; j < (BNL + CW - 1) / CW; ++j) {
              constexpr int CPG = (SL::GB_ROWS + CW - 1) / CW;   // chunks per column group
              const int in = w.b_col + (j / CPG) * 256 + (j % CPG) * CW;
              if (b_mid) tma_load(sb + j * (BKE * 128), bmap, in, b_sc, kc);
              else tma_load(sb + j * (BKE * 128), bmap, in, kc, b_sc);
            }
          } else {
#pragma unroll
            for (int g = 0; g < SL::NG; ++g) {
              const int row = w.b_col + g * 256;
              if (b_mid) tma_load(sb + g * (SL::GB_ROWS * 128), bmap, kc, b_sc, row);
              else tma_load(sb + g * (SL::GB_ROWS * 128), bmap, kc, row, b_sc);
            }
          }
        }
        __syncwarp();
        --tile_left;
        if (++sub == n_sub) {
          sub = 0;
          if (++grp == groups) { grp = 0; phase ^= 1u; }
        }
      }
      }
    }
    if (!ok && rank == 0 && load_a) {
      // Unwinding: let the copies already issued land before the CTA's shared memory goes away.
      for (int st = 0; st < groups; ++st) {
        if (!((armed >> st) & 1u)) continue;
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try_wait(full_bar(st), (armed_phase >> st) & 1u)) {
          if (globaltimer_ns() - t0 > 2000000ull) break;   // 2 ms
        }
      }
    }
  } else if (warp == 1 && rank == 0) {
    // ------------------------------------------------------------------ MMA issuer (even CTA of a pair)
    // One thread runs the whole role: it waits for a round of the ring (UNIT k-blocks), issues their MMAs and
    // hands the round back with one commit.
    constexpr uint32_t idesc = make_idesc<TM, SL::UMMA_N, A_MN, B_MN, EB>();
    if (lane == 0) {
      int grp = 0;
      uint32_t phase = 0;
      bool ok = true;
      Work w;
      for (int i = 0; ok && get_work<TM, BN>(p, i, bid, G, w); ++i) {
        const int buf = i % SL::NBUF;
        const uint32_t bphase = (uint32_t)(i / SL::NBUF) & 1u;
        ok = mbar_wait(tempty_bar(buf), bphase ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA);
        if (!ok) break;
        tc_fence_after();   // the epilogue's tensor-memory loads of this accumulator set are complete
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int kb = 0; kb < w.kblocks; kb += unit) {
          const int n_sub = min(unit, w.kblocks - kb);
          ok = mbar_wait(full_bar(grp), phase, abort_flag, p.status, STATUS_TIMEOUT_MMA);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int sub = 0; sub < SL::UNIT; ++sub) {
            if (sub < n_sub) {
              const uint32_t sa = smem_base + (uint32_t)(grp * unit + sub) * SL::STAGE_BYTES;
              const uint32_t sb = sa + SL::A_BYTES;
              const uint64_t adesc = make_smem_desc<A_MN, EB>(sa);
              const uint64_t bdesc = make_smem_desc<B_MN, EB>(sb);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {   // four tcgen05.mma of 32 bytes of reduction each per k-block
#pragma unroll
                for (int g = 0; g < SL::NG; ++g) {
                  const uint32_t d = d_tmem + (uint32_t)(g * SL::UMMA_N);
                  const uint64_t ad = adesc + (uint64_t)((kk * desc_k_advance<A_MN, EB>()) >> 4);
                  const uint64_t bd = bdesc + (uint64_t)((g * SL::GB_ROWS * 128 + kk * desc_k_advance<B_MN, EB>()) >> 4);
                  const uint32_t acc = (kb + sub > 0 || kk > 0) ? 1u : 0u;
                  if (EB == 2 && SL::NG == 2 && g == 0) umma_bf16<CTA2, 1>(d, ad, bd, idesc, acc);
                  else if (EB == 2 && SL::NG == 2 && g == 1) umma_bf16<CTA2, 2>(d, ad, bd, idesc, acc);
                  else if (EB == 2) umma_bf16<CTA2>(d, ad, bd, idesc, acc);
                  else umma_f8<CTA2>(d, ad, bd, idesc, acc);
                }
              }
            }
          }
          umma_commit<CTA2>(empty_bar(grp));                               // frees the round when its MMAs retire
          if (kb + unit >= w.kblocks) umma_commit<CTA2>(tfull_bar(buf));   // accumulator complete
          if (++grp == groups) { grp = 0; phase ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue
    // Each warp owns 32 rows of the tile and two 4 KB staging buffers (32 rows x 128 bytes, 128-byte
    // swizzle).  Outputs leave as TMA stores (or reduce-adds) of 32 x 128-byte boxes, which the
    // tensor maps clip at the end of the matrix or of the slice.  The carry of a summed output:
    // slice 0 stores the fp32 partial, later slices reduce-add theirs into it (the addition is
    // done by the memory system, nothing is read back), the last slice prefetches the carry
    // with TMA loads, adds its own partial and writes the final result.
    const int quarter = warp & 3;
    const int wg = (warp - 4) >> 2;                 // which share of the tile's columns this warp drains
    constexpr int EG = SL::EPI_WARPS / 4;
    constexpr uint32_t NB = SL::STG_BUFS;
    const uint32_t stg = smem_base + SL::STG_OFFSET + (uint32_t)(warp - 4) * (NB * 4096u);
    const uint32_t row_off = (uint32_t)lane * 128u;
    const uint32_t swz = (uint32_t)(lane & 7);
    const bool out_sliced = (p.mode == MODE_COLS) || (p.mode == MODE_ROWS);
    const bool out_mid = (p.mode == MODE_COLS);
    // first row, in the carry's box-by-box layout, of the box that holds rows row .. row + 31, columns col .. col + 31
    auto carry_box = [&](int row, int col) { return ((row >> 5) * p.carry_cb + (col >> 5)) << 5; };
    uint32_t n_store = 0;   // staged boxes issued by this warp (selects the staging buffer)
    uint32_t n_cload = 0;   // carry boxes loaded by this warp
    bool ok = true;
    Work w;
    for (int i = 0; ok && get_work<TM, BN>(p, i, bid, G, w); ++i) {
      w.a_row += (int)rank * BM;
      w.row0 += (int)rank * BM;
      if (i == 0 && p.tma_epilogue && p.epi.gz && lane == 0)   // this CTA's first tile: while its main loop runs
        tma_prefetch_l2_3d(&p.gz_pf_map, w.b_col, w.a_row + quarter * 32, 0);
      const int buf = i % SL::NBUF;
      const uint32_t bphase = (uint32_t)(i / SL::NBUF) & 1u;
      ok = mbar_wait(tfull_bar(buf), bphase, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE);
      if (!ok) break;
      tc_fence_after();
      const int wrow0 = w.row0 + quarter * 32;
      const long long row = (long long)wrow0 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN);
      // Hands the accumulator set back to the MMA thread: at the end of the tile's epilogue, or, where one tile
      // fills the tensor memory (nothing else for the tensor pipe to do meanwhile), as soon as this warp's last
      // columns are in registers, so that converting and storing them overlaps the next tile's first k-blocks.
      bool released = false;
      auto release_accumulator = [&]() {
        if (released) return;
        released = true;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CTA2 && rank != 0) mbar_arrive_remote(tempty_bar(buf), 0);   // the even CTA's MMA thread waits on it
          else mbar_arrive(tempty_bar(buf));
        }
      };
      if (p.tma_epilogue && p.mode == MODE_RED && lane == 0) {
        // The carry of this CTA's next tile is touched one main loop from now: have it in L2 by then.
        Work nx;
        if (get_work<TM, BN>(p, i + 1, bid, G, nx) && nx.carry_in)
          tma_prefetch_l2_3d(&p.carry_pf_map, 0, carry_box(nx.row0 + (int)rank * BM + quarter * 32, nx.col0), 0);
      }
      if (p.tma_epilogue && p.epi.gz && lane == 0) {
        // likewise the next tile's rows of gz
        Work nx;
        if (get_work<TM, BN>(p, i + 1, bid, G, nx))
          tma_prefetch_l2_3d(&p.gz_pf_map, nx.b_col, nx.a_row + (int)rank * BM + quarter * 32, 0);
      }
      if (!p.tma_epilogue) {
        // direct stores from registers (used when the epilogue also reads a second tensor)
#pragma unroll 1
        for (int c = wg * (BN / 32 / EG); c < (wg + 1) * (BN / 32 / EG); ++c) {
          const int cbase = w.col0 + c * 32;
          if (cbase >= w.col_end) break;
          uint32_t v[32];
          tmem_ld_x32(taddr + (uint32_t)(c * 32), v);
          tmem_ld_wait();
          scale_acc(v, p.epi.scale);
          if (row < w.row_end) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const int col = cbase + g * 8;
              if (col < w.col_end) {
                float f[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[g * 8 + j]);
                epilogue8(p.epi, row, col, f, w.carry_in, w.carry_out);
              }
            }
          }
        }
      } else if (wrow0 < w.row_end) {
        const bool tail = (w.s == p.k_total - 1);
        const int sc = (out_sliced && !tail) ? w.s * p.out_sc_mul : 0;
        const CUtensorMap *omap = (out_sliced && !tail) ? &p.out_main : &p.out_tail;
        const CUtensorMap *zmap = (out_sliced && !tail) ? &p.z_main : &p.z_tail;
        const int r_in = w.a_row + quarter * 32;
        // One staged box: wait until the buffer's previous box has been read, fill it, hand it to TMA.
        auto stage_begin = [&]() -> uint32_t {
          if (lane == 0) bulk_wait_read<NB - 1>();
          __syncwarp();
          return stg + (n_store % NB) * 4096u;
        };
        auto stage_issue = [&](const CUtensorMap *map, uint32_t src, int col_in, bool reduce) {
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (p.n_peers > 0 && (map == &p.out_main || map == &p.out_tail)) {
              // the owner of this 32-row box (rows_per_peer is a multiple of 32, so a box has one owner)
              const int q = r_in / p.rows_per_peer;
              const int rl = r_in - q * p.rows_per_peer;
              if (out_mid) tma_reduce_add_3d(&p.peer_out[q], src, col_in, 0, rl);
              else tma_reduce_add_3d(&p.peer_out[q], src, col_in, rl, 0);
            } else if (out_mid && map != &p.carry_map) {
              if (reduce) tma_reduce_add_3d(map, src, col_in, sc, r_in);
              else tma_store_3d(map, src, col_in, sc, r_in);
            } else if (map == &p.carry_map) {
              if (reduce) tma_reduce_add_3d(map, src, 0, carry_box(r_in, col_in), 0);
              else tma_store_3d(map, src, 0, carry_box(r_in, col_in), 0);
            } else {
              if (reduce) tma_reduce_add_3d(map, src, col_in, r_in, sc);
              else tma_store_3d(map, src, col_in, r_in, sc);
            }
            bulk_commit();
          }
          ++n_store;
        };
        // bf16 running sum kept in the output itself: slice 0 stores, every later slice reduce-adds.
        const bool inplace_add = p.carry_bf16 && p.mode == MODE_RED && w.s > 0;
        const bool skip_bias = p.carry_bf16 && p.mode == MODE_RED && w.s > 0;   // bias enters once, with slice 0
        if (w.first_of_slice && (w.carry_in || inplace_add)) {
          // Slice boundary: everything this warp sent for the previous slice must have landed
          // before the same addresses are added to (or read) again.
          if (lane == 0) bulk_wait_all();
          __syncwarp();
        }
        if (w.carry_out) {
          // fp32 partial -> carry, 32 columns (128 bytes per row) per box
#pragma unroll 1
          for (int c = wg * (BN / 32 / EG); c < (wg + 1) * (BN / 32 / EG); ++c) {
            const int cbase = w.col0 + c * 32;
            if (cbase >= w.col_end) break;
            uint32_t v[32];
            tmem_ld_x32(taddr + (uint32_t)(c * 32), v);
            tmem_ld_wait();
            scale_acc(v, p.epi.scale);
            const uint32_t dst = stage_begin();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              st_shared_v4(dst + row_off + (((uint32_t)j ^ swz) << 4), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            stage_issue(&p.carry_map, dst, cbase, w.carry_in != 0);
          }
        } else if (w.carry_in) {
          // Last slice: carry + accumulator -> bias/act -> out.  The carry box of the next 32 columns is
          // fetched by TMA while this one is worked on; a box that has been read into registers is
          // overwritten in place with the bf16 results (64 bytes per row; z_save in its second half) and
          // leaves as a TMA store, so the buffer takes its next carry box once that store has read it.
          const uint32_t cbar = bar_base + 8u * (2 * SL::STAGES + 5 + (warp - 4) * NB);
          int nchunks = (w.col_end - w.col0 + 31) / 32;
          if (nchunks > BN / 32) nchunks = BN / 32;
          const int c_lo = wg * (BN / 32 / EG);                       // this warp's share of the columns
          const int c_hi = min((wg + 1) * (BN / 32 / EG), nchunks);
          const bool staged_out = !p.epi.out_fp32;
          auto issue_load = [&](int c) {
            if (lane == 0) {
              if (staged_out) bulk_wait_read<0>();   // the store that last left from this buffer
              const uint32_t b = n_cload % NB;
              mbar_expect_tx(cbar + 8u * b, 4096u);
              tma_load_3d(stg + b * 4096u, &p.carry_map, cbar + 8u * b, 0, carry_box(wrow0, w.col0 + c * 32), 0);
            }
            ++n_cload;
          };
          const uint32_t first = n_cload;
          if (lane == 0) bulk_wait_read<0>();
          __syncwarp();
          for (int c = c_lo; c < c_lo + (int)NB - 1 && c < c_hi; ++c) issue_load(c);
#pragma unroll 1
          for (int c = c_lo; c < c_hi; ++c) {
            if (c + (int)NB - 1 < c_hi) issue_load(c + (int)NB - 1);
            uint32_t v[32];
            tmem_ld_x32(taddr + (uint32_t)(c * 32), v);
            tmem_ld_wait();
            scale_acc(v, p.epi.scale);
            const uint32_t n = first + (uint32_t)(c - c_lo);
            ok = mbar_wait(cbar + 8u * (n % NB), (n / NB) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE);
            if (!ok) break;
            const uint32_t buf0 = stg + (n % NB) * 4096u;
            const uint32_t src = buf0 + row_off;
            const int cbase = w.col0 + c * 32;
            float f[32];
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const float4 cv = ld_shared_f4(src + (((uint32_t)g ^ swz) << 4));
              f[4 * g + 0] = __uint_as_float(v[4 * g + 0]) + cv.x;
              f[4 * g + 1] = __uint_as_float(v[4 * g + 1]) + cv.y;
              f[4 * g + 2] = __uint_as_float(v[4 * g + 2]) + cv.z;
              f[4 * g + 3] = __uint_as_float(v[4 * g + 3]) + cv.w;
            }
            if (!staged_out) {
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                const int col = cbase + g * 8;
                if (row < w.row_end && col < w.col_end) {
                  float e8[8];
#pragma unroll
                  for (int j = 0; j < 8; ++j) e8[j] = f[g * 8 + j];
                  epilogue8(p.epi, row, col, e8, 0, 0);
                }
              }
              __syncwarp();   // the buffer may be refilled once every lane has read it
              continue;
            }
            if (p.epi.bias) {
#pragma unroll
              for (int g = 0; g < 8; ++g) {
                if (cbase + g * 4 < w.col_end) {
                  const float4 b0 = *reinterpret_cast<const float4 *>(p.epi.bias + cbase + g * 4);
                  f[4 * g + 0] += b0.x; f[4 * g + 1] += b0.y; f[4 * g + 2] += b0.z; f[4 * g + 3] += b0.w;
                }
              }
            }
            __syncwarp();   // every lane has read its carry row: the box may now be overwritten
            if (p.epi.z_save) {
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                float e8[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) e8[j] = f[g * 8 + j];
                const uint4 pk = pack_bf16x8(e8);
                st_shared_v4(buf0 + 2048u + (uint32_t)lane * 64u + (uint32_t)g * 16u, pk.x, pk.y, pk.z, pk.w);
              }
            }
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              float e8[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) e8[j] = f[g * 8 + j];
              gelu_array(e8, p.epi.act);
              const uint4 pk = pack_bf16x8(e8);
              st_shared_v4(buf0 + (uint32_t)lane * 64u + (uint32_t)g * 16u, pk.x, pk.y, pk.z, pk.w);
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tma_store_3d(&p.out32_map, buf0, w.b_col + c * 32, r_in, 0);
              if (p.epi.z_save) tma_store_3d(&p.z32_map, buf0 + 2048u, w.b_col + c * 32, r_in, 0);
              bulk_commit();
            }
          }
          if (!ok) break;
        } else if (p.epi.gz) {
          // out = acc (.) act'(gz), act_out = act(gz): the gz box of the next 32 columns is fetched by TMA
          // while this one is worked on; the results overwrite the consumed box (act_out in the
          // buffer's second half) and leave as TMA stores.  Unsliced launches only.
          const uint32_t cbar = bar_base + 8u * (2 * SL::STAGES + 5 + (warp - 4) * NB);
          int nchunks = (w.col_end - w.col0 + 31) / 32;
          if (nchunks > BN / 32) nchunks = BN / 32;
          const int c_lo = wg * (BN / 32 / EG);                       // this warp's share of the columns
          const int c_hi = min((wg + 1) * (BN / 32 / EG), nchunks);
          auto issue_load = [&](int c) {
            if (lane == 0) {
              bulk_wait_read<0>();   // the stores that last left from this buffer
              const uint32_t b = n_cload % NB;
              mbar_expect_tx(cbar + 8u * b, 2048u);
              tma_load_3d(stg + b * 4096u, &p.gz32_map, cbar + 8u * b, w.b_col + c * 32, r_in, 0);
            }
            ++n_cload;
          };
          const uint32_t first = n_cload;
          for (int c = c_lo; c < c_lo + (int)NB - 1 && c < c_hi; ++c) issue_load(c);
#pragma unroll 1
          for (int c = c_lo; c < c_hi; ++c) {
            if (c + (int)NB - 1 < c_hi) issue_load(c + (int)NB - 1);
            uint32_t v[32];
            tmem_ld_x32(taddr + (uint32_t)(c * 32), v);
            tmem_ld_wait();
            scale_acc(v, p.epi.scale);
            const uint32_t n = first + (uint32_t)(c - c_lo);
            ok = mbar_wait(cbar + 8u * (n % NB), (n / NB) & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPILOGUE);
            if (!ok) break;
            const uint32_t buf0 = stg + (n % NB) * 4096u;
            const uint32_t mine = buf0 + (uint32_t)lane * 64u;
            float4 zq[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) zq[g] = ld_shared_f4(mine + (uint32_t)g * 16u);
            __syncwarp();   // every lane has read its row of gz: the box may now be overwritten
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              float z[8], f[8];
              uint4 zb;
              zb.x = __float_as_uint(zq[g].x); zb.y = __float_as_uint(zq[g].y);
              zb.z = __float_as_uint(zq[g].z); zb.w = __float_as_uint(zq[g].w);
              unpack_bf16x8(zb, z);
              gelu_grad_and_value_array(z, f, p.epi.gz_act);   // f = act'(z), z = act(z)
#pragma unroll
              for (int j = 0; j < 8; ++j) f[j] *= __uint_as_float(v[g * 8 + j]);
              const uint4 pk = pack_bf16x8(f);
              st_shared_v4(mine + (uint32_t)g * 16u, pk.x, pk.y, pk.z, pk.w);
              if (p.epi.act_out) {
                const uint4 pa = pack_bf16x8(z);
                st_shared_v4(mine + 2048u + (uint32_t)g * 16u, pa.x, pa.y, pa.z, pa.w);
              }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tma_store_3d(&p.out32_map, buf0, w.b_col + c * 32, r_in, 0);
              if (p.epi.act_out) tma_store_3d(&p.z32_map, buf0 + 2048u, w.b_col + c * 32, r_in, 0);
              bulk_commit();
            }
          }
          if (!ok) break;
        } else if (p.epi.out_fp32) {
          // fp32 output, 32 columns per box; += is a reduce-add
#pragma unroll 1
          for (int c = wg * (BN / 32 / EG); c < (wg + 1) * (BN / 32 / EG); ++c) {
            const int cbase = w.col0 + c * 32;
            if (cbase >= w.col_end) break;
            uint32_t v[32];
            tmem_ld_x32(taddr + (uint32_t)(c * 32), v);
            tmem_ld_wait();
            if (SL::NBUF == 1 && (c + 1 == (wg + 1) * (BN / 32 / EG) || cbase + 32 >= w.col_end)) release_accumulator();
            scale_acc(v, p.epi.scale);
            if (p.epi.bias) {
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                if (cbase + g * 8 < w.col_end) {
                  const float4 b0 = *reinterpret_cast<const float4 *>(p.epi.bias + cbase + g * 8);
                  const float4 b1 = *reinterpret_cast<const float4 *>(p.epi.bias + cbase + g * 8 + 4);
                  v[g * 8 + 0] = __float_as_uint(__uint_as_float(v[g * 8 + 0]) + b0.x);
                  v[g * 8 + 1] = __float_as_uint(__uint_as_float(v[g * 8 + 1]) + b0.y);
                  v[g * 8 + 2] = __float_as_uint(__uint_as_float(v[g * 8 + 2]) + b0.z);
                  v[g * 8 + 3] = __float_as_uint(__uint_as_float(v[g * 8 + 3]) + b0.w);
                  v[g * 8 + 4] = __float_as_uint(__uint_as_float(v[g * 8 + 4]) + b1.x);
                  v[g * 8 + 5] = __float_as_uint(__uint_as_float(v[g * 8 + 5]) + b1.y);
                  v[g * 8 + 6] = __float_as_uint(__uint_as_float(v[g * 8 + 6]) + b1.z);
                  v[g * 8 + 7] = __float_as_uint(__uint_as_float(v[g * 8 + 7]) + b1.w);
                }
              }
            }
            if (p.epi.act != ACT_NONE) {
              float a32[32];
#pragma unroll
              for (int j = 0; j < 32; ++j) a32[j] = __uint_as_float(v[j]);
              gelu_array(a32, p.epi.act);
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(a32[j]);
            }
            const uint32_t dst = stage_begin();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              st_shared_v4(dst + row_off + (((uint32_t)j ^ swz) << 4), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            stage_issue(omap, dst, w.b_col + c * 32, p.epi.accumulate != 0);
          }
        } else {
          // bf16 output, 64 columns (128 bytes per row) per box
#pragma unroll 1
          for (int c = wg * ((BN + 63) / 64 / EG); c < (wg + 1) * ((BN + 63) / 64 / EG); ++c) {
            const int cbase = w.col0 + c * 64;
            if (cbase >= w.col_end) break;
            uint32_t v[64];
            {
              uint32_t lo[32], hi[32];
              tmem_ld_x32(taddr + (uint32_t)(c * 64), lo);
              if (BN >= 64) tmem_ld_x32(taddr + (uint32_t)(c * 64 + 32), hi);
              tmem_ld_wait();
              if (SL::NBUF == 1 && (c + 1 == (wg + 1) * ((BN + 63) / 64 / EG) || cbase + 64 >= w.col_end)) release_accumulator();
              scale_acc(lo, p.epi.scale);
              if (BN >= 64) scale_acc(hi, p.epi.scale);
#pragma unroll
              for (int j = 0; j < 32; ++j) { v[j] = lo[j]; v[32 + j] = hi[j]; }
            }
            uint4 packed[8];
            if (p.epi.bias && !skip_bias) {
#pragma unroll
              for (int g = 0; g < 8; ++g) {
                if (cbase + g * 8 < w.col_end) {
                  const float4 b0 = *reinterpret_cast<const float4 *>(p.epi.bias + cbase + g * 8);
                  const float4 b1 = *reinterpret_cast<const float4 *>(p.epi.bias + cbase + g * 8 + 4);
                  v[g * 8 + 0] = __float_as_uint(__uint_as_float(v[g * 8 + 0]) + b0.x);
                  v[g * 8 + 1] = __float_as_uint(__uint_as_float(v[g * 8 + 1]) + b0.y);
                  v[g * 8 + 2] = __float_as_uint(__uint_as_float(v[g * 8 + 2]) + b0.z);
                  v[g * 8 + 3] = __float_as_uint(__uint_as_float(v[g * 8 + 3]) + b0.w);
                  v[g * 8 + 4] = __float_as_uint(__uint_as_float(v[g * 8 + 4]) + b1.x);
                  v[g * 8 + 5] = __float_as_uint(__uint_as_float(v[g * 8 + 5]) + b1.y);
                  v[g * 8 + 6] = __float_as_uint(__uint_as_float(v[g * 8 + 6]) + b1.z);
                  v[g * 8 + 7] = __float_as_uint(__uint_as_float(v[g * 8 + 7]) + b1.w);
                }
              }
            }
            if (p.epi.z_save) {
#pragma unroll
              for (int g = 0; g < 8; ++g) {
                float f[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[g * 8 + j]);
                packed[g] = pack_bf16x8(f);
              }
              const uint32_t dstz = stage_begin();
#pragma unroll
              for (int g = 0; g < 8; ++g)
                st_shared_v4(dstz + row_off + (((uint32_t)g ^ swz) << 4), packed[g].x, packed[g].y, packed[g].z, packed[g].w);
              stage_issue(zmap, dstz, w.b_col + c * 64, false);
            }
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              float f[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[g * 8 + j]);
              gelu_array(f, p.epi.act);
              packed[g] = pack_bf16x8(f);
            }
            const uint32_t dst = stage_begin();
#pragma unroll
            for (int g = 0; g < 8; ++g)
              st_shared_v4(dst + row_off + (((uint32_t)g ^ swz) << 4), packed[g].x, packed[g].y, packed[g].z, packed[g].w);
            stage_issue(omap, dst, w.b_col + c * 64, p.epi.accumulate != 0 || inplace_add);
          }
        }
      }
      release_accumulator();
    }
    // Nothing this warp handed to TMA may still be reading shared memory at exit.  (The writes themselves are
    // complete and visible when the grid is: waiting for them here would only put their latency in front of
    // the next kernel on the stream.)
    if (lane == 0) bulk_wait_read<0>();
    __syncwarp();
  }

  tc_fence_before();
  __syncthreads();
  if (CTA2) cluster_sync_all();   // neither CTA of a pair leaves while the other may still touch its memory
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc<CTA2>(tmem_base, SL::TMEM_COLS);
  }
}

// Diagnostic: one warp waits, with the same bounded wait the GEMM uses, on a barrier that nothing
// ever signals.  The wait gives up after limit_ns, records STATUS_TIMEOUT_PROBE and the kernel returns.
enum : int { STATUS_TIMEOUT_PROBE = 199 };
__global__ void wait_probe_kernel(int *status, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  mbar_wait(smem_u32(&bar), 0, &abort_flag, status, STATUS_TIMEOUT_PROBE, limit_ns);
}

}  // namespace osdp
