// hola_verify.cu - sm_100a kernels and C ABI for the entropy-aware verify step of Hierarchical Speculative
// Decoding (HSD section, Eq. 1, the HSD loop of Algorithm 1).  See include/hola_verify.h for the contract.
//
// Kernels
//   lm_head_entropy_kernel      persistent, warp-specialised weight-streaming GEMM run by pairs of CTAs (clusters of
//       two).  The vocabulary lies on the 128 tensor-memory lanes of each CTA, the verify positions on the N
//       dimension of the MMA:  D[v, r] = sum_h W_lm[v, h] * hidden[r, h].  A pair owns up to 256 vocabulary rows
//       per tile; each CTA streams its (up to 128) rows of W_lm and HALF of the hidden rows per K block with TMA, and one
//       thread of the leader CTA issues tcgen05.mma.cta_group::2 (bf16 x bf16 -> fp32 in tensor memory) that reads
//       both halves.  Sixteen epilogue warps copy finished accumulators to the fp32 logits buffer and, from the
//       same registers transposed through a small shared-memory buffer, keep per verify position the running
//       softmax statistics (m, s, t) = (max, sum e^(l-m), sum e^(l-m)(l-m)) and the arg-max in registers, in the
//       shadow of the next tile's MMAs.  W_lm is read from HBM once; the logits are never read back.  More verify
//       rows than one pass holds (at most 512): all passes run in the same launch, on groups of neighbouring pairs
//       that walk the same vocabulary tiles in step, one pass each, so that a tile still leaves HBM once and reaches
//       the other pairs of its group out of the L2.
//       With 257..384 verify rows the accumulators rotate over the four 128-column units of the tensor memory and a
//       unit is handed back as soon as its chunk has gone to the logits buffer and a staging buffer.  In its
//       on-chip-expansion mode the kernel streams groups of 256 vocabulary rows stored at 4, 8 or 16 bits and
//       converter warps (groups of two, each owning whole K blocks) expand the codes exactly to bf16 (mixed-precision
//       quantiser of the Lo-Bi Optimization section).
//   quantize_rows_int8_kernel   8-bit case of the Lo-Bi quantiser, per row (W_lm ahead of time, hidden rows per call).
//   quantize_rows_w4_kernel     4-bit case: codes in [-7, 7] with one shared exponent per sub-block of 128 channels.
//   bounded_wait_selftest_kernel  a wait that is made to run out, to exercise the give-up path without breaking anything.
//   draft_entropy_kernel        H(q_j) of the draft rows, for the gate on the draft distribution.
//   shard_record_kernel         vocabulary-parallel form: a rank's statistics record for the first all-gather.
//   finalize_kernel             merges the per-CTA statistics:  logZ = m + ln s,  H = ln s - t/s  (entropy
//       definition of the HSD section, rearranged around the running maximum).
//   accept_sample_kernel        one cluster of CTAs per sequence: merges the statistics for its k+1 positions (warp
//       shuffles), applies the entropy gate and the ratio test in draft order, then makes one vectorised pass
//       over the logits row and the draft row of the first rejected position: residual max(0, p - q), per-chunk
//       sums, a scan, and the inverse-CDF pick with the supplied uniform.
//
// Every on-chip wait is bounded: when a wait runs out the CTA raises HOLA_FLAG_TIMEOUT, leaves its loops,
// releases its tensor memory and returns.

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cooperative_groups.h>

#include <mutex>

#include "../../include/hola_verify.h"

namespace cg = cooperative_groups;

namespace {

// ------------------------------------------------------------------------------------------------ constants
constexpr int kBlockK = 64;                      // bf16 elements per K block = one 128-byte swizzle row
constexpr int kLanes = 128;                      // vocabulary rows per CTA per tile = tensor-memory lanes
constexpr int kPairTile = 2 * kLanes;            // vocabulary rows per CTA pair per tile
constexpr int kWBlockBytes = kLanes * kBlockK * 2;
constexpr int kMaxN = 256;                       // verify rows per MMA
constexpr int kMaxRowsPerPass = 2 * kMaxN;       // two MMAs per K step fill the 512 tensor-memory columns
constexpr int kEpiWarps = 16;                    // warps 2..17: tensor memory -> logits buffer + softmax statistics
constexpr int kK1Warps = 2 + kEpiWarps;          // warp 0 TMA, warp 1 MMA + tensor-memory owner
constexpr int kK1Threads = kK1Warps * 32;
constexpr int kEpiSlots = 4;                     // 32-column chunks of a tile one epilogue warp handles at most
constexpr int kTransRows = 16;                   // verify rows per transposition step of an epilogue warp
constexpr int kTransBytes = kTransRows * 32 * 4; // its staging buffer: [16 rows][32 vocabulary entries] fp32
// 8-bit W_lm, expanded on chip (mode 1): the int8 tile of a K block lands in a raw block of the ring slot and
// converter warps expand it to the bf16 tile the MMA reads.  Warps 2..9 are epilogue warps, warps 10..17 convert (and
// the first lane of a group also fetches the hidden blocks of the K blocks the group owns).
constexpr int kRawBlockBytes = kLanes * kBlockK;  // int8 [128][64]
constexpr int kSubBlock = 128;                    // hidden channels per 4-bit sub-block (one shared exponent each)
constexpr int kGroupRows = 256;                   // vocabulary rows per group of one width
constexpr int kW8EpiWarps = 8;
constexpr int kConvWarps = kK1Warps - 2 - kW8EpiWarps;   // 8
constexpr int kTmemCols = 512;
constexpr int kMaxStages = 12;
constexpr int kMaxPaceGroups = 128;              // groups of CTA pairs of a launch that holds all passes
constexpr int kSmemBudget = 227 * 1024;          // dynamic shared memory per CTA on sm_100
constexpr int kBarrierBytes = 512;
constexpr long long kWaitLimitCycles = 4000000000ll;   // about 2 s of SM clock per wait, far above any legitimate wait

constexpr int kK3Threads = 256;
constexpr int kK3Warps = kK3Threads / 32;
constexpr int kK3MaxPerSm = 4;                   // CTAs of the accept/sample kernel an SM holds (register budget: 64 per thread)
constexpr int kChunk = 128;                      // vocabulary entries per warp step (32 lanes x 4)
constexpr int kMaxChunks = 4096;                 // => V <= 524288
constexpr int kMaxK1 = 64;                       // k + 1 <= 64
constexpr int kK3Unroll = 4;                     // vocabulary chunks a warp has in flight per step

constexpr int kHqSlices = 8;                     // CTAs that share one draft row in draft_entropy_kernel

constexpr float kLog2e = 1.4426950408889634f;

struct K1Params {
  int M;          // total verify rows B(k+1)
  int row0;       // first row of this pass
  int rows;       // rows of this pass (<= n_sub * N)
  int n_pass;     // > 1: all passes in this launch; CTA pair i works on pass i % n_pass (rows from row0 + that many
  int rows_per_pass;   // times rows_per_pass on) and shares the vocabulary tiles with the pairs i / n_pass, see the kernel
  int V, n_ptiles, n_kblocks, stages, nbuf;
  int n_sub, N;   // MMAs per K step and their N (verify rows each; multiple of 16)
  int rot;        // 1: three MMAs of N <= 128 per K step whose accumulators rotate over the four 128-column units
  int pair256;    // rot with N = 128 exactly: two of the three units of a tile are adjacent and take ONE MMA of N = 256
  int conv_group; // (on-chip expansion) converter warps that share one K block
  int tile_rows;  // vocabulary rows per CTA per tile (<= 128, multiple of 4): balances the tiles over the pairs
  int ldl;        // row pitch of the logits buffer, in floats
  const float* w_scale;   // 8-bit W_lm: fp32 scale per vocabulary row, applied to the accumulators
  const float* h_scale;   // 8-bit activations (modes 2, 3): fp32 scale per verify row (mode 3: of the coarse plane)
  const float* h_scale2;  // mode 3: scale of the second plane
  // Mode 1 with vocabulary groups of mixed width (null: every row is 8-bit and lives at its own index in W_lm): width
  // (4, 8 or 16) of each group of 256 vocabulary rows, first row of the group inside the buffer of its width, and the
  // exponents of the 4-bit sub-blocks, [sub-block][row of the 4-bit buffer].
  const uint8_t* group_width;
  const int* group_row;
  const uint8_t* shift4;
  int rows4;
  int stream_logits;      // 1: store the logits with the streaming hint (they exceed what the L2 keeps until they are read)
  float* logits;
  float4* partials;   // [grid][part_stride] (m, s, t, arg-max index)
  int part_stride;
  unsigned* status;
  unsigned* pace;     // n_pass > 1: one counter per group of pairs (zero at launch), by which the group keeps in step
};

struct K3Params {
  int B, k, V, ldl;
  const float* logits;
  const float4* partials;
  int nparts, part_stride, combine;
  const int* tok;
  const void* q;
  int q_dtype;
  const float* q_tok;           // optional fp32 [B][k]: q_j(x_j) already gathered (then q is read at row n only)
  const void* q_far;            // optional: the same draft tensor in pinned HOST memory, as the device sees it; rows
  int q_far_from;               //   n >= q_far_from of a sequence are read from there (rows before it were copied to q)
  int inputs_settled;           // 1: launched right behind this call's own GEMM kernel, whose CTAs have waited for the
                                // kernel before the call: tokens, uniforms and draft probabilities may be read
                                // before this grid's dependency wait.  0: wait first.
  int phase;                    // 0: the whole step; 1: stop after the accept test (accept_len, statistics written);
                                // vocabulary-parallel form: 3: stop after the masses of row n inside this shard,
                                // 4: the draw, by the shard that holds the point u * R
  // Vocabulary-parallel form (shard_world > 0): V, logits and q cover this rank's V entries starting at v_offset;
  // draft tokens and next_tok are global indices below V_global.
  int shard_world, shard_rank, v_offset, V_global;
  const float* lx_all;          // [world] records, rec_stride floats apart: logit of x_j where its owner found it, else -inf
  int rec_stride;               // floats from one rank's record to the next
  double* mass_out;             // phase 3: [B][2] mass of max(0, p_n - q_n) and of p_n inside this shard
  const double* mass_all;       // phase 4: [world][B][2], the same from every rank
  const float* u;
  float tau;
  int gate_source;          // hola_gate_source
  int fallback;             // hola_fallback
  const double* hq_part;        // [B][k][kHqSlices] slice sums of q ln q, read when the draft entropy gates
  float* draft_entropy;         // [B][k] optional output of H(q_j)
  int* accept_len;
  int* next_tok;
  float* entropy;
  float* logZ;
  unsigned* status;
};

// ------------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address, in the cluster's shared window, of the same shared-memory offset in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// Execution barrier only: orders no memory operations.  For the end of the kernel, where the point is that the peer CTA
// has stopped using this CTA's barriers and tensor memory; a release here would make every thread wait until its last
// stores of logits (hundreds of KB per CTA) have drained to L2 before the CTA may leave.
__device__ __forceinline__ void cluster_sync_execution_only() {
  asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory");
  asm volatile("barrier.cluster.wait;" ::: "memory");
}

// True in exactly one lane of a converged warp.  Unlike a lane-id test, the compiler knows that a single thread
// runs the guarded region, so TMA / tcgen05 operands can stay in uniform registers.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n .reg .pred P;\n elect.sync _|P, 0xffffffff;\n selp.u32 %0, 1, 0, P;\n}" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Arrivals on a barrier that may live in the peer CTA (address from map_to_cta).  Default (CTA-scope release)
// semantics on purpose: a cluster-scope release here acts as a fence that waits for the thread's earlier
// outstanding operations and serialises the pipeline.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred P1;\n mbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n selp.u32 %0, 1, 0, P1;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out of time).
// The clock is the SM's cycle counter (cheap to read), looked at only every 256 unsuccessful polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          unsigned* status, long long limit_cycles = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = 0;
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 255u) == 0u) {
      if (*abort_flag) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      if (now - t0 > limit_cycles) {
        *abort_flag = 1u;
        if (status) atomicOr(status, HOLA_FLAG_TIMEOUT);
        return false;
      }
    }
  }
}

// Whole-warp form: lane 0 polls, every lane gets the same answer (and, through the shuffle, the same ordering).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                               unsigned* status, long long limit_cycles = kWaitLimitCycles) {
  int r = 1;
  if ((threadIdx.x & 31) == 0) r = mbar_wait(bar, parity, abort_flag, status, limit_cycles) ? 1 : 0;
  r = __shfl_sync(0xffffffffu, r, 0);
  return r != 0;
}

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// 2-D tiled TMA load, global -> this CTA's shared memory.  The completion is counted on an mbarrier that may
// live in either CTA of the pair (cta_group::2 form); no multicast: each CTA fetches its own bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int x, int y,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(x), "r"(y), "l"(policy)
      : "memory");
}

// All passes in one launch: the pairs of a group read the same tile of W_lm, and only those that read it within the
// few tens of microseconds a line stays in the L2 are spared the trip to HBM.  So before a new tile every producer
// thread of the group counts itself in and waits, for a bounded time, until the others have done so too.  A pace
// maker, not a barrier: when the time is up the thread goes on, and nothing depends on the others having arrived.
constexpr long long kPaceLimitCycles = 60000;
__device__ __forceinline__ void keep_pace(unsigned* counter, unsigned target) {
  atomicAdd(counter, 1u);
  const long long t0 = clock64();
  while (true) {
    unsigned seen;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
    if (seen >= target || clock64() - t0 > kPaceLimitCycles) break;
  }
}

// Programmatic dependent launch: the grid may have been started while the kernel before it in the stream was still
// running.  grid_dependency_wait returns once that kernel has completed and its writes are visible; it must precede
// every global-memory access of the calling thread that could touch what that kernel reads or writes.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Tensor memory of the CTA pair: executed by one warp of EACH CTA of the pair.
__device__ __forceinline__ void tmem_alloc(uint32_t holder_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem of both CTAs] (+)= A[smem of both CTAs] * B[smem of both CTAs]^T.  bf16 inputs with fp32 accumulation
// (K = 16 per instruction) or, with kInt8, signed 8-bit inputs with int32 accumulation (K = 32 per instruction).
// Issued by one thread of the pair's leader CTA; descriptors are shared-memory offsets valid in both CTAs.
template <bool kInt8>
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                     uint32_t accumulate) {
  if (kInt8) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
// The mbarrier at this shared-memory offset in BOTH CTAs of the pair gets one arrival once every MMA issued so far
// by this thread has completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}

// 32 consecutive fp32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// 16 consecutive 32-bit columns of this thread's tensor-memory lane, as raw words (no wait: the caller waits once
// for all loads it has issued).
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor: K-major tile whose rows are 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart (stride byte offset), descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);      // start address, 16-byte units
  d |= static_cast<uint64_t>(1) << 16;                          // leading byte offset: unused with swizzled K-major
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                  // stride byte offset
  d |= static_cast<uint64_t>(1) << 46;                          // version
  d |= static_cast<uint64_t>(2) << 61;                          // layout: 128-byte swizzle
  return d;
}

// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, M = 256 (the pair), N = n.
__device__ __forceinline__ uint32_t make_idesc_bf16_m256(uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((256u >> 4) << 24);
}
// Instruction descriptor, kind::i8: D int32, A and B signed 8-bit, both K-major, M = 256, N = n (multiple of 32).
__device__ __forceinline__ uint32_t make_idesc_s8_m256(uint32_t n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((256u >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------ softmax statistics
// Statistics of a set of logits around its maximum m:  s = sum e^(l-m),  t = sum e^(l-m) (l-m).
// logZ = m + ln s;  H = -sum p ln p = ln s - t/s.
struct Stats {
  float m, s, t;
  int arg;        // vocabulary index of the maximum (lowest index among equals): the greedy verifier's token
};
__device__ __forceinline__ Stats stats_empty() { return Stats{-CUDART_INF_F, 0.f, 0.f, 0x7fffffff}; }

__device__ __forceinline__ Stats stats_merge(Stats a, Stats b) {
  if (b.m == -CUDART_INF_F) return a;
  if (a.m == -CUDART_INF_F) return b;
  const float m = fmaxf(a.m, b.m);
  const float da = a.m - m, db = b.m - m;
  const float ea = __expf(da), eb = __expf(db);
  Stats r;
  r.m = m;
  r.s = ea * a.s + eb * b.s;
  r.t = ea * (a.t + da * a.s) + eb * (b.t + db * b.s);
  r.arg = a.m > b.m ? a.arg : (b.m > a.m ? b.arg : min(a.arg, b.arg));
  return r;
}

// Fold the first `n` (1..16) of sixteen logits into the running statistics; element i is vocabulary entry vocab0 + i.
template <bool kFull>
__device__ __forceinline__ void stats_fold16(const float* v, int n, int vocab0, Stats& st) {
  float cmax = v[0];
#pragma unroll
  for (int i = 1; i < 16; ++i)
    if (kFull || i < n) cmax = fmaxf(cmax, v[i]);
  if (cmax > st.m) {
    if (st.m != -CUDART_INF_F) {
      const float d = st.m - cmax;
      const float sc = ex2_approx(d * kLog2e);
      st.t = sc * (st.t + d * st.s);
      st.s *= sc;
    }
    st.m = cmax;
    int first = 0;
#pragma unroll
    for (int i = 15; i > 0; --i)
      if ((kFull || i < n) && v[i] == cmax) first = i;
    if (v[0] == cmax) first = 0;
    st.arg = vocab0 + first;
  }
  const float m = st.m;
  const float mneg2 = -m * kLog2e;
  float s = st.s, t = st.t;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    if (kFull || i < n) {
      const float e = ex2_approx(fmaf(v[i], kLog2e, mneg2));
      s += e;
      t = fmaf(e, v[i] - m, t);
    }
  }
  st.s = s;
  st.t = t;
}

// Two fp32 values in one 64-bit register, for the packed fp32 instructions of sm_100 (two results per issue slot).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t r, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// stats_fold16<true> with half the issue slots: the maximum by three-input comparisons, the exponents' arguments, the
// sum of the exponentials and the sum of e * l two at a time.  The centred sum of the sixteen entries,
// sum e (l - m), is taken as  sum e l - m sum e : both terms are of size |m| * (sum e), so the rounding of the
// difference is about 1e-7 |m| relative to s, far inside the tolerance on H = ln s - t / s.
__device__ __forceinline__ void stats_fold16_packed(const float* v, int vocab0, Stats& st) {
  const float c0 = max3(v[0], v[1], v[2]), c1 = max3(v[3], v[4], v[5]), c2 = max3(v[6], v[7], v[8]),
              c3 = max3(v[9], v[10], v[11]), c4 = max3(v[12], v[13], v[14]);
  const float cmax = fmaxf(max3(c0, c1, c2), max3(c3, c4, v[15]));
  if (cmax > st.m) {
    if (st.m != -CUDART_INF_F) {
      const float d = st.m - cmax;
      const float sc = ex2_approx(d * kLog2e);
      st.t = sc * (st.t + d * st.s);
      st.s *= sc;
    }
    st.m = cmax;
    int first = 0;
#pragma unroll
    for (int i = 15; i > 0; --i)
      if (v[i] == cmax) first = i;
    if (v[0] == cmax) first = 0;
    st.arg = vocab0 + first;
  }
  const float m = st.m;
  const float mneg2 = -m * kLog2e;
  const uint64_t l2e = pack2(kLog2e, kLog2e), mn = pack2(mneg2, mneg2);
  uint64_t s2 = pack2(0.f, 0.f), a2 = pack2(0.f, 0.f);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint64_t vp = pack2(v[2 * j], v[2 * j + 1]);
    float x0, x1;
    unpack2(fma2(vp, l2e, mn), x0, x1);
    const uint64_t ep = pack2(ex2_approx(x0), ex2_approx(x1));
    s2 = add2(s2, ep);
    a2 = fma2(ep, vp, a2);
  }
  float sa, sb, aa, ab;
  unpack2(s2, sa, sb);
  unpack2(a2, aa, ab);
  const float sc = sa + sb;
  st.s += sc;
  st.t += fmaf(-m, sc, aa + ab);
}

// Integer codes to bf16 without conversion instructions: 0x4300 | n is the bf16 number 128 + n for 0 <= n < 128 (seven
// mantissa bits, unit steps), two such numbers sit in one register, and one packed bf16 subtraction or multiply-add
// (exact: every intermediate is an integer of at most eight bits) leaves the codes themselves.
__device__ __forceinline__ uint32_t bf16x2_sub(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf16x2_fma(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Sixteen int8 values (one 16-byte piece of a row of the raw block) -> sixteen bf16 values, written as the two 16-byte
// chunks d0, d1 of the 128-byte-swizzled K-major tile that the caller has located.
__device__ __forceinline__ void expand_int8x16(const uint4 x, uint8_t* d0, uint8_t* d1) {
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
  uint32_t o[8];
  // byte b = (128 + its low seven bits) - (256 if its sign bit is set, else 128); as bf16 bit patterns the minuend is
  // 0x4300 | low bits and the subtrahend 0x4300 | sign bit (0x4380 = 256), so one byte permutation each puts two of
  // them in a register next to the constant high byte 0x43
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t lo = w[j] & 0x7F7F7F7Fu, sg = w[j] & 0x80808080u;
    o[2 * j] = bf16x2_sub(__byte_perm(lo, 0x43434343u, 0x4140), __byte_perm(sg, 0x43434343u, 0x4140));       // bytes 0, 1
    o[2 * j + 1] = bf16x2_sub(__byte_perm(lo, 0x43434343u, 0x4342), __byte_perm(sg, 0x43434343u, 0x4342));   // bytes 2, 3
  }
  *reinterpret_cast<uint4*>(d0) = make_uint4(o[0], o[1], o[2], o[3]);
  *reinterpret_cast<uint4*>(d1) = make_uint4(o[4], o[5], o[6], o[7]);
}

// Thirty-two 4-bit codes (one 16-byte piece of a row of the raw block; two's complement nibbles, even entry in the low
// nibble) -> thirty-two bf16 values  code << shift, written as four 16-byte chunks of the 128-byte-swizzled K-major
// tile: chunk j goes to d + ((16 j) ^ x3), d and x3 = 16 (row % 4) located by the caller.  Every value (magnitude
// <= 7 * 2^4) is exact in bf16.
__device__ __forceinline__ void expand_int4x32(const uint4 x, uint8_t* d, uint32_t x3, int shift) {
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
  // nibble n with its sign bit flipped is code + 8; (128 + code + 8) * 2^shift - 136 * 2^shift = code * 2^shift
  const uint32_t mul1 = static_cast<uint32_t>(127 + shift) << 7;           // bf16 bits of 2^shift
  const uint32_t mul = mul1 | (mul1 << 16);
  const uint32_t sub1 = 0xC308u + (static_cast<uint32_t>(shift) << 7);     // bf16 bits of -136 * 2^shift
  const uint32_t sub = sub1 | (sub1 << 16);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    // entries (0,4), (1,5), (2,6), (3,7) of this word side by side in 16-bit lanes; flipping the sign bit of the nibble
    // and setting the bits of 128 are one exclusive-or with 0x4308 (the masked nibble has no bits there)
    const uint32_t u = w[j];
    const uint32_t r0 = bf16x2_fma((u & 0x000F000Fu) ^ 0x43084308u, mul, sub);
    const uint32_t r1 = bf16x2_fma(((u >> 4) & 0x000F000Fu) ^ 0x43084308u, mul, sub);
    const uint32_t r2 = bf16x2_fma(((u >> 8) & 0x000F000Fu) ^ 0x43084308u, mul, sub);
    const uint32_t r3 = bf16x2_fma(((u >> 12) & 0x000F000Fu) ^ 0x43084308u, mul, sub);
    // back into channel order: (0,1) (2,3) (4,5) (6,7)
    *reinterpret_cast<uint4*>(d + ((16u * j) ^ x3)) =
        make_uint4(__byte_perm(r0, r1, 0x5410), __byte_perm(r2, r3, 0x5410), __byte_perm(r0, r1, 0x7632),
                   __byte_perm(r2, r3, 0x7632));
  }
}

// A logit on its way to the buffer.  Only one verify row per sequence is ever read back (row accept_len, by the
// accept/sample kernel); when the buffer is much larger than the L2 the streaming hint lets the lines leave early
// instead of displacing what the next kernel reads.
__device__ __forceinline__ void store_logit(float* dst, float x, int streaming) {
  if (streaming) __stcs(dst, x);
  else *dst = x;
}

// One accumulator on its way to the logits buffer.  Mode 0: as is.  Mode 1: times the scale of the vocabulary row.
// Mode 2: the accumulator is an int32 (bit pattern in `acc`); times the scales of the vocabulary row and of the
// verify row.
template <int kMode>
__device__ __forceinline__ float scaled(float acc, float w_scale, const float* h_scale, int row) {
  if (kMode == 1) return acc * w_scale;
  if (kMode == 2) return static_cast<float>(__float_as_int(acc)) * (w_scale * h_scale[row]);
  return acc;
}

// ------------------------------------------------------------------------------------------------ K1
// Shared memory: `stages` ring slots of [W_lm block 128 x 64 | hidden block(s) n_sub x (N/2) x 64], then the
// barrier area.  Barriers (8 bytes each, offsets in the barrier area):
//   full[12]   @0    leader CTA's copy is the live one: 2 arrivals (one producer per CTA) + the bytes of both CTAs
//   empty[12]  @96   per CTA: the MMAs that read this slot have completed (commit, delivered to both CTAs)
//   tfull[2]   @192  per CTA: the accumulators of a tile are complete (commit, delivered to both CTAs)
//   tempty[4]  @208  leader's copy: all epilogue warps of the pair have read their accumulators (per buffer; per
//                    128-column unit when the accumulators rotate)
//   tensor-memory base @256, abort flag @260
//   8-bit W_lm only: rawfull[12] @272 per CTA: the int8 tile of the slot has landed; rawempty[12] @368 per CTA: the
//   converter warps have expanded it.  full[] then collects, besides the hidden bytes, one arrival per converter warp.
// After the barrier area: one 2 KB transposition buffer per epilogue warp (reused for the final merge of the
// statistics of the four tensor-memory lane quarters).
// kMode 3 is kMode 2 with every verify row present twice in the hidden operand (coarse 8-bit plane and the plane of
// its remainder, in alternating blocks of 32 rows): the epilogue adds the two int32 sums with their scales.
// kMode: 0 bf16 x bf16; 1 int8 W_lm expanded to bf16 on chip (exact); 2 int8 W_lm x int8 hidden on the 8-bit MMA
// kind (K blocks of 128 elements, so that a block is 128 bytes per row exactly as in mode 0; int32 accumulators).
// kRot: 257..384 rows per pass, three MMAs of N <= 128 per K step on rotating 128-column accumulator units (a
// specialisation of its own because its epilogue holds a different set of values in registers).
template <int kMode, bool kRot>
__global__ void __launch_bounds__(kK1Threads, 1)
lm_head_entropy_kernel(const __grid_constant__ CUtensorMap tmap_hidden, const __grid_constant__ CUtensorMap tmap_w,
                       const __grid_constant__ CUtensorMap tmap_w4, const __grid_constant__ CUtensorMap tmap_w16,
                       const K1Params p) {
  constexpr bool kW8 = kMode == 1;
  constexpr bool kI8 = kMode >= 2;                       // both operands 8-bit, 8-bit MMA kind
  constexpr bool kTwoPlane = kMode == 3;                 // hidden rows as two 8-bit planes, 64 operand rows per 32 verify rows
  constexpr int kKStep = kI8 ? 2 * kBlockK : kBlockK;    // elements of K per ring slot
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;          // 128-byte swizzle wants 1024-byte aligned tiles
  uint8_t* smem = smem_raw + (base - raw);

  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);   // same value in all lanes, and the compiler knows it
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();              // 0 = leader of the pair
  // One pass per launch: pair i of npairs takes the vocabulary tiles i, i + npairs, ...  All passes in one launch
  // (n_pass > 1): n_pass neighbouring pairs form a group that walks the same tiles at the same time, one pass of the
  // verify rows each, so that a tile of W_lm comes from HBM once and reaches the other pairs of the group out of the L2.
  const int pair_of_grid = blockIdx.x >> 1;
  const int pair = p.n_pass > 1 ? pair_of_grid / p.n_pass : pair_of_grid;          // which tiles
  const int npairs = p.n_pass > 1 ? (gridDim.x >> 1) / p.n_pass : gridDim.x >> 1;
  const int row0 = p.n_pass > 1 ? (pair_of_grid - pair * p.n_pass) * p.rows_per_pass : p.row0;
  const int rows = p.n_pass > 1 ? min(p.rows_per_pass, p.M - row0) : p.rows;
  const int half_n = p.N >> 1;                           // hidden rows this CTA supplies per MMA
  const uint32_t hid_block_bytes = static_cast<uint32_t>(half_n) * 128u;
  const uint32_t raw_off = kWBlockBytes + p.n_sub * hid_block_bytes;     // int8 block of the slot (8-bit W_lm only)
  const uint32_t stage_bytes = raw_off + (kW8 ? kRawBlockBytes : 0);
  const uint32_t hid_tx_bytes = p.n_sub * hid_block_bytes;
  const uint32_t tx_bytes = static_cast<uint32_t>(p.tile_rows) * 128u + hid_tx_bytes;   // bf16 W_lm: per CTA and slot
  const uint32_t raw_tx_bytes = static_cast<uint32_t>(p.tile_rows) * 64u;
  const int pair_rows = 2 * p.tile_rows;                 // vocabulary rows of a pair's tile
  const uint32_t bar_base = base + p.stages * stage_bytes;
  const uint32_t full_bar = bar_base, empty_bar = bar_base + 96, tfull_bar = bar_base + 192,
                 tempty_bar = bar_base + 208, rawfull_bar = bar_base + 272, rawempty_bar = bar_base + 368;
  constexpr int kNumEpi = kW8 ? kW8EpiWarps : kEpiWarps;      // epilogue warps 2 .. 2 + kNumEpi - 1
  constexpr int kGroups = kNumEpi / 4;                        // warps per tensor-memory lane quarter
  constexpr int kWarpTransBytes = kRot ? 2 * kTransBytes : kTransBytes;   // rotating units: a whole 32-row chunk at once
  float* trans_base = reinterpret_cast<float*>(smem + p.stages * stage_bytes + kBarrierBytes);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + p.stages * stage_bytes + 256);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + p.stages * stage_bytes + 260);

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.stages; ++i) {
      mbar_init(full_bar + 8 * i, kW8 ? 2 + 2 * p.conv_group : 2);   // + the converter warps of a K block, both CTAs
      mbar_init(empty_bar + 8 * i, 1);
      if (kW8) {
        mbar_init(rawfull_bar + 8 * i, 1);
        mbar_init(rawempty_bar + 8 * i, p.conv_group);
      }
    }
    for (int i = 0; i < 2; ++i) mbar_init(tfull_bar + 8 * i, 1);
    for (int i = 0; i < 4; ++i) mbar_init(tempty_bar + 8 * i, 2 * kNumEpi);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_hidden) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_w) : "memory");
  }
  __syncwarp();
  if (warp == 1) tmem_alloc(smem_u32(tmem_holder), kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // the peer's barriers are initialised too
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  const int my_tiles = (p.n_ptiles - pair + npairs - 1) / npairs;
  const int sub_chunks = (p.N + 31) >> 5;                // 32-column chunks per MMA's accumulator
  // Accumulators.  rot == 0: MMA s of buffer b starts at column b * 256 + s * 256 (two buffers only when
  // n_sub == 1; with two MMAs the next tile waits until the whole tile has been read out).  rot == 1 (257..384 rows):
  // three MMAs of N <= 128; MMA s of tile t owns the 128-column unit (3 t + s) % 4, so a tile's first unit is always
  // free and its second and third are the first two the epilogue of the tile before it reads out: the tensor pipe
  // restarts after one epilogue round instead of after the whole read-out.

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one per CTA)
    if (elect_one()) {
      // W_lm is streamed once.  (With all passes in one launch the other pairs of the group read the tile out of the L2
      // within microseconds, the group keeping in step; measured, the lines still do best as the first to be evicted:
      // they then never displace the hidden rows, which every pair re-reads for every tile.)
      const uint64_t pol_w = l2_policy_evict_first();
      const uint64_t pol_h = l2_policy_evict_last();     // hidden is re-read for every tile
      const uint32_t leader_full = map_to_cta(full_bar, 0);
      const uint32_t own_rawfull = map_to_cta(rawfull_bar, rank);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      grid_dependency_wait();                            // W_lm and the hidden rows may come from the kernel before
      if (kW8) {
        // On-chip expansion: only the raw W_lm blocks.  The raw block of a slot may be refilled as soon as the
        // converters have read it (16-bit rows, which go straight into the tile the MMA reads: once the MMAs of the
        // slot's previous use are done as well).  The hidden blocks of a slot are fetched by the converter group that
        // owns the K block, which waits for those MMAs anyway.
        for (int t = 0; t < my_tiles && ok; ++t) {
          if (p.n_pass > 1 && p.pace && t > 0) keep_pace(p.pace + pair, static_cast<unsigned>(2 * p.n_pass * t));
          int tile_width = 8;                              // width of this tile's rows and where they are stored
          int w_row = (pair + t * npairs) * pair_rows + static_cast<int>(rank) * p.tile_rows;
          if (p.group_width) {
            const int g = pair + t * npairs;
            tile_width = p.group_width[g];
            w_row = p.group_row[g] + static_cast<int>(rank) * p.tile_rows;
          }
          int kx = 0;
          for (int kb = 0; kb < p.n_kblocks; ++kb, kx += kKStep) {
            if (!mbar_wait(rawempty_bar + 8 * stage, phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
            const uint32_t sa = base + stage * stage_bytes;
            const uint32_t rb = own_rawfull + 8 * stage;
            if (tile_width == 8) {
              mbar_expect_tx_cluster(rb, raw_tx_bytes);
              tma_load_2d(sa + raw_off, &tmap_w, rb, kx, w_row, pol_w);
            } else if (tile_width == 4) {                  // two codes per byte: 32 bytes per row and K block
              mbar_expect_tx_cluster(rb, raw_tx_bytes >> 1);
              tma_load_2d(sa + raw_off, &tmap_w4, rb, kx >> 1, w_row, pol_w);
            } else {
              if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
              mbar_expect_tx_cluster(rb, raw_tx_bytes << 1);
              tma_load_2d(sa, &tmap_w16, rb, kx, w_row, pol_w);
            }
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
          }
        }
      } else
      for (int t = 0; t < my_tiles && ok; ++t) {
        const int v0 = (pair + t * npairs) * pair_rows + static_cast<int>(rank) * p.tile_rows;
        if (p.n_pass > 1 && p.pace && t > 0) keep_pace(p.pace + pair, static_cast<unsigned>(2 * p.n_pass * t));
        int kx = 0;                                      // K coordinate of the block, in elements
        for (int kb = 0; kb < p.n_kblocks; ++kb, kx += kKStep) {
          const uint32_t sa = base + stage * stage_bytes;
          if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          const uint32_t fb = leader_full + 8 * stage;
          mbar_expect_tx_cluster(fb, tx_bytes);
          tma_load_2d(sa, &tmap_w, fb, kx, v0, pol_w);
          if (kRot && p.pair256) {
            // Row blocks 0, 1, 2 (128 rows each) sit on units (3t, 3t+1, 3t+2) mod 4.  Two of them that are adjacent
            // without wrapping (blocks 0, 1, or blocks 1, 2 when the tile starts on unit 3) share one MMA of N = 256:
            // this CTA then supplies ONE of the two blocks whole, and its half of the third block as before.
            const bool late_pair = ((3 * t) & 3) == 3;
            const int pair_row = (late_pair ? 128 : 0) + static_cast<int>(rank) * 128;
            const int single_row = (late_pair ? 0 : 256) + static_cast<int>(rank) * 64;
            tma_load_2d(sa + kWBlockBytes, &tmap_hidden, fb, kx, row0 + pair_row, pol_h);
            tma_load_2d(sa + kWBlockBytes + hid_block_bytes, &tmap_hidden, fb, kx, row0 + pair_row + 64, pol_h);
            tma_load_2d(sa + kWBlockBytes + 2 * hid_block_bytes, &tmap_hidden, fb, kx, row0 + single_row, pol_h);
          } else {
            for (int s = 0; s < p.n_sub; ++s)
              tma_load_2d(sa + kWBlockBytes + s * hid_block_bytes, &tmap_hidden, fb, kx,
                          (kTwoPlane ? 2 : 1) * row0 + s * p.N + static_cast<int>(rank) * half_n, pol_h);
          }
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (rank == 0 && elect_one()) {
      const uint32_t idesc = kI8 ? make_idesc_s8_m256(static_cast<uint32_t>(p.N))
                                 : make_idesc_bf16_m256(static_cast<uint32_t>(p.N));
      const uint32_t idesc_pair = kI8 ? make_idesc_s8_m256(256u) : make_idesc_bf16_m256(256u);
      const uint64_t desc0 = make_kmajor_sw128_desc(base);
      const bool two_mmas = p.n_sub == 2;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      if (kRot) {
        uint32_t used = 0;                               // bit u: parity of the number of tiles that used unit u
        for (int t = 0; t < my_tiles && ok; ++t) {
          for (int kb = 0; kb < p.n_kblocks && ok; ++kb) {
            if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            const uint64_t adesc = desc0 + ((stage * stage_bytes) >> 4);
            const uint64_t bdesc0 = adesc + (kWBlockBytes >> 4);
            if (p.pair256) {
              // one MMA of N = 256 over the two adjacent units, one of N = 128 over the third: the W_lm block is read
              // from shared memory twice per K step instead of three times
              const uint32_t a0 = static_cast<uint32_t>(3 * t) & 3u;
              const bool late_pair = a0 == 3u;
              const uint32_t unit_pair = late_pair ? 0u : a0, unit_single = late_pair ? 3u : ((a0 + 2u) & 3u);
              if (kb == 0) {                             // the epilogue must have read these units' previous tiles
#pragma unroll
                for (int u = 0; u < 3; ++u) {
                  const uint32_t unit = (a0 + u) & 3u;
                  const uint32_t par = (used >> unit) & 1u;
                  if (!mbar_wait(tempty_bar + 8 * unit, par ^ 1u, abort_flag, p.status)) { ok = false; break; }
                  used ^= 1u << unit;
                }
                if (!ok) break;
                tc_fence_after();
              }
              const uint32_t acc = kb != 0 ? 1u : 0u;
              const uint32_t dp = tmem_base + unit_pair * 128u, ds = tmem_base + unit_single * 128u;
              const uint64_t bdesc_s = bdesc0 + 2 * (hid_block_bytes >> 4);
#pragma unroll
              for (int kk = 0; kk < kBlockK / 16; ++kk) {
                umma<kI8>(dp, adesc + 2 * kk, bdesc0 + 2 * kk, idesc_pair, kk == 0 ? acc : 1u);
                umma<kI8>(ds, adesc + 2 * kk, bdesc_s + 2 * kk, idesc, kk == 0 ? acc : 1u);
              }
            } else
#pragma unroll
            for (int u = 0; u < 3; ++u) {
              const uint32_t unit = static_cast<uint32_t>(3 * t + u) & 3u;
              if (kb == 0) {                             // the epilogue must have read this unit's previous tile
                const uint32_t par = (used >> unit) & 1u;
                if (!mbar_wait(tempty_bar + 8 * unit, par ^ 1u, abort_flag, p.status)) { ok = false; break; }
                used ^= 1u << unit;
                tc_fence_after();
              }
              const uint32_t d = tmem_base + unit * 128u;
              const uint64_t bdesc = bdesc0 + u * (hid_block_bytes >> 4);
              umma<kI8>(d, adesc, bdesc, idesc, kb != 0 ? 1u : 0u);
#pragma unroll
              for (int kk = 1; kk < kBlockK / 16; ++kk) umma<kI8>(d, adesc + 2 * kk, bdesc + 2 * kk, idesc, 1u);
            }
            if (!ok) break;
            umma_commit_pair(empty_bar + 8 * stage);
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
          }
          if (ok) umma_commit_pair(tfull_bar);           // all three units of this tile are complete in both CTAs
        }
      } else
      for (int t = 0; t < my_tiles && ok; ++t) {
        const int buf = t % p.nbuf;
        const uint32_t acc_phase = static_cast<uint32_t>(t / p.nbuf) & 1u;
        if (!mbar_wait(tempty_bar + 8 * buf, acc_phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d0 = tmem_base + buf * 256;
        for (int kb = 0; kb < p.n_kblocks; ++kb) {
          if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          // descriptors of this slot: only the 14-bit address field changes (16-byte units)
          const uint64_t adesc = desc0 + ((stage * stage_bytes) >> 4);
          const uint64_t bdesc0 = adesc + (kWBlockBytes >> 4);
          const uint32_t acc = kb != 0 ? 1u : 0u;
          // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in 16-byte address units
          if (two_mmas) {
            const uint64_t bdesc1 = bdesc0 + (hid_block_bytes >> 4);
            umma<kI8>(d0, adesc, bdesc0, idesc, acc);
            umma<kI8>(d0 + 256, adesc, bdesc1, idesc, acc);
#pragma unroll
            for (int kk = 1; kk < kBlockK / 16; ++kk) {
              umma<kI8>(d0, adesc + 2 * kk, bdesc0 + 2 * kk, idesc, 1u);
              umma<kI8>(d0 + 256, adesc + 2 * kk, bdesc1 + 2 * kk, idesc, 1u);
            }
          } else {
            umma<kI8>(d0, adesc, bdesc0, idesc, acc);
#pragma unroll
            for (int kk = 1; kk < kBlockK / 16; ++kk) umma<kI8>(d0, adesc + 2 * kk, bdesc0 + 2 * kk, idesc, 1u);
          }
          umma_commit_pair(empty_bar + 8 * stage);       // frees the slot in both CTAs once these MMAs have read it
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(tfull_bar + 8 * buf);   // accumulators of this tile are complete in both CTAs
      }
    }
  } else if (warp < 2 + kNumEpi) {
    // ------------------------------------------------------------------ epilogue warps
    // Tensor memory -> registers (thread = vocabulary entry, register = verify row) -> logits buffer, and the same
    // values, transposed through a small shared-memory buffer 16 rows at a time (thread = verify row and half of the
    // warp's 32 vocabulary entries), into thread-private softmax statistics that live in registers for the whole
    // kernel.  A warp owns one lane quarter (fixed by its id) and every kGroups-th 32-column chunk (with rotating
    // accumulators: chunk `group` of every unit, so that all warps read unit after unit and free each at once).
    const int quarter = warp & 3;                        // tensor-memory lanes 32*quarter .. +31
    const int group = (warp - 2) >> 2;
    const uint32_t leader_tempty = map_to_cta(tempty_bar, 0);
    const int n_chunks = p.n_sub * sub_chunks;
    constexpr bool rot = kRot;
    const int my_chunks = rot ? (group < sub_chunks ? p.n_sub : 0)
                              : (group < n_chunks ? (n_chunks - 1 - group) / kGroups + 1 : 0);
    float* tbuf = trans_base + (warp - 2) * (kWarpTransBytes / 4);
    const int trow = lane & 15, thalf = lane >> 4;       // row of a transposition step; which 16 of the 32 entries
    constexpr int kSlots = kRot ? 3 : kEpiSlots;         // chunks per tile this warp keeps statistics for
    Stats st[kSlots][2];
#pragma unroll
    for (int i = 0; i < kSlots; ++i) { st[i][0] = stats_empty(); st[i][1] = stats_empty(); }
    bool ok = true;
    grid_dependency_wait();                              // the logits buffer may still be read by the kernel before
    for (int t = 0; t < my_tiles && ok; ++t) {
      const int buf = t % p.nbuf;
      const uint32_t acc_phase = static_cast<uint32_t>(t / p.nbuf) & 1u;
      if (!mbar_wait_warp(tfull_bar + 8 * buf, acc_phase, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      const int vbase = (pair + t * npairs) * pair_rows + static_cast<int>(rank) * p.tile_rows;
      const int tile_lane = quarter * 32 + lane;         // lanes at or beyond tile_rows hold nothing
      const int vocab = vbase + tile_lane;
      const bool vocab_ok = tile_lane < p.tile_rows && vocab < p.V;
      // vocabulary entries of this quarter that exist (a prefix of its 32 lanes), and of this thread's 16
      const int nv = max(0, min(32, min(p.tile_rows, p.V - vbase) - quarter * 32));
      const int n16 = max(0, min(16, nv - thalf * 16));
      const int vocab16 = vbase + quarter * 32 + thalf * 16;
      const float w_scale = ((kW8 || kI8) && vocab_ok) ? p.w_scale[vocab] : 1.f;   // 8-bit W_lm: the row's scale
      const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      if (kTwoPlane) {
        // Two planes: 64 consecutive accumulator columns hold the coarse-plane sums (first 32) and the remainder-plane
        // sums (last 32) of the same 32 verify rows.  Read 16 + 16 columns at a time, add them with their scales, and
        // go on as in the other modes (16 rows are exactly one transposition step).
        const int n_pairs = p.n_sub * p.N / 64;
        const int my_pairs = group < n_pairs ? (n_pairs - 1 - group) / kGroups + 1 : 0;
        if (my_pairs == 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * buf);
        }
#pragma unroll
        for (int slot = 0; slot < 2; ++slot) {
          if (slot < my_pairs) {
            const int pr = group + slot * kGroups;
            const int sub = (64 * pr) / p.N, col = 64 * pr - sub * p.N;
            const uint32_t taddr = lane_addr + buf * 256 + sub * 256 + col;
            const int vr0 = row0 + 32 * pr;            // verify row of the pair's first column
            const int n_ok = min(32, p.M - vr0);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t a[16], c[16];
              __syncwarp();
              tmem_ld16_nowait(taddr + 16 * half, a);
              tmem_ld16_nowait(taddr + 32 + 16 * half, c);
              tmem_ld_wait();
              if (slot == my_pairs - 1 && half == 1) {   // this warp's accumulators may be overwritten
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * buf);
              }
              const int rows_here = n_ok - 16 * half;    // real rows among these 16
              if (rows_here > 0) {
                float f[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                  f[i] = 0.f;
                  if (i < rows_here) {
                    const int r = vr0 + 16 * half + i;
                    f[i] = fmaf(static_cast<float>(static_cast<int>(c[i])), w_scale * p.h_scale2[r],
                                static_cast<float>(static_cast<int>(a[i])) * (w_scale * p.h_scale[r]));
                  }
                }
                if (vocab_ok) {
                  float* dst = p.logits + static_cast<size_t>(vr0 + 16 * half) * p.ldl + vocab;
#pragma unroll
                  for (int i = 0; i < 16; ++i)
                    if (i < rows_here) store_logit(dst + static_cast<size_t>(i) * p.ldl, f[i], p.stream_logits);
                }
                if (nv > 0) {
                  __syncwarp();
#pragma unroll
                  for (int i = 0; i < kTransRows; ++i)
                    tbuf[i * 32 + ((((lane >> 2) ^ (i & 7))) << 2) + (lane & 3)] = f[i];
                  __syncwarp();
                  float e[16];
#pragma unroll
                  for (int jj = 0; jj < 4; ++jj) {
                    const float4 x = *reinterpret_cast<const float4*>(
                        tbuf + trow * 32 + (((thalf * 4 + jj) ^ (trow & 7)) << 2));
                    e[4 * jj] = x.x; e[4 * jj + 1] = x.y; e[4 * jj + 2] = x.z; e[4 * jj + 3] = x.w;
                  }
                  if (n16 == 16) stats_fold16_packed(e, vocab16, st[slot][half]);
                  else if (n16 > 0) stats_fold16<false>(e, n16, vocab16, st[slot][half]);
                }
              }
            }
          }
        }
        continue;
      }
      if (my_chunks == 0) {                              // nothing to read: the accumulators are free as far as this
        tc_fence_before();                               // warp is concerned
        __syncwarp();
        if (lane == 0) {
          if (rot) {
            for (int u = 0; u < p.n_sub; ++u) mbar_arrive_cluster(leader_tempty + 8 * ((3 * t + u) & 3));
          } else {
            mbar_arrive_cluster(leader_tempty + 8 * buf);
          }
        }
      }
      if (kRot) {
        // Rotating units.  The next tile's MMAs wait for this tile's first two units, so a unit is read and handed back
        // as early as possible: a chunk goes from the registers to the logits buffer and, whole, into the warp's
        // 4 KB staging buffer; the registers then take the next unit's chunk at once, and the statistics of the chunk
        // before are folded from the staging buffer while that unit is already free.
        if (my_chunks > 0) {
          float v[32];
          __syncwarp();
          tmem_ld32(lane_addr + ((3 * t) & 3) * 128 + group * 32, v);
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * ((3 * t) & 3));
#pragma unroll
          for (int slot = 0; slot < 3; ++slot) {
            const int c0 = group * 32;                   // first column of the chunk inside its MMA
            const int r0 = row0 + slot * p.N + c0;     // verify row of column c0
            const int n_ok = min(32, min(p.N - c0, p.M - r0));   // columns that are real rows
            if (n_ok > 0) {
#pragma unroll
              for (int i0 = 0; i0 < 32; i0 += 8) {
#pragma unroll
                for (int i = i0; i < i0 + 8; ++i)
                  if (i < n_ok) v[i] = scaled<kMode>(v[i], w_scale, p.h_scale, r0 + i);
                if (kMode >= 2) asm volatile("" ::: "memory");   // the row scales eight at a time, not all 32 ahead
              }
              if (vocab_ok) {
                float* dst = p.logits + static_cast<size_t>(r0) * p.ldl + vocab;
                if (n_ok == 32 && p.stream_logits) {
#pragma unroll
                  for (int i = 0; i < 32; ++i) __stcs(dst + static_cast<size_t>(i) * p.ldl, v[i]);
                } else if (n_ok == 32) {
#pragma unroll
                  for (int i = 0; i < 32; ++i) dst[static_cast<size_t>(i) * p.ldl] = v[i];
                } else {
#pragma unroll
                  for (int i = 0; i < 32; ++i)
                    if (i < n_ok) store_logit(dst + static_cast<size_t>(i) * p.ldl, v[i], p.stream_logits);
                }
              }
            }
            const bool fold = n_ok > 0 && nv > 0;
            __syncwarp();                                // every lane has folded the chunk before out of the buffer
            if (fold) {
              // two blocks of 16 rows, each laid out as in the 16-row scheme: entry (row i, vocabulary lane l) at
              // 16-byte group (l / 4) ^ (i % 8) of row i
#pragma unroll
              for (int i = 0; i < 32; ++i)
                tbuf[i * 32 + ((((lane >> 2) ^ (i & 7))) << 2) + (lane & 3)] = v[i];
            }
            __syncwarp();
            if (slot < 2) {                              // the registers are free: take the next unit's chunk, free the unit
              const int unit = (3 * t + slot + 1) & 3;
              tmem_ld32(lane_addr + unit * 128 + group * 32, v);
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * unit);
            }
            if (fold) {
#pragma unroll
              for (int half = 0; half < 2; ++half) {
                if (half * kTransRows < n_ok) {
                  float e[16];
#pragma unroll
                  for (int jj = 0; jj < 4; ++jj) {
                    const float4 x = *reinterpret_cast<const float4*>(
                        tbuf + (half * kTransRows + trow) * 32 + (((thalf * 4 + jj) ^ (trow & 7)) << 2));
                    e[4 * jj] = x.x; e[4 * jj + 1] = x.y; e[4 * jj + 2] = x.z; e[4 * jj + 3] = x.w;
                  }
                  if (n16 == 16) stats_fold16_packed(e, vocab16, st[slot][half]);
                  else if (n16 > 0) stats_fold16<false>(e, n16, vocab16, st[slot][half]);
                }
              }
            }
          }
        }
        continue;
      }
#pragma unroll
      for (int slot = 0; slot < kSlots; ++slot) {
        if (slot < my_chunks) {
          const int ch = rot ? slot * sub_chunks + group : group + slot * kGroups;
          const int sub = ch / sub_chunks, j = ch - sub * sub_chunks;
          const int unit = (3 * t + slot) & 3;           // (rotating accumulators only)
          float v[32];
          __syncwarp();                                  // tcgen05.ld is warp-collective: reconverge first
          tmem_ld32(lane_addr + (rot ? unit * 128 : buf * 256 + sub * 256) + j * 32, v);
          if (rot || slot == my_chunks - 1) {            // this warp's accumulators (of this unit) may be overwritten
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_tempty + 8 * (rot ? unit : buf));
          }
          const int c0 = j * 32;                         // first column of the chunk inside its MMA
          const int r0 = row0 + sub * p.N + c0;        // verify row of column c0
          const int n_ok = min(32, min(p.N - c0, p.M - r0));   // columns that are real rows
          if (n_ok > 0) {
#pragma unroll
            for (int i0 = 0; i0 < 32; i0 += 8) {
#pragma unroll
              for (int i = i0; i < i0 + 8; ++i)
                if (i < n_ok) v[i] = scaled<kMode>(v[i], w_scale, p.h_scale, r0 + i);
              if (kMode >= 2) asm volatile("" ::: "memory");     // the row scales eight at a time, not all 32 ahead
            }
            if (vocab_ok) {
              float* dst = p.logits + static_cast<size_t>(r0) * p.ldl + vocab;
              if (n_ok == 32 && p.stream_logits) {       // (the common cases without a test per store)
#pragma unroll
                for (int i = 0; i < 32; ++i) __stcs(dst + static_cast<size_t>(i) * p.ldl, v[i]);
              } else if (n_ok == 32) {
#pragma unroll
                for (int i = 0; i < 32; ++i) dst[static_cast<size_t>(i) * p.ldl] = v[i];
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (i < n_ok) store_logit(dst + static_cast<size_t>(i) * p.ldl, v[i], p.stream_logits);
              }
            }
            if (nv > 0) {
#pragma unroll
              for (int half = 0; half < 2; ++half) {
                if (half * kTransRows < n_ok) {
                  // entry (row i, vocabulary lane l) at 16-byte group (l / 4) ^ (i % 8) of row i: stores of one
                  // row and the 16-byte loads of eight neighbouring rows both touch every bank once
                  __syncwarp();
#pragma unroll
                  for (int i = 0; i < kTransRows; ++i)
                    tbuf[i * 32 + ((((lane >> 2) ^ (i & 7))) << 2) + (lane & 3)] = v[half * kTransRows + i];
                  __syncwarp();
                  float e[16];
#pragma unroll
                  for (int jj = 0; jj < 4; ++jj) {
                    const float4 x = *reinterpret_cast<const float4*>(
                        tbuf + trow * 32 + (((thalf * 4 + jj) ^ (trow & 7)) << 2));
                    e[4 * jj] = x.x; e[4 * jj + 1] = x.y; e[4 * jj + 2] = x.z; e[4 * jj + 3] = x.w;
                  }
                  // (rows at or beyond n_ok fold whatever the unused columns held; they are never written out)
                  if (n16 == 16) stats_fold16_packed(e, vocab16, st[slot][half]);
                  else if (n16 > 0) stats_fold16<false>(e, n16, vocab16, st[slot][half]);
                }
              }
            }
          }
        }
      }
    }
    // ---- the CTA's statistics of every row: first the two halves of a quarter (lanes L and L ^ 16), then, after
    // all epilogue warps are done with their buffers, the quarters side by side in shared memory
    asm volatile("bar.sync 1, %0;" ::"n"(kNumEpi * 32) : "memory");
    float4* merge = reinterpret_cast<float4*>(trans_base);          // [4 quarters][rows of the pass]
#pragma unroll
    for (int slot = 0; slot < kSlots; ++slot) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        Stats a = st[slot][half], o;
        o.m = __shfl_xor_sync(0xffffffffu, a.m, 16);
        o.s = __shfl_xor_sync(0xffffffffu, a.s, 16);
        o.t = __shfl_xor_sync(0xffffffffu, a.t, 16);
        o.arg = __shfl_xor_sync(0xffffffffu, a.arg, 16);
        a = stats_merge(a, o);
        if (kTwoPlane) {
          const int r = 32 * (group + slot * kGroups) + half * kTransRows + trow;   // row inside the pass
          if (slot < 2 && thalf == 0 && r < rows)
            merge[quarter * rows + r] = make_float4(a.m, a.s, a.t, __int_as_float(a.arg));
        } else if (slot < my_chunks && thalf == 0) {
          const int ch = rot ? slot * sub_chunks + group : group + slot * kGroups;
          const int sub = ch / sub_chunks, j = ch - sub * sub_chunks;
          const int c = j * 32 + half * kTransRows + trow;           // column inside its MMA
          const int r = sub * p.N + c;                               // row inside the pass
          if (c < p.N && r < rows) merge[quarter * rows + r] = make_float4(a.m, a.s, a.t, __int_as_float(a.arg));
        }
      }
    }
  } else if (kW8) {
    // ------------------------------------------------------------------ 8-bit W_lm: converter warps
    // int8 [tile_rows][64] (row pitch 64 bytes) -> bf16 [tile_rows][64] in the 128-byte-swizzled K-major layout the
    // MMA reads: 16-byte chunk c of row r sits at chunk position c ^ (r % 8) of its 128-byte row.  Every int8 value is
    // exact in bf16; the row's scale is applied to the accumulators by the epilogue warps.
    // The converter warps form groups of conv_group warps; each group owns whole K blocks, every ngroups-th one of the
    // CTA's sequence of blocks.  The waits, the expansion and the fence of one block are a chain of dependent steps:
    // several groups run such chains side by side (ring slots permitting), several warps in a group shorten the chain.
    const int cw = warp - (2 + kW8EpiWarps);
    const uint32_t leader_full = map_to_cta(full_bar, 0);
    const int units = p.tile_rows * 4;                   // 16-byte pieces of the int8 tile
    const uint64_t pol_h = l2_policy_evict_last();       // hidden is re-read for every tile
    const int total_blocks = my_tiles * p.n_kblocks;
    grid_dependency_wait();                              // the width table and the exponents may come from the kernel before
    // No more groups than ring slots take part: a group that starts block i has finished block i - ngroups, whose slot
    // had been freed by the MMAs of block i - ngroups - stages, so with ngroups <= stages every barrier it waits on is at
    // most one phase behind and the parity waits below cannot mistake "two trips round the ring ago" for "done".
    const int G = p.conv_group;
    const int ngroups = min(kConvWarps / G, p.stages);
    const int grp = cw / G, mem = cw - grp * G;          // warps beyond ngroups * G groups stay idle
    const int step = 32 * G;                             // pieces the group expands per trip of its loops
    const int first = mem * 32 + lane;                   // this lane's first piece
    int t = 0, kb = grp;                                 // block i = t * n_kblocks + kb of the sequence, i % ngroups == grp
    while (kb >= p.n_kblocks && t < my_tiles) { kb -= p.n_kblocks; ++t; }
    // Where this lane's pieces go does not change from block to block.  8-bit: piece u is the 16 bytes c = u % 4 of row
    // u / 4 and becomes chunks 2c, 2c+1 of the row's 128 bytes in the tile, each XOR-ed with row % 8 (128-byte swizzle;
    // the row itself starts at row * 128); a step of the loop moves on by a multiple of 8 rows.  4-bit: piece u is half
    // c = u % 2 of row u / 2 and becomes chunks 4c .. 4c+3.
    const uint32_t off8 = static_cast<uint32_t>(first >> 2) * 128u + (((2u * (first & 3)) ^ ((first >> 2) & 7u)) << 4);
    const uint32_t off4 = static_cast<uint32_t>(first >> 1) * 128u + (((4u * (first & 1)) ^ ((first >> 1) & 4u)) << 4);
    const uint32_t x3 = ((first >> 1) & 3u) << 4;
    const uint32_t raw_step = static_cast<uint32_t>(step) * 16u;          // bytes of the raw block per step
    const uint32_t tile_step8 = static_cast<uint32_t>(step) * 32u;        // 8 G rows of the tile
    const uint32_t tile_step4 = static_cast<uint32_t>(step) * 64u;        // 16 G rows of the tile
    // Width of a tile's rows and where they start in the buffer of that width (4-bit: for the exponents).
    auto tile_info = [&](int tt, int& width, int& wrow) {
      width = 8; wrow = 0;
      if (p.group_width) {
        const int g = pair + tt * npairs;
        width = p.group_width[g];
        wrow = p.group_row[g] + static_cast<int>(rank) * p.tile_rows;
      }
    };
    // (4-bit) the exponents of this lane's rows in K block kkb: a sub-block of 128 hidden channels spans two K blocks
    auto fetch_shifts = [&](int kkb, int width, int wrow, uint32_t (&e)[8]) {
      const uint8_t* sh = p.shift4 + static_cast<size_t>(kkb >> 1) * p.rows4;
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        const int row = (first + step * n) >> 1;
        const int r4 = wrow + row;
        e[n] = (width == 4 && row < p.tile_rows && r4 >= 0 && r4 < p.rows4) ? sh[r4] : 0u;
      }
    };
    int tile_width, w_row;
    uint32_t e[8];
    if (grp < ngroups && grp < total_blocks) {
      tile_info(t, tile_width, w_row);
      if (tile_width == 4) fetch_shifts(kb, tile_width, w_row, e);
    }
    int stage = grp;                                     // ring slot and phase of block i (grp < ngroups <= stages)
    uint32_t phase = 0;
    for (int i = grp; i < total_blocks && grp < ngroups; i += ngroups) {
      uint8_t* slot = smem + stage * stage_bytes;
      uint32_t shifts = 0;                               // one nibble per step
      if (tile_width == 4) {
#pragma unroll
        for (int n = 0; n < 8; ++n) shifts |= min(e[n], 4u) << (4 * n);
      }
      // the group's next block: its exponents are fetched while this block is waited for and expanded
      int t2 = t, kb2 = kb + ngroups, width2 = tile_width, w_row2 = w_row;
      while (kb2 >= p.n_kblocks) { kb2 -= p.n_kblocks; ++t2; }
      if (i + ngroups < total_blocks) {
        if (t2 != t) tile_info(t2, width2, w_row2);
        if (width2 == 4) fetch_shifts(kb2, width2, w_row2, e);
      }
      // first the slot's previous use (which implies that its raw block's previous phase is over), then this block's bytes
      if (!mbar_wait_warp(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.status)) break;
      if (mem == 0 && lane == 0) {                       // the slot is free: its hidden blocks arrive while the W_lm block is expanded
        const uint32_t sa = base + stage * stage_bytes;
        const uint32_t fb = leader_full + 8 * stage;
        mbar_expect_tx_cluster(fb, hid_tx_bytes);
        for (int sb = 0; sb < p.n_sub; ++sb)
          tma_load_2d(sa + kWBlockBytes + sb * hid_block_bytes, &tmap_hidden, fb, kb * kKStep,
                      row0 + sb * p.N + static_cast<int>(rank) * half_n, pol_h);
      }
      if (!mbar_wait_warp(rawfull_bar + 8 * stage, phase, abort_flag, p.status)) break;
      // Two pieces per trip of a loop that is kept rolled: the expansion of a whole block written out is some ten
      // thousand bytes of straight-line code per width, which a warp would fetch anew for every block (measured: rolled
      // is faster, and four pieces per trip are no faster than two).
      const uint8_t* src = slot + raw_off + first * 16;
      if (tile_width == 8) {
        uint32_t o = off8;
#pragma unroll 1
        for (int u0 = first; u0 < units; u0 += 2 * step, src += 2 * raw_step, o += 2 * tile_step8) {
          const bool two = u0 + step < units;
          const uint4 x0 = *reinterpret_cast<const uint4*>(src);
          const uint4 x1 = two ? *reinterpret_cast<const uint4*>(src + raw_step) : make_uint4(0u, 0u, 0u, 0u);
          expand_int8x16(x0, slot + o, slot + (o ^ 16u));
          if (two) expand_int8x16(x1, slot + o + tile_step8, slot + ((o + tile_step8) ^ 16u));
        }
      } else if (tile_width == 4) {
        uint32_t o = off4;
#pragma unroll 1
        for (int n = 0; n < 8; n += 2, src += 2 * raw_step, o += 2 * tile_step4) {   // 32-byte rows: two pieces per row
          const int u0 = first + step * n;
          if (u0 >= (units >> 1)) break;
          const bool two = u0 + step < (units >> 1);
          const uint4 x0 = *reinterpret_cast<const uint4*>(src);
          const uint4 x1 = two ? *reinterpret_cast<const uint4*>(src + raw_step) : make_uint4(0u, 0u, 0u, 0u);
          expand_int4x32(x0, slot + o, x3, static_cast<int>((shifts >> (4 * n)) & 15u));
          if (two) expand_int4x32(x1, slot + o + tile_step4, x3, static_cast<int>((shifts >> (4 * n + 4)) & 15u));
        }
      }
      // (16-bit rows were loaded into the tile as they are)
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes, read by the MMA
      __syncwarp();
      if (lane == 0) {
        mbar_arrive_cluster(leader_full + 8 * stage);    // this warp's share of the bf16 tile is in place
        mbar_arrive(rawempty_bar + 8 * stage);           // and the raw block may be refilled
      }
      t = t2; kb = kb2; tile_width = width2; w_row = w_row2;
      stage += ngroups;
      if (stage >= p.stages) { stage -= p.stages; phase ^= 1u; }
    }
  }

  // ------------------------------------------------------------------ common tail
  __syncwarp();                                          // warps 0 and 1 ran one lane apart from the others
  tc_fence_before();
  __syncthreads();
  grid_dependency_wait();                                // (every thread that writes below; long since satisfied)
  if (!*abort_flag) {
    // one partial per CTA and row: the four quarters merged
    const float4* merge = reinterpret_cast<const float4*>(trans_base);
    for (int r = threadIdx.x; r < rows; r += kK1Threads) {
      Stats a = stats_empty();
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 x = merge[q * rows + r];
        a = stats_merge(a, Stats{x.x, x.y, x.z, __float_as_int(x.w)});
      }
      p.partials[static_cast<size_t>(blockIdx.x) * p.part_stride + row0 + r] =
          make_float4(a.m, a.s, a.t, __int_as_float(a.arg));
    }
    if (p.n_pass > 1) {
      // the accept/sample kernel merges the partials of every CTA for every row: this CTA has seen only its pass
      const Stats none = stats_empty();
      const float4 blank = make_float4(none.m, none.s, none.t, __int_as_float(none.arg));
      for (int r = threadIdx.x; r < p.M; r += kK1Threads)
        if (r < row0 || r >= row0 + rows) p.partials[static_cast<size_t>(blockIdx.x) * p.part_stride + r] = blank;
    }
  }
  cluster_sync_execution_only();                         // the peer no longer signals this CTA's barriers or tensor memory
  if (warp == 1) {
    if (*abort_flag) __nanosleep(200000);                // let copies already in flight land before leaving
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------ self-test
// The way a GEMM CTA pair gives up, in miniature and on purpose: a pair of CTAs sets up barriers and tensor memory as
// the GEMM kernel does, then one thread and one whole warp of each CTA wait (with the limit given) on a barrier that
// nothing ever arrives on.  The wait must run out, raise HOLA_FLAG_TIMEOUT and the CTA's abort flag, the other waiters
// must see that flag, and every thread must reach the common tail, where the tensor memory is released.
// out[0] counts the threads that got there, out[1] the waits that returned "give up".
__global__ void __launch_bounds__(64, 1) bounded_wait_selftest_kernel(long long limit_cycles, unsigned* status,
                                                                      unsigned* out) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_holder;
  __shared__ uint32_t abort_word;
  volatile uint32_t* abort_flag = &abort_word;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_word = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (warp == 1) tmem_alloc(smem_u32(&tmem_holder), 32);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_holder;
  unsigned gave_up = 0;
  if (warp == 0) {
    if (lane == 0) gave_up = mbar_wait(smem_u32(&bar), 0u, abort_flag, status, limit_cycles) ? 0u : 1u;
  } else {
    gave_up = mbar_wait_warp(smem_u32(&bar), 0u, abort_flag, status, limit_cycles) ? 0u : (lane == 0 ? 1u : 0u);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (gave_up) atomicAdd(out + 1, 1u);
  atomicAdd(out, 1u);
  cluster_sync_execution_only();
  if (warp == 1) tmem_dealloc(tmem_base, 32);
}

// ------------------------------------------------------------------------------------------------ K2
__device__ __forceinline__ Stats warp_merge_partials(const float4* partials, int nparts, int part_stride, int row,
                                                     int lane) {
  Stats st = stats_empty();
  // six loads per lane in flight (192 partials per round: one round on a 148-SM part), then the merges in index order
  for (int base = 0; base < nparts; base += 192) {
    float4 x[6];
#pragma unroll
    for (int u = 0; u < 6; ++u) {
      const int i = base + lane + 32 * u;
      x[u] = i < nparts ? partials[static_cast<size_t>(i) * part_stride + row]
                        : make_float4(-CUDART_INF_F, 0.f, 0.f, __int_as_float(0x7fffffff));
    }
#pragma unroll
    for (int u = 0; u < 6; ++u) st = stats_merge(st, Stats{x[u].x, x[u].y, x[u].z, __float_as_int(x[u].w)});
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    Stats o;
    o.m = __shfl_xor_sync(0xffffffffu, st.m, off);
    o.s = __shfl_xor_sync(0xffffffffu, st.s, off);
    o.t = __shfl_xor_sync(0xffffffffu, st.t, off);
    o.arg = __shfl_xor_sync(0xffffffffu, st.arg, off);
    // merge in a fixed (lower lane first) order so that every lane holds bit-identical results
    st = ((lane & off) == 0) ? stats_merge(st, o) : stats_merge(o, st);
  }
  return st;
}

__device__ __forceinline__ void stats_to_outputs(Stats st, float* logZ, float* H) {
  const float ls = logf(st.s);
  *logZ = st.m + ls;
  *H = fmaxf(0.f, ls - st.t / st.s);
}

__global__ void __launch_bounds__(256) finalize_kernel(const float4* partials, int nparts, int part_stride, int M,
                                                       float* logZ, float* entropy) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  Stats st = warp_merge_partials(partials, nparts, part_stride, row, lane);
  if (lane == 0) stats_to_outputs(st, &logZ[row], &entropy[row]);
}

// Vocabulary-parallel form, first exchange record of a rank: per verify row the statistics of this shard's logits
// (m, s, t, arg-max as a GLOBAL vocabulary index), then per draft position the logit of the draft token if this shard
// owns it (-inf otherwise).  Blocks 0 .. ceil(M/8)-1 merge the per-CTA partials, the others gather the logits.
__global__ void __launch_bounds__(256) shard_record_kernel(const float4* partials, int nparts, int part_stride, int M,
                                                           int v_offset, int V, const float* logits, int ldl,
                                                           const int* tok, int B, int k, float4* stats_out,
                                                           float* lx_out) {
  const int row_blocks = (M + 7) / 8;
  if (static_cast<int>(blockIdx.x) < row_blocks) {
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= M) return;
    Stats st = warp_merge_partials(partials, nparts, part_stride, row, lane);
    if (lane == 0) {
      const int arg = st.arg == 0x7fffffff ? st.arg : st.arg + v_offset;
      stats_out[row] = make_float4(st.m, st.s, st.t, __int_as_float(arg));
    }
  } else {
    const int i = (blockIdx.x - row_blocks) * 256 + threadIdx.x;
    if (i >= B * k) return;
    const int b = i / k, j = i - b * k;
    const int x = tok[i] - v_offset;
    lx_out[i] = (x >= 0 && x < V) ? logits[static_cast<size_t>(b * (k + 1) + j) * ldl + x] : -CUDART_INF_F;
  }
}

// ------------------------------------------------------------------------------------------------ K3
__device__ __forceinline__ double warp_sum_f64(double x) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

// Four sums over the warp at once (lanes 8 i .. 8 i + 7 return the sum of v[i]): the first two rounds halve the
// number of values a lane carries instead of adding all of them everywhere, six shuffles in all.
__device__ __forceinline__ float warp_sum4_f32(const float v[4], int lane) {
  const bool hi16 = (lane & 16) != 0;
  const float a = (hi16 ? v[2] : v[0]) + __shfl_xor_sync(0xffffffffu, hi16 ? v[0] : v[2], 16);
  const float b = (hi16 ? v[3] : v[1]) + __shfl_xor_sync(0xffffffffu, hi16 ? v[1] : v[3], 16);
  const bool hi8 = (lane & 8) != 0;
  float c = (hi8 ? b : a) + __shfl_xor_sync(0xffffffffu, hi8 ? a : b, 8);
#pragma unroll
  for (int off = 4; off > 0; off >>= 1) c += __shfl_xor_sync(0xffffffffu, c, off);
  return c;
}

// Logits and draft probabilities of vocabulary entries base..base+3 of one row (q = 0 when the row is drawn
// from p itself; entries at or beyond V get l = -inf, q = 0 and so no mass).  Loads only: a caller can issue
// several of these before using any, which keeps more requests in flight.
template <bool kVec>
__device__ __forceinline__ void fetch4(const float* lrow, const void* qrow, int q_dtype, bool residual, int base,
                                       int V, float l[4], float q[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) q[i] = 0.f;
  if (kVec && base + 3 < V) {
    const float4 l4 = *reinterpret_cast<const float4*>(lrow + base);
    l[0] = l4.x; l[1] = l4.y; l[2] = l4.z; l[3] = l4.w;
    if (residual) {
      if (q_dtype == HOLA_Q_BF16) {
        const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(qrow) + base);
        q[0] = __uint_as_float(raw.x << 16); q[1] = __uint_as_float(raw.x & 0xFFFF0000u);
        q[2] = __uint_as_float(raw.y << 16); q[3] = __uint_as_float(raw.y & 0xFFFF0000u);
      } else {
        const float4 q4 = *reinterpret_cast<const float4*>(static_cast<const float*>(qrow) + base);
        q[0] = q4.x; q[1] = q4.y; q[2] = q4.z; q[3] = q4.w;
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int v = base + i;
      l[i] = -CUDART_INF_F;
      if (v < V) {
        l[i] = lrow[v];
        if (residual)
          q[i] = (q_dtype == HOLA_Q_BF16) ? __bfloat162float(static_cast<const __nv_bfloat16*>(qrow)[v])
                                          : static_cast<const float*>(qrow)[v];
      }
    }
  }
}

// The four residual masses  r = max(0, p - q)  with  p = e^(l - logZ)  (q = 0: r = p).  The exponential is the
// hardware's 2^x on (l - logZ) log2 e: relative error about 1e-6 at l - logZ = -30, against a decision margin of 1e-4
// on the cumulative mass; the pass over the row and the final search inside a chunk both come through here.
__device__ __forceinline__ void resid4(const float l[4], const float q[4], float logZ, float r[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) r[i] = fmaxf(0.f, ex2_approx((l[i] - logZ) * kLog2e) - q[i]);
}

template <bool kVec>
__device__ __forceinline__ void load_r4(const float* lrow, const void* qrow, int q_dtype, bool residual, int base,
                                        int V, float logZ, float r[4]) {
  float l[4], q[4];
  fetch4<kVec>(lrow, qrow, q_dtype, residual, base, V, l, q);
  resid4(l, q, logZ, r);
}

__device__ __forceinline__ float clamp_uniform(float u, unsigned& flags) {
  if (!(u >= 0.f)) { flags |= HOLA_FLAG_BAD_UNIFORM; return 0.f; }
  if (u >= 1.f) { flags |= HOLA_FLAG_BAD_UNIFORM; return 1.f - 5.9604645e-8f; }   // 1 - 2^-24
  return u;
}

// One cluster of S CTAs per sequence.  Every CTA derives accept_len on its own (same inputs, same arithmetic,
// same result), sums the residual mass of its slice of the vocabulary chunk by chunk, and publishes its slice
// total to all CTAs of the cluster through distributed shared memory.  After one cluster barrier each CTA knows
// the total mass R and which slice holds the point u*R; that CTA alone finishes the inverse-CDF search.
template <bool kVec>
__global__ void __launch_bounds__(kK3Threads, kK3MaxPerSm) accept_sample_kernel(const K3Params p) {
  extern __shared__ double csum[];                       // per-chunk residual mass of this CTA's slice
  __shared__ double sh_tot[2][8];                        // slice totals of the whole cluster, per attempt
  __shared__ float sh_logZ[kMaxK1], sh_H[kMaxK1], sh_lx[kMaxK1], sh_qx[kMaxK1], sh_u[kMaxK1], sh_Hq[kMaxK1];
  __shared__ int sh_x[kMaxK1], sh_amax[kMaxK1];
  __shared__ int sh_n;
  __shared__ unsigned sh_flags;

  // The next kernel in the stream (normally the next call's GEMM kernel, which waits for this grid before it touches
  // memory) may be scheduled from now on: its launch and prologue then hide behind this kernel.
  grid_dependency_release();
  cg::cluster_group cluster = cg::this_cluster();
  const int S = static_cast<int>(cluster.num_blocks());
  const int rank = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / S;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k = p.k, V = p.V;
  const int row_first = b * (k + 1);

  // ---- gather the k draft-token logits, draft probabilities and the uniforms (independent of the statistics).
  // These come from the caller, not from the GEMM kernel.  Behind this call's own GEMM kernel they are known to be in
  // place (its CTAs waited for whatever ran before the call) and are fetched before this grid's dependency wait; in
  // every other launch the wait comes first.
  if (!p.inputs_settled) grid_dependency_wait();
  for (int j = threadIdx.x; j <= k; j += kK3Threads) sh_u[j] = p.u[b * (k + 1) + j];
  int x_mine = -1;                                       // (k <= 63 < kK3Threads: one draft position per thread)
  float qx_mine = 0.f;
  const bool shard = p.shard_world > 0;
  const int Vtok = shard ? p.V_global : V;               // range of valid token ids
  if (threadIdx.x < k) {
    const int j = threadIdx.x;
    x_mine = p.tok[b * k + j];
    if (x_mine >= 0 && x_mine < Vtok) {
      const size_t qi = (static_cast<size_t>(b) * k + j) * V + x_mine;
      if (p.q_tok) qx_mine = p.q_tok[b * k + j];
      else qx_mine = (p.q_dtype == HOLA_Q_BF16) ? __bfloat162float(static_cast<const __nv_bfloat16*>(p.q)[qi])
                                                : static_cast<const float*>(p.q)[qi];
    }
  }
  // From here on the GEMM kernel's results are read.
  if (p.inputs_settled) grid_dependency_wait();
  for (int j = threadIdx.x; j < k; j += kK3Threads) {
    const int x = x_mine;
    sh_x[j] = x;
    float lx = 0.f;
    const float qx = qx_mine;
    if (x >= 0 && x < Vtok) {
      if (shard) {                                       // exactly one shard owns x and left its logit there
        lx = -CUDART_INF_F;
        for (int r = 0; r < p.shard_world; ++r) lx = fmaxf(lx, p.lx_all[static_cast<size_t>(r) * p.rec_stride + b * k + j]);
      } else {
        lx = p.logits[static_cast<size_t>(row_first + j) * p.ldl + x];
      }
    }
    sh_lx[j] = lx; sh_qx[j] = qx;
    float hq = 0.f;
    if (p.gate_source == HOLA_GATE_DRAFT_ENTROPY) {
      double tot = 0.0;
      for (int sl = 0; sl < kHqSlices; ++sl) tot += p.hq_part[(static_cast<size_t>(b) * k + j) * kHqSlices + sl];
      hq = fmaxf(0.f, static_cast<float>(-tot));
      if (rank == 0 && p.draft_entropy) p.draft_entropy[b * k + j] = hq;
    }
    sh_Hq[j] = hq;
  }
  // ---- softmax statistics of this sequence's k+1 positions
  if (p.combine) {
    // (rows are dealt to the warps from the last warp down: warp 0, whose threads are still waiting for the gathers
    // above, gets a row only when there are more than seven)
    for (int j = kK3Warps - 1 - warp; j <= k; j += kK3Warps) {
      Stats st = warp_merge_partials(p.partials, p.nparts, p.part_stride, row_first + j, lane);
      if (lane == 0) {
        float lz, h;
        stats_to_outputs(st, &lz, &h);
        sh_logZ[j] = lz; sh_H[j] = h; sh_amax[j] = st.arg;
        if (rank == 0) { p.logZ[row_first + j] = lz; p.entropy[row_first + j] = h; }
      }
    }
  } else {
    for (int j = threadIdx.x; j <= k; j += kK3Threads) {
      sh_logZ[j] = p.logZ[row_first + j];
      sh_H[j] = p.entropy[row_first + j];
    }
  }
  __syncthreads();

  // ---- gate and ratio test in draft order; stop at the first position that is not accepted
  if (threadIdx.x == 0) {
    unsigned flags = 0;
    int n = k;
    for (int j = 0; j < k; ++j) {
      const int x = sh_x[j];
      if (x < 0 || x >= Vtok) { flags |= HOLA_FLAG_BAD_TOKEN; n = j; break; }
      const float gate_value = p.gate_source == HOLA_GATE_DRAFT_ENTROPY ? sh_Hq[j] : sh_H[j];
      if (gate_value < p.tau) continue;                  // entropy gate: fast path keeps the draft token
      if (p.fallback == HOLA_FALLBACK_GREEDY) {          // the verifier's own token, or the run ends here
        if (x != sh_amax[j]) { n = j; break; }
        continue;
      }
      const float u = clamp_uniform(sh_u[j], flags);
      const float px = expf(sh_lx[j] - sh_logZ[j]);
      const float qx = sh_qx[j];
      const bool accept = (qx > 0.f) ? (u * qx < px) : (px > 0.f);
      if (!accept) { n = j; break; }
    }
    sh_n = n;
    sh_flags = flags;
    if (rank == 0) {
      p.accept_len[b] = n;
      if (p.fallback == HOLA_FALLBACK_GREEDY) {          // greedy: argmax p_n follows the accepted run; no draw
        p.next_tok[b] = min(max(sh_amax[n], 0), Vtok - 1);
        if (flags && p.status) atomicOr(p.status, flags);
      } else if (p.phase == 1 && flags && p.status) {
        atomicOr(p.status, flags);
      }
    }
  }
  __syncthreads();
  if (p.fallback == HOLA_FALLBACK_GREEDY || p.phase == 1) return;   // same decision in every CTA of the cluster

  // ---- this CTA's slice of row n: per-chunk residual mass
  const int n = sh_n;
  const float logZ = sh_logZ[n];
  const float* lrow = p.logits + static_cast<size_t>(row_first + n) * p.ldl;
  const size_t q_elem = (p.q_dtype == HOLA_Q_BF16) ? 2 : 4;
  const char* qbase = static_cast<const char*>((p.q_far && n >= p.q_far_from) ? p.q_far : p.q);
  const void* qrow = (n < k) ? static_cast<const void*>(qbase + (static_cast<size_t>(b) * k + n) * V * q_elem) : nullptr;
  const int nchunks = (V + kChunk - 1) / kChunk;
  const int cpc = (nchunks + S - 1) / S;                 // chunks per CTA
  const int c_first = rank * cpc;
  const int mine = max(0, min(nchunks, c_first + cpc) - c_first);
  const int per_lane = (mine + 31) / 32;
  bool residual = n < k;

  // Vocabulary-parallel draw: every rank holds every rank's two masses of row n, so all of them agree on which mass
  // counts (the residual's unless it vanishes everywhere), on the total R and on the shard that holds the point u * R.
  double shard_target = 0.0;
  if (shard && p.phase == 4) {
    const double* mass = p.mass_all + static_cast<size_t>(b) * 2;
    const size_t rs = static_cast<size_t>(p.B) * 2;
    double tot_res = 0.0;
    for (int r = 0; r < p.shard_world; ++r) tot_res += mass[r * rs];
    const bool use_p = !residual || !(tot_res > 0.0);
    if (use_p && residual) {
      residual = false;
      if (threadIdx.x == 0) sh_flags |= HOLA_FLAG_R_ZERO;
    }
    const int idx = use_p ? 1 : 0;
    double total = 0.0;
    for (int r = 0; r < p.shard_world; ++r) total += mass[r * rs + idx];
    unsigned uflags = 0;
    const double target = static_cast<double>(clamp_uniform(sh_u[k], uflags)) * total;
    int owner = -1, last_mass = 0;
    double before = 0.0, cum = 0.0;
    for (int r = 0; r < p.shard_world; ++r) {
      const double m = mass[r * rs + idx];
      if (m > 0.0) last_mass = r;
      if (owner < 0 && cum + m > target) { owner = r; before = cum; }
      cum += m;
    }
    shard_target = target - before;
    if (owner < 0) { owner = last_mass; shard_target = CUDART_INF; }     // rounding: the last entry with mass
    if (owner != p.shard_rank) {
      if (rank == 0 && threadIdx.x == 0) p.next_tok[b] = -1;
      return;                                            // same decision in every CTA of the cluster
    }
    __syncthreads();
  }

  for (int attempt = 0; attempt < 2; ++attempt) {
    for (int c0 = warp; c0 < mine; c0 += kK3Unroll * kK3Warps) {
      float l[kK3Unroll][4], q[kK3Unroll][4];
#pragma unroll
      for (int i = 0; i < kK3Unroll; ++i) {              // all loads of this step first
        const int c = c0 + i * kK3Warps;
        if (c < mine) fetch4<kVec>(lrow, qrow, p.q_dtype, residual, (c_first + c) * kChunk + lane * 4, V, l[i], q[i]);
      }
      // the mass of each chunk in fp32 (128 non-negative terms added pairwise: relative error a few 1e-7), kept as
      // fp64 for the scans that follow; lanes 0, 8, 16, 24 end up with chunks 0, 1, 2, 3 of this step
      float part[kK3Unroll];
#pragma unroll
      for (int i = 0; i < kK3Unroll; ++i) {
        const int c = c0 + i * kK3Warps;
        part[i] = 0.f;
        if (c < mine) {
          float r[4];
          resid4(l[i], q[i], logZ, r);
          part[i] = (r[0] + r[1]) + (r[2] + r[3]);
        }
      }
      const float sum = warp_sum4_f32(part, lane);
      const int c = c0 + (lane >> 3) * kK3Warps;
      if ((lane & 7) == 0 && c < mine) csum[c] = static_cast<double>(sum);
    }
    __syncthreads();
    // warp 0: scan of the slice; lane L owns chunks [lo, hi)
    double tot = 0.0, incl = 0.0;
    const int lo = lane * per_lane, hi = min(mine, lo + per_lane);
    if (warp == 0) {
      for (int c = lo; c < hi; ++c) tot += csum[c];
      incl = tot;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const double o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
      }
      const double slice_total = __shfl_sync(0xffffffffu, incl, 31);
      if (lane < S) *cluster.map_shared_rank(&sh_tot[attempt][rank], lane) = slice_total;
    }
    cluster.sync();
    // every CTA: total mass and the slice that holds u * R (identical arithmetic everywhere)
    double R = 0.0;
    for (int r2 = 0; r2 < S; ++r2) R += sh_tot[attempt][r2];
    if (shard && p.phase == 3) {
      // the shard's masses of row n: of the residual, then (second pass, q taken as 0) of p itself
      if (rank == 0 && threadIdx.x == 0) {
        p.mass_out[b * 2 + attempt] = R;
        if (!residual && attempt == 0) p.mass_out[b * 2 + 1] = R;          // bonus position: both are the mass of p
        const unsigned fl = sh_flags;
        if (fl && p.status && (attempt == 1 || !residual)) atomicOr(p.status, fl);
      }
      if (residual) {
        residual = false;
        __syncthreads();
        continue;
      }
      return;
    }
    if (!(R > 0.0) && residual && !shard) {              // p <= q everywhere: draw from p instead
      residual = false;
      if (threadIdx.x == 0) sh_flags |= HOLA_FLAG_R_ZERO;
      __syncthreads();
      continue;
    }
    unsigned uflags = 0;
    const float uk = clamp_uniform(sh_u[k], uflags);
    const double target = shard ? shard_target : static_cast<double>(uk) * R;
    int rstar = -1, last_mass = 0;
    double before_slice = 0.0;
    {
      double cum = 0.0;
      for (int r2 = 0; r2 < S; ++r2) {
        const double t = sh_tot[attempt][r2];
        if (t > 0.0) last_mass = r2;
        if (rstar < 0 && cum + t > target) { rstar = r2; before_slice = cum; }
        cum += t;
      }
    }
    bool take_last = false;
    if (rstar < 0) {                                     // rounding left the running sum a hair below u*R
      rstar = last_mass;
      take_last = true;
    }
    if (rank == rstar && warp == 0) {
      const unsigned over = __ballot_sync(0xffffffffu, before_slice + incl > target);
      const unsigned has_mass = __ballot_sync(0xffffffffu, tot > 0.0);
      int L;
      if (over && !take_last) L = __ffs(over) - 1;
      else { L = has_mass ? 31 - __clz(has_mass) : 0; take_last = true; }
      int cstar = -1;
      double before = 0.0;
      if (lane == L) {
        double cum = before_slice + (incl - tot);
        int last_pos = lo;
        for (int c = lo; c < hi; ++c) {
          if (csum[c] > 0.0) last_pos = c;
          if (!take_last && cum + csum[c] > target) { cstar = c; before = cum; break; }
          cum += csum[c];
        }
        if (cstar < 0) { cstar = last_pos; before = cum - csum[last_pos]; take_last = true; }
      }
      cstar = __shfl_sync(0xffffffffu, cstar, L);
      before = __shfl_sync(0xffffffffu, before, L);
      take_last = __shfl_sync(0xffffffffu, take_last ? 1 : 0, L) != 0;
      // inside the chunk: lane prefix, then the lane's four entries in ascending order
      float r4[4];
      load_r4<kVec>(lrow, qrow, p.q_dtype, residual, (c_first + cstar) * kChunk + lane * 4, V, logZ, r4);
      const double mine4 = ((static_cast<double>(r4[0]) + r4[1]) + r4[2]) + r4[3];
      double lincl = mine4;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const double o = __shfl_up_sync(0xffffffffu, lincl, off);
        if (lane >= off) lincl += o;
      }
      double cum = before + (lincl - mine4);
      int found = -1, last4 = -1;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        cum += r4[i];
        if (r4[i] > 0.f) last4 = i;
        if (found < 0 && !take_last && cum > target) found = i;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, found >= 0);
      const unsigned mass = __ballot_sync(0xffffffffu, last4 >= 0);
      int src, idx;
      if (hit) { src = __ffs(hit) - 1; idx = found; }
      else { src = mass ? 31 - __clz(mass) : 0; idx = last4 < 0 ? 0 : last4; }
      idx = __shfl_sync(0xffffffffu, idx, src);
      if (lane == 0) {
        int tokn = (c_first + cstar) * kChunk + src * 4 + idx;
        if (tokn >= V) tokn = V - 1;
        p.next_tok[b] = tokn + (shard ? p.v_offset : 0);
        const unsigned fl = sh_flags | uflags;
        if (fl && p.status) atomicOr(p.status, fl);
      }
    }
    break;
  }
}

// ------------------------------------------------------------------------------------------------ 8-bit quantiser
// The 8-bit case of the Lo-Bi quantiser on the LM head (Lo-Bi Optimization section; the quantiser itself is not
// spelled out there): one vocabulary row per sub-block, symmetric integers in [-127, 127], one fp32 scale per row,
//   scale = max|w| / 127 (1 for an all-zero row),  q = clip(rint(w / scale)),  all in fp32, ties to even.
// One CTA per row.
__global__ void __launch_bounds__(256) quantize_rows_int8_kernel(const __nv_bfloat16* W, int H, signed char* q,
                                                                 float* scale) {
  __shared__ float sh_max[8];
  __shared__ float sh_scale;
  grid_dependency_wait();                                // (no-op unless launched with programmatic serialization)
  const size_t row = blockIdx.x;
  const __nv_bfloat16* wr = W + row * H;
  float amax = 0.f;
  for (int h = threadIdx.x; h < H; h += 256) amax = fmaxf(amax, fabsf(__bfloat162float(wr[h])));
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
  if ((threadIdx.x & 31) == 0) sh_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < 8; ++i) m = fmaxf(m, sh_max[i]);
    const float sc = m > 0.f ? __fdiv_rn(m, 127.f) : 1.f;
    sh_scale = sc;
    scale[row] = sc;
  }
  __syncthreads();
  const float sc = sh_scale;
  for (int h = threadIdx.x; h < H; h += 256) {
    const float r = rintf(__fdiv_rn(__bfloat162float(wr[h]), sc));
    q[row * H + h] = static_cast<signed char>(fminf(127.f, fmaxf(-127.f, r)));
  }
}

// The 4-bit case of the Lo-Bi quantiser on the LM head (reading: a sub-block is 128 hidden channels of one vocabulary
// row; symmetric codes in [-7, 7]; the sub-block's scale is the row's fp32 scale times a power of two):
//   s = max|w| / 112 (1 for an all-zero row);  e_b = the smallest e in 0..4 with  7 * 2^e * s >= max_{h in b} |w|  (else 4);
//   c = clip(rint(w / (s * 2^e_b)), -7, 7),  every step one fp32 operation, ties to even.
// Two codes per byte (even channel in the low nibble, 4-bit two's complement).  Exponents go to
// shift[b * shift_stride + row].  One CTA per row; warp w takes sub-blocks w, w + 8, ...; a lane holds four channels.
__global__ void __launch_bounds__(256) quantize_rows_w4_kernel(const __nv_bfloat16* W, int H, uint8_t* packed,
                                                               uint8_t* shift, int shift_stride, float* scale) {
  __shared__ float sh_max[8];
  __shared__ float sh_scale;
  const size_t row = blockIdx.x;
  const __nv_bfloat16* wr = W + row * H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float amax = 0.f;
  for (int h = threadIdx.x; h < H; h += 256) amax = fmaxf(amax, fabsf(__bfloat162float(wr[h])));
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
  if (lane == 0) sh_max[warp] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < 8; ++i) m = fmaxf(m, sh_max[i]);
    const float sc = m > 0.f ? __fdiv_rn(m, 112.f) : 1.f;
    sh_scale = sc;
    scale[row] = sc;
  }
  __syncthreads();
  const float sc = sh_scale;
  for (int b = warp; b < H / kSubBlock; b += 8) {
    float w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) w[i] = __bfloat162float(wr[b * kSubBlock + lane * 4 + i]);
    float bmax = fmaxf(fmaxf(fabsf(w[0]), fabsf(w[1])), fmaxf(fabsf(w[2]), fabsf(w[3])));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, off));
    int e = 4;
#pragma unroll
    for (int c = 3; c >= 0; --c)
      if (__fmul_rn(sc, static_cast<float>(7 << c)) >= bmax) e = c;
    const float step = sc * static_cast<float>(1 << e);              // exact
    uint32_t bits = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float r = fminf(7.f, fmaxf(-7.f, rintf(__fdiv_rn(w[i], step))));
      bits |= (static_cast<uint32_t>(static_cast<int>(r)) & 0xFu) << (4 * i);
    }
    *reinterpret_cast<uint16_t*>(packed + row * (H / 2) + b * (kSubBlock / 2) + lane * 2) = static_cast<uint16_t>(bits);
    if (lane == 0) shift[static_cast<size_t>(b) * shift_stride + row] = static_cast<uint8_t>(e);
  }
}

// Hidden rows as two 8-bit planes (16-bit-class activations for the 8-bit MMA kind): per verify row
//   s1 = max|x| / 127 (1 if zero), q1 = clip(rint(x / s1));  r = x - s1 q1;  s2 = s1 / 254, q2 = clip(rint(r / s2)),
// every step one fp32 operation.  Operand layout: blocks of 32 verify rows, each block as 32 rows of q1 followed by
// 32 rows of q2 (so that 64 consecutive accumulator columns hold both sums of the same 32 rows); rows past M are
// written as zeros.  One CTA per (padded) verify row.
__global__ void __launch_bounds__(256) quantize_rows_two_plane_kernel(const __nv_bfloat16* X, int M, int H,
                                                                      signed char* q, float* s1, float* s2) {
  __shared__ float sh_max[8];
  __shared__ float sh_scale;
  grid_dependency_wait();
  const int row = blockIdx.x;
  signed char* q1 = q + (static_cast<size_t>(64) * (row >> 5) + (row & 31)) * H;
  signed char* q2 = q1 + static_cast<size_t>(32) * H;
  if (row >= M) {
    for (int h = threadIdx.x; h < H; h += 256) { q1[h] = 0; q2[h] = 0; }
    return;
  }
  const __nv_bfloat16* xr = X + static_cast<size_t>(row) * H;
  float amax = 0.f;
  for (int h = threadIdx.x; h < H; h += 256) amax = fmaxf(amax, fabsf(__bfloat162float(xr[h])));
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
  if ((threadIdx.x & 31) == 0) sh_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < 8; ++i) m = fmaxf(m, sh_max[i]);
    const float sc = m > 0.f ? __fdiv_rn(m, 127.f) : 1.f;
    sh_scale = sc;
    s1[row] = sc;
    s2[row] = __fdiv_rn(sc, 254.f);
  }
  __syncthreads();
  const float sc = sh_scale, sc2 = __fdiv_rn(sc, 254.f);
  for (int h = threadIdx.x; h < H; h += 256) {
    const float x = __bfloat162float(xr[h]);
    const float a = fminf(127.f, fmaxf(-127.f, rintf(__fdiv_rn(x, sc))));
    const float rem = __fsub_rn(x, __fmul_rn(sc, a));                  // no fused multiply-add: two roundings
    const float b = fminf(127.f, fmaxf(-127.f, rintf(__fdiv_rn(rem, sc2))));
    q1[h] = static_cast<signed char>(a);
    q2[h] = static_cast<signed char>(b);
  }
}

// ------------------------------------------------------------------------------------------------ draft entropy
// H(q) = -sum_v q ln q of each draft row (one CTA per row): the gate value when the gate looks at the draft
// distribution, as the HSD section words it.  q is used as stored; entries with q <= 0 contribute nothing.
// q ln q for q > 0, else 0.  The fast logarithm (absolute error about 2^-21 near 1, a few ulp elsewhere) is
// ample here: every term is weighted by q <= 1 and the sum is compared at 1e-4.
__device__ __forceinline__ float qlnq(float a) { return a > 0.f ? a * __logf(a) : 0.f; }
__device__ __forceinline__ float qlnq8(const uint4 raw) {     // sum over eight bf16 values
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  float part = 0.f;
#pragma unroll
  for (int j = 0; j < 4; ++j) part += qlnq(__uint_as_float(w[j] << 16)) + qlnq(__uint_as_float(w[j] & 0xFFFF0000u));
  return part;
}
__device__ __forceinline__ float qlnq4(const float4 x) { return (qlnq(x.x) + qlnq(x.y)) + (qlnq(x.z) + qlnq(x.w)); }

// Grid (rows, kHqSlices): CTA (r, s) sums slice s of row r and leaves the partial sum in part[r][s]; the
// accept/sample kernel adds the slices in index order.  Small CTAs of 32 registers per thread on purpose: the pass
// runs on a side stream while the GEMM kernel holds every SM, and only a CTA of this size fits into the registers
// that kernel leaves free (a persistent form with eight loads in flight per thread, 100 registers, could not start
// before the GEMM kernel had finished and made the step 45 us longer).
__global__ void __launch_bounds__(256) draft_entropy_kernel(const void* q, int q_dtype, int V, double* part) {
  __shared__ double sh_part[8];
  const size_t row = blockIdx.x;
  const int slice = blockIdx.y;
  double acc = 0.0;
  constexpr int kInFlight = 4;                           // independent 16-byte loads per thread and step
  if (q_dtype == HOLA_Q_BF16) {
    const __nv_bfloat16* qr = static_cast<const __nv_bfloat16*>(q) + row * V;
    const bool vec = (reinterpret_cast<uintptr_t>(qr) & 15u) == 0;
    const int nvec = vec ? V / 8 : 0;
    const uint4* q16 = reinterpret_cast<const uint4*>(qr);
    const int per = (nvec + kHqSlices - 1) / kHqSlices, end = min(nvec, (slice + 1) * per);
    int i = slice * per + threadIdx.x;
    for (; i + (kInFlight - 1) * 256 < end; i += kInFlight * 256) {
      uint4 raw[kInFlight];
#pragma unroll
      for (int u = 0; u < kInFlight; ++u) raw[u] = q16[i + u * 256];
#pragma unroll
      for (int u = 0; u < kInFlight; ++u) acc += qlnq8(raw[u]);
    }
    for (; i < end; i += 256) acc += qlnq8(q16[i]);
    for (int v = nvec * 8 + threadIdx.x; slice == 0 && v < V; v += 256) {    // scalar tail (or whole row): slice 0
      acc += qlnq(__bfloat162float(qr[v]));
    }
  } else {
    const float* qr = static_cast<const float*>(q) + row * V;
    const bool vec = (reinterpret_cast<uintptr_t>(qr) & 15u) == 0;
    const int nvec = vec ? V / 4 : 0;
    const float4* q16 = reinterpret_cast<const float4*>(qr);
    const int per = (nvec + kHqSlices - 1) / kHqSlices, end = min(nvec, (slice + 1) * per);
    int i = slice * per + threadIdx.x;
    for (; i + (kInFlight - 1) * 256 < end; i += kInFlight * 256) {
      float4 raw[kInFlight];
#pragma unroll
      for (int u = 0; u < kInFlight; ++u) raw[u] = q16[i + u * 256];
#pragma unroll
      for (int u = 0; u < kInFlight; ++u) acc += qlnq4(raw[u]);
    }
    for (; i < end; i += 256) acc += qlnq4(q16[i]);
    for (int v = nvec * 4 + threadIdx.x; slice == 0 && v < V; v += 256) {
      acc += qlnq(qr[v]);
    }
  }
  acc = warp_sum_f64(acc);
  if ((threadIdx.x & 31) == 0) sh_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int i = 0; i < 8; ++i) tot += sh_part[i];
    part[row * kHqSlices + slice] = tot;
  }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Plan {
  int n_sub, N, rows_per_pass, passes, grid, stages, nbuf, rot, n_ptiles, n_kblocks, smem_bytes, tile_rows;
  int fused;            // all passes in one launch, groups of `passes` CTA pairs sharing the vocabulary tiles
  double est_seconds;   // rough duration of all passes (the cost the split was chosen by)
};

}  // namespace

// What a call needs besides its arguments, kept from one call to the next: the launch geometry of a (rows, weight
// mode) pair and the two tensor maps of a (hidden pointer, W_lm pointer, rows, weight mode) quadruple.
struct PlanEntry { int valid, M, w_dtype; Plan pl; };
struct MapEntry { int valid, M, w_dtype; const void* hidden; const void* W; const void* W4; const void* W16;
                  CUtensorMap th, tw, tw4, tw16; };
constexpr int kPlanCache = 8, kMapCache = 8;

struct hola_ctx {
  int device, num_sms, maxB, maxK, H, V, ldl, max_rows;
  EncodeTiledFn encode;
  PlanEntry plans[kPlanCache];
  MapEntry maps[kMapCache];
  int plan_next, map_next;
  char* ws;                 // one device allocation, carved below
  size_t ws_bytes;
  float* logits;            // [max_rows][ldl]
  float4* partials;         // [num_sms][max_rows]
  unsigned* status;         // [1]
  unsigned* pace;           // [kMaxPaceGroups] counters of the groups of pairs when all passes share a launch
  double* hq;               // [max_rows][kHqSlices] slice sums of q ln q over the draft rows
  signed char* hid8;        // [max_rows][H] int8 hidden rows (8-bit activation mode)
  float* hid_scale;         // [max_rows]
  // staging for hola_verify_host
  void* st_hidden; int* st_tok; void* st_q; float* st_u;
  unsigned char* st_out;      // device block of one call's outputs (status, accept_len, next_tok, entropy, logZ, ...)
  unsigned char* h_out;       // pinned host mirror: the outputs come back in ONE copy
  int force_stages;
  int no_rot;                 // tuning override: never use the rotating accumulator units
  int force_passes;           // tuning override: passes over W_lm (0: chosen by cost)
  int no_pair256;             // tuning override: rotating units always as three MMAs of N = 128
  int no_fuse;                // tuning override: several passes always as one launch each
  int no_pace;                // tuning override: the groups of pairs of a fused launch do not keep in step
  int conv_group;             // tuning override (0 = by plan): converter warps per K block in the on-chip expansion
  int host_in_place;          // hola_verify_host: read draft rows not sent ahead in place from pinned host memory
  cudaStream_t copy_stream;   // hola_verify_host: the draft tensor travels here while the GEMM runs
  cudaEvent_t copy_done;
  cudaEvent_t fork_point;     // verify_device: where the side stream branches off the caller's stream
  int hq_ready;               // the draft-row entropies of this call are already being made on the side stream
  int host_overlap;           // 1: copy the draft tensor on copy_stream while the GEMM runs
  int host_lazy_q;            // hola_verify_host copies only the draft rows the step reads: 0 never, 1 always,
                              // -1 when the whole tensor would not fit under the GEMM (the default)
  float* st_qtok;             // device fp32 [maxB][maxK]: q_j(x_j) gathered on the host
  float* h_qtok;              // pinned host: the same values before the copy (inside h_small)
  unsigned char* h_small;     // pinned host mirror of the workspace span [st_tok, st_qtok + ...): tokens, uniforms, q_tok
  size_t small_u_off, small_qtok_off, small_span;   // offsets of the uniforms and of q_tok inside that span; its size
  int* h_accept;              // pinned host int32 [maxB]: accept_len read back between the two phases
  unsigned long long last_h2d, last_d2h;   // bytes the last hola_verify_host call moved
  // optional per-kernel timing (hola_profile_begin / hola_profile_end)
  cudaEvent_t* prof_ev;     // 3 events per recorded call: before the GEMM, after it, after accept/sample
  int prof_cap, prof_n, prof_on;
  char last_error[256];
};

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Where one call's outputs sit inside the output block of hola_verify_host (16-byte aligned pieces, packed for the
// call's own B and k so that one copy brings them all back).
struct OutBlock {
  size_t status, accept, next, entropy, logZ, dent, total;
};
OutBlock out_block(int B, int k) {
  const size_t rows = static_cast<size_t>(B) * (k + 1);
  OutBlock o;
  o.status = 0;
  o.accept = 16;
  o.next = o.accept + align_up(static_cast<size_t>(B) * 4, 16);
  o.entropy = o.next + align_up(static_cast<size_t>(B) * 4, 16);
  o.logZ = o.entropy + align_up(rows * 4, 16);
  o.dent = o.logZ + align_up(rows * 4, 16);
  o.total = o.dent + align_up(static_cast<size_t>(B) * (k > 0 ? k : 1) * 4, 16);
  return o;
}

struct WsLayout {
  size_t logits, partials, status, pace, hq, hid8, hid_scale, st_hidden, st_tok, st_q, st_u, st_out, st_qtok, st_small_end, total;
};

WsLayout ws_layout(int maxB, int maxK, int H, int V, int num_sms) {
  const size_t rows = static_cast<size_t>(maxB) * (maxK + 1);
  const size_t ldl = align_up(static_cast<size_t>(V), 4);
  WsLayout w;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.logits = take(rows * ldl * 4);
  w.partials = take(static_cast<size_t>(num_sms) * rows * 16);
  w.status = take(4);
  w.pace = take(4 * kMaxPaceGroups);
  w.hq = take(rows * kHqSlices * 8);
  w.hid8 = take(2 * align_up(rows, 32) * static_cast<size_t>(H));     // one or two 8-bit planes of the hidden rows
  w.hid_scale = take(2 * rows * 4);                                   // their scales (second plane after the first)
  w.st_hidden = take(rows * H * 2);
  // the three small per-step inputs side by side: hola_verify_host sends them as one copy
  w.st_tok = take(static_cast<size_t>(maxB) * maxK * 4);
  w.st_u = take(rows * 4);
  w.st_qtok = take(static_cast<size_t>(maxB) * (maxK > 0 ? maxK : 1) * 4);
  w.st_small_end = off;
  w.st_q = take(static_cast<size_t>(maxB) * maxK * V * 4);
  w.st_out = take(out_block(maxB, maxK).total);
  w.total = off;
  return w;
}

constexpr int kAssumedSms = 148;

void set_error(hola_ctx* ctx, const char* what, cudaError_t e) {
  snprintf(ctx->last_error, sizeof ctx->last_error, "%s: %s", what, cudaGetErrorString(e));
}

int round_up(int x, int a) { return (x + a - 1) / a * a; }

// Splits M verify rows into passes over W_lm and each pass into one or two MMAs per K step.
// A pass holds at most 512 rows (two MMAs of N <= 256 fill the tensor memory); N is a multiple of 16.
// Cost per pass: the slower of streaming W_lm once and the padded rows' tensor time, plus a fixed launch cost.
Plan make_plan(const hola_ctx* ctx, int M, int w_dtype = HOLA_W_BF16) {
  const bool mixed = w_dtype == HOLA_W_MIXED;    // vocabulary groups of 4-, 8- and 16-bit rows, expanded on chip
  const bool w8 = w_dtype == HOLA_W_INT8 || mixed;   // int8 W_lm expanded on chip
  const bool two = w_dtype == HOLA_W8A16;        // as W8A8, with two operand rows per verify row
  const bool i8 = w_dtype == HOLA_W8A8 || two;   // 8-bit MMA: N a multiple of 32, K blocks of 128, twice the rate
  Plan best{};
  double best_cost = 1e300;
  const int rows = M > 0 ? M : 1;
  // 8-bit W_lm: one MMA per K step (at most 256 rows per pass), and the slot also holds the int8 block
  const int max_rows_per_pass = (w8 || two) ? kMaxN : kMaxRowsPerPass;
  const int p_min = (rows + max_rows_per_pass - 1) / max_rows_per_pass;
  const double t_hbm = (w8 || i8 ? 1.0 : 2.0) * ctx->V * static_cast<double>(ctx->H) / 6.4e12;
  const int p_max = ctx->force_passes > p_min + 3 ? ctx->force_passes : p_min + 3;
  for (int passes = p_min; passes <= p_max; ++passes) {
    if (ctx->force_passes && passes != ctx->force_passes && ctx->force_passes >= p_min) continue;
    const int r = (rows + passes - 1) / passes;
    // up to 256 rows: one MMA, two accumulator buffers; up to 384: three MMAs of N <= 128 on rotating 128-column
    // units; beyond: two MMAs of N <= 256 that fill the tensor memory
    int n_sub = (r > 3 * 128 || (ctx->no_rot && r > kMaxN)) ? 2 : (r > kMaxN ? 3 : 1);
    int N = round_up((r + n_sub - 1) / n_sub, i8 ? 32 : 16);
    if (two) {                                     // operand rows: 64 per 32 verify rows; one or two MMAs, N % 64 == 0
      const int r8 = 2 * round_up(r, 32);
      n_sub = r8 > kMaxN ? 2 : 1;
      N = round_up(r8 / n_sub, 64);
    }
    const double t_mma = 2.0 * n_sub * N * static_cast<double>(ctx->V) * ctx->H / (i8 ? 2.8e15 : 1.4e15);
    const double cost = passes * ((t_mma > t_hbm ? t_mma : t_hbm) + 6e-6);
    if (cost < best_cost) {
      best_cost = cost;
      best.n_sub = n_sub; best.N = N; best.rows_per_pass = two ? n_sub * N / 2 : n_sub * N; best.passes = passes;
      best.est_seconds = cost;
    }
  }
  // a pass may end up empty when rows_per_pass * (passes - 1) already covers M
  best.passes = (rows + best.rows_per_pass - 1) / best.rows_per_pass;
  const int stage_bytes = kWBlockBytes + best.n_sub * (best.N / 2) * 128 + (w8 ? kRawBlockBytes : 0);
  // (rotating units: every epilogue warp stages a whole 32-row chunk, twice the bytes)
  const int trans_bytes = (w8 ? kW8EpiWarps : kEpiWarps) * kTransBytes * (best.n_sub == 3 ? 2 : 1);
  int stages = (kSmemBudget - 1024 - kBarrierBytes - trans_bytes) / stage_bytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (ctx->force_stages && ctx->force_stages < stages) stages = ctx->force_stages;
  best.stages = stages;
  best.nbuf = best.n_sub == 1 ? 2 : 1;
  best.rot = best.n_sub == 3 ? 1 : 0;
  // Vocabulary rows per CTA per tile: the smallest multiple of 4 that covers V in the fewest whole rounds over
  // all pairs, so that every pair streams the same number of bytes (V = 32000 on 74 pairs: 2 rounds of 112 + 112
  // rows instead of 1.69 rounds of 128 + 128).
  const int all_pairs = ctx->num_sms / 2 > 0 ? ctx->num_sms / 2 : 1;
  // Several passes: one launch in which `passes` neighbouring pairs walk the same tiles together, one pass each (W_lm
  // then leaves HBM once, not once per pass), as long as every pass gets a pair.
  best.fused = (best.passes > 1 && !ctx->no_fuse && all_pairs / best.passes >= 1) ? 1 : 0;
  const int pairs = best.fused ? all_pairs / best.passes : all_pairs;     // pairs that divide the tiles among them
  const int rounds = (ctx->V + pairs * kPairTile - 1) / (pairs * kPairTile);
  int tile_rows = round_up((ctx->V + 2 * pairs * rounds - 1) / (2 * pairs * rounds), 4);
  if (tile_rows < 8) tile_rows = 8;
  if (tile_rows > kLanes) tile_rows = kLanes;
  if (mixed) tile_rows = kLanes;                 // a pair's tile is one group of 256 rows of one width
  best.tile_rows = tile_rows;
  best.n_ptiles = (ctx->V + 2 * tile_rows - 1) / (2 * tile_rows);
  best.grid = 2 * (best.n_ptiles < pairs ? best.n_ptiles : pairs) * (best.fused ? best.passes : 1);
  best.n_kblocks = i8 ? (ctx->H + 2 * kBlockK - 1) / (2 * kBlockK) : (ctx->H + kBlockK - 1) / kBlockK;
  best.smem_bytes = stages * stage_bytes + kBarrierBytes + trans_bytes + 1024;
  return best;
}

// make_plan through the context's cache (the geometry depends on the context's shape and tuning options, on the number
// of verify rows and on the weight mode only).
const Plan& plan_for(hola_ctx* ctx, int M, int w_dtype) {
  for (int i = 0; i < kPlanCache; ++i)
    if (ctx->plans[i].valid && ctx->plans[i].M == M && ctx->plans[i].w_dtype == w_dtype) return ctx->plans[i].pl;
  PlanEntry& e = ctx->plans[ctx->plan_next];
  ctx->plan_next = (ctx->plan_next + 1) % kPlanCache;
  e.pl = make_plan(ctx, M, w_dtype);
  e.M = M; e.w_dtype = w_dtype; e.valid = 1;
  return e.pl;
}

// K-major 2-D tensor map with a box of 64 elements x box_rows.  bf16: 128-byte swizzle (the layout the MMA reads);
// int8: plain rows of 64 bytes (the converter warps read them).
// int8 with swizzle (8-bit MMA): box of 128 elements = 128 bytes, 128-byte swizzle, the same bytes as a bf16 block.
// `packed4`: rows of cols / 2 bytes holding two 4-bit codes each; box of 32 bytes (64 codes) x box_rows, plain rows.
hola_status encode_map(hola_ctx* ctx, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols,
                       uint32_t box_rows, bool int8 = false, bool int8_swizzled = false, bool packed4 = false) {
  if (packed4) { cols /= 2; int8 = true; int8_swizzled = false; }
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * (int8 ? 1u : 2u)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(packed4 ? kBlockK / 2 : (int8_swizzled ? 2 * kBlockK : kBlockK)),
                             box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = ctx->encode(map, int8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                                 const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                 (int8 && !int8_swizzled) ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof ctx->last_error, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return HOLA_ERR_CUDA;
  }
  return HOLA_OK;
}

hola_status check_common(const hola_ctx* ctx, const hola_verify_args* a) {
  if (!ctx || !a) return HOLA_ERR_INVALID_ARG;
  if (a->B < 0 || a->k < 0 || a->H <= 0 || a->V <= 0) return HOLA_ERR_INVALID_ARG;
  if (a->H != ctx->H || a->V != ctx->V || a->B > ctx->maxB || a->k > ctx->maxK) return HOLA_ERR_UNSUPPORTED_SHAPE;
  if (a->q_dtype != HOLA_Q_BF16 && a->q_dtype != HOLA_Q_F32) return HOLA_ERR_INVALID_ARG;
  if (a->gate_source != HOLA_GATE_TARGET_ENTROPY && a->gate_source != HOLA_GATE_DRAFT_ENTROPY)
    return HOLA_ERR_INVALID_ARG;
  if (a->fallback != HOLA_FALLBACK_SAMPLE && a->fallback != HOLA_FALLBACK_GREEDY) return HOLA_ERR_INVALID_ARG;
  return HOLA_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Steps 1-2: the LM-head GEMM with fused statistics, one launch (clusters of two CTAs) per pass over W_lm.
hola_status run_lm_head(hola_ctx* ctx, const hola_verify_args* a, float* logits, int ldl, const Plan& pl,
                        cudaStream_t stream) {
  const int M = a->B * (a->k + 1);
  const bool mixed = a->w_dtype == HOLA_W_MIXED;
  const bool w8 = a->w_dtype == HOLA_W_INT8 || mixed, two = a->w_dtype == HOLA_W8A16,
             i8 = a->w_dtype == HOLA_W8A8 || two;
  const hola_wmix* mx = mixed ? a->wmix : nullptr;
  // (mixed widths: W_lm of the arguments is not read; the 8-bit buffer takes its place in the cache key and the map)
  const void* w_main = mixed ? (mx->rows8 > 0 ? mx->W8 : (mx->rows4 > 0 ? mx->W4 : mx->W16)) : a->W_lm;
  hola_status s;
  // 8-bit activations: the hidden operand is the context's own buffer of 8-bit planes, filled per call below
  const void* hid_src = (two || i8) ? static_cast<const void*>(ctx->hid8) : a->hidden;
  if ((two || i8) && !ctx->hid8) return HOLA_ERR_INVALID_ARG;   // (the entry point without a context has no room for it)
  if (two || i8) {
    // the same per-row quantiser as for W_lm (one plane), or the two-plane form in blocks of 32 rows
    const int padded = round_up(M, 32);
    cudaLaunchConfig_t qc = {};
    qc.gridDim = dim3(static_cast<unsigned>(two ? padded : M)); qc.blockDim = dim3(256); qc.stream = stream;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // launch latency hides behind the call before
    qa[0].val.programmaticStreamSerializationAllowed = 1;
    qc.attrs = qa; qc.numAttrs = 1;
    const cudaError_t qe =
        two ? cudaLaunchKernelEx(&qc, quantize_rows_two_plane_kernel, static_cast<const __nv_bfloat16*>(a->hidden), M,
                                 a->H, ctx->hid8, ctx->hid_scale, ctx->hid_scale + ctx->max_rows)
            : cudaLaunchKernelEx(&qc, quantize_rows_int8_kernel, static_cast<const __nv_bfloat16*>(a->hidden), a->H,
                                 ctx->hid8, ctx->hid_scale);
    if (qe != cudaSuccess) { set_error(ctx, "launch of the hidden-row quantiser", qe); return HOLA_ERR_CUDA; }
  }
  MapEntry* me = nullptr;
  for (int i = 0; i < kMapCache; ++i) {
    MapEntry& c = ctx->maps[i];
    if (c.valid && c.hidden == hid_src && c.W == w_main && c.M == M && c.w_dtype == a->w_dtype &&
        (!mixed || (c.W4 == mx->W4 && c.W16 == mx->W16))) { me = &c; break; }
  }
  if (!me) {
    me = &ctx->maps[ctx->map_next];
    ctx->map_next = (ctx->map_next + 1) % kMapCache;
    me->valid = 0;
    if (two)
      s = encode_map(ctx, &me->th, hid_src, static_cast<uint64_t>(2 * round_up(M, 32)), static_cast<uint64_t>(a->H),
                     static_cast<uint32_t>(pl.N / 2), true, true);
    else if (i8)
      s = encode_map(ctx, &me->th, hid_src, static_cast<uint64_t>(M), static_cast<uint64_t>(a->H),
                     static_cast<uint32_t>(pl.N / 2), true, true);
    else
      s = encode_map(ctx, &me->th, hid_src, static_cast<uint64_t>(M), static_cast<uint64_t>(a->H),
                     static_cast<uint32_t>(pl.N / 2));
    if (s != HOLA_OK) return s;
    const uint32_t trows = static_cast<uint32_t>(pl.tile_rows);
    if (!mixed) {
      s = encode_map(ctx, &me->tw, a->W_lm, static_cast<uint64_t>(a->V), static_cast<uint64_t>(a->H), trows, w8 || i8, i8);
      if (s != HOLA_OK) return s;
      me->tw4 = me->tw; me->tw16 = me->tw;               // (never read outside the mixed-width form)
      me->W4 = nullptr; me->W16 = nullptr;
    } else {
      // one map per width that occurs; a width that does not occur gets a copy of one that does (never used)
      bool have = false;
      if (mx->rows8 > 0) {
        s = encode_map(ctx, &me->tw, mx->W8, static_cast<uint64_t>(mx->rows8), static_cast<uint64_t>(a->H), trows, true);
        if (s != HOLA_OK) return s;
        have = true;
      }
      if (mx->rows4 > 0) {
        s = encode_map(ctx, &me->tw4, mx->W4, static_cast<uint64_t>(mx->rows4), static_cast<uint64_t>(a->H), trows, true,
                       false, true);
        if (s != HOLA_OK) return s;
        if (!have) me->tw = me->tw4;
        have = true;
      }
      if (mx->rows16 > 0) {
        s = encode_map(ctx, &me->tw16, mx->W16, static_cast<uint64_t>(mx->rows16), static_cast<uint64_t>(a->H), trows);
        if (s != HOLA_OK) return s;
        if (!have) me->tw = me->tw16;
        have = true;
      }
      if (mx->rows4 <= 0) me->tw4 = me->tw;
      if (mx->rows16 <= 0) me->tw16 = me->tw;
      me->W4 = mx->W4; me->W16 = mx->W16;
    }
    me->hidden = hid_src; me->W = w_main; me->M = M; me->w_dtype = a->w_dtype; me->valid = 1;
  }
  const CUtensorMap& th = me->th;
  const CUtensorMap& tw = me->tw;
  const CUtensorMap& tw4 = me->tw4;
  const CUtensorMap& tw16 = me->tw16;
  K1Params kp;
  kp.M = M; kp.V = a->V; kp.n_ptiles = pl.n_ptiles; kp.n_kblocks = pl.n_kblocks;
  kp.pair256 = (pl.rot && pl.N == 128 && !ctx->no_pair256) ? 1 : 0;
  kp.conv_group = ctx->conv_group > 0 ? ctx->conv_group : 2;
  kp.stages = pl.stages; kp.nbuf = pl.nbuf; kp.rot = pl.rot; kp.n_sub = pl.n_sub; kp.N = pl.N; kp.tile_rows = pl.tile_rows; kp.ldl = ldl;
  kp.logits = logits; kp.partials = ctx->partials; kp.part_stride = ctx->max_rows;
  kp.status = a->status_word ? a->status_word : ctx->status;
  kp.w_scale = a->w_scale;
  kp.h_scale = ctx->hid_scale;
  kp.h_scale2 = ctx->hid_scale ? ctx->hid_scale + ctx->max_rows : nullptr;
  kp.stream_logits = static_cast<double>(M) * a->V * 4.0 > 96e6 ? 1 : 0;     // beyond ~3/4 of the L2
  kp.group_width = mixed ? mx->group_width : nullptr;
  kp.group_row = mixed ? mx->group_row : nullptr;
  kp.shift4 = mixed ? mx->shift4 : nullptr;
  kp.rows4 = mixed ? mx->rows4 : 0;
  cudaError_t e = cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(pl.grid));
  cfg.blockDim = dim3(kK1Threads);
  cfg.dynamicSmemBytes = static_cast<size_t>(pl.smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // may start while the kernel before it in the stream drains (its threads wait for that kernel before they touch
  // global memory): launch, barrier set-up and tensor-memory allocation hide behind the previous call's last kernel
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  kp.n_pass = pl.fused ? pl.passes : 1;
  kp.rows_per_pass = pl.rows_per_pass;
  kp.pace = nullptr;
  if (pl.fused && ctx->pace && !ctx->no_pace && pl.grid / (2 * pl.passes) <= kMaxPaceGroups) {
    kp.pace = ctx->pace;
    e = cudaMemsetAsync(ctx->pace, 0, sizeof(unsigned) * static_cast<size_t>(pl.grid / (2 * pl.passes)), stream);
    if (e != cudaSuccess) { set_error(ctx, "reset of the pace counters", e); return HOLA_ERR_CUDA; }
  }
  for (int pass = 0; pass < (pl.fused ? 1 : pl.passes); ++pass) {
    kp.row0 = pass * pl.rows_per_pass;
    kp.rows = M - kp.row0 < pl.rows_per_pass ? M - kp.row0 : pl.rows_per_pass;
    if (kp.rows <= 0) break;
    e = two ? cudaLaunchKernelEx(&cfg, lm_head_entropy_kernel<3, false>, th, tw, tw4, tw16, kp)
      : i8 ? (pl.rot ? cudaLaunchKernelEx(&cfg, lm_head_entropy_kernel<2, true>, th, tw, tw4, tw16, kp)
                     : cudaLaunchKernelEx(&cfg, lm_head_entropy_kernel<2, false>, th, tw, tw4, tw16, kp))
      : w8 ? cudaLaunchKernelEx(&cfg, lm_head_entropy_kernel<1, false>, th, tw, tw4, tw16, kp)
           : (pl.rot ? cudaLaunchKernelEx(&cfg, lm_head_entropy_kernel<0, true>, th, tw, tw4, tw16, kp)
                     : cudaLaunchKernelEx(&cfg, lm_head_entropy_kernel<0, false>, th, tw, tw4, tw16, kp));
    if (e != cudaSuccess) { set_error(ctx, "launch lm_head_entropy_kernel", e); return HOLA_ERR_CUDA; }
  }
  return HOLA_OK;
}

// What the accept/sample kernel needs to know in the vocabulary-parallel form.
struct ShardLaunch {
  int world, rank, v_offset, V_global;
  const float4* stats_all;   // world records (statistics, then draft-token logits)
  int rec_floats;            // floats per record
  double* mass_out;
  const double* mass_all;
};

// `settled`: the launch sits right behind this call's own GEMM kernel (see K3Params::inputs_settled).
hola_status run_accept_sample(hola_ctx* ctx, const hola_verify_args* a, const float* logits, int ldl, int combine,
                              int nparts, cudaStream_t stream, const float* q_tok = nullptr, int phase = 0,
                              const ShardLaunch* sh = nullptr, bool settled = false, const void* q_far = nullptr,
                              int q_far_from = 0) {
  K3Params kp{};
  kp.q_far = q_far; kp.q_far_from = q_far_from;
  kp.q_tok = q_tok; kp.phase = phase; kp.inputs_settled = settled ? 1 : 0;
  kp.B = a->B; kp.k = a->k; kp.V = a->V; kp.ldl = ldl; kp.logits = logits;
  kp.partials = ctx->partials; kp.nparts = nparts; kp.part_stride = ctx->max_rows; kp.combine = combine;
  kp.tok = a->draft_tok; kp.q = a->draft_q; kp.q_dtype = a->q_dtype; kp.u = a->uniforms; kp.tau = a->tau;
  kp.gate_source = a->gate_source; kp.fallback = a->fallback; kp.hq_part = nullptr; kp.draft_entropy = a->draft_entropy;
  if (a->gate_source == HOLA_GATE_DRAFT_ENTROPY && a->k > 0) {
    // one more pass over the draft rows: H(q_j) for every (sequence, draft position) - unless the caller has put it
    // on the side stream already, next to the GEMM
    if (!ctx->hq_ready) {
      draft_entropy_kernel<<<dim3(static_cast<unsigned>(a->B * a->k), kHqSlices), 256, 0, stream>>>(
          a->draft_q, a->q_dtype, a->V, ctx->hq);
      const cudaError_t e0 = cudaGetLastError();
      if (e0 != cudaSuccess) { set_error(ctx, "launch draft_entropy_kernel", e0); return HOLA_ERR_CUDA; }
    }
    kp.hq_part = ctx->hq;
  }
  kp.accept_len = a->accept_len; kp.next_tok = a->next_tok; kp.entropy = a->entropy; kp.logZ = a->logZ;
  kp.status = a->status_word ? a->status_word : ctx->status;
  if (sh) {
    kp.shard_world = sh->world; kp.shard_rank = sh->rank; kp.v_offset = sh->v_offset; kp.V_global = sh->V_global;
    kp.lx_all = reinterpret_cast<const float*>(sh->stats_all) + 4 * static_cast<size_t>(a->B) * (a->k + 1);
    kp.rec_stride = sh->rec_floats;
    kp.mass_out = sh->mass_out; kp.mass_all = sh->mass_all;
    if (combine) { kp.partials = sh->stats_all; kp.nparts = sh->world; kp.part_stride = sh->rec_floats / 4; }
  }
  const bool vec = (a->V % 4 == 0) && (ldl % 4 == 0) && aligned16(logits) && (a->k == 0 || aligned16(a->draft_q));
  // cluster size: as many CTAs per sequence as keeps the grid within a few waves of the SMs
  const int nchunks = (a->V + kChunk - 1) / kChunk;
  int S = 8;
  while (S > 1 && (a->B * S > kK3MaxPerSm * ctx->num_sms || nchunks / S < 8)) S >>= 1;   // one wave of CTAs
  if (phase == 1) S = 1;                                 // no vocabulary pass: one CTA per sequence
  const int cpc = (nchunks + S - 1) / S;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(a->B * S));
  cfg.blockDim = dim3(kK3Threads);
  cfg.dynamicSmemBytes = static_cast<size_t>(cpc) * sizeof(double);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(S);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // May be scheduled as soon as every CTA of the kernel before it in the stream has exited; it waits for that
  // kernel's results itself.  (The GEMM kernel does not release its dependents earlier: their CTAs would then pile
  // up on whichever SMs its first CTAs leave, and the 8-CTA clusters of a large batch run unbalanced.)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const cudaError_t e = vec ? cudaLaunchKernelEx(&cfg, accept_sample_kernel<true>, kp)
                            : cudaLaunchKernelEx(&cfg, accept_sample_kernel<false>, kp);
  if (e != cudaSuccess) { set_error(ctx, "launch accept_sample_kernel", e); return HOLA_ERR_CUDA; }
  return HOLA_OK;
}

hola_status check_lm_head_args(const hola_ctx* ctx, const hola_verify_args* a) {
  if (a->w_dtype < HOLA_W_BF16 || a->w_dtype > HOLA_W_MIXED) return HOLA_ERR_INVALID_ARG;
  if (a->w_dtype == HOLA_W_MIXED) {
    // vocabulary groups of mixed width: the weights come through args->wmix, W_lm is not read
    const hola_wmix* mx = a->wmix;
    if (!a->hidden || !aligned16(a->hidden) || !mx || !a->w_scale) return HOLA_ERR_INVALID_ARG;
    if (a->H % kSubBlock != 0) return HOLA_ERR_UNSUPPORTED_SHAPE;          // whole sub-blocks of 128 hidden channels
    if (mx->rows4 < 0 || mx->rows8 < 0 || mx->rows16 < 0 || !mx->group_width || !mx->group_row) return HOLA_ERR_INVALID_ARG;
    if (static_cast<long long>(mx->rows4) + mx->rows8 + mx->rows16 < a->V) return HOLA_ERR_INVALID_ARG;
    if ((mx->rows4 > 0 && (!mx->W4 || !mx->shift4 || !aligned16(mx->W4))) || (mx->rows8 > 0 && (!mx->W8 || !aligned16(mx->W8))) ||
        (mx->rows16 > 0 && (!mx->W16 || !aligned16(mx->W16))))
      return HOLA_ERR_INVALID_ARG;
    return HOLA_OK;
  }
  if (!a->hidden || !a->W_lm) return HOLA_ERR_INVALID_ARG;
  if (!aligned16(a->hidden) || !aligned16(a->W_lm)) return HOLA_ERR_INVALID_ARG;
  if (a->H % 8 != 0) return HOLA_ERR_UNSUPPORTED_SHAPE;
  if (a->w_dtype != HOLA_W_BF16) {
    if (!a->w_scale) return HOLA_ERR_INVALID_ARG;
    if (a->H % 16 != 0) return HOLA_ERR_UNSUPPORTED_SHAPE;     // int8 row pitch must be a multiple of 16 bytes
  }
  (void)ctx;
  return HOLA_OK;
}

hola_status check_sample_args(const hola_verify_args* a) {
  if (!a->uniforms || !a->accept_len || !a->next_tok || !a->entropy || !a->logZ) return HOLA_ERR_INVALID_ARG;
  if (a->k > 0 && (!a->draft_tok || !a->draft_q)) return HOLA_ERR_INVALID_ARG;
  return HOLA_OK;
}

// Once per context (and once per device for the entry point without one), with the device current: the kernels that
// ask for more dynamic shared memory than the default limit are told so here, not on every call.
cudaError_t configure_kernels() {
  cudaError_t e = cudaSuccess;
  const void* kernels[] = {reinterpret_cast<const void*>(lm_head_entropy_kernel<0, false>),
                           reinterpret_cast<const void*>(lm_head_entropy_kernel<0, true>),
                           reinterpret_cast<const void*>(lm_head_entropy_kernel<1, false>),
                           reinterpret_cast<const void*>(lm_head_entropy_kernel<2, false>),
                           reinterpret_cast<const void*>(lm_head_entropy_kernel<2, true>),
                           reinterpret_cast<const void*>(lm_head_entropy_kernel<3, false>)};
  for (const void* k : kernels)
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
  return e;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

// ------------------------------------------------------------------------------------------------ C ABI
extern "C" {

const char* hola_version(void) { return "0.1"; }

const char* hola_strerror(hola_status s) {
  switch (s) {
    case HOLA_OK: return "ok";
    case HOLA_ERR_INVALID_ARG: return "invalid argument (null pointer, bad size or misaligned buffer)";
    case HOLA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (H % 8 != 0, or sizes beyond the context's limits)";
    case HOLA_ERR_WORKSPACE: return "workspace allocation failed";
    case HOLA_ERR_CUDA: return "CUDA call failed (see hola_last_cuda_error)";
    case HOLA_ERR_NO_DEVICE: return "no usable sm_100 device";
    case HOLA_ERR_STATIC_LIMIT:
      return "problem too large for the fixed scratch of hola_lm_head_entropy_static (more than 512 verify rows)";
    default: return "unknown status";
  }
}

const char* hola_last_cuda_error(const hola_ctx* ctx) { return ctx ? ctx->last_error : ""; }

size_t hola_workspace_bytes(int maxB, int maxK, int H, int V) {
  if (maxB <= 0 || maxK < 0 || H <= 0 || V <= 0) return 0;
  return ws_layout(maxB, maxK, H, V, kAssumedSms).total;
}

hola_status hola_create(hola_ctx** out, int device, int maxB, int maxK, int H, int V) {
  if (!out) return HOLA_ERR_INVALID_ARG;
  *out = nullptr;
  if (maxB <= 0 || maxK < 0 || H <= 0 || V <= 0) return HOLA_ERR_INVALID_ARG;
  if (H % 8 != 0 || maxK + 1 > kMaxK1 || V > kMaxChunks * kChunk) return HOLA_ERR_UNSUPPORTED_SHAPE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return HOLA_ERR_NO_DEVICE;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return HOLA_ERR_NO_DEVICE;
  if (prop.major != 10) return HOLA_ERR_NO_DEVICE;       // the kernels are sm_100a only; there is no fallback
  DeviceGuard guard(device);
  if (!guard.ok) return HOLA_ERR_NO_DEVICE;

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return HOLA_ERR_NO_DEVICE;

  hola_ctx* ctx = static_cast<hola_ctx*>(calloc(1, sizeof(hola_ctx)));
  if (!ctx) return HOLA_ERR_WORKSPACE;
  ctx->device = device; ctx->num_sms = prop.multiProcessorCount; ctx->maxB = maxB; ctx->maxK = maxK;
  ctx->H = H; ctx->V = V; ctx->ldl = static_cast<int>(align_up(static_cast<size_t>(V), 4));
  ctx->max_rows = maxB * (maxK + 1);
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  ctx->host_overlap = 1;
  ctx->host_lazy_q = -1;
  ctx->host_in_place = 1;
  if (configure_kernels() != cudaSuccess) { free(ctx); return HOLA_ERR_CUDA; }
  const WsLayout w = ws_layout(maxB, maxK, H, V, ctx->num_sms);
  const cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->ws), w.total);
  if (e != cudaSuccess) { free(ctx); return HOLA_ERR_WORKSPACE; }
  ctx->ws_bytes = w.total;
  ctx->logits = reinterpret_cast<float*>(ctx->ws + w.logits);
  ctx->partials = reinterpret_cast<float4*>(ctx->ws + w.partials);
  ctx->status = reinterpret_cast<unsigned*>(ctx->ws + w.status);
  ctx->pace = reinterpret_cast<unsigned*>(ctx->ws + w.pace);
  ctx->hq = reinterpret_cast<double*>(ctx->ws + w.hq);
  ctx->hid8 = reinterpret_cast<signed char*>(ctx->ws + w.hid8);
  ctx->hid_scale = reinterpret_cast<float*>(ctx->ws + w.hid_scale);
  ctx->st_hidden = ctx->ws + w.st_hidden; ctx->st_tok = reinterpret_cast<int*>(ctx->ws + w.st_tok);
  ctx->st_q = ctx->ws + w.st_q; ctx->st_u = reinterpret_cast<float*>(ctx->ws + w.st_u);
  ctx->st_out = reinterpret_cast<unsigned char*>(ctx->ws + w.st_out);
  ctx->st_qtok = reinterpret_cast<float*>(ctx->ws + w.st_qtok);
  cudaMemset(ctx->status, 0, 4);
  const size_t n_qtok = static_cast<size_t>(maxB) * (maxK > 0 ? maxK : 1);
  void* pinned = nullptr;
  if (cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&ctx->copy_done, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&ctx->fork_point, cudaEventDisableTiming) != cudaSuccess ||
      cudaHostAlloc(&pinned, (w.st_small_end - w.st_tok) + maxB * 4 + 16 + out_block(maxB, maxK).total,
                    cudaHostAllocDefault) != cudaSuccess) {
    if (ctx->copy_done) cudaEventDestroy(ctx->copy_done);
    if (ctx->fork_point) cudaEventDestroy(ctx->fork_point);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    cudaFree(ctx->ws);
    free(ctx);
    return HOLA_ERR_CUDA;
  }
  ctx->h_small = static_cast<unsigned char*>(pinned);
  ctx->small_u_off = w.st_u - w.st_tok;
  ctx->small_qtok_off = w.st_qtok - w.st_tok;
  ctx->small_span = w.st_small_end - w.st_tok;
  ctx->h_qtok = reinterpret_cast<float*>(ctx->h_small + ctx->small_qtok_off);
  ctx->h_accept = reinterpret_cast<int*>(ctx->h_small + ctx->small_span);
  (void)n_qtok;
  ctx->h_out = reinterpret_cast<unsigned char*>(align_up(reinterpret_cast<size_t>(ctx->h_accept + maxB), 16));
  *out = ctx;
  return HOLA_OK;
}

hola_status hola_destroy(hola_ctx* ctx) {
  if (!ctx) return HOLA_OK;
  DeviceGuard guard(ctx->device);
  for (int i = 0; i < 3 * ctx->prof_cap; ++i) cudaEventDestroy(ctx->prof_ev[i]);
  free(ctx->prof_ev);
  if (ctx->copy_done) cudaEventDestroy(ctx->copy_done);
  if (ctx->fork_point) cudaEventDestroy(ctx->fork_point);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  if (ctx->h_small) cudaFreeHost(ctx->h_small);
  cudaFree(ctx->ws);
  free(ctx);
  return HOLA_OK;
}

hola_status hola_plan_for_shape(int num_sms, int H, int V, int rows, int w_dtype, hola_plan_info* out) {
  if (!out || num_sms < 2 || H <= 0 || V <= 0 || rows <= 0) return HOLA_ERR_INVALID_ARG;
  if (w_dtype < HOLA_W_BF16 || w_dtype > HOLA_W_MIXED) return HOLA_ERR_INVALID_ARG;
  if (H % 8 != 0 || V > kMaxChunks * kChunk) return HOLA_ERR_UNSUPPORTED_SHAPE;
  hola_ctx* c = static_cast<hola_ctx*>(calloc(1, sizeof(hola_ctx)));     // only the fields make_plan reads
  if (!c) return HOLA_ERR_WORKSPACE;
  c->num_sms = num_sms; c->H = H; c->V = V;
  const Plan pl = make_plan(c, rows, w_dtype);
  free(c);
  out->tile_v = 2 * pl.tile_rows; out->grid = pl.grid; out->stages = pl.stages; out->rows_per_pass = pl.rows_per_pass;
  out->passes = pl.passes; out->kernels_per_call = (pl.fused ? 1 : pl.passes) + 1;
  return HOLA_OK;
}

hola_status hola_plan_ex(const hola_ctx* ctx, int B, int k, int w_dtype, hola_plan_info* out) {
  if (!ctx || !out || B < 0 || k < 0) return HOLA_ERR_INVALID_ARG;
  if (w_dtype < HOLA_W_BF16 || w_dtype > HOLA_W_MIXED) return HOLA_ERR_INVALID_ARG;
  if (B > ctx->maxB || k > ctx->maxK) return HOLA_ERR_UNSUPPORTED_SHAPE;
  const Plan pl = make_plan(ctx, B * (k + 1), w_dtype);
  out->tile_v = 2 * pl.tile_rows; out->grid = pl.grid; out->stages = pl.stages; out->rows_per_pass = pl.rows_per_pass;
  out->passes = pl.passes; out->kernels_per_call = (pl.fused ? 1 : pl.passes) + 1;
  return HOLA_OK;
}

hola_status hola_plan(const hola_ctx* ctx, int B, int k, hola_plan_info* out) {
  return hola_plan_ex(ctx, B, k, HOLA_W_BF16, out);
}

hola_status hola_set_option(hola_ctx* ctx, int option, int value) {
  if (!ctx) return HOLA_ERR_INVALID_ARG;
  switch (option) {
    case HOLA_OPT_RING_SLOTS:
      if (value != 0 && (value < 2 || value > kMaxStages)) return HOLA_ERR_INVALID_ARG;
      ctx->force_stages = value;
      break;
    case HOLA_OPT_ROTATING_UNITS: ctx->no_rot = value == 0; break;
    case HOLA_OPT_PAIR_MMA: ctx->no_pair256 = value == 0; break;
    case HOLA_OPT_HOST_IN_PLACE: ctx->host_in_place = value != 0; break;
    case HOLA_OPT_FUSED_PASSES:
      if (value < 0 || value > 2) return HOLA_ERR_INVALID_ARG;
      ctx->no_fuse = value == 0;
      ctx->no_pace = value == 2;
      break;
    case HOLA_OPT_CONVERTER_GROUP:
      if (value < 0 || value > kConvWarps) return HOLA_ERR_INVALID_ARG;
      ctx->conv_group = value;
      break;
    case HOLA_OPT_PASSES:
      if (value < 0 || value > 64) return HOLA_ERR_INVALID_ARG;
      ctx->force_passes = value;
      break;
    case HOLA_OPT_HOST_OVERLAP: ctx->host_overlap = value != 0; break;
    case HOLA_OPT_HOST_ROWS_ON_DEMAND:
      if (value < -1 || value > 1) return HOLA_ERR_INVALID_ARG;
      ctx->host_lazy_q = value;
      break;
    default: return HOLA_ERR_INVALID_ARG;
  }
  for (int i = 0; i < kPlanCache; ++i) ctx->plans[i].valid = 0;     // the launch geometry may have changed
  for (int i = 0; i < kMapCache; ++i) ctx->maps[i].valid = 0;
  return HOLA_OK;
}

hola_status hola_selftest_bounded_wait(hola_ctx* ctx, long long limit_cycles, uint32_t* status_word,
                                       uint32_t* counters, void* cuda_stream) {
  if (!ctx || !status_word || !counters) return HOLA_ERR_INVALID_ARG;
  if (limit_cycles < 1000 || limit_cycles > 200000000ll) return HOLA_ERR_INVALID_ARG;   // at most ~0.1 s of SM clock
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(counters, 0, 2 * sizeof(uint32_t), stream) != cudaSuccess) return HOLA_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2); cfg.blockDim = dim3(64); cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, bounded_wait_selftest_kernel, limit_cycles,
                                           static_cast<unsigned*>(status_word), static_cast<unsigned*>(counters));
  if (e != cudaSuccess) { set_error(ctx, "launch bounded_wait_selftest_kernel", e); return HOLA_ERR_CUDA; }
  return HOLA_OK;
}

hola_status hola_lm_head_entropy(hola_ctx* ctx, const hola_verify_args* a, void* cuda_stream) {
  hola_status s = check_common(ctx, a);
  if (s != HOLA_OK) return s;
  if (a->B == 0) return HOLA_OK;
  if ((s = check_lm_head_args(ctx, a)) != HOLA_OK) return s;
  if (!a->entropy || !a->logZ) return HOLA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int M = a->B * (a->k + 1);
  const Plan& pl = plan_for(ctx, M, a->w_dtype);
  float* logits = a->logits_out ? a->logits_out : ctx->logits;
  const int ldl = a->logits_out ? a->V : ctx->ldl;
  if ((s = run_lm_head(ctx, a, logits, ldl, pl, stream)) != HOLA_OK) return s;
  finalize_kernel<<<(M + 7) / 8, 256, 0, stream>>>(ctx->partials, pl.grid, ctx->max_rows, M, a->logZ, a->entropy);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_error(ctx, "launch finalize_kernel", e); return HOLA_ERR_CUDA; }
  return HOLA_OK;
}

hola_status hola_accept_sample(hola_ctx* ctx, const hola_verify_args* a, void* cuda_stream) {
  hola_status s = check_common(ctx, a);
  if (s != HOLA_OK) return s;
  if (a->B == 0) return HOLA_OK;
  if ((s = check_sample_args(a)) != HOLA_OK) return s;
  if (!a->logits_out) return HOLA_ERR_INVALID_ARG;
  if (a->fallback == HOLA_FALLBACK_GREEDY) return HOLA_ERR_INVALID_ARG;   // needs the arg-max of the fused path
  DeviceGuard guard(ctx->device);
  return run_accept_sample(ctx, a, a->logits_out, a->V, 0, 0, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

namespace {

// The whole step on device buffers.  `before_sample`, when given, is an event the accept/sample part waits for
// (the draft tensor still being copied in by hola_verify_host).
hola_status verify_device(hola_ctx* ctx, const hola_verify_args* a, cudaStream_t stream, cudaEvent_t before_sample) {
  const Plan& pl = plan_for(ctx, a->B * (a->k + 1), a->w_dtype);
  float* logits = a->logits_out ? a->logits_out : ctx->logits;
  const int ldl = a->logits_out ? a->V : ctx->ldl;
  const bool prof = ctx->prof_on && ctx->prof_n < ctx->prof_cap;
  cudaEvent_t* ev = prof ? ctx->prof_ev + 3 * ctx->prof_n : nullptr;
  if (prof) cudaEventRecord(ev[0], stream);
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) capturing = cudaStreamCaptureStatusActive;
  // The pass over the draft rows (draft-entropy gate) depends on nothing the GEMM makes, and its small CTAs fit on the
  // SMs beside the GEMM's: it runs on the context's side stream (behind the copy of the draft tensor, when the host
  // entry put one there), branching off the caller's stream before the GEMM and joining it again before the
  // accept/sample kernel.  It is launched AFTER the GEMM so that the GEMM's CTAs get their SMs first.
  // (While the caller records a graph everything stays on the caller's stream.)
  const bool side = a->gate_source == HOLA_GATE_DRAFT_ENTROPY && a->k > 0 &&
                    (before_sample || capturing == cudaStreamCaptureStatusNone);
  if (side && !before_sample && cudaEventRecord(ctx->fork_point, stream) != cudaSuccess) return HOLA_ERR_CUDA;
  hola_status s = run_lm_head(ctx, a, logits, ldl, pl, stream);
  if (s != HOLA_OK) return s;
  if (prof) cudaEventRecord(ev[1], stream);
  if (side) {
    cudaError_t e = cudaSuccess;
    if (!before_sample) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->fork_point, 0);
    if (e == cudaSuccess) {
      draft_entropy_kernel<<<dim3(static_cast<unsigned>(a->B * a->k), kHqSlices), 256, 0, ctx->copy_stream>>>(
          a->draft_q, a->q_dtype, a->V, ctx->hq);
      e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaEventRecord(ctx->copy_done, ctx->copy_stream);
    if (e != cudaSuccess) { set_error(ctx, "draft_entropy_kernel on the side stream", e); return HOLA_ERR_CUDA; }
    before_sample = ctx->copy_done;
  }
  if (before_sample && cudaStreamWaitEvent(stream, before_sample, 0) != cudaSuccess) return HOLA_ERR_CUDA;
  ctx->hq_ready = side ? 1 : 0;
  // (behind the GEMM kernel: the caller's inputs are settled; an event wait in between makes it an ordinary launch)
  s = run_accept_sample(ctx, a, logits, ldl, 1, pl.grid, stream, nullptr, 0, nullptr, true);
  ctx->hq_ready = 0;
  if (prof) { cudaEventRecord(ev[2], stream); ctx->prof_n++; }
  return s;
}

// hola_verify_host while the target entropy gates.  Of the draft tensor the step then reads k single probabilities
// per sequence (q_j(x_j), gathered here on the host) and at most ONE row per sequence: row accept_len, and none when
// every draft token was kept or the fallback is greedy.  Rows 0 .. ahead-1 of every sequence (as many as the bus
// carries while the GEMM runs, at least one) are sent ahead on the context's own stream; after the accept test the
// accept lengths come back and only the rows still missing follow.  Same kernels, same arithmetic and so the same
// results as the whole-tensor copy.
constexpr double kHostBusBytesPerSecond = 50e9;          // what a pinned host-to-device copy reaches here

// Draft rows per sequence that can cross the bus while the GEMM of this call runs.
int rows_under_gemm(hola_ctx* ctx, const hola_verify_args* a) {
  const Plan& pl = plan_for(ctx, a->B * (a->k + 1), a->w_dtype);
  const double group = static_cast<double>(a->B) * a->V * (a->q_dtype == HOLA_Q_BF16 ? 2 : 4);
  const double n = pl.est_seconds * kHostBusBytesPerSecond / group;
  return n > 1e6 ? 1000000 : static_cast<int>(n);
}

hola_status verify_host_lazy(hola_ctx* ctx, const hola_verify_args* a, cudaStream_t stream, int ahead) {
  const int B = a->B, k = a->k, V = a->V;
  const size_t rows = static_cast<size_t>(B) * (k + 1);
  const size_t q_elem = a->q_dtype == HOLA_Q_BF16 ? 2 : 4;
  const size_t row_bytes = static_cast<size_t>(V) * q_elem;
  const bool sample = a->fallback != HOLA_FALLBACK_GREEDY;
  cudaError_t e = cudaSuccess;
  unsigned long long up = 0, down = 0;
  auto h2d = [&](void* dst, const void* src, size_t bytes, cudaStream_t st) {
    if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st);
    up += bytes;
  };
  auto d2h = [&](void* dst, const void* src, size_t bytes) {
    if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, stream);
    down += bytes;
  };
  for (int b = 0; b < B; ++b)
    for (int j = 0; j < k; ++j) {
      const int x = a->draft_tok[b * k + j];
      float qx = 0.f;
      if (x >= 0 && x < V) {
        const size_t qi = (static_cast<size_t>(b) * k + j) * V + x;
        if (a->q_dtype == HOLA_Q_BF16) {
          const uint32_t bits = static_cast<uint32_t>(static_cast<const uint16_t*>(a->draft_q)[qi]) << 16;
          memcpy(&qx, &bits, 4);
        } else {
          qx = static_cast<const float*>(a->draft_q)[qi];
        }
      }
      ctx->h_qtok[b * k + j] = qx;
    }
  h2d(ctx->st_hidden, a->hidden, rows * a->H * 2, stream);
  // tokens, uniforms and the gathered probabilities: into the pinned mirror, then one copy of the span in use
  memcpy(ctx->h_small, a->draft_tok, static_cast<size_t>(B) * k * 4);
  memcpy(ctx->h_small + ctx->small_u_off, a->uniforms, rows * 4);
  h2d(ctx->st_tok, ctx->h_small, ctx->small_qtok_off + static_cast<size_t>(B) * k * 4, stream);
  const OutBlock ob = out_block(B, k);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->st_out, 0, 4, stream);
  const size_t seq_pitch = static_cast<size_t>(k) * row_bytes;   // from row (b, 0) to row (b + 1, 0)
  ahead = ahead < 1 ? 1 : (ahead > k ? k : ahead);
  const size_t ahead_bytes = static_cast<size_t>(ahead) * row_bytes;     // rows 0 .. ahead-1 of a sequence are adjacent
  if (sample) {
    if (seq_pitch < (1ull << 31)) {
      if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(ctx->st_q, seq_pitch, a->draft_q, seq_pitch, ahead_bytes, static_cast<size_t>(B),
                              cudaMemcpyHostToDevice, ctx->copy_stream);
      up += static_cast<size_t>(B) * ahead_bytes;
    } else {
      for (int b = 0; b < B; ++b)
        h2d(static_cast<char*>(ctx->st_q) + b * seq_pitch, static_cast<const char*>(a->draft_q) + b * seq_pitch,
            ahead_bytes, ctx->copy_stream);
    }
    if (e == cudaSuccess) e = cudaEventRecord(ctx->copy_done, ctx->copy_stream);
  }
  if (e != cudaSuccess) { set_error(ctx, "host-to-device copy", e); return HOLA_ERR_CUDA; }
  hola_verify_args d = *a;
  d.hidden = ctx->st_hidden; d.draft_tok = ctx->st_tok; d.draft_q = ctx->st_q; d.uniforms = ctx->st_u;
  d.accept_len = reinterpret_cast<int*>(ctx->st_out + ob.accept);
  d.next_tok = reinterpret_cast<int*>(ctx->st_out + ob.next);
  d.entropy = reinterpret_cast<float*>(ctx->st_out + ob.entropy);
  d.logZ = reinterpret_cast<float*>(ctx->st_out + ob.logZ);
  d.logits_out = nullptr; d.status_word = reinterpret_cast<uint32_t*>(ctx->st_out); d.draft_entropy = nullptr;
  hola_status s = check_lm_head_args(ctx, &d);
  if (s != HOLA_OK) return s;
  const Plan& pl = plan_for(ctx, B * (k + 1), a->w_dtype);
  if ((s = run_lm_head(ctx, &d, ctx->logits, ctx->ldl, pl, stream)) != HOLA_OK) return s;
  // Where the caller's draft tensor is pinned host memory that the device can address, the rows still missing after the
  // accept test are not copied at all: the accept/sample kernel reads row accept_len of a sequence in place, over the
  // bus, when that row is not among the ones sent ahead.  One launch, no read-back in the middle of the call.
  const void* q_far = nullptr;
  if (sample && ctx->host_in_place) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, a->draft_q) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer)
      q_far = at.devicePointer;
    else
      cudaGetLastError();                                // (an unregistered pointer is not an error of this call)
  }
  if (!sample) {
    if ((s = run_accept_sample(ctx, &d, ctx->logits, ctx->ldl, 1, pl.grid, stream, ctx->st_qtok, 0)) != HOLA_OK) return s;
  } else if (q_far) {
    if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->copy_done, 0);
    if (e != cudaSuccess) { set_error(ctx, "wait for the draft rows sent ahead", e); return HOLA_ERR_CUDA; }
    if ((s = run_accept_sample(ctx, &d, ctx->logits, ctx->ldl, 1, pl.grid, stream, ctx->st_qtok, 0, nullptr, false, q_far,
                               ahead)) != HOLA_OK)
      return s;
  } else {
    if ((s = run_accept_sample(ctx, &d, ctx->logits, ctx->ldl, 1, pl.grid, stream, ctx->st_qtok, 1)) != HOLA_OK) return s;
    d2h(ctx->h_accept, d.accept_len, static_cast<size_t>(B) * 4);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) { set_error(ctx, "accept lengths to host", e); return HOLA_ERR_CUDA; }
    for (int b = 0; b < B; ++b) {
      const int n = ctx->h_accept[b];
      if (n >= ahead && n < k) {
        const size_t off = (static_cast<size_t>(b) * k + n) * row_bytes;
        h2d(static_cast<char*>(ctx->st_q) + off, static_cast<const char*>(a->draft_q) + off, row_bytes, stream);
      }
    }
    if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->copy_done, 0);
    if (e != cudaSuccess) { set_error(ctx, "host-to-device copy of draft rows", e); return HOLA_ERR_CUDA; }
    // statistics and accept lengths are in place: this launch repeats the (cheap) accept test and draws the token
    if ((s = run_accept_sample(ctx, &d, ctx->logits, ctx->ldl, 0, 0, stream, ctx->st_qtok, 0)) != HOLA_OK) return s;
  }
  d2h(ctx->h_out, ctx->st_out, ob.dent);                 // every output in one copy
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) { set_error(ctx, "device-to-host copy", e); return HOLA_ERR_CUDA; }
  memcpy(a->accept_len, ctx->h_out + ob.accept, static_cast<size_t>(B) * 4);
  memcpy(a->next_tok, ctx->h_out + ob.next, static_cast<size_t>(B) * 4);
  memcpy(a->entropy, ctx->h_out + ob.entropy, rows * 4);
  memcpy(a->logZ, ctx->h_out + ob.logZ, rows * 4);
  if (a->status_word) memcpy(a->status_word, ctx->h_out + ob.status, 4);
  if (q_far) {                                           // rows the kernel read over the bus count as bytes sent
    for (int b = 0; b < B; ++b) {
      const int n = a->accept_len[b];
      if (n >= ahead && n < k) up += row_bytes;
    }
  }
  ctx->last_h2d = up; ctx->last_d2h = down;
  return HOLA_OK;
}

}  // namespace

extern "C" {

hola_status hola_verify(hola_ctx* ctx, const hola_verify_args* a, void* cuda_stream) {
  hola_status s = check_common(ctx, a);
  if (s != HOLA_OK) return s;
  if (a->B == 0) return HOLA_OK;
  if ((s = check_lm_head_args(ctx, a)) != HOLA_OK) return s;
  if ((s = check_sample_args(a)) != HOLA_OK) return s;
  DeviceGuard guard(ctx->device);
  return verify_device(ctx, a, static_cast<cudaStream_t>(cuda_stream), nullptr);
}

hola_status hola_profile_begin(hola_ctx* ctx, int max_calls) {
  if (!ctx || max_calls <= 0 || max_calls > 4096) return HOLA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (ctx->prof_cap < max_calls) {
    cudaEvent_t* ev = static_cast<cudaEvent_t*>(calloc(static_cast<size_t>(3) * max_calls, sizeof(cudaEvent_t)));
    if (!ev) return HOLA_ERR_WORKSPACE;
    for (int i = 0; i < 3 * max_calls; ++i) {
      const cudaError_t e = cudaEventCreate(&ev[i]);
      if (e != cudaSuccess) { set_error(ctx, "cudaEventCreate", e); free(ev); return HOLA_ERR_CUDA; }
    }
    for (int i = 0; i < 3 * ctx->prof_cap; ++i) cudaEventDestroy(ctx->prof_ev[i]);
    free(ctx->prof_ev);
    ctx->prof_ev = ev;
    ctx->prof_cap = max_calls;
  }
  ctx->prof_n = 0;
  ctx->prof_on = 1;
  return HOLA_OK;
}

hola_status hola_profile_end(hola_ctx* ctx, void* cuda_stream, double* lm_head_ms, double* accept_sample_ms,
                             int* calls) {
  if (!ctx || !lm_head_ms || !accept_sample_ms || !calls) return HOLA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  ctx->prof_on = 0;
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) { set_error(ctx, "cudaStreamSynchronize", e); return HOLA_ERR_CUDA; }
  double a = 0.0, b = 0.0;
  for (int i = 0; i < ctx->prof_n; ++i) {
    float ms1 = 0.f, ms2 = 0.f;
    e = cudaEventElapsedTime(&ms1, ctx->prof_ev[3 * i], ctx->prof_ev[3 * i + 1]);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms2, ctx->prof_ev[3 * i + 1], ctx->prof_ev[3 * i + 2]);
    if (e != cudaSuccess) { set_error(ctx, "cudaEventElapsedTime", e); return HOLA_ERR_CUDA; }
    a += ms1; b += ms2;
  }
  *lm_head_ms = a; *accept_sample_ms = b; *calls = ctx->prof_n;
  return HOLA_OK;
}

hola_status hola_verify_host(hola_ctx* ctx, const hola_verify_args* a, void* cuda_stream) {
  hola_status s = check_common(ctx, a);
  if (s != HOLA_OK) return s;
  if (a->B == 0) return HOLA_OK;
  if (!a->hidden || (!a->W_lm && a->w_dtype != HOLA_W_MIXED)) return HOLA_ERR_INVALID_ARG;
  if ((s = check_sample_args(a)) != HOLA_OK) return s;
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t rows = static_cast<size_t>(a->B) * (a->k + 1);
  const size_t q_elem = a->q_dtype == HOLA_Q_BF16 ? 2 : 4;
  if (ctx->host_lazy_q && a->k > 0 && a->gate_source == HOLA_GATE_TARGET_ENTROPY) {
    // when the whole draft tensor crosses the bus under the GEMM anyway, the plain copy below has one launch and
    // one synchronisation fewer
    const int ahead = rows_under_gemm(ctx, a);
    if (ctx->host_lazy_q > 0 || ahead < a->k) return verify_host_lazy(ctx, a, stream, ahead);
  }
  cudaError_t e = cudaSuccess;
  unsigned long long up = 0, down = 0;
  auto h2d = [&](void* dst, const void* src, size_t bytes) {
    if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, stream);
    up += bytes;
  };
  auto d2h = [&](void* dst, const void* src, size_t bytes) {
    if (e == cudaSuccess && bytes) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, stream);
    down += bytes;
  };
  // The small inputs go first (copies queue on the DMA engine in issue order).  The draft tensor is by far the
  // largest input and only the accept/sample part reads it: it travels on the context's own stream while the
  // GEMM runs on the caller's.  (The previous call synchronised before returning, so the staging is free.)
  h2d(ctx->st_hidden, a->hidden, rows * a->H * 2);
  memcpy(ctx->h_small, a->draft_tok, static_cast<size_t>(a->B) * a->k * 4);
  memcpy(ctx->h_small + ctx->small_u_off, a->uniforms, rows * 4);
  h2d(ctx->st_tok, ctx->h_small, ctx->small_u_off + rows * 4);
  const size_t q_bytes = static_cast<size_t>(a->B) * a->k * a->V * q_elem;
  const bool overlap = q_bytes && ctx->host_overlap;
  if (overlap) {
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->st_q, a->draft_q, q_bytes, cudaMemcpyHostToDevice, ctx->copy_stream);
    if (e == cudaSuccess) e = cudaEventRecord(ctx->copy_done, ctx->copy_stream);
    up += q_bytes;
  } else {
    h2d(ctx->st_q, a->draft_q, q_bytes);
  }
  const OutBlock ob = out_block(a->B, a->k);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->st_out, 0, 4, stream);
  if (e != cudaSuccess) { set_error(ctx, "host-to-device copy", e); return HOLA_ERR_CUDA; }
  hola_verify_args d = *a;
  d.hidden = ctx->st_hidden; d.draft_tok = ctx->st_tok; d.draft_q = ctx->st_q; d.uniforms = ctx->st_u;
  d.accept_len = reinterpret_cast<int*>(ctx->st_out + ob.accept);
  d.next_tok = reinterpret_cast<int*>(ctx->st_out + ob.next);
  d.entropy = reinterpret_cast<float*>(ctx->st_out + ob.entropy);
  d.logZ = reinterpret_cast<float*>(ctx->st_out + ob.logZ);
  d.logits_out = nullptr; d.status_word = reinterpret_cast<uint32_t*>(ctx->st_out);
  const bool want_dent = a->draft_entropy && a->gate_source == HOLA_GATE_DRAFT_ENTROPY;
  d.draft_entropy = a->draft_entropy ? reinterpret_cast<float*>(ctx->st_out + ob.dent) : nullptr;
  if ((s = check_lm_head_args(ctx, &d)) != HOLA_OK) return s;
  if ((s = verify_device(ctx, &d, stream, overlap ? ctx->copy_done : nullptr)) != HOLA_OK) return s;
  d2h(ctx->h_out, ctx->st_out, want_dent ? ob.total : ob.dent);      // every output in one copy
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) { set_error(ctx, "device-to-host copy", e); return HOLA_ERR_CUDA; }
  memcpy(a->accept_len, ctx->h_out + ob.accept, static_cast<size_t>(a->B) * 4);
  memcpy(a->next_tok, ctx->h_out + ob.next, static_cast<size_t>(a->B) * 4);
  memcpy(a->entropy, ctx->h_out + ob.entropy, rows * 4);
  memcpy(a->logZ, ctx->h_out + ob.logZ, rows * 4);
  if (a->status_word) memcpy(a->status_word, ctx->h_out + ob.status, 4);
  if (want_dent) memcpy(a->draft_entropy, ctx->h_out + ob.dent, static_cast<size_t>(a->B) * a->k * 4);
  ctx->last_h2d = up; ctx->last_d2h = down;
  return HOLA_OK;
}

// ---- vocabulary-parallel form: three calls per step with two small all-gathers between them (made by the caller)
size_t hola_shard_record_bytes(int B, int k) {
  if (B <= 0 || k < 0) return 0;
  const size_t rows = static_cast<size_t>(B) * (k + 1);
  return rows * 16 + align_up(static_cast<size_t>(B) * k * 4, 16);
}

static hola_status check_shard(const hola_ctx* ctx, const hola_verify_args* a, const hola_shard_args* sh) {
  if (!sh || sh->world < 1 || sh->rank < 0 || sh->rank >= sh->world) return HOLA_ERR_INVALID_ARG;
  if (sh->v_offset < 0 || sh->V_global < sh->v_offset + a->V) return HOLA_ERR_INVALID_ARG;
  if (a->gate_source != HOLA_GATE_TARGET_ENTROPY) return HOLA_ERR_INVALID_ARG;   // H(q_j) would need q of all shards
  (void)ctx;
  return HOLA_OK;
}

static ShardLaunch shard_launch(const hola_verify_args* a, const hola_shard_args* sh) {
  ShardLaunch l;
  l.world = sh->world; l.rank = sh->rank; l.v_offset = sh->v_offset; l.V_global = sh->V_global;
  l.stats_all = static_cast<const float4*>(sh->records);
  l.rec_floats = static_cast<int>(hola_shard_record_bytes(a->B, a->k) / 4);
  l.mass_out = sh->mass_out; l.mass_all = sh->masses;
  return l;
}

hola_status hola_shard_lm_head(hola_ctx* ctx, const hola_verify_args* a, const hola_shard_args* sh, void* cuda_stream) {
  hola_status s = check_common(ctx, a);
  if (s != HOLA_OK) return s;
  if (a->B == 0) return HOLA_OK;
  if ((s = check_lm_head_args(ctx, a)) != HOLA_OK) return s;
  if ((s = check_shard(ctx, a, sh)) != HOLA_OK) return s;
  if (!sh->record_out || !aligned16(sh->record_out) || (a->k > 0 && !a->draft_tok)) return HOLA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int M = a->B * (a->k + 1);
  const Plan& pl = plan_for(ctx, M, a->w_dtype);
  float* logits = a->logits_out ? a->logits_out : ctx->logits;
  const int ldl = a->logits_out ? a->V : ctx->ldl;
  if ((s = run_lm_head(ctx, a, logits, ldl, pl, stream)) != HOLA_OK) return s;
  float4* stats_out = static_cast<float4*>(sh->record_out);
  float* lx_out = reinterpret_cast<float*>(stats_out + M);
  const int blocks = (M + 7) / 8 + (a->B * a->k + 255) / 256;
  shard_record_kernel<<<blocks, 256, 0, stream>>>(ctx->partials, pl.grid, ctx->max_rows, M, sh->v_offset, a->V, logits,
                                                  ldl, a->draft_tok, a->B, a->k, stats_out, lx_out);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { set_error(ctx, "launch shard_record_kernel", e); return HOLA_ERR_CUDA; }
  return HOLA_OK;
}

static hola_status shard_phase(hola_ctx* ctx, const hola_verify_args* a, const hola_shard_args* sh, void* cuda_stream,
                               int phase) {
  hola_status s = check_common(ctx, a);
  if (s != HOLA_OK) return s;
  if (a->B == 0) return HOLA_OK;
  if ((s = check_sample_args(a)) != HOLA_OK) return s;
  if ((s = check_shard(ctx, a, sh)) != HOLA_OK) return s;
  if (!sh->records || !aligned16(sh->records) || (a->k > 0 && !sh->q_tok)) return HOLA_ERR_INVALID_ARG;
  if (phase == 3 && !sh->mass_out) return HOLA_ERR_INVALID_ARG;
  if (phase == 4 && (!sh->masses || a->fallback == HOLA_FALLBACK_GREEDY)) return HOLA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  const float* logits = a->logits_out ? a->logits_out : ctx->logits;
  const int ldl = a->logits_out ? a->V : ctx->ldl;
  const ShardLaunch l = shard_launch(a, sh);
  return run_accept_sample(ctx, a, logits, ldl, phase == 3 ? 1 : 0, 0, static_cast<cudaStream_t>(cuda_stream),
                           sh->q_tok, phase, &l);
}

hola_status hola_shard_accept(hola_ctx* ctx, const hola_verify_args* a, const hola_shard_args* sh, void* cuda_stream) {
  return shard_phase(ctx, a, sh, cuda_stream, 3);
}

hola_status hola_shard_sample(hola_ctx* ctx, const hola_verify_args* a, const hola_shard_args* sh, void* cuda_stream) {
  return shard_phase(ctx, a, sh, cuda_stream, 4);
}

hola_status hola_host_traffic(const hola_ctx* ctx, unsigned long long* h2d_bytes, unsigned long long* d2h_bytes) {
  if (!ctx || !h2d_bytes || !d2h_bytes) return HOLA_ERR_INVALID_ARG;
  *h2d_bytes = ctx->last_h2d; *d2h_bytes = ctx->last_d2h;
  return HOLA_OK;
}

hola_status hola_quantize_w4(const void* W_bf16, int rows, int H, void* packed_out, uint8_t* shift_out, int shift_stride,
                             float* scale_out, void* cuda_stream) {
  if (!W_bf16 || !packed_out || !shift_out || !scale_out || rows <= 0 || H <= 0 || shift_stride < rows)
    return HOLA_ERR_INVALID_ARG;
  if (H % kSubBlock != 0) return HOLA_ERR_UNSUPPORTED_SHAPE;
  quantize_rows_w4_kernel<<<static_cast<unsigned>(rows), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const __nv_bfloat16*>(W_bf16), H, static_cast<uint8_t*>(packed_out), shift_out, shift_stride, scale_out);
  return cudaGetLastError() == cudaSuccess ? HOLA_OK : HOLA_ERR_CUDA;
}

hola_status hola_quantize_w8(const void* W_bf16, int V, int H, void* q_out, float* scale_out, void* cuda_stream) {
  if (!W_bf16 || !q_out || !scale_out || V <= 0 || H <= 0) return HOLA_ERR_INVALID_ARG;
  quantize_rows_int8_kernel<<<static_cast<unsigned>(V), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const __nv_bfloat16*>(W_bf16), H, static_cast<signed char*>(q_out), scale_out);
  return cudaGetLastError() == cudaSuccess ? HOLA_OK : HOLA_ERR_CUDA;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------ no-allocation entry
// hola_lm_head_entropy_static: steps 1-2 for callers that must not allocate device memory.  The per-CTA softmax
// statistics, which hola_lm_head_entropy keeps in the context's cudaMalloc'ed workspace, live here in a fixed
// array inside the library image; logits, entropy and logZ go to the caller's buffers as usual.

namespace {

constexpr int kStaticMaxRows = 512;    // verify rows B(k+1) one call may have
constexpr int kStaticMaxCtas = 160;    // CTAs of the GEMM kernel that may leave statistics (one per SM; B200 has 148)
constexpr size_t kStaticStatusBytes = 256;
constexpr size_t kStaticScratchBytes =
    kStaticStatusBytes + static_cast<size_t>(kStaticMaxCtas) * kStaticMaxRows * sizeof(float4);   // 1 310 976 bytes

}  // namespace

// Every GPU that loads the library holds this array until the process exits.  In host code the name is only a
// handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

constexpr int kStaticMaxDevices = 64;
std::mutex g_static_mu;
hola_ctx g_static_ctx[kStaticMaxDevices];      // host-side descriptors only; they own no memory
bool g_static_ready[kStaticMaxDevices];

// Once per device, with that device current: where the array lives on this device, the tensor-map encoder of the
// driver, and the SM count.  Allocates nothing.
hola_status static_setup(int dev, hola_ctx* out) {
  std::lock_guard<std::mutex> lock(g_static_mu);
  hola_ctx* c = &g_static_ctx[dev];
  if (!g_static_ready[dev]) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess || prop.major != 10) return HOLA_ERR_NO_DEVICE;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return HOLA_ERR_NO_DEVICE;
    void* base = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&base, g_static_scratch);
    if (e != cudaSuccess || !base) return HOLA_ERR_CUDA;
    if (configure_kernels() != cudaSuccess) return HOLA_ERR_CUDA;
    memset(c, 0, sizeof *c);
    c->device = dev;
    c->num_sms = prop.multiProcessorCount;
    c->encode = reinterpret_cast<EncodeTiledFn>(fn);
    c->status = reinterpret_cast<unsigned*>(base);
    c->partials = reinterpret_cast<float4*>(static_cast<unsigned char*>(base) + kStaticStatusBytes);
    c->max_rows = kStaticMaxRows;
    g_static_ready[dev] = true;
  }
  *out = *c;
  return HOLA_OK;
}

}  // namespace

extern "C" hola_status hola_lm_head_entropy_static(const hola_verify_args* a, void* cuda_stream) {
  if (!a) return HOLA_ERR_INVALID_ARG;
  if (a->B < 0 || a->k < 0 || a->H <= 0 || a->V <= 0) return HOLA_ERR_INVALID_ARG;
  if (a->B == 0) return HOLA_OK;
  if (!a->hidden || !a->W_lm || !a->logits_out || !a->entropy || !a->logZ) return HOLA_ERR_INVALID_ARG;
  if (!aligned16(a->hidden) || !aligned16(a->W_lm)) return HOLA_ERR_INVALID_ARG;
  if (a->H % 8 != 0) return HOLA_ERR_UNSUPPORTED_SHAPE;
  const long long rows = static_cast<long long>(a->B) * (a->k + 1);
  if (rows > kStaticMaxRows) return HOLA_ERR_STATIC_LIMIT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return HOLA_ERR_NO_DEVICE;
  hola_ctx local;                      // a per-call copy: concurrent host threads do not share host state
  hola_status s = static_setup(dev, &local);
  if (s != HOLA_OK) return s;
  local.H = a->H; local.V = a->V; local.maxB = a->B; local.maxK = a->k;
  const int M = static_cast<int>(rows);
  if (a->w_dtype != HOLA_W_BF16) return HOLA_ERR_INVALID_ARG;   // the 8-bit weight modes need a context's workspace
  const Plan pl = make_plan(&local, M, a->w_dtype);
  if (pl.grid > kStaticMaxCtas) return HOLA_ERR_STATIC_LIMIT;
  // a timed-out wait must be visible to the caller: the kernels report to the caller's status word when there is one
  // (run_lm_head picks it), else to the word inside the array, which nobody outside can read
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // The array keeps whatever the last call left.  The statistics slots are fully overwritten for the rows of this
  // call before they are read; the internal status word is the one thing that must start at zero.
  if (cudaMemsetAsync(local.status, 0, sizeof(unsigned), stream) != cudaSuccess) return HOLA_ERR_CUDA;
  if ((s = run_lm_head(&local, a, a->logits_out, a->V, pl, stream)) != HOLA_OK) return s;
  finalize_kernel<<<(M + 7) / 8, 256, 0, stream>>>(local.partials, pl.grid, local.max_rows, M, a->logZ, a->entropy);
  return cudaGetLastError() == cudaSuccess ? HOLA_OK : HOLA_ERR_CUDA;
}
