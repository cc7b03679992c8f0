// Device-side building blocks for sm_100a: mbarrier, TMA, tcgen05 (MMA, TMEM) wrappers.
// Every wait is bounded: on expiry it records an error word and lets the caller bail out.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace lg {

// ---- workspace header (first 256 bytes of every workspace) ---------------------------
struct WsHeader {
  unsigned int error_word;         // 0 = ok; else (code << 24) | site.  code 1: a wait gave up, 2: shared memory
                                   // misaligned, 3: the workspace does not hold the lists the call was told it holds,
                                   // 4: a schedule value out of range (checked builds only)
  unsigned int latched;            // an error word that a later call found unread and kept for lg_last_status
  unsigned long long magic;        // kWsMagic once the header has been initialised by a call
  unsigned long long fingerprint;  // which pattern the lists and schedules below were built for (0: none)
  unsigned int pad[58];
};
constexpr int kDqEntInts = 5;   // ints per entry of the schedule of the dQ pass that reads dS back (dq_sched_kernel)
constexpr unsigned long long kWsMagic = 0x4c47575348445231ull;   // "LGWSHDR1"
static_assert(sizeof(WsHeader) == 256, "header size");

// A call that was told its workspace holds prepared lists checks, before it reads any of them,
// that the header carries a fingerprint it accepts; otherwise the CTA records code 3 and returns.
__device__ __forceinline__ bool lists_match(unsigned int* error_word, unsigned long long fp, unsigned long long fp2,
                                            unsigned int site) {
  if (fp == 0) return true;
  const unsigned long long have = reinterpret_cast<const volatile WsHeader*>(error_word)->fingerprint;
  if (have == fp || have == fp2) return true;
  if (threadIdx.x == 0) atomicCAS(error_word, 0u, (3u << 24) | site);
  return false;
}

// Checked builds (-DLG_DEBUG): every value read from a schedule or list that is later used as an index, an
// offset or an address passes through here.  A value outside [lo, hi] is recorded in the status word
// (code 4, with the site) and replaced by the nearest bound, so that a damaged workspace shows up as a
// status instead of a fault.  In normal builds this is the identity.
__device__ __forceinline__ int checked(int v, int lo, int hi, unsigned int* error_word, unsigned int site) {
#ifdef LG_DEBUG
  if (v < lo || v > hi) {
    atomicCAS(error_word, 0u, (4u << 24) | site);
    return v < lo ? lo : hi;
  }
#else
  (void)lo; (void)hi; (void)error_word; (void)site;
#endif
  return v;
}

constexpr long long kWaitLimitCycles = 4000000000ll;   // ~2 s of SM clock: a wait that long gave up

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31; }

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---- mbarrier -------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (after recording `site` in the error word) if the phase
// never completed; callers then skip the rest of their work and fall through to cleanup.
// The first probe is inlined: a wait that is already satisfied costs one try_wait.
static __device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, unsigned int* error_word,
                                                   uint32_t site, long long limit_cycles = kWaitLimitCycles) {
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int it = 0; it < 256; ++it) {
      if (mbar_try_wait(bar, parity)) return true;
    }
    if (clock64() - t0 > limit_cycles) break;
  }
  if (error_word) atomicCAS(error_word, 0u, (1u << 24) | site);
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned int* error_word,
                                          uint32_t site) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, error_word, site);
}
// Whole-warp wait: one lane watches the barrier, the others wait at the warp barrier (which
// also orders their later reads after the lane's observation).  Returns the same value in
// every lane.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, unsigned int* error_word,
                                               uint32_t site) {
  // common case: the phase is over already and every lane sees that with one probe of its own
  if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
  bool ok = true;
  if (lane_id() == 0) ok = mbar_wait(bar, parity, error_word, site);
  ok = __all_sync(0xffffffffu, ok);
  __syncwarp();
  return ok;
}

// ---- TMA (tiled bulk tensor copies, no multicast) ------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const void* tmap, uint64_t* bar, int c0, int c1,
                                            int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(bar)), "r"(c0), "r"(c1),
      "r"(c2), "r"(c3)
      : "memory");
}
// ask for a tile to be brought into the L2 (no shared memory, no barrier: nothing to wait for)
__device__ __forceinline__ void tma_prefetch_l2_4d(const void* tmap, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(
                   reinterpret_cast<uint64_t>(tmap)),
               "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}
// untiled bulk copy global -> shared (addresses 16-byte aligned, size a multiple of 16 bytes)
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// the same with an L2 cache policy for the source lines
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
// generic-proxy smem writes -> visible to the async proxy (tcgen05.mma operands read from shared memory)
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---- tcgen05: TMEM allocation ---------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_slot, uint32_t ncols) {  // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- tcgen05: descriptors -------------------------------------------------------------
// Instruction descriptor for kind::f16 with bf16 operands and fp32 accumulation.
// a_mn / b_mn: operand is MN-major (1) or K-major (0).
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn) << 15) |
         (static_cast<uint32_t>(b_mn) << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// Shared-memory matrix descriptors (128-byte swizzle, rows of 128 bytes packed in groups of 8 =
// 1024-byte atoms), given as (low word, high word).  The high word (stride between 8-row groups,
// descriptor version, swizzle mode) is constant for an operand kind and the low word is
// (address >> 4) | (leading-dimension field << 16) -- the leading dimension being the distance
// between 64-element column groups of an MN-major operand (ignored for K-major) -- so stepping
// through the K slices of a tile costs the issuing thread one 32-bit add per operand.
// mma_ss2: D[tmem] (+)= A[smem] * B[smem];  mma_ts2: D[tmem] (+)= A[tmem] * B[smem].
// (layout: 2 = 128-byte swizzle, 0 = none -- core matrices of 8 rows x 16 bytes placed by the two offsets)
__device__ __forceinline__ uint32_t desc_hi(uint32_t sbo_bytes, uint32_t layout = 2) {
  return ((sbo_bytes >> 4) & 0x3FFF) | (1u << 14) | (layout << 29);
}
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
  return ((smem_addr & 0x3FFFF) >> 4) | (((lbo_bytes >> 4) & 0x3FFF) << 16);
}
__device__ __forceinline__ void mma_ss2(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the same with a descriptor high word of its own for A (an operand in another shared-memory layout)
__device__ __forceinline__ void mma_ss2x(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                         uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_ts2(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives once all tcgen05 operations issued so far by this thread completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// ---- tcgen05: TMEM <-> registers (each thread: its own lane, consecutive columns) -----
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]),
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
      "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- which (head, launch rank) a CTA works ----------------------------------------------
// CTAs start in the order of their linear index (x fastest).  With x = head, the CTAs that run at one time
// spread over all heads, a handful of tiles each, and the operand tiles that neighbouring tiles of one
// head share (the window's K / V in the forward, its Q / dO in the dK/dV pass) have to stay in the L2 for
// every head at once: 80 MB at 32 heads, more than the L2 holds of it (measured at cfg 3: 22.9 GB of DRAM
// reads in the dK/dV pass against 4.3 GB of operands; 4.6 GB with groups of four).  Heads can therefore be
// taken in groups of `group`: linear index w -> group w / (group * n_y), and inside a group the heads
// alternate and the ranks advance, so that 148 CTAs cover ~ 37 neighbouring tiles of 4 heads.  The host
// asks for it where the tiles of a head take about the same time (sink + window well below the sequence
// length), and for full causal attention, where every tile of a head streams the same rows from the same
// end (K / V from the first key in the forward and the dQ pass, Q / dO from the last query in the dK/dV
// pass): with two heads at a time the tiles that run together share what they stream, and the DRAM reads
// of the three kernels at 128K fall from 0.5 / 1.1 / 0.5 TB to 5 / 8 / 7 GB (fwd + bwd 664 -> 523 ms).
// Strided combs keep all heads side by side (group = n_x): a few very long tiles per head make the
// longest-first launch order over all heads worth more; only the dK/dV pass takes its comb tiles two or four
// heads at a time (cta_coords2).
constexpr int kHeadGroup = 4;
constexpr int kHeadGroupCombs = 2;     // strided pattern, dK/dV pass: the comb tiles of this many kv heads at a time
constexpr int kHeadGroupCombsGqa = 4;  // the same with grouped queries
constexpr int kHeadGroupFull = 2;   // full causal attention: every tile of a head streams the same rows from the same end
__device__ __forceinline__ void cta_coords(long long w, int n_x, int n_y, int group, int& x, int& y) {
  const long long per_group = static_cast<long long>(group) * n_y;
  const int grp = static_cast<int>(w / per_group);
  const int rem = static_cast<int>(w - grp * per_group);
  const int size = min(group, n_x - grp * group);   // the last group may be smaller
  x = grp * group + rem % size;
  y = rem / size;
}
// The same with two regions of launch ranks: the first n_long ranks in groups of `group` heads, the rest with
// all heads side by side (a strided pattern's few long comb tiles per head, and the many short ones behind
// them, which fill the tail whatever head the last long tile belongs to).
__device__ __forceinline__ void cta_coords2(long long w, int n_x, int n_y, int group, int n_long, int& x, int& y) {
  const long long first = static_cast<long long>(n_x) * n_long;
  if (n_long >= n_y || w < first) { cta_coords(w, n_x, n_long < n_y ? n_long : n_y, group, x, y); return; }
  x = static_cast<int>((w - first) % n_x);
  y = n_long + static_cast<int>((w - first) / n_x);
}

// ---- small math helpers --------------------------------------------------------------
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// packed pairs of fp32 (one instruction for two lanes of work on sm_100)
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Epilogue of an accumulator tile: fp32 columns [taddr, taddr + 64) of this warp's 32 tensor-memory lanes
// (lane = row), times `mul`, as bf16 to global rows.  A thread holds a whole row, so storing straight from its
// registers makes every store instruction of the warp touch 32 rows (32 separate 16-byte pieces); the
// rows go through `stage` (4 KB of shared memory of this warp's own, 16-byte chunks XOR-swizzled by the row)
// instead, and every store instruction then writes four whole 128-byte rows.  row_ptr(r) = where the 64
// columns of row r (0 .. 31 of this warp) go, or nullptr for a row that is not stored.  The whole warp calls.
template <typename RowPtr>
__device__ __forceinline__ void store_acc_64cols(uint32_t taddr, uint8_t* stage, float mul, RowPtr row_ptr) {
  const uint32_t lane = lane_id();
  const uint32_t sbase = smem_u32(stage);
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    uint32_t reg[32];
    tmem_ld32(taddr + c * 32, reg);
    tmem_ld_wait();
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const uint32_t w0 = pack_bf16(__uint_as_float(reg[8 * x + 0]) * mul, __uint_as_float(reg[8 * x + 1]) * mul);
      const uint32_t w1 = pack_bf16(__uint_as_float(reg[8 * x + 2]) * mul, __uint_as_float(reg[8 * x + 3]) * mul);
      const uint32_t w2 = pack_bf16(__uint_as_float(reg[8 * x + 4]) * mul, __uint_as_float(reg[8 * x + 5]) * mul);
      const uint32_t w3 = pack_bf16(__uint_as_float(reg[8 * x + 6]) * mul, __uint_as_float(reg[8 * x + 7]) * mul);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbase + lane * 128 + (((4 * c + x) ^ (lane & 7)) << 4)),
                   "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
    }
  }
  __syncwarp();
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t row = 4 * k + (lane >> 3), ch = lane & 7;
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(sbase + row * 128 + ((ch ^ (row & 7)) << 4)) : "memory");
    __nv_bfloat16* dst = row_ptr(static_cast<int>(row));
    if (dst) *reinterpret_cast<uint4*>(dst + ch * 8) = v;
  }
  __syncwarp();   // the stage may be written again
}


}  // namespace lg
