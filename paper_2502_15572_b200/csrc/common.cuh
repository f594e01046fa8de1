// Device-side building blocks shared by the retrieval kernels (sm_100a).
//
//  * candidate packing: (score, id) -> one u64 whose unsigned order is
//    "score descending, then id ascending" (Eq. 3's arg max extended to the
//    n best, ties to the lower row index);
//  * warp-wide bitonic sort / merge of such words held one per lane;
//  * WarpTopN: a warp-private running top-n list with a candidate queue;
//  * mbarrier + TMA (cp.async.bulk.tensor) wrappers with BOUNDED waits.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dresd {

constexpr int kListLen = 32;            // lanes of one warp-held list (>= top_n)
constexpr int kQueueCap = 32;           // pending candidates per (warp, query)
constexpr int kMergeLevel = 16;         // merge the queue once it holds this many
constexpr int kStatusTimeout = -5;      // value of DRESD_ERR_TIMEOUT
constexpr long long kWaitCycles = 4000000000LL;  // ~2-3 s at B200 clocks

// ---------------------------------------------------------------------------
// (score, id) <-> orderable u64.  0 is "empty" and sorts below every candidate.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t float_to_ordered(float f)      // monotone float -> uint, never 0
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_float(uint32_t u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}
__device__ __forceinline__ unsigned long long pack_candidate(float score, uint32_t id)
{
    score += 0.0f;                                   // -0.0 -> +0.0: one zero
    return (static_cast<unsigned long long>(float_to_ordered(score)) << 32) | (0xFFFFFFFFu - id);
}
__device__ __forceinline__ float candidate_score(unsigned long long p)
{
    return ordered_to_float(static_cast<uint32_t>(p >> 32));
}

// Grid-wide filter: every CTA's n-th best score is a lower bound of the final n-th
// best, so the maximum over CTAs (kept per query in global memory, ordered-uint
// encoded, 0 = nothing known) may be used by all of them to reject rows early.
// The filter only rejects rows that cannot be in the result, so the result does not
// depend on when a CTA sees an update.
__device__ __forceinline__ float share_tau(unsigned int *gtau, float local)
{
    if (!(local > -INFINITY)) {
        const unsigned int g = *reinterpret_cast<volatile unsigned int *>(gtau);
        return g ? ordered_to_float(g) : local;
    }
    const unsigned int mine = float_to_ordered(local);
    const unsigned int old = atomicMax(gtau, mine);
    return old > mine ? ordered_to_float(old) : local;
}
__device__ __forceinline__ float peek_tau(const unsigned int *gtau, float current)
{
    const unsigned int g = *reinterpret_cast<const volatile unsigned int *>(gtau);
    const float t = g ? ordered_to_float(g) : -INFINITY;
    return t > current ? t : current;
}
__device__ __forceinline__ uint32_t candidate_id(unsigned long long p)
{
    return 0xFFFFFFFFu - static_cast<uint32_t>(p);
}

__device__ __forceinline__ unsigned long long shfl_xor_u64(unsigned long long v, int m)
{
    return __shfl_xor_sync(0xFFFFFFFFu, v, m);
}
__device__ __forceinline__ unsigned long long shfl_u64(unsigned long long v, int src)
{
    return __shfl_sync(0xFFFFFFFFu, v, src);
}
__device__ __forceinline__ unsigned long long umax64(unsigned long long a, unsigned long long b)
{
    return a > b ? a : b;
}
__device__ __forceinline__ unsigned long long umin64(unsigned long long a, unsigned long long b)
{
    return a < b ? a : b;
}

// Sort 32 words (one per lane) so that lane 0 holds the largest.
__device__ __forceinline__ unsigned long long warp_sort_desc(unsigned long long x, int lane)
{
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            unsigned long long o = shfl_xor_u64(x, j);
            bool desc_block = (lane & k) == 0;       // k == 32: always true
            bool lower = (lane & j) == 0;
            x = (lower == desc_block) ? umax64(x, o) : umin64(x, o);
        }
    }
    return x;
}
// Turn a bitonic sequence (one word per lane) into descending order.
__device__ __forceinline__ unsigned long long warp_bitonic_merge_desc(unsigned long long x, int lane)
{
#pragma unroll
    for (int j = 16; j > 0; j >>= 1) {
        unsigned long long o = shfl_xor_u64(x, j);
        x = ((lane & j) == 0) ? umax64(x, o) : umin64(x, o);
    }
    return x;
}
// Top 32 of the union of two descending lists a, b (one word per lane each).
__device__ __forceinline__ unsigned long long warp_merge_top32(unsigned long long a,
                                                               unsigned long long b, int lane)
{
    unsigned long long rb = shfl_u64(b, 31 - lane);  // ascending copy of b
    return warp_bitonic_merge_desc(umax64(a, rb), lane);
}

// ---------------------------------------------------------------------------
// WarpTopN: running top-n of one (warp, query) pair.  All state is in shared
// memory owned by ONE warp, so no CTA-wide synchronisation is ever needed in
// the streaming loop.  Candidates that pass the cheap score filter are queued;
// the queue is folded into the sorted list kMergeLevel at a time.
// ---------------------------------------------------------------------------
struct WarpTopN {
    unsigned long long list[kListLen];   // sorted descending; slots >= n are 0
    unsigned long long queue[kQueueCap];
    int count;                           // entries waiting in queue
    float tau;                           // filter: score of the n-th best so far
};

__device__ __forceinline__ void warp_topn_init(WarpTopN *s, int lane)
{
    s->list[lane] = 0ull;
    if (lane == 0) {
        s->count = 0;
        s->tau = -INFINITY;
    }
    __syncwarp();
}

// Fold the queue into the sorted list and tighten the filter score (-inf while
// fewer than n candidates are known).  Call with all 32 lanes.
static __device__ __noinline__ void warp_topn_merge(WarpTopN *s, int n, int lane)
{
    int count = s->count;
    unsigned long long x = lane < count ? s->queue[lane] : 0ull;
    x = warp_sort_desc(x, lane);
    unsigned long long m = warp_merge_top32(s->list[lane], x, lane);
    if (lane >= n) m = 0ull;
    unsigned long long nth = shfl_u64(m, n - 1);
    __syncwarp();
    s->list[lane] = m;
    if (lane == 0) {
        s->count = 0;
        s->tau = nth ? candidate_score(nth) : -INFINITY;
    }
    __syncwarp();
}

// Append this lane's candidate (if `take`) to the queue of one (warp, query).
// Call with all 32 lanes.  Overflow is handled by merging first; the queue is
// merged again once it reaches kMergeLevel so the filter stays tight.
static __device__ __noinline__ void warp_topn_push(WarpTopN *s, int n, int lane, bool take, float score,
                                            uint32_t id)
{
    unsigned m = __ballot_sync(0xFFFFFFFFu, take);
    if (m == 0) return;
    int incoming = __popc(m);
    if (s->count + incoming > kQueueCap) warp_topn_merge(s, n, lane);
    int count = s->count;
    if (take) s->queue[count + __popc(m & ((1u << lane) - 1u))] = pack_candidate(score, id);
    __syncwarp();
    if (lane == 0) s->count = count + incoming;
    __syncwarp();
    if (count + incoming >= kMergeLevel) warp_topn_merge(s, n, lane);
}

// ---------------------------------------------------------------------------
// mbarrier / TMA wrappers.  Every wait is bounded: after kWaitCycles the
// caller gets `false`, records a timeout and leaves its loop.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
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
// Bounded wait; false = gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, long long limit = kWaitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}
// 2-D tiled TMA load global -> shared, completion on `bar`.  x is the
// innermost (element) coordinate and must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y,
                                            uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];" ::"r"(smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// ---------------------------------------------------------------------------
// Programmatic dependent launch: the kernels of one retrieve call form a chain (K1 -> scan ->
// merge).  A kernel launched with launch_dependent() may start while its predecessor still
// runs: it sets up (barriers, TMEM) and then blocks in pdl_wait() until the predecessor has
// completed and its writes are visible; a kernel calls pdl_launch_dependents() as early as it
// likes to let its successor be scheduled.  Both are no-ops in a kernel launched the plain way.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args &&...args)
{
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------------------
// tcgen05 / TMEM wrappers (5th-generation tensor cores)
// ---------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t *smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Same for 8-bit operands (E4M3 here): K = 32 per instruction, still 32 bytes of a row.
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// E4M3 conversions (round to nearest even, saturating at +-448) and the two-term 8-bit query:
// h1 = e4m3(256 q), h2 = e4m3(16 (256 q - h1)).  Rows 2b / 2b+1 of the operand hold h1 / h2 of
// query b; in the packed form (two 64-byte keys per 128-byte store row) rows 4b .. 4b+3 hold
// (h1|0), (h2|0), (0|h1), (0|h2).
__device__ __forceinline__ uint32_t to_e4m3(float x)
{
    return (uint32_t)__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3);
}
__device__ __forceinline__ float from_e4m3(uint32_t c)
{
    const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3);
    return __half2float(*reinterpret_cast<const __half *>(&h));
}
__device__ __forceinline__ void store_query_e4m3(uint8_t *qsplit8, int dpad8, int pack2, int b, int c, float q)
{
    const float q256 = 256.f * q;
    const uint32_t c1 = to_e4m3(q256);
    const uint32_t c2 = to_e4m3(16.f * (q256 - from_e4m3(c1)));
    if (pack2) {
        if (c >= 64) return;
        uint8_t *r0 = qsplit8 + (size_t)(4 * b) * dpad8;
        r0[c] = (uint8_t)c1;
        r0[64 + c] = 0;
        r0[dpad8 + c] = (uint8_t)c2;
        r0[dpad8 + 64 + c] = 0;
        r0[2 * dpad8 + c] = 0;
        r0[2 * dpad8 + 64 + c] = (uint8_t)c1;
        r0[3 * dpad8 + c] = 0;
        r0[3 * dpad8 + 64 + c] = (uint8_t)c2;
    } else {
        uint8_t *h1 = qsplit8 + (size_t)(2 * b) * dpad8;
        h1[c] = (uint8_t)c1;
        h1[dpad8 + c] = (uint8_t)c2;
    }
}

// Element-type tag of the 8-bit copy of a datastore: the scan kernels see such a store as rows
// of d/2 two-byte units (TMA moves bytes) and only switch the instruction kind.
struct E4M3Keys {};
// K-major operand, 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t *r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld1(uint32_t taddr, uint32_t &v0)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v0) : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld2(uint32_t taddr, uint32_t &v0, uint32_t &v1)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"(v0), "=r"(v1) : "r"(taddr));
}

// ---- CTA pairs (cta_group::2): one MMA spans two SMs of a cluster ------------------------
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t *smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish2()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// TMA load into this CTA's shared memory whose completion bytes are counted on a barrier of
// the pair's leader CTA (`bar_cluster_addr` from mapa_rank); the data go to this CTA only.
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, int x, int y,
                                                 uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];" ::"r"(smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster_addr)
        : "memory");
}

__device__ __forceinline__ void report_timeout(int *status_word)
{
    atomicExch(status_word, kStatusTimeout);
}

// Bounds-checked debug build (-DDRESD_DEBUG_BOUNDS, libdresd_debug.so): every global index and every
// pipeline-ring slot that the kernels form is checked where it is formed; a violation records
// -(1000 + site) in the status word (the first one wins) and the caller SKIPS the access.  In the
// release build the function is the constant `true` and the checks compile to nothing.
constexpr int kStatusBoundsBase = -1000;
#ifdef DRESD_DEBUG_BOUNDS
__device__ __forceinline__ bool debug_check(bool ok, int *status_word, int site)
{
    if (!ok && status_word) atomicCAS(status_word, 0, kStatusBoundsBase - site);
    return ok;
}
#else
__device__ __forceinline__ bool debug_check(bool, int *, int) { return true; }
#endif

}  // namespace dresd
