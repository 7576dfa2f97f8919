// Thread-level building blocks of the barrier-free AllReduce kernels: scoped
// memory operations, bounded polling, element widening/narrowing and the
// data+flag (LL) send/receive on a per-slot, double-buffered scratch region
// (paper Sec. IV "LL", "Bidirectional Communication & Double Buffering";
// Sec. V: send, recv, recvUnrolled, recvReduce, bcast, advanceEpoch).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "symar_layout.h"

namespace symar {

// ---- bounds-checking debug build (-DSYMAR_CHECK) -------------------------------------
// Every global-memory helper below passes its address through SYMAR_PTR(p, bytes, regions):
// in the regular build that is `p`; in the checking build the access must lie wholly inside one
// of the named regions of some rank's segment (for the user region: inside THIS call's input
// or output range), else the violation is recorded -- SYMAR_ERR_INVAL in the heap's status word
// with the rank, the CTA slot and the regions the access was meant for -- and the access is
// SKIPPED: it is redirected to a small sink array, so that nothing outside the sink is read or
// written.  Stands in for a memory checker where none can be run.
enum : uint32_t { kRegIn = 1, kRegOut = 2, kRegLL = 4, kRegSn = 8, kRegAt = 16, kRegReady = 32, kRegDone = 64,
                  kRegCtr = 128 };
#ifdef SYMAR_CHECK
struct CheckCtx {
    const char *base;            // rank 0's segment (nullptr: no heap); the ranges below repeat every `stride`
    uint64_t    stride;
    uint32_t    nranks, nreg, nabs;
    uint64_t    lo[8], hi[8];    // segment-relative byte ranges
    uint32_t    kind[8];
    const char *alo[4], *ahi[4]; // absolute ranges (buffers outside a heap)
    uint32_t    akind[4];
    uint32_t   *ctl;             // heap status words, or nullptr
    uint32_t   *status;          // a caller's status word, or nullptr
};
static __device__ __align__(32) unsigned char g_check_sink[64 * 32];
__device__ __forceinline__ CheckCtx &check_ctx()
{
    __shared__ CheckCtx ctx;
    return ctx;
}
static __device__ __noinline__ void check_fail(const CheckCtx &c, uint32_t allowed)
{
    if (c.ctl && atomicCAS(&c.ctl[kCtlCode], 0u, (uint32_t)SYMAR_ERR_INVAL) == 0u) {
        c.ctl[kCtlRank] = blockIdx.y;
        c.ctl[kCtlPeer] = allowed;
        c.ctl[kCtlCta]  = blockIdx.x;
        __threadfence();
    }
    if (c.status) atomicCAS(c.status, 0u, (uint32_t)SYMAR_ERR_INVAL);
}
static __device__ __noinline__ bool check_range(const void *p, uint64_t bytes, uint32_t allowed)
{
    const CheckCtx &c = check_ctx();
    const char *q     = reinterpret_cast<const char *>(p);
    bool ok           = false;
    if (c.base && q >= c.base && (uint64_t)(q - c.base) < c.stride * c.nranks) {
        const uint64_t o = (uint64_t)(q - c.base) % c.stride;
        for (uint32_t i = 0; i < c.nreg; ++i) ok = ok || ((c.kind[i] & allowed) && o >= c.lo[i] && o + bytes <= c.hi[i]);
    }
    for (uint32_t i = 0; i < c.nabs; ++i) ok = ok || ((c.akind[i] & allowed) && q >= c.alo[i] && q + bytes <= c.ahi[i]);
    if (!ok) check_fail(c, allowed);
    return ok;
}
template <typename T>
__device__ __forceinline__ T *check_ptr(T *p, uint64_t bytes, uint32_t allowed)
{
    if (check_range(p, bytes, allowed)) return p;
    return reinterpret_cast<T *>(g_check_sink + (threadIdx.x & 63u) * 32u);
}
// First statement of every kernel on a heap (all threads): the regions of this call.
__device__ __forceinline__ void check_begin(const KArgs &a, int nranks, uint64_t in_bytes, uint64_t out_bytes)
{
    if (threadIdx.x == 0) {
        CheckCtx &c = check_ctx();
        c.base   = a.seg0;
        c.stride = a.stride;
        c.nranks = (uint32_t)nranks;
        c.nabs   = 0;
        c.ctl    = a.ctl;
        c.status = nullptr;
        const uint64_t lo[8]   = {a.in_off, a.out_off, a.ll_off, a.sn_off, a.at_off, a.ready_off, a.done_off, a.epoch_off};
        const uint64_t hi[8]   = {a.in_off + (in_bytes + 15) / 16 * 16,   // whole vectors are read (the region is padded)
                                  a.out_off + out_bytes, a.sn_off, a.at_off, a.ready_off, a.done_off, a.epoch_off,
                                  a.epoch_off + (uint64_t)kPairBytes};
        const uint32_t kind[8] = {kRegIn, kRegOut, kRegLL, kRegSn, kRegAt, kRegReady, kRegDone, kRegCtr};
        c.nreg = 8;
        for (int i = 0; i < 8; ++i) {
            c.lo[i]   = lo[i];
            c.hi[i]   = hi[i];
            c.kind[i] = kind[i];
        }
    }
    __syncthreads();
}
// message bytes of an AllReduce call
__device__ __forceinline__ uint64_t check_message_bytes(const KArgs &a)
{
    return a.tail_bytes ? (a.nvec - 1) * 16 + a.tail_bytes : a.nvec * 16;
}
#define SYMAR_CHECK_BEGIN(a, nranks, in_bytes, out_bytes) symar::check_begin(a, nranks, in_bytes, out_bytes)
#define SYMAR_CHECK_BEGIN_ALLREDUCE(a, nranks) \
    symar::check_begin(a, nranks, symar::check_message_bytes(a), symar::check_message_bytes(a))
#define SYMAR_PTR(p, bytes, regions) symar::check_ptr(p, bytes, regions)
#define SYMAR_RANGE_OK(p, bytes, regions) symar::check_range(p, bytes, regions)
#else
#define SYMAR_CHECK_BEGIN(a, nranks, in_bytes, out_bytes) ((void)0)
#define SYMAR_CHECK_BEGIN_ALLREDUCE(a, nranks) ((void)0)
#define SYMAR_PTR(p, bytes, regions) (p)
#define SYMAR_RANGE_OK(p, bytes, regions) true
#endif

// ---- memory operations -------------------------------------------------------
// On one device `.gpu` scope is sufficient; a multi-GPU build of the same
// protocol would use `.sys`.  Compiling with -DSYMAR_SCOPE_SYS gives that build
// (every flag, signal and data+flag access at system scope), so that its cost
// can be timed beside the default.
#ifdef SYMAR_SCOPE_SYS
#define SYMAR_SCOPE "sys"
#else
#define SYMAR_SCOPE "gpu"
#endif

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    p = SYMAR_PTR(p, 4, kRegReady | kRegDone);
    uint32_t v;
    asm volatile("ld.acquire." SYMAR_SCOPE ".global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t *p, uint32_t v)
{
    p = SYMAR_PTR(p, 4, kRegReady | kRegDone);
    asm volatile("st.release." SYMAR_SCOPE ".global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p)
{
    p = SYMAR_PTR(p, 4, kRegCtr | kRegIn);
    uint32_t v;
    asm volatile("ld.relaxed." SYMAR_SCOPE ".global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Signal: add 1 to a peer's flag word; release orders every earlier write of
// this thread (and, through the preceding CTA barrier, of its CTA) before it.
__device__ __forceinline__ void red_release_inc_u32(uint32_t *p)
{
    p = SYMAR_PTR(p, 4, kRegReady | kRegDone);
    asm volatile("red.release." SYMAR_SCOPE ".global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
__device__ __forceinline__ void red_relaxed_inc_u32(uint32_t *p)
{
    p = SYMAR_PTR(p, 4, kRegReady | kRegDone);
    asm volatile("red.relaxed." SYMAR_SCOPE ".global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
__device__ __forceinline__ void fence_acq_rel()
{
    asm volatile("fence.acq_rel." SYMAR_SCOPE ";" ::: "memory");
}
__device__ __forceinline__ uint64_t ld_relaxed_u64(const uint64_t *p)
{
    p = SYMAR_PTR(p, 8, kRegCtr);
    uint64_t v;
    asm volatile("ld.relaxed." SYMAR_SCOPE ".global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// 16-byte transfer made of two 8-byte elements.  Each 8-byte element {payload,
// flag} is a single aligned 64-bit access, hence observed whole; the two
// elements need not arrive together because each carries its own flag.
struct __align__(16) U64x2 { uint64_t a, b; };

__device__ __forceinline__ void st_relaxed_v2u64(void *p, uint64_t a, uint64_t b)
{
    p = SYMAR_PTR(p, 16, kRegLL);
    asm volatile("st.relaxed." SYMAR_SCOPE ".global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(a), "l"(b)
                 : "memory");
}
__device__ __forceinline__ U64x2 ld_relaxed_v2u64(const void *p)
{
    p = SYMAR_PTR(p, 16, kRegLL);
    U64x2 v;
    asm volatile("ld.relaxed." SYMAR_SCOPE ".global.v2.u64 {%0, %1}, [%2];"
                 : "=l"(v.a), "=l"(v.b)
                 : "l"(p)
                 : "memory");
    return v;
}

// 16-byte strong accesses of four 32-bit elements (each element a single access)
__device__ __forceinline__ void st_relaxed_v4(void *p, const uint4 &v)
{
    p = SYMAR_PTR(p, 16, kRegSn | kRegAt);
    asm volatile("st.relaxed." SYMAR_SCOPE ".global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y),
                 "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ uint4 ld_relaxed_v4(const void *p)
{
    p = SYMAR_PTR(p, 16, kRegSn | kRegAt);
    uint4 v;
    asm volatile("ld.relaxed." SYMAR_SCOPE ".global.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p)
                 : "memory");
    return v;
}

// A rank's OWN input is written before its kernel starts and never during it:
// read-only path, no L1 allocation.
__device__ __forceinline__ uint4 ld_own(const void *p)
{
    p = SYMAR_PTR(p, 16, kRegIn);
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
// A PEER's input is read only after that peer's "ready" signal was observed: a
// strong (L1-bypassing) load issued after the poll, so it cannot return a line
// cached before the signal.
__device__ __forceinline__ uint4 ld_peer(const void *p)
{
    p = SYMAR_PTR(p, 16, kRegIn);
    uint4 v;
    asm volatile("ld.relaxed." SYMAR_SCOPE ".global.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p)
                 : "memory");
    return v;
}
// Outputs are written once and not re-read by this kernel.
__device__ __forceinline__ void st_output(void *p, uint4 v)
{
    p = SYMAR_PTR(p, 16, kRegOut);
    asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

// 32-byte accesses (two adjacent 16-byte vectors), 32-byte aligned.  Issued
// after this warp's acquire poll, which already dropped any stale L1 line, so
// an ordinary load is enough.
struct U32B { uint4 lo, hi; };
__device__ __forceinline__ U32B ld_peer_32B(const void *p)
{
    p = SYMAR_PTR(p, 32, kRegIn);
    U32B v;
    asm volatile("ld.global.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v.lo.x), "=r"(v.lo.y), "=r"(v.lo.z), "=r"(v.lo.w), "=r"(v.hi.x), "=r"(v.hi.y),
                   "=r"(v.hi.z), "=r"(v.hi.w)
                 : "l"(p)
                 : "memory");
    return v;
}
__device__ __forceinline__ void st_output_32B(void *p, const U32B &v)
{
    p = SYMAR_PTR(p, 32, kRegOut);
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v.lo.x), "r"(v.lo.y),
                 "r"(v.lo.z), "r"(v.lo.w), "r"(v.hi.x), "r"(v.hi.y), "r"(v.hi.z), "r"(v.hi.w)
                 : "memory");
}

__device__ __forceinline__ uint64_t globaltimer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// ---- programmatic dependent launch ------------------------------------------------
// With the launch attribute set, the next kernel of the stream may be made
// resident while this one still runs; it blocks in pdl_wait() until this grid
// has completed and its writes are visible.  Without the attribute both calls
// do nothing.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// The same, with addresses that are to be ready BEFORE the wait: a kernel made
// resident early computes them while its predecessor still runs.
__device__ __forceinline__ void pdl_wait_holding(const void *p0, const void *p1, const void *p2)
{
    asm volatile("griddepcontrol.wait;" ::"l"(p0), "l"(p1), "l"(p2) : "memory");
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

// L2 prefetch hint.  Safe on memory that an earlier kernel may still be writing: no data
// is returned, and L2 is the point of coherence, so a later write simply updates the line.
__device__ __forceinline__ void prefetch_l2(const void *p)
{
    p = SYMAR_PTR(p, 1, kRegIn);
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// a short, bounded pause (holding back a poll that would only arrive before its data)
__device__ __forceinline__ void idle_cycles(uint32_t cycles)
{
    if (cycles == 0) return;
    const uint32_t c0 = (uint32_t)clock();
    while ((uint32_t)clock() - c0 < cycles) { /* bounded by `cycles` */ }
}

// ---- bounded waiting ------------------------------------------------------------
// Counts polls in a register; every 256th poll reads the nanosecond timer.  The
// first reading starts the clock, so the fast path never touches the timer.
struct Spin {
    uint32_t n  = 0;
    uint64_t t0 = 0;
    __device__ __forceinline__ bool due() { return (++n & 0xffu) == 0; }
    __device__ __forceinline__ bool expired(uint64_t limit_ns)
    {
        uint64_t now = globaltimer_ns();
        if (t0 == 0) {
            t0 = now;
            return false;
        }
        return now - t0 > limit_ns;
    }
};

// First error wins; the kernel then leaves through its normal exit.
static __device__ __noinline__ void report_timeout(uint32_t *ctl, int rank, int peer, int cta)
{
    if (atomicCAS(&ctl[kCtlCode], 0u, (uint32_t)SYMAR_ERR_TIMEOUT) == 0u) {
        ctl[kCtlRank] = (uint32_t)rank;
        ctl[kCtlPeer] = (uint32_t)peer;
        ctl[kCtlCta]  = (uint32_t)cta;
        __threadfence();
    }
}

// ---- per-slot iteration counter ("epoch") ----------------------------------------
// The counter n is 64-bit and private to one (rank, CTA slot).  The 32-bit flag
// sent with the data is 1 + n mod (2^32 - 1): never 0 (0 = "never written"),
// and consecutive iterations always differ in parity n & 1, also across the
// 32-bit wrap.
// (2^32 = 1 mod 2^32 - 1, so the remainder is the folded sum of the two halves;
// no 64-bit division on the critical path.)
__device__ __forceinline__ uint32_t flag_of(uint64_t n)
{
    uint64_t x = (n & 0xffffffffull) + (n >> 32);      // < 2^33
    x = (x & 0xffffffffull) + (x >> 32);               // <= 2^32
    if (x >= 0xffffffffull) x -= 0xffffffffull;        // n mod (2^32 - 1)
    return (uint32_t)x + 1u;
}

// ---- element types ---------------------------------------------------------------
struct F32 {
    static constexpr int kEpv = 4;   // elements per 16-byte vector
    __device__ static __forceinline__ void widen(const uint4 &v, float (&f)[kEpv])
    {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ uint4 narrow(const float (&f)[kEpv])
    {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                          __float_as_uint(f[3]));
    }
};

struct BF16 {
    static constexpr int kEpv = 8;
    __device__ static __forceinline__ void widen(const uint4 &v, float (&f)[kEpv])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i]     = __uint_as_float(w[i] << 16);          // low half = even element
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);  // high half = odd element
        }
    }
    __device__ static __forceinline__ uint4 narrow(const float (&f)[kEpv])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);   // RNE
            w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// Rank-ordered sum of P vectors with a binary32 accumulator that starts as the
// rank-0 value; one narrowing at the end (recvReduce's accumulate-and-convert).
template <typename E, int P>
__device__ __forceinline__ uint4 reduce_in_rank_order(const uint4 (&x)[P])
{
    float acc[E::kEpv];
    E::widen(x[0], acc);
#pragma unroll
    for (int q = 1; q < P; ++q) {
        float t[E::kEpv];
        E::widen(x[q], t);
#pragma unroll
        for (int j = 0; j < E::kEpv; ++j) acc[j] = __fadd_rn(acc[j], t[j]);
    }
    return E::narrow(acc);
}

// ---- narrow units: W 32-bit words per thread (W = 1, 2 or 4) --------------------------
// For small messages the per-thread instruction count, not bandwidth, sets the
// latency; giving a thread 4 or 8 bytes instead of 16 shortens its unpack/add
// chain and spreads the message over more warps.
template <int W> struct Words { uint32_t w[W]; };

template <int W>
__device__ __forceinline__ Words<W> ld_peer_words(const void *p)
{
    p = SYMAR_PTR(p, 4 * W, kRegIn);
    Words<W> v;
    if (W == 1)
        asm volatile("ld.relaxed." SYMAR_SCOPE ".global.u32 %0, [%1];" : "=r"(v.w[0]) : "l"(p) : "memory");
    else if (W == 2)
        asm volatile("ld.relaxed." SYMAR_SCOPE ".global.v2.u32 {%0, %1}, [%2];"
                     : "=r"(v.w[0]), "=r"(v.w[W > 1 ? 1 : 0])
                     : "l"(p)
                     : "memory");
    else
        asm volatile("ld.relaxed." SYMAR_SCOPE ".global.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v.w[0]), "=r"(v.w[W > 1 ? 1 : 0]), "=r"(v.w[W > 2 ? 2 : 0]), "=r"(v.w[W > 3 ? 3 : 0])
                     : "l"(p)
                     : "memory");
    return v;
}

// rank-ordered binary32 sum of P units, one narrowing at the end
template <typename E, int P, int W>
__device__ __forceinline__ Words<W> reduce_words_in_rank_order(const Words<W> (&x)[P])
{
    Words<W> out;
    if (E::kEpv == 4) {          // fp32: one element per word
#pragma unroll
        for (int i = 0; i < W; ++i) {
            float acc = __uint_as_float(x[0].w[i]);
#pragma unroll
            for (int q = 1; q < P; ++q) acc = __fadd_rn(acc, __uint_as_float(x[q].w[i]));
            out.w[i] = __float_as_uint(acc);
        }
    } else {                     // bf16: two elements per word, low half first
#pragma unroll
        for (int i = 0; i < W; ++i) {
            float lo = __uint_as_float(x[0].w[i] << 16), hi = __uint_as_float(x[0].w[i] & 0xffff0000u);
#pragma unroll
            for (int q = 1; q < P; ++q) {
                lo = __fadd_rn(lo, __uint_as_float(x[q].w[i] << 16));
                hi = __fadd_rn(hi, __uint_as_float(x[q].w[i] & 0xffff0000u));
            }
            __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
            out.w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
    }
    return out;
}

// store of a unit of which only `valid` bytes (a multiple of 2, 1..4W) belong to the message
template <int W>
__device__ __forceinline__ void store_words(char *dst, const Words<W> &v, uint32_t valid)
{
    dst = SYMAR_PTR(dst, valid, kRegOut);
    if (valid >= 4u * W) {
        if (W == 1) asm volatile("st.global.u32 [%0], %1;" ::"l"(dst), "r"(v.w[0]) : "memory");
        else if (W == 2)
            asm volatile("st.global.v2.u32 [%0], {%1, %2};" ::"l"(dst), "r"(v.w[0]), "r"(v.w[W > 1 ? 1 : 0]) : "memory");
        else
            asm volatile("st.global.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(v.w[0]), "r"(v.w[W > 1 ? 1 : 0]),
                         "r"(v.w[W > 2 ? 2 : 0]), "r"(v.w[W > 3 ? 3 : 0])
                         : "memory");
    } else {
        uint16_t *d = reinterpret_cast<uint16_t *>(dst);
#pragma unroll
        for (int b = 0; b < 2 * W; ++b)
            if ((uint32_t)(2 * b) < valid) d[b] = (uint16_t)(v.w[b >> 1] >> ((b & 1) * 16));
    }
}

// Store of output vector v; the last vector of a message may be partial.  The
// partial store peels 2-byte pieces out of registers with compile-time indices
// (no address of `val` is taken, so it never lives in local memory).
__device__ __forceinline__ void store_result(char *out, uint64_t v, const uint4 &val, uint64_t nvec,
                                             uint32_t tail_bytes)
{
    if (tail_bytes != 0 && v == nvec - 1) {
        uint16_t *dst = SYMAR_PTR(reinterpret_cast<uint16_t *>(out + v * 16), tail_bytes, kRegOut);
        const uint32_t w[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
        for (int b = 0; b < 8; ++b)
            if ((uint32_t)b < tail_bytes / 2) dst[b] = (uint16_t)(w[b >> 1] >> ((b & 1) * 16));
    } else {
        st_output(out + v * 16, val);
    }
}

// ---- test hook: in-kernel span (first CTA in -> last CTA out, nanosecond timer) --------
__device__ __forceinline__ void debug_stamp_in(const KArgs &a)
{
    if (a.dbg_span && threadIdx.x == 0)
        atomicMin(reinterpret_cast<unsigned long long *>(a.ctl + kCtlSpanIn), (unsigned long long)globaltimer_ns());
}
// every thread of the CTA calls it as its last action
__device__ __forceinline__ void debug_stamp_out(const KArgs &a)
{
    if (!a.dbg_span) return;
    __syncthreads();
    if (threadIdx.x == 0)
        atomicMax(reinterpret_cast<unsigned long long *>(a.ctl + kCtlSpanOut), (unsigned long long)globaltimer_ns());
}

// ---- test hook: phase stamps ------------------------------------------------------------
// Thread 0 of every CTA stamps the device's nanosecond timer when it reaches phase k; the
// control block keeps, per phase, the earliest and the latest stamp over all CTAs and the
// (wrapping) sum, from which the host derives the mean.  A warp issues in order, so a stamp
// placed after an instruction that consumes a load's result is taken after that load returned.
__device__ __forceinline__ void debug_phase(const KArgs &a, int k)
{
    if (!a.dbg_span || threadIdx.x != 0) return;
    const unsigned long long now = globaltimer_ns();
    unsigned long long *w = reinterpret_cast<unsigned long long *>(a.ctl);
    atomicMin(w + kCtlPhaseMin / 2 + k, now);
    atomicMax(w + kCtlPhaseMax / 2 + k, now);
    atomicAdd(w + kCtlPhaseSum / 2 + k, now);
    atomicAdd(w + kCtlPhaseCnt / 2 + k, 1ull);
}

// ---- test hook: seeded start delay (also stamps the CTA's start for the span hook) ----
__device__ __forceinline__ void debug_delay(const KArgs &a, int rank, int cta)
{
    debug_stamp_in(a);
    if (a.dbg_delay_ns == 0) return;
    uint32_t h = a.dbg_seed ^ (uint32_t)(rank * 0x9E3779B1u) ^ (uint32_t)(cta * 0x85EBCA77u);
    h ^= h >> 16;
    h *= 0x7feb352dU;
    h ^= h >> 15;
    h *= 0x846ca68bU;
    h ^= h >> 16;
    const uint64_t wait = h % a.dbg_delay_ns;
    const uint64_t t0   = globaltimer_ns();
    while (globaltimer_ns() - t0 < wait) { /* bounded by dbg_delay_ns */ }
}

// ---- the copy of a flag or counter that is homed on this SM's half of the chip ------------------
__device__ __forceinline__ uint32_t my_half(const KArgs &a)
{
    uint32_t smid;
    asm("mov.u32 %0, %%smid;" : "=r"(smid));
    const uint64_t w = smid < 64u ? a.sm_half[0] : (smid < 128u ? a.sm_half[1] : (smid < 192u ? a.sm_half[2] : a.sm_half[3]));
    return (uint32_t)(w >> (smid & 63u)) & 1u;
}
__device__ __forceinline__ uint32_t near_copy(const KArgs &a, uint32_t half, int rank, int pair)
{
    return half ^ ((uint32_t)(a.home >> (rank * kPairsPerRank + pair)) & 1u);
}
// the counters of (rank r, slot c), copy k
__device__ __forceinline__ char *counters_at(const KArgs &a, int r, int c, uint32_t k)
{
    return a.seg0 + (size_t)r * a.stride + a.epoch_off + counters_off(c, k);
}
// the copy to READ (this SM's half)
__device__ __forceinline__ const char *counters_near(const KArgs &a, int r, int c)
{
    return counters_at(a, r, c, near_copy(a, my_half(a), r, kPairCounters));
}
// WRITE a counter: threads 0 and 1 of the CTA store the two copies
__device__ __forceinline__ void publish_u32(const KArgs &a, int r, int c, size_t which, uint32_t v)
{
    if (threadIdx.x < 2) *SYMAR_PTR(reinterpret_cast<uint32_t *>(counters_at(a, r, c, threadIdx.x) + which), 4, kRegCtr) = v;
}
__device__ __forceinline__ void publish_u64(const KArgs &a, int r, int c, size_t which, uint64_t v)
{
    if (threadIdx.x < 2) *SYMAR_PTR(reinterpret_cast<uint64_t *>(counters_at(a, r, c, threadIdx.x) + which), 8, kRegCtr) = v;
}

// ---- one synchronisation of Table I ---------------------------------------------------
// Slot c of rank r signals slot c of every peer and waits for every peer's
// signal.
//
// A signal is an atomic increment of the receiver's flag word for this sender,
// so the sender needs no sequence number.  The receiver compares against its
// own count of exchanges on this slot (a word private to (rank, slot) that the
// caller advances), whose load travels together with the first poll.  Lane q
// polls peer q's flag with an acquire load, so all P polls are in flight
// together and one round trip observes them all.
//
// RELEASE says whether the signal must order this CTA's earlier writes (the
// "chunk done" handoff: yes, after a CTA barrier).  The "input ready" signal
// orders nothing written by this kernel -- the input was complete before the
// kernel started, and a kernel boundary makes it visible to every later reader
// -- so it is a relaxed increment and costs no fence on the critical path.
// `want` receives the count to publish.  Returns false if the wait ran out.
// The addresses one exchange touches, computable before the kernel may touch memory.
struct ExchangePtrs {
    uint32_t       *signal;   // thread t < 2P: this rank's word in copy t / P of peer (t mod P)'s flag group
    const uint32_t *mine;     // lane q: peer q's word in this rank's flag group, the copy homed on this SM's half
};
// `pair` = kPairReady or kPairDone, matching flags_off
template <int P>
__device__ __forceinline__ ExchangePtrs exchange_ptrs(const KArgs &a, uint64_t flags_off, int pair, int r, int c)
{
    const uint32_t t    = threadIdx.x;
    const uint32_t lane = t & 31u;
    const uint32_t peer = t & (uint32_t)(P - 1), copy = (t / P) & 1u;
    ExchangePtrs p;
    p.signal = reinterpret_cast<uint32_t *>(a.seg0 + (size_t)peer * a.stride + flags_off + flag_group_off(c, copy)) + r;
    const uint32_t nc = near_copy(a, my_half(a), r, pair + c / kFlagSlotsPerPair);
    p.mine   = reinterpret_cast<const uint32_t *>(a.seg0 + (size_t)r * a.stride + flags_off + flag_group_off(c, nc)) +
             (lane < P ? lane : 0);
    return p;
}

// STAMP >= 0 (instrumented instantiations only): phase stamp once this thread's signal is issued,
// i.e. for a release signal once its fence has completed.
struct NoHook {
    __device__ __forceinline__ void operator()(uint32_t) const {}
};

// `after_count(want)` runs on every thread once the count has been read and the signals are on their way,
// before the first poll: the place to publish counters whose stores should drain during the wait.
template <int P, bool RELEASE, int STAMP = -1, typename Hook = NoHook>
__device__ __forceinline__ bool flag_exchange_at(const KArgs &a, const ExchangePtrs &p, const uint32_t *count, int r,
                                                 int c, bool silent, bool all_warps, uint32_t &want,
                                                 Hook after_count = Hook())
{
    const uint32_t t    = threadIdx.x;
    const uint32_t lane = t & 31u;
    if (t < 2 * P && !silent) {              // both copies of every peer's flag word
        if (RELEASE) red_release_inc_u32(p.signal);
        else red_relaxed_inc_u32(p.signal);
    }
    if (STAMP >= 0) debug_phase(a, STAMP);
    const uint32_t n = ld_relaxed_u32(count);
    after_count(n + 1);
    if (!all_warps && t >= 32) {
        want = n + 1;
        return true;
    }
    Spin spin;
    for (;;) {
        const uint32_t f = ld_acquire_u32(p.mine);
        want = n + 1;
        // ">= want": a peer may already have signalled its next call
        const unsigned late = __ballot_sync(0xffffffffu, lane < P && (int32_t)(f - want) < 0);
        if (late == 0) return true;
        if (spin.due() && __any_sync(0xffffffffu, spin.expired(a.spin_ns))) {
            if (lane == 0) report_timeout(a.ctl, r, __ffs(late) - 1, c);
            return false;
        }
    }
}

template <int P, bool RELEASE, int STAMP = -1, typename Hook = NoHook>
__device__ __forceinline__ bool flag_exchange(const KArgs &a, uint64_t flags_off, int pair, const uint32_t *count,
                                              int r, int c, bool silent, bool all_warps, uint32_t &want,
                                              Hook after_count = Hook())
{
    return flag_exchange_at<P, RELEASE, STAMP, Hook>(a, exchange_ptrs<P>(a, flags_off, pair, r, c), count, r, c, silent,
                                                     all_warps, want, after_count);
}

// Reduce-scatter + all-gather of one 16-byte vector: P loads, the rank-ordered
// sum, then the result goes straight from registers into every rank's output.
template <typename E, int P>
__device__ __forceinline__ void twoshot_vector(const KArgs &a, uint64_t v)
{
    uint4 x[P];
#pragma unroll
    for (int q = 0; q < P; ++q) x[q] = ld_peer(a.seg0 + (size_t)q * a.stride + a.in_off + v * 16);
    const uint4 res = reduce_in_rank_order<E, P>(x);
#pragma unroll
    for (int q = 0; q < P; ++q)
        store_result(a.seg0 + (size_t)q * a.stride + a.out_off, v, res, a.nvec, a.tail_bytes);
}


}  // namespace symar
