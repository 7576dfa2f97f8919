// The AllReduce kernels built from per-thread loads and stores.  One launch
// emulates all P ranks: blockIdx.y is the rank, blockIdx.x the CTA slot of that
// rank.  CTAs of different ranks meet only through the symmetric heap, as GPUs
// of one NVLink domain would.
//
//   oneshot_kernel       Sec. III-A.1 (pull): exchange "input ready" signals with
//                        every peer, read all P inputs, reduce, write the own output.
//   twoshot_kernel       Sec. III-A.2: the same exchange, reduce only the owned
//                        vectors, store them into every rank's output (all-gather
//                        from registers), then hand off with "done" signals.
//   ll_kernel            Sec. IV "LL" + Sec. V example kernel: push every input word
//                        to every peer's scratch as {payload, flag} 8-byte stores,
//                        poll the own scratch, reduce, write the own output; scratch
//                        is double-buffered by iteration parity.
//   ll_small_kernel      the same for messages that one iteration covers with one
//                        unit per thread: straight-line code, all peers polled at once.
//   sentinel_kernel      Sec. IV "Sentinel": the same push with bare payload into
//                        scratch that holds a sentinel word; the receiver polls
//                        until every word has changed and restores the sentinel.
//   twoshot_push_kernel  Table I "Two-shot (LL)" / "Two-shot (Sentinel)": reduce-
//                        scatter and all-gather both pushed through the scratch,
//                        synchronised by the data itself.
//
// (Elsewhere: the two-shot kernel of the bandwidth regime on bulk asynchronous
// copies in symar_bulk.cu, the atomic two-shot in symar_atomic.cu, the sibling
// collectives in symar_coll.cu.)
//
// No kernel contains a grid-wide barrier; every wait is one-directional (a CTA
// waits for data or a signal FROM each peer) and bounded.
#include "symar_device.cuh"
#include "symar_internal.h"

namespace symar {

// One-shot data phase with W words per thread: unit u covers bytes [4W u, 4W u + 4W).
// For small messages the loads are issued BEFORE the CTA barrier that lets threads 0 and 1 publish
// the exchange count, so that the barrier and the publication cost nothing while the data
// travels (measured -0.03 us of 1.72 us at 16 KiB).
// (Measured and dropped: two units per thread in half as many CTAs, +0.1 to +0.3 us at 16 KiB;
// leaving the trigger of the dependent launch to the kernel's end, +0.1 us at every size.)
template <typename E, int P, int W, bool DBG>
__device__ __forceinline__ void oneshot_data(const KArgs &a, char *out, uint64_t first, uint64_t step, bool ok,
                                             int r, int c, uint32_t want)
{
    const uint64_t bytes  = a.tail_bytes ? (a.nvec - 1) * 16 + a.tail_bytes : a.nvec * 16;
    const uint64_t nunits = (bytes + 4 * W - 1) / (4 * W);
    const bool have = ok && first < nunits;
    Words<W> x[P];
    // ... when one pass covers the message; with several passes per thread the barrier would sit
    // between the passes' loads and cost more than it hides (measured +0.13 us at 64 KiB)
    const bool late = nunits > step;
    if (have && !late) {
#pragma unroll
        for (int q = 0; q < P; ++q)
            x[q] = ld_peer_words<W>(a.seg0 + (size_t)q * a.stride + a.in_off + first * (4 * W));
    }
    // Every warp has consumed the count: publish the next one now, so that its store drains
    // while the data is in flight.
    __syncthreads();
    publish_u32(a, r, c, kCtrReady, want);
    if (have && late) {
#pragma unroll
        for (int q = 0; q < P; ++q)
            x[q] = ld_peer_words<W>(a.seg0 + (size_t)q * a.stride + a.in_off + first * (4 * W));
    }
    if (have) {
        const uint64_t left = bytes - first * (4 * W);
        store_words<W>(out + first * (4 * W), reduce_words_in_rank_order<E, P, W>(x),
                       left < 4u * W ? (uint32_t)left : 4u * W);
    }
    if (DBG) debug_phase(a, 2);               // this thread's loads are back, reduced and on their way out
    if (!ok) return;
    for (uint64_t u = first + step; u < nunits; u += step) {
#pragma unroll
        for (int q = 0; q < P; ++q)
            x[q] = ld_peer_words<W>(a.seg0 + (size_t)q * a.stride + a.in_off + u * (4 * W));
        const uint64_t left = bytes - u * (4 * W);
        store_words<W>(out + u * (4 * W), reduce_words_in_rank_order<E, P, W>(x),
                       left < 4u * W ? (uint32_t)left : 4u * W);
    }
}

template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kMaxThreads) oneshot_kernel(const KArgs a)
{
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, P);
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r = a.seg0 + (size_t)r * a.stride;
    const uint32_t *count = reinterpret_cast<const uint32_t *>(counters_near(a, r, c) + kCtrReady);
    const ExchangePtrs xp = exchange_ptrs<P>(a, a.ready_off, kPairReady, r, c);
    if (a.pdl) {
        // Made resident early, this CTA has time while its predecessor still runs: pull the peers'
        // input lines of its first passes towards L2 (a hint only -- if a line is still being written,
        // the write lands in L2 all the same).  One thread per 128-byte line.
        const uint32_t ub = 16u >> ((a.variant >> 8) & 3u);                    // bytes per thread and pass
        uint64_t off = ((uint64_t)c * T + t) * ub;
        for (int pass = 0; pass < 4 && off < a.nvec * 16; ++pass, off += (uint64_t)C * T * ub) {
            if ((off & 127u) != 0) break;                                       // T * ub is a multiple of 128
#pragma unroll
            for (int q = 0; q < P; ++q) prefetch_l2(a.seg0 + (size_t)q * a.stride + a.in_off + off);
        }
        pdl_wait_holding(xp.signal, xp.mine, count);   // the previous call has left the heap
        // The successor may take its seats at once: it then has this whole call for its own address
        // arithmetic and prefetch hints before its wait ends.  (Measured against a trigger after the
        // exchange, with flag reads placed on the near L2 half: 1.53 -> 1.43 us at 128 B, 1.72 -> 1.62 us
        // at 16 KiB, 2.04 -> 1.90 us at 64 KiB, 2.34 -> 2.01 us per call of the decode-step graph; the
        // same early trigger gains nothing in the two-shot kernel and costs 0.1-0.2 us in the LL kernel,
        // which have no such prologue.)
        pdl_launch_dependents();
    }
    if (DBG) debug_delay(a, r, c);
    if (DBG && a.dbg_mute == r) return;       // test hook: this rank never joins
    if (DBG) debug_phase(a, 0);

    // Variant bit 14: the prior-art form that the method replaces (Sec. III-B), for comparison only --
    // a memory-ordering barrier before the data phase (release signals) and a second one before
    // returning, as a pull kernel needs when nothing else keeps inputs from being overwritten.
    // Variant bit 15: release on the "input ready" signal and nothing else changed -- what the
    // exchange costs when the signal itself has to publish the input, as it must where no kernel
    // boundary common to all ranks does (Sec. II-B: remote writes visible to polling); comparison only.
    // (Measured and dropped: only warp 0 polls while the other warps wait at a CTA barrier, +0.03 to
    // +0.06 us: the barrier costs more than three more warps' polls of the same sector.)
    const bool prior_art = a.variant & 0x4000u;
    const bool release   = prior_art || (a.variant & 0x8000u);
    uint32_t want;
    // (Measured and dropped: holding back the first poll as the LL kernel does.  Up to 500 cycles of
    // delay change nothing, more only add: the exchange waits for the peers' increments to become
    // visible, about 550 cycles after they were issued, not for a poll that came too early.)
    const bool ok = release ? flag_exchange_at<P, true>(a, xp, count, r, c, false, true, want)
                            : flag_exchange_at<P, false>(a, xp, count, r, c, false, true, want);
    if (DBG) debug_phase(a, 1);
    char *out = seg_r + a.out_off;
    const uint64_t first = (uint64_t)c * T + t, step = (uint64_t)C * T;
    const uint32_t narrow = (a.variant >> 8) & 3u;     // bytes per thread: 16, 8 or 4
    if (narrow == 2) oneshot_data<E, P, 1, DBG>(a, out, first, step, ok, r, c, want);
    else if (narrow == 1) oneshot_data<E, P, 2, DBG>(a, out, first, step, ok, r, c, want);
    else oneshot_data<E, P, 4, DBG>(a, out, first, step, ok, r, c, want);
    if (prior_art) {
        const uint32_t *dcount = reinterpret_cast<const uint32_t *>(counters_near(a, r, c) + kCtrDone);
        uint32_t dwant;
        __syncthreads();
        flag_exchange<P, true>(a, a.done_off, kPairDone, dcount, r, c, !ok, false, dwant);
        publish_u32(a, r, c, kCtrDone, dwant);
    }
    if (DBG) {
        debug_stamp_out(a);
        debug_phase(a, 7);
    }
}

// The same for two adjacent vectors moved as one 32-byte access per peer.
template <typename E, int P>
__device__ __forceinline__ void twoshot_vector_pair(const KArgs &a, uint64_t v)
{
    U32B x[P];
#pragma unroll
    for (int q = 0; q < P; ++q) x[q] = ld_peer_32B(a.seg0 + (size_t)q * a.stride + a.in_off + v * 16);
    uint4 lo[P], hi[P];
#pragma unroll
    for (int q = 0; q < P; ++q) {
        lo[q] = x[q].lo;
        hi[q] = x[q].hi;
    }
    U32B res;
    res.lo = reduce_in_rank_order<E, P>(lo);
    res.hi = reduce_in_rank_order<E, P>(hi);
#pragma unroll
    for (int q = 0; q < P; ++q) st_output_32B(a.seg0 + (size_t)q * a.stride + a.out_off + v * 16, res);
}

template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kMaxThreads) twoshot_kernel(const KArgs a)
{
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, P);
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    const uint32_t *rcount = reinterpret_cast<const uint32_t *>(counters_near(a, r, c) + kCtrReady);
    const uint32_t *dcount = reinterpret_cast<const uint32_t *>(counters_near(a, r, c) + kCtrDone);
    if (a.pdl) pdl_wait();                    // the previous call has left the heap
    if (DBG) debug_delay(a, r, c);
    if (DBG && a.dbg_mute == r) return;       // test hook: this rank never joins

    // reduce-scatter: which vectors rank r owns
    uint32_t rwant, dwant;
    if (DBG) debug_phase(a, 0);
    bool ok = flag_exchange<P, false>(a, a.ready_off, kPairReady, rcount, r, c, false, true, rwant);
    if (a.pdl) pdl_launch_dependents();
    if (DBG) debug_phase(a, 1);               // every peer's input is ready
    if (ok) {
        const uint64_t step = (uint64_t)C * T;
        if (a.blk_log2 == kOneChunk) {
            // small and medium messages: rank r owns the contiguous chunk r
            const uint64_t chv = (a.nvec + P - 1) / P;
            const uint64_t lo  = (uint64_t)r * chv;
            const uint64_t hi  = (lo + chv < a.nvec) ? lo + chv : a.nvec;
            if (a.variant & 0x40u) {
                // 8 bytes per thread and trip instead of 16: twice the threads share a chunk, each with half
                // the unpack-add-store chain (what made the one-shot kernel faster below 128 KiB)
                const uint64_t bytes = a.tail_bytes ? (a.nvec - 1) * 16 + a.tail_bytes : a.nvec * 16;
                for (uint64_t u = 2 * lo + (uint64_t)c * T + t; u < 2 * hi; u += step) {
                    if (u * 8 >= bytes) break;
                    Words<2> x[P];
#pragma unroll
                    for (int q = 0; q < P; ++q) x[q] = ld_peer_words<2>(a.seg0 + (size_t)q * a.stride + a.in_off + u * 8);
                    const Words<2> res  = reduce_words_in_rank_order<E, P, 2>(x);
                    const uint64_t left = bytes - u * 8;
#pragma unroll
                    for (int q = 0; q < P; ++q)
                        store_words<2>(a.seg0 + (size_t)q * a.stride + a.out_off + u * 8, res, left < 8u ? (uint32_t)left : 8u);
                }
            } else {
                for (uint64_t v = lo + (uint64_t)c * T + t; v < hi; v += step) twoshot_vector<E, P>(a, v);
            }
        } else {
            // large messages: blocks of 2^blk_log2 vectors are dealt to the ranks
            // round-robin, so that at any moment all P * C CTAs stream through the
            // same neighbourhood of each buffer (fewer open DRAM pages than P
            // far-apart chunks).  Rank r owns blocks r, r + P, r + 2P, ...
            const uint32_t sh   = a.blk_log2;
            const uint64_t nblk = (a.nvec + (1ull << sh) - 1) >> sh;
            const uint64_t mine = (nblk + P - 1 - r) / P;
            if (a.wide) {
                const uint64_t total = mine << (sh - 1);            // 32-byte steps
                const uint64_t mask  = (1ull << (sh - 1)) - 1;
                for (uint64_t w = (uint64_t)c * T + t; w < total; w += step) {
                    const uint64_t v = (((w >> (sh - 1)) * P + r) << sh) + 2 * (w & mask);
                    if (v + 2 < a.nvec) twoshot_vector_pair<E, P>(a, v);   // never the (maybe partial) last vector
                    else {
                        if (v < a.nvec) twoshot_vector<E, P>(a, v);
                        if (v + 1 < a.nvec) twoshot_vector<E, P>(a, v + 1);
                    }
                }
            } else {
                const uint64_t total = mine << sh;
                const uint64_t mask  = (1ull << sh) - 1;
                for (uint64_t w = (uint64_t)c * T + t; w < total; w += step) {
                    const uint64_t v = (((w >> sh) * P + r) << sh) + (w & mask);
                    if (v < a.nvec) twoshot_vector<E, P>(a, v);
                }
            }
        }
    }
    // handoff: this CTA's part of rank r's vectors has landed everywhere -> tell
    // every peer; then wait until every peer's CTA c has delivered its part here.
    if (DBG) debug_phase(a, 2);               // thread 0's share reduced, its stores issued
    __syncthreads();
    if (DBG) debug_phase(a, 3);               // the whole CTA's stores issued
    // Both counts are published once the "done" signals are on their way and before the first poll: their
    // stores (one copy each on the other half of the L2) drain during the wait instead of after it.  (Not
    // earlier: before the handoff the release fence would have to wait for them too, measured +0.1 us
    // between two ranks.)
    auto publish = [&](uint32_t done_want) {
        publish_u32(a, r, c, kCtrReady, rwant);
        publish_u32(a, r, c, kCtrDone, done_want);
    };
    if (DBG) flag_exchange<P, true, 5>(a, a.done_off, kPairDone, dcount, r, c, !ok, false, dwant, publish);   // 5: release fence done, signal sent
    else flag_exchange<P, true>(a, a.done_off, kPairDone, dcount, r, c, !ok, false, dwant, publish);
    if (DBG) debug_phase(a, 4);               // every peer's part has landed here
    if (DBG) {
        debug_stamp_out(a);
        debug_phase(a, 7);
    }
}

// LL with 8 bytes of payload per thread: one 16-byte {w0,f,w1,f} store per peer and
// one 16-byte poll per peer and round.  Half the instructions per thread of the
// 16-byte form and twice the threads; same scratch layout (unit u = half u&1 of
// vector u>>1), so both forms can alternate on one heap.
template <typename E, int P>
__device__ __forceinline__ bool ll_iteration_narrow(const KArgs &a, int r, int c, uint32_t e, uint64_t region,
                                                    uint64_t v0, uint32_t cnt, Words<2> &kept)
{
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r       = a.seg0 + (size_t)r * a.stride;
    const char *in    = seg_r + a.in_off;
    char *out         = seg_r + a.out_off;
    const uint64_t hi_e = (uint64_t)e << 32;
    const uint32_t units = 2 * cnt;
    // bytes of unit u that belong to the message (0 = the unit lies past its end)
    auto valid_of = [&](uint32_t u) -> uint32_t {
        const uint64_t v = v0 + (u >> 1);
        const uint32_t vb = (a.tail_bytes != 0 && v == a.nvec - 1) ? a.tail_bytes : 16u;
        const uint32_t lo = (u & 1u) * 8u;
        return vb > lo ? (vb - lo < 8u ? vb - lo : 8u) : 0u;
    };
    for (uint32_t u = t; u < units; u += T) {
        if (valid_of(u) == 0) continue;
        const size_t off = (size_t)(u & 1u) * kLLSlotVecs * 16 + (size_t)(u >> 1) * 16;
        Words<2> x;
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];"
                     : "=r"(x.w[0]), "=r"(x.w[1])
                     : "l"(SYMAR_PTR(in + (v0 + (u >> 1)) * 16 + (u & 1u) * 8, 8, kRegIn)));
        if (u == t) kept = x;
        const uint64_t d0 = hi_e | x.w[0], d1 = hi_e | x.w[1];
        char *dst = a.seg0 + region + (size_t)r * kLLSenderBytes + off;
#pragma unroll
        for (int q = 0; q < P; ++q) {
            if (q != r) st_relaxed_v2u64(dst, d0, d1);
            dst += a.stride;
        }
    }
    for (uint32_t u = t; u < units; u += T) {
        const uint32_t valid = valid_of(u);
        if (valid == 0) continue;
        const size_t off = (size_t)(u & 1u) * kLLSlotVecs * 16 + (size_t)(u >> 1) * 16;
        const char *src  = seg_r + region + off;
        Words<2> x[P];
        unsigned need = ((1u << P) - 1u) & ~(1u << r);
        Spin spin;
        while (need != 0) {
            U64x2 d[P];
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (need >> q & 1u) d[q] = ld_relaxed_v2u64(src + (size_t)q * kLLSenderBytes);
#pragma unroll
            for (int q = 0; q < P; ++q) {
                if ((need >> q & 1u) && (uint32_t)(d[q].a >> 32) == e && (uint32_t)(d[q].b >> 32) == e) {
                    x[q].w[0] = (uint32_t)d[q].a;
                    x[q].w[1] = (uint32_t)d[q].b;
                    need &= ~(1u << q);
                }
            }
            if (need != 0 && spin.due() && spin.expired(a.spin_ns)) {
                report_timeout(a.ctl, r, __ffs(need) - 1, c);
                return false;
            }
        }
        Words<2> own;
        if (u == t) own = kept;
        else
            asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];"
                         : "=r"(own.w[0]), "=r"(own.w[1])
                         : "l"(SYMAR_PTR(in + (v0 + (u >> 1)) * 16 + (u & 1u) * 8, 8, kRegIn)));
#pragma unroll
        for (int q = 0; q < P; ++q)
            if (q == r) x[q] = own;
        store_words<2>(out + (v0 + (u >> 1)) * 16 + (u & 1u) * 8, reduce_words_in_rank_order<E, P, 2>(x), valid);
    }
    return true;
}

template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kLLMaxThreads) ll_kernel(const KArgs a)
{
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, P);
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r  = a.seg0 + (size_t)r * a.stride;
    const uint64_t *ep = reinterpret_cast<const uint64_t *>(counters_near(a, r, c) + kCtrLL);
    if (a.pdl) {
        pdl_wait();                           // the previous call has left the heap
        pdl_launch_dependents();
    }
    const uint64_t n0 = ld_relaxed_u64(ep);
    if (DBG) debug_delay(a, r, c);
    if (DBG && a.dbg_mute == r) return;       // test hook: this rank never joins
    // Every thread has read the counter, and where it will stand after this call is known: publish it now,
    // so that its stores drain during the call and not after it.
    __syncthreads();
    publish_u64(a, r, c, kCtrLL, n0 + a.iters);
    if (DBG) debug_phase(a, 0);

    const char *in = seg_r + a.in_off;
    char *out      = seg_r + a.out_off;
    bool failed    = false;
    uint4 kept     = make_uint4(0u, 0u, 0u, 0u);   // own vector of the first trip stays in registers
    Words<2> kept2 = {{0u, 0u}};

    for (uint32_t it = 0; it < a.iters && !failed; ++it) {
        const uint64_t n   = n0 + 1 + it;            // advanceEpoch: flag value and sub-buffer
        const uint32_t e   = flag_of(n);
        const uint64_t v0  = ((uint64_t)it * C + c) * a.cv;
        const uint32_t cnt = v0 < a.nvec ? (uint32_t)(a.nvec - v0 < a.cv ? a.nvec - v0 : a.cv) : 0u;
        const uint64_t region = a.ll_off + ((uint64_t)(n & 1) * kLLSlots + c) * P * kLLSenderBytes;
        const uint64_t hi_e   = (uint64_t)e << 32;

        if (a.variant & 0x100u) {            // 8 bytes of payload per thread
            failed = !ll_iteration_narrow<E, P>(a, r, c, e, region, v0, cnt, kept2);
            continue;
        }
        // bcast: {payload word, flag} pairs into every PEER's scratch, sender row r.
        // The own contribution stays in registers (same bits as a round trip
        // through the own scratch row would return).
        for (uint32_t k = t; k < cnt; k += T) {
            const uint4 x = ld_own(in + (v0 + k) * 16);
            if (k == t) kept = x;
            const uint64_t d0 = hi_e | x.x, d1 = hi_e | x.y, d2 = hi_e | x.z, d3 = hi_e | x.w;
#pragma unroll
            for (int q = 0; q < P; ++q) {
                if (q == r) continue;
                char *dst = a.seg0 + (size_t)q * a.stride + region + (size_t)r * kLLSenderBytes + (size_t)k * 16;
                st_relaxed_v2u64(dst, d0, d1);
                st_relaxed_v2u64(dst + (size_t)kLLSlotVecs * 16, d2, d3);
            }
        }
        if (DBG && it == 0) debug_phase(a, 1);     // counter and input were back, first trip's stores issued
        // recvReduce: poll the P-1 peer rows together; a row that has arrived is
        // not polled again
        for (uint32_t k = t; k < cnt && !failed; k += T) {
            const char *src = seg_r + region + (size_t)k * 16;
            uint4 x[P];
            const uint4 own = (k == t) ? kept : ld_own(in + (v0 + k) * 16);
            unsigned need   = ((1u << P) - 1u) & ~(1u << r);
            Spin spin;
            while (need != 0) {
                U64x2 lo[P], hi[P];
#pragma unroll
                for (int q = 0; q < P; ++q) {
                    if (need >> q & 1u) {
                        lo[q] = ld_relaxed_v2u64(src + (size_t)q * kLLSenderBytes);
                        hi[q] = ld_relaxed_v2u64(src + (size_t)q * kLLSenderBytes + (size_t)kLLSlotVecs * 16);
                    }
                }
#pragma unroll
                for (int q = 0; q < P; ++q) {
                    if (need >> q & 1u) {
                        const bool here = (uint32_t)(lo[q].a >> 32) == e && (uint32_t)(lo[q].b >> 32) == e &&
                                          (uint32_t)(hi[q].a >> 32) == e && (uint32_t)(hi[q].b >> 32) == e;
                        if (here) {
                            x[q] = make_uint4((uint32_t)lo[q].a, (uint32_t)lo[q].b, (uint32_t)hi[q].a,
                                              (uint32_t)hi[q].b);
                            need &= ~(1u << q);
                        }
                    }
                }
                if (need != 0 && spin.due() && spin.expired(a.spin_ns)) {
                    report_timeout(a.ctl, r, __ffs(need) - 1, c);
                    failed = true;
                    break;
                }
            }
            if (failed) break;
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (q == r) x[q] = own;
            store_result(out, v0 + k, reduce_in_rank_order<E, P>(x), a.nvec, a.tail_bytes);
        }
        if (DBG && it == 0) debug_phase(a, 4);     // first iteration received, reduced and stored
        // No CTA barrier between iterations: position k is sent and received by
        // the same thread index on every rank, and a thread sends iteration i+1
        // only after its own receive of iteration i, which needed the peer
        // thread's send of iteration i, issued after that thread's receive of
        // iteration i-1 -- so the sub-buffer of parity (i+1)&1 is free.
    }
    if (DBG) {
        debug_stamp_out(a);
        debug_phase(a, 7);
    }
}

// LL for a message that one iteration covers with ONE unit of W words per thread (Sec. V example
// kernel; Sec. VII Obs. 1: LL owes its small-message lead to compile-time unrolling and to polling
// all peers in parallel): no loop over units or iterations, no run-time choice of the unit width,
// the counter load and the input load in flight together, P - 1 stores, then polls of all P - 1 rows
// at once.  Unit t of CTA c sits at byte t * 16 of the sender's row (W = 2: {w0,f,w1,f}) and, for
// W = 4, also in the second plane of the row ({w2,f,w3,f}); the flag is the slot's own
// iteration counter, so this kernel and ll_kernel can alternate on one heap.
//
// Polling.  A poll of a line that a peer has just written returns after several hundred cycles, and
// a poll that reaches L2 a moment before the data costs that round trip again while it competes
// with the peers' stores for L2.  The first poll is therefore held back by `gap` cycles (64 cycles x
// variant bits 12-15; a default per size, refined by the tuner): measured at P = 8, 2.8 -> 2.3 us at
// 16 KiB with 768 cycles (about one store-to-poll hop), no gain below 1 KiB.  Keeping two polls per
// row in flight instead (a second one issued half a round trip after the first) was measured
// slower at every size (+0.4 us).
//
// (Measured and dropped: writing every row twice, 4 KiB apart, so that the receiver can poll a copy on its
// own half of the L2 -- what pays for flags and counters.  The second set of stores costs more than the
// nearer poll gains: +0.06 to +0.5 us from 16 B to 2 KiB at P = 2, 4 and 8.  And once a slot's ranks are
// launched as one cluster, writer and reader share a half and the row's home no longer shows: moving all
// rows by 4 KiB, onto lines homed on the other half, changed at most 0.03 us.)
//
// Dependent launch.  The kernel never triggers its dependent early: the next call then starts when
// this grid has drained, overlapping only its launch with this grid's completion.  Measured against
// a trigger before the stores, after them or after the polls: 1.56 instead of 1.81 us at 128 B,
// equal or better at every size up to 64 KiB (an early-resident successor only sits in its wait).
template <int W> struct LLRaw { U64x2 v[W / 2]; };

template <int W>
__device__ __forceinline__ LLRaw<W> ll_row_load(const char *p)
{
    LLRaw<W> d;
    d.v[0] = ld_relaxed_v2u64(p);
    if (W == 4) d.v[W / 2 - 1] = ld_relaxed_v2u64(p + (size_t)kLLSlotVecs * 16);
    return d;
}
template <int W>
__device__ __forceinline__ bool ll_row_take(const LLRaw<W> &d, uint32_t e, Words<W> &x)
{
    bool here = (uint32_t)(d.v[0].a >> 32) == e && (uint32_t)(d.v[0].b >> 32) == e;
    if (W == 4) here = here && (uint32_t)(d.v[W / 2 - 1].a >> 32) == e && (uint32_t)(d.v[W / 2 - 1].b >> 32) == e;
    if (here) {
        x.w[0] = (uint32_t)d.v[0].a;
        x.w[1] = (uint32_t)d.v[0].b;
        if (W == 4) {
            x.w[W - 2] = (uint32_t)d.v[W / 2 - 1].a;
            x.w[W - 1] = (uint32_t)d.v[W / 2 - 1].b;
        }
    }
    return here;
}

template <typename E, int P, int W, bool DBG>
__global__ void __launch_bounds__(kLLMaxThreads) ll_small_kernel(const KArgs a)
{
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, P);
    const int c = blockIdx.x, r = blockIdx.y;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r  = a.seg0 + (size_t)r * a.stride;
    const uint64_t *ep = reinterpret_cast<const uint64_t *>(counters_near(a, r, c) + kCtrLL);
    const uint64_t bytes = a.tail_bytes ? (a.nvec - 1) * 16 + a.tail_bytes : a.nvec * 16;
    const uint64_t lo    = ((uint64_t)c * T + t) * (4 * W);
    const uint32_t valid = lo < bytes ? (bytes - lo < 4u * W ? (uint32_t)(bytes - lo) : 4u * W) : 0u;
    const char *in  = seg_r + a.in_off + lo;
    const size_t pos = (size_t)t * 16;
    const uint32_t gap = ((a.variant >> 12) & 15u) * 64u;
    if (a.pdl) pdl_wait_holding(ep, in, seg_r);       // the previous call has left the heap
    const uint64_t n = ld_relaxed_u64(ep) + 1;        // advanceEpoch: flag value and sub-buffer
    Words<W> own;
#pragma unroll
    for (int i = 0; i < W; ++i) own.w[i] = 0u;
    if (valid) {
        // the last 16-byte vector of a message lies inside the user region even when it is partial
        if (W == 2)
            asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];"
                         : "=r"(own.w[0]), "=r"(own.w[1])
                         : "l"(SYMAR_PTR(in, 8, kRegIn)));
        else
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(own.w[0]), "=r"(own.w[1]), "=r"(own.w[W - 2]), "=r"(own.w[W - 1])
                         : "l"(SYMAR_PTR(in, 16, kRegIn)));
    }
    if (DBG) debug_delay(a, r, c);
    if (DBG && a.dbg_mute == r) return;       // test hook: this rank never joins
    if (DBG) debug_phase(a, 0);

    const uint32_t e      = flag_of(n);
    const uint64_t region = a.ll_off + ((uint64_t)(n & 1) * kLLSlots + c) * P * kLLSenderBytes;
    bool failed = false;
    // Every thread has read the counter: publish the next value now, so that its stores (one of them to the
    // other half of the L2) drain while the rows travel instead of after the output (-0.03 to -0.06 us at
    // every size and rank count).
    __syncthreads();
    publish_u64(a, r, c, kCtrLL, n);
    if (valid) {
        const uint64_t hi_e = (uint64_t)e << 32;
        char *dst = a.seg0 + region + (size_t)r * kLLSenderBytes + pos;      // my row in rank 0's region
#pragma unroll
        for (int q = 0; q < P; ++q) {
            if (q != r) {
                st_relaxed_v2u64(dst, hi_e | own.w[0], hi_e | own.w[1]);
                if (W == 4) st_relaxed_v2u64(dst + (size_t)kLLSlotVecs * 16, hi_e | own.w[W - 2], hi_e | own.w[W - 1]);
            }
            dst += a.stride;
        }
        if (DBG) debug_phase(a, 1);           // counter and input were back, all stores issued
        const char *src = seg_r + region + pos;                              // row q of my region: + q * kLLSenderBytes
        Words<W> x[P];
        unsigned need = ((1u << P) - 1u) & ~(1u << r);
        Spin spin;
        idle_cycles(gap);
        while (need != 0) {
            LLRaw<W> d[P];
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (need >> q & 1u) d[q] = ll_row_load<W>(src + (size_t)q * kLLSenderBytes);
#pragma unroll
            for (int q = 0; q < P; ++q)
                if ((need >> q & 1u) && ll_row_take<W>(d[q], e, x[q])) need &= ~(1u << q);
            if (need != 0 && spin.due() && spin.expired(a.spin_ns)) {
                report_timeout(a.ctl, r, __ffs(need) - 1, c);
                failed = true;
                break;
            }
        }
        if (DBG) debug_phase(a, 3);           // every peer's row seen
        if (!failed) {
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (q == r) x[q] = own;
            store_words<W>(seg_r + a.out_off + lo, reduce_words_in_rank_order<E, P, W>(x), valid);
        }
        if (DBG) debug_phase(a, 4);
    }
    if (DBG) {
        debug_stamp_out(a);
        debug_phase(a, 7);
    }
}

// One-shot push with sentinel synchronisation (Sec. IV "Sentinel"; Sec. V send / recv with
// Reset / reset).  The receiving scratch holds the sentinel word everywhere; a sender
// stores bare payload vectors (full payload bandwidth, half of LL's scratch); the
// receiver polls a slot until none of its four words is the sentinel, takes the data
// and stores the sentinel back.  A payload word that happens to equal the sentinel
// (a NaN with all bits set) is sent with its lowest bit cleared: still a NaN, and
// a sum with a NaN is a NaN either way, so no input value is forbidden.
// Double buffering by iteration parity as in the LL kernel; with more than one
// iteration per call a fence per iteration makes the restored sentinels visible
// before a peer can target the same sub-buffer again (between calls the kernel
// boundary does that).
template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kMaxThreads) sentinel_kernel(const KArgs a)
{
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, P);
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r  = a.seg0 + (size_t)r * a.stride;
    const uint64_t *ep = reinterpret_cast<const uint64_t *>(counters_near(a, r, c) + kCtrLL);
    if (a.pdl) {
        pdl_wait();
        pdl_launch_dependents();
    }
    const uint64_t n0 = ld_relaxed_u64(ep);
    if (DBG) debug_delay(a, r, c);
    if (DBG && a.dbg_mute == r) return;       // test hook: this rank never joins
    // Every thread has read the counter, and where it will stand after this call is known: publish it now,
    // so that its stores drain during the call and not after it.
    __syncthreads();
    publish_u64(a, r, c, kCtrLL, n0 + a.iters);

    const char *in = seg_r + a.in_off;
    char *out      = seg_r + a.out_off;
    bool failed    = false;
    uint4 kept     = make_uint4(0u, 0u, 0u, 0u);
    const uint4 sentinel = make_uint4(kSentinelWord, kSentinelWord, kSentinelWord, kSentinelWord);
    auto clean = [](uint32_t w) { return w == kSentinelWord ? (kSentinelWord & ~1u) : w; };

    for (uint32_t it = 0; it < a.iters && !failed; ++it) {
        const uint64_t n   = n0 + 1 + it;
        const uint64_t v0  = ((uint64_t)it * C + c) * a.cv;
        const uint32_t cnt = v0 < a.nvec ? (uint32_t)(a.nvec - v0 < a.cv ? a.nvec - v0 : a.cv) : 0u;
        const uint64_t region = a.sn_off + ((uint64_t)(n & 1) * kLLSlots + c) * P * kSnSenderBytes;

        for (uint32_t k = t; k < cnt; k += T) {          // bcast
            uint4 x = ld_own(in + (v0 + k) * 16);
            x = make_uint4(clean(x.x), clean(x.y), clean(x.z), clean(x.w));
            if (k == t) kept = x;
            char *dst = a.seg0 + region + (size_t)r * kSnSenderBytes + (size_t)k * 16;
#pragma unroll
            for (int q = 0; q < P; ++q) {
                if (q != r) st_relaxed_v4(dst, x);
                dst += a.stride;
            }
        }
        for (uint32_t k = t; k < cnt && !failed; k += T) {   // recvReduce with reset
            char *src = seg_r + region + (size_t)k * 16;
            uint4 x[P];
            unsigned need = ((1u << P) - 1u) & ~(1u << r);
            Spin spin;
            while (need != 0) {
                uint4 d[P];
#pragma unroll
                for (int q = 0; q < P; ++q)
                    if (need >> q & 1u) d[q] = ld_relaxed_v4(src + (size_t)q * kSnSenderBytes);
#pragma unroll
                for (int q = 0; q < P; ++q) {
                    if ((need >> q & 1u) && d[q].x != kSentinelWord && d[q].y != kSentinelWord &&
                        d[q].z != kSentinelWord && d[q].w != kSentinelWord) {
                        x[q] = d[q];
                        st_relaxed_v4(src + (size_t)q * kSnSenderBytes, sentinel);      // reset for reuse
                        need &= ~(1u << q);
                    }
                }
                if (need != 0 && spin.due() && spin.expired(a.spin_ns)) {
                    report_timeout(a.ctl, r, __ffs(need) - 1, c);
                    failed = true;
                    break;
                }
            }
            if (failed) break;
            uint4 own = kept;
            if (k != t) {
                own = ld_own(in + (v0 + k) * 16);
                own = make_uint4(clean(own.x), clean(own.y), clean(own.z), clean(own.w));
            }
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (q == r) x[q] = own;
            store_result(out, v0 + k, reduce_in_rank_order<E, P>(x), a.nvec, a.tail_bytes);
        }
        if (a.iters > 1) fence_acq_rel();
    }
    if (DBG) {
        debug_stamp_out(a);
        debug_phase(a, 7);
    }
}

// ---- two-shot over the push buffers (the paper's AllReduce_LLBuffer_Twoshot; Table I rows
//      "Two-shot (LL)" and "Two-shot (Sentinel)") ------------------------------------------
// Rank r pushes vector p of chunk q of its input into rank q's scratch, every rank
// reduces the chunk it owns, pushes the reduced vector into every peer's scratch and
// collects the other chunks from its own scratch.  Two synchronisations, both carried
// by the data (LL flag words or the sentinel), none by a barrier; per-rank volume
// 2 (P-1) M / P payload bytes (twice that with LL flags).  The first half of a scratch
// row takes the reduce-scatter traffic, the second half the all-gather traffic.
template <bool SENT>
struct PushRow {
    static constexpr size_t kRowBytes = SENT ? kSnSenderBytes : kLLSenderBytes;
    __device__ static __forceinline__ void send(char *row, uint32_t j, const uint4 &x, uint32_t e)
    {
        if (SENT) {
            st_relaxed_v4(row + (size_t)j * 16, x);
        } else {
            const uint64_t hi_e = (uint64_t)e << 32;
            st_relaxed_v2u64(row + (size_t)j * 16, hi_e | x.x, hi_e | x.y);
            st_relaxed_v2u64(row + (size_t)kLLSlotVecs * 16 + (size_t)j * 16, hi_e | x.z, hi_e | x.w);
        }
    }
    // Receiving is split into load / check so that a caller can put the loads of all
    // peers in flight before it looks at any of them.
    struct Raw { U64x2 lo, hi; };        // sentinel mode uses `lo` only (one 16-byte vector)
    __device__ static __forceinline__ Raw load(const char *row, uint32_t j)
    {
        Raw d;
        if (SENT) {
            const uint4 v = ld_relaxed_v4(row + (size_t)j * 16);
            d.lo.a = (uint64_t)v.y << 32 | v.x;
            d.lo.b = (uint64_t)v.w << 32 | v.z;
            d.hi   = d.lo;
        } else {
            d.lo = ld_relaxed_v2u64(row + (size_t)j * 16);
            d.hi = ld_relaxed_v2u64(row + (size_t)kLLSlotVecs * 16 + (size_t)j * 16);
        }
        return d;
    }
    // true when the vector has arrived (sentinel mode then restores the sentinel)
    __device__ static __forceinline__ bool check(char *row, uint32_t j, const Raw &d, uint32_t e, uint4 &x)
    {
        if (SENT) {
            const uint4 v = make_uint4((uint32_t)d.lo.a, (uint32_t)(d.lo.a >> 32), (uint32_t)d.lo.b,
                                       (uint32_t)(d.lo.b >> 32));
            if (v.x == kSentinelWord || v.y == kSentinelWord || v.z == kSentinelWord || v.w == kSentinelWord)
                return false;
            x = v;
            st_relaxed_v4(row + (size_t)j * 16,
                          make_uint4(kSentinelWord, kSentinelWord, kSentinelWord, kSentinelWord));
            return true;
        } else {
            if ((uint32_t)(d.lo.a >> 32) != e || (uint32_t)(d.lo.b >> 32) != e || (uint32_t)(d.hi.a >> 32) != e ||
                (uint32_t)(d.hi.b >> 32) != e)
                return false;
            x = make_uint4((uint32_t)d.lo.a, (uint32_t)d.lo.b, (uint32_t)d.hi.a, (uint32_t)d.hi.b);
            return true;
        }
    }
    // sentinel mode cannot carry a word equal to the sentinel: clear its lowest bit (still a NaN)
    __device__ static __forceinline__ uint4 clean(const uint4 &x)
    {
        if (!SENT) return x;
        auto c = [](uint32_t w) { return w == kSentinelWord ? (kSentinelWord & ~1u) : w; };
        return make_uint4(c(x.x), c(x.y), c(x.z), c(x.w));
    }
};

template <typename E, int P, bool SENT, bool DBG>
__global__ void __launch_bounds__(kPushTwoshotMaxThreads) twoshot_push_kernel(const KArgs a)
{
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, P);
    using Row = PushRow<SENT>;
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r  = a.seg0 + (size_t)r * a.stride;
    const uint64_t *ep = reinterpret_cast<const uint64_t *>(counters_near(a, r, c) + kCtrLL);
    if (a.pdl) {
        pdl_wait();
        pdl_launch_dependents();
    }
    const uint64_t n0 = ld_relaxed_u64(ep);
    if (DBG) debug_delay(a, r, c);
    if (DBG && a.dbg_mute == r) return;       // test hook: this rank never joins
    // Every thread has read the counter, and where it will stand after this call is known: publish it now,
    // so that its stores drain during the call and not after it.
    __syncthreads();
    publish_u64(a, r, c, kCtrLL, n0 + a.iters);

    const char *in = seg_r + a.in_off;
    char *out      = seg_r + a.out_off;
    const uint64_t chv  = (a.nvec + P - 1) / P;            // vectors per chunk; chunk q = [q chv, (q+1) chv)
    const uint32_t half = kLLSlotVecs / 2;                 // all-gather positions start here
    bool failed = false;

    for (uint32_t it = 0; it < a.iters && !failed; ++it) {
        const uint64_t n  = n0 + 1 + it;
        const uint32_t e  = flag_of(n);
        const uint64_t p0 = ((uint64_t)it * C + c) * a.cv;             // first chunk position of this CTA
        const uint32_t cnt = p0 < chv ? (uint32_t)(chv - p0 < a.cv ? chv - p0 : a.cv) : 0u;
        const uint64_t region = (SENT ? a.sn_off : a.ll_off) + ((uint64_t)(n & 1) * kLLSlots + c) * P * Row::kRowBytes;
        auto valid = [&](int q, uint64_t p) { return (uint64_t)q * chv + p < a.nvec; };
        // my row r in rank q's region / rank q's row in my region
        auto peer_row = [&](int q) { return a.seg0 + (size_t)q * a.stride + region + (size_t)r * Row::kRowBytes; };
        auto my_row   = [&](int q) { return seg_r + region + (size_t)q * Row::kRowBytes; };

        for (uint32_t k = t; k < cnt; k += T) {                        // reduce-scatter: push
            uint4 mine[P];
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (q != r && valid(q, p0 + k)) mine[q] = ld_own(in + ((uint64_t)q * chv + p0 + k) * 16);
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (q != r && valid(q, p0 + k)) Row::send(peer_row(q), k, Row::clean(mine[q]), e);
        }
        for (uint32_t k = t; k < cnt && !failed; k += T) {
            const uint64_t p = p0 + k;
            if (valid(r, p)) {                                          // reduce the owned vector
                uint4 x[P];
                unsigned need = ((1u << P) - 1u) & ~(1u << r);
                Spin spin;
                while (need != 0) {
                    typename Row::Raw d[P];
#pragma unroll
                    for (int q = 0; q < P; ++q)
                        if (need >> q & 1u) d[q] = Row::load(my_row(q), k);
#pragma unroll
                    for (int q = 0; q < P; ++q)
                        if ((need >> q & 1u) && Row::check(my_row(q), k, d[q], e, x[q])) need &= ~(1u << q);
                    if (need != 0 && spin.due() && spin.expired(a.spin_ns)) {
                        report_timeout(a.ctl, r, __ffs(need) - 1, c);
                        failed = true;
                        break;
                    }
                }
                if (failed) break;
                const uint4 own = Row::clean(ld_own(in + ((uint64_t)r * chv + p) * 16));
#pragma unroll
                for (int q = 0; q < P; ++q)
                    if (q == r) x[q] = own;
                const uint4 res = Row::clean(reduce_in_rank_order<E, P>(x));
#pragma unroll
                for (int q = 0; q < P; ++q)                             // all-gather: push
                    if (q != r) Row::send(peer_row(q), half + k, res, e);
                store_result(out, (uint64_t)r * chv + p, res, a.nvec, a.tail_bytes);
            }
            unsigned need = 0;                                          // all-gather: collect
#pragma unroll
            for (int q = 0; q < P; ++q)
                if (q != r && valid(q, p)) need |= 1u << q;
            Spin spin;
            while (need != 0) {
                typename Row::Raw d[P];
#pragma unroll
                for (int q = 0; q < P; ++q)
                    if (need >> q & 1u) d[q] = Row::load(my_row(q), half + k);
#pragma unroll
                for (int q = 0; q < P; ++q) {
                    uint4 v;
                    if ((need >> q & 1u) && Row::check(my_row(q), half + k, d[q], e, v)) {
                        store_result(out, (uint64_t)q * chv + p, v, a.nvec, a.tail_bytes);
                        need &= ~(1u << q);
                    }
                }
                if (need != 0 && spin.due() && spin.expired(a.spin_ns)) {
                    report_timeout(a.ctl, r, __ffs(need) - 1, c);
                    failed = true;
                    break;
                }
            }
        }
        if (SENT && a.iters > 1) fence_acq_rel();      // restored sentinels before the sub-buffer's next use
    }
    if (DBG) {
        debug_stamp_out(a);
        debug_phase(a, 7);
    }
}

// ---- self-test of the bounds-checking build ------------------------------------------------
// One CTA of rank 0 declares a 64-byte call and makes one store inside its output range and one
// just beyond it -- an address that is still inside the heap's user region, so the store is
// harmless even where nothing checks it.  The checking build must record the second one and
// keep it from landing.
__global__ void check_selftest_kernel(const KArgs a)
{
    SYMAR_CHECK_BEGIN_ALLREDUCE(a, 1);
    if (threadIdx.x != 0) return;
    char *out = a.seg0 + a.out_off;
    st_output(out, make_uint4(1u, 2u, 3u, 4u));              // inside [out, out + 64)
    st_output(out + 64, make_uint4(5u, 6u, 7u, 8u));         // beyond it
}

cudaError_t launch_check_selftest(const KArgs &args, cudaStream_t stream)
{
#ifdef SYMAR_CHECK
    check_selftest_kernel<<<1, 32, 0, stream>>>(args);
    return cudaGetLastError();
#else
    (void)args;
    (void)stream;
    return cudaErrorNotSupported;
#endif
}

// ---- dispatch ---------------------------------------------------------------------

template <typename E, int P, bool DBG>
static KernelFn pick_algo(int algo)
{
    switch (algo) {
        case SYMAR_ONESHOT: return oneshot_kernel<E, P, DBG>;
        case SYMAR_TWOSHOT: return twoshot_kernel<E, P, DBG>;
        case SYMAR_LL:      return ll_kernel<E, P, DBG>;
        case SYMAR_SENTINEL: return sentinel_kernel<E, P, DBG>;
        case SYMAR_TWOSHOT_LL: return twoshot_push_kernel<E, P, false, DBG>;
        case SYMAR_TWOSHOT_SENTINEL: return twoshot_push_kernel<E, P, true, DBG>;
    }
    return nullptr;
}

template <typename E, bool DBG>
static KernelFn pick_ranks(int algo, int P)
{
    switch (P) {
        case 1: return pick_algo<E, 1, DBG>(algo);
        case 2: return pick_algo<E, 2, DBG>(algo);
        case 4: return pick_algo<E, 4, DBG>(algo);
        case 8: return pick_algo<E, 8, DBG>(algo);
    }
    return nullptr;
}

KernelFn kernel_for(int algo, int dtype, int P, bool dbg)
{
    if (dtype == SYMAR_F32) return dbg ? pick_ranks<F32, true>(algo, P) : pick_ranks<F32, false>(algo, P);
    if (dtype == SYMAR_BF16) return dbg ? pick_ranks<BF16, true>(algo, P) : pick_ranks<BF16, false>(algo, P);
    return nullptr;
}

template <typename E, bool DBG>
static KernelFn pick_ll_small_ranks(int P, int words)
{
    switch (P) {
        case 1: return words == 2 ? ll_small_kernel<E, 1, 2, DBG> : ll_small_kernel<E, 1, 4, DBG>;
        case 2: return words == 2 ? ll_small_kernel<E, 2, 2, DBG> : ll_small_kernel<E, 2, 4, DBG>;
        case 4: return words == 2 ? ll_small_kernel<E, 4, 2, DBG> : ll_small_kernel<E, 4, 4, DBG>;
        case 8: return words == 2 ? ll_small_kernel<E, 8, 2, DBG> : ll_small_kernel<E, 8, 4, DBG>;
    }
    return nullptr;
}

KernelFn ll_small_kernel_for(int dtype, int P, int words, bool dbg)
{
    if (dtype == SYMAR_F32) return dbg ? pick_ll_small_ranks<F32, true>(P, words) : pick_ll_small_ranks<F32, false>(P, words);
    if (dtype == SYMAR_BF16) return dbg ? pick_ll_small_ranks<BF16, true>(P, words) : pick_ll_small_ranks<BF16, false>(P, words);
    return nullptr;
}

// `cluster`: the P CTAs of a slot (one per rank) are launched as one thread-block cluster, which puts them
// on SMs of one GPC, i.e. on one half of the chip.  Nothing of a cluster is used in the kernels -- no
// distributed shared memory, no cluster barrier: the ranks still meet through flags in global memory
// only -- it is a statement about where the CTAs that signal one another run.
static void launch_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute attr[2], int P, int ctas_per_rank, int threads,
                          size_t smem_bytes, bool pdl, bool cluster, cudaStream_t stream)
{
    cfg                  = cudaLaunchConfig_t{};
    cfg.gridDim          = dim3((unsigned)ctas_per_rank, (unsigned)P, 1);
    cfg.blockDim         = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream           = stream;
    cfg.attrs            = attr;
    cfg.numAttrs         = 0;
    if (pdl) {
        attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
        ++cfg.numAttrs;
    }
    if (cluster && P > 1) {
        attr[cfg.numAttrs].id               = cudaLaunchAttributeClusterDimension;
        attr[cfg.numAttrs].val.clusterDim.x = 1;
        attr[cfg.numAttrs].val.clusterDim.y = (unsigned)P;
        attr[cfg.numAttrs].val.clusterDim.z = 1;
        ++cfg.numAttrs;
    }
}

cudaError_t launch_kernel(KernelFn fn, int P, int ctas_per_rank, int threads, size_t smem_bytes,
                          const KArgs &args, cudaStream_t stream, bool cluster)
{
    if (!args.pdl && !(cluster && P > 1)) {
        fn<<<dim3((unsigned)ctas_per_rank, (unsigned)P, 1), dim3((unsigned)threads, 1, 1), smem_bytes, stream>>>(args);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    launch_config(cfg, attr, P, ctas_per_rank, threads, smem_bytes, args.pdl != 0, cluster, stream);
    return cudaLaunchKernelEx(&cfg, fn, args);
}

// Clusters of P CTAs (one slot's ranks) of `fn` that the device holds at once; 0 or minus the CUDA error
// if such a cluster cannot be launched at all.
int max_resident_clusters(KernelFn fn, int P, int threads, size_t smem_bytes)
{
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    launch_config(cfg, attr, P, 1, threads, smem_bytes, false, true, nullptr);
    int n = 0;
    const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, fn, &cfg);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return -(int)e;                 // not launchable as clusters (the caller logs why)
    }
    return n;
}

}  // namespace symar
