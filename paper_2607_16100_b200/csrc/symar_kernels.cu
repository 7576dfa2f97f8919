// The three AllReduce kernels.  One launch emulates all P ranks: blockIdx.y is
// the rank, blockIdx.x the CTA slot of that rank.  CTAs of different ranks meet
// only through the symmetric heap, as GPUs of one NVLink domain would.
//
//   oneshot_kernel  Sec. III-A.1 (pull): exchange "input ready" flags with every
//                   peer, read all P inputs, reduce, write the own output.
//   twoshot_kernel  Sec. III-A.2: the same exchange, reduce only the own chunk,
//                   store it into every rank's output (all-gather from
//                   registers), then hand off with "chunk done" flags.
//   ll_kernel       Sec. IV "LL" + Sec. V example kernel: push every input word
//                   to every peer's scratch as {payload, flag} 8-byte stores,
//                   poll the own scratch, reduce, write the own output; scratch
//                   is double-buffered by iteration parity.
//
// No kernel contains a grid-wide barrier; every wait is one-directional (a CTA
// waits for data or a flag FROM each peer) and bounded.
#include "symar_device.cuh"
#include "symar_internal.h"

namespace symar {

// "Input ready" exchange shared by one-shot and two-shot (one synchronisation,
// Table I).  Lane q of warp 0 raises this rank's flag at peer q; then every
// warp polls the P flags of its own rank with lane q watching peer q, so all P
// polls are in flight together.  Returns false if the wait ran out.
template <int P, bool DBG>
__device__ __forceinline__ bool exchange_flags(const KArgs &a, uint64_t flags_off, int r, int c,
                                               uint32_t e, bool muted, bool all_warps)
{
    const uint32_t t    = threadIdx.x;
    const uint32_t lane = t & 31u;
    if (t < P && !muted) {
        uint32_t *dst =
            reinterpret_cast<uint32_t *>(a.seg0 + t * a.stride + flags_off + (size_t)c * kFlagGroup) + r;
        st_release_u32(dst, e);
    }
    if (P == 1) return true;
    if (!all_warps && t >= 32) return true;
    const uint32_t *mine =
        reinterpret_cast<const uint32_t *>(a.seg0 + (size_t)r * a.stride + flags_off + (size_t)c * kFlagGroup) +
        (lane < P ? lane : 0);
    Spin spin;
    for (;;) {
        const uint32_t f = ld_acquire_u32(mine);
        const unsigned late = __ballot_sync(0xffffffffu, lane < P && f != e);
        if (late == 0) return true;
        if (spin.due()) {
            if (__any_sync(0xffffffffu, spin.expired(a.spin_ns))) {
                if (lane == 0) report_timeout(a.ctl, r, __ffs(late) - 1, c);
                return false;
            }
        }
    }
}

template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kMaxThreads) oneshot_kernel(const KArgs a)
{
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r  = a.seg0 + (size_t)r * a.stride;
    uint64_t *ep = reinterpret_cast<uint64_t *>(seg_r + a.epoch_off) + c;
    const uint64_t n = ld_relaxed_u64(ep) + 1;   // this call's iteration number of slot c
    if (DBG) debug_delay(a, r, c);
    const bool muted = DBG && a.dbg_mute == r;

    const bool ok = exchange_flags<P, DBG>(a, a.ready_off, r, c, flag_of(n), muted, true);

    if (ok) {
        char *out = seg_r + a.out_off;
        for (uint64_t v = (uint64_t)c * T + t; v < a.nvec; v += (uint64_t)C * T) {
            uint4 x[P];
#pragma unroll
            for (int q = 0; q < P; ++q) x[q] = ld_peer(a.seg0 + (size_t)q * a.stride + a.in_off + v * 16);
            store_result(out, v, reduce_in_rank_order<E, P>(x), a.nvec, a.tail_bytes);
        }
    }
    __syncthreads();          // every thread has read the counter before it moves
    if (t == 0) *ep = n;
}

template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kMaxThreads) twoshot_kernel(const KArgs a)
{
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r  = a.seg0 + (size_t)r * a.stride;
    uint64_t *ep = reinterpret_cast<uint64_t *>(seg_r + a.epoch_off) + c;
    const uint64_t n = ld_relaxed_u64(ep) + 1;
    if (DBG) debug_delay(a, r, c);
    const bool muted  = DBG && a.dbg_mute == r;
    const uint32_t e  = flag_of(n);

    // reduce-scatter: rank r owns chunk r = vectors [lo, hi)
    bool ok = exchange_flags<P, DBG>(a, a.ready_off, r, c, e, muted, true);
    if (ok) {
        const uint64_t chv = (a.nvec + P - 1) / P;
        const uint64_t lo  = (uint64_t)r * chv;
        const uint64_t hi  = (lo + chv < a.nvec) ? lo + chv : a.nvec;
        for (uint64_t v = lo + (uint64_t)c * T + t; v < hi; v += (uint64_t)C * T) {
            uint4 x[P];
#pragma unroll
            for (int q = 0; q < P; ++q) x[q] = ld_peer(a.seg0 + (size_t)q * a.stride + a.in_off + v * 16);
            const uint4 res = reduce_in_rank_order<E, P>(x);
            // all-gather straight from registers into every rank's output
#pragma unroll
            for (int q = 0; q < P; ++q)
                store_result(a.seg0 + (size_t)q * a.stride + a.out_off, v, res, a.nvec, a.tail_bytes);
        }
    }
    // handoff: this CTA's part of chunk r has landed everywhere -> tell every
    // peer; then wait until every peer's CTA c has delivered its part here.
    __syncthreads();
    if (ok) ok = exchange_flags<P, DBG>(a, a.done_off, r, c, e, muted, false);
    if (t == 0) *ep = n;
}

template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kMaxThreads) ll_kernel(const KArgs a)
{
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    char *seg_r  = a.seg0 + (size_t)r * a.stride;
    uint64_t *ep = reinterpret_cast<uint64_t *>(seg_r + a.epoch_off) + c;
    const uint64_t n0 = ld_relaxed_u64(ep);
    if (DBG) debug_delay(a, r, c);
    const bool muted = DBG && a.dbg_mute == r;

    const char *in = seg_r + a.in_off;
    char *out      = seg_r + a.out_off;
    bool failed    = false;

    for (uint32_t it = 0; it < a.iters && !failed; ++it) {
        const uint64_t n   = n0 + 1 + it;            // advanceEpoch: flag value and sub-buffer
        const uint32_t e   = flag_of(n);
        const uint64_t v0  = ((uint64_t)it * C + c) * a.cv;
        const uint32_t cnt = v0 < a.nvec ? (uint32_t)(a.nvec - v0 < a.cv ? a.nvec - v0 : a.cv) : 0u;
        const uint64_t region = a.ll_off + ((uint64_t)(n & 1) * kLLSlots + c) * P * kLLSenderBytes;
        const uint64_t hi_e   = (uint64_t)e << 32;

        // bcast: {payload word, flag} pairs into every rank's scratch, sender row r
        if (!muted) {
            for (uint32_t k = t; k < cnt; k += T) {
                const uint4 x = ld_own(in + (v0 + k) * 16);
                const uint64_t d0 = hi_e | x.x, d1 = hi_e | x.y, d2 = hi_e | x.z, d3 = hi_e | x.w;
#pragma unroll
                for (int q = 0; q < P; ++q) {
                    char *dst = a.seg0 + (size_t)q * a.stride + region + (size_t)r * kLLSenderBytes + (size_t)k * 16;
                    st_relaxed_v2u64(dst, d0, d1);
                    st_relaxed_v2u64(dst + (size_t)kLLSlotVecs * 16, d2, d3);
                }
            }
        }
        // recvReduce: poll all P sender rows together until every flag matches
        for (uint32_t k = t; k < cnt && !failed; k += T) {
            const char *src = seg_r + region + (size_t)k * 16;
            U64x2 lo[P], hi[P];
            Spin spin;
            for (;;) {
                bool ready = true;
#pragma unroll
                for (int q = 0; q < P; ++q) {
                    lo[q] = ld_relaxed_v2u64(src + (size_t)q * kLLSenderBytes);
                    hi[q] = ld_relaxed_v2u64(src + (size_t)q * kLLSenderBytes + (size_t)kLLSlotVecs * 16);
                }
#pragma unroll
                for (int q = 0; q < P; ++q)
                    ready = ready && (uint32_t)(lo[q].a >> 32) == e && (uint32_t)(lo[q].b >> 32) == e &&
                            (uint32_t)(hi[q].a >> 32) == e && (uint32_t)(hi[q].b >> 32) == e;
                if (ready) break;
                if (spin.due() && spin.expired(a.spin_ns)) {
                    int late = 0;
#pragma unroll
                    for (int q = P - 1; q >= 0; --q)
                        if ((uint32_t)(lo[q].a >> 32) != e || (uint32_t)(hi[q].b >> 32) != e) late = q;
                    report_timeout(a.ctl, r, late, c);
                    failed = true;
                    break;
                }
            }
            if (failed) break;
            uint4 x[P];
#pragma unroll
            for (int q = 0; q < P; ++q)
                x[q] = make_uint4((uint32_t)lo[q].a, (uint32_t)lo[q].b, (uint32_t)hi[q].a, (uint32_t)hi[q].b);
            store_result(out, v0 + k, reduce_in_rank_order<E, P>(x), a.nvec, a.tail_bytes);
        }
        // No CTA barrier between iterations: position k is sent and received by
        // the same thread index on every rank, and a thread sends iteration i+1
        // only after its own receive of iteration i, which needed the peer
        // thread's send of iteration i, issued after that thread's receive of
        // iteration i-1 -- so the sub-buffer of parity (i+1)&1 is free.
    }
    __syncthreads();
    if (t == 0) *ep = n0 + a.iters;
}

// ---- dispatch ---------------------------------------------------------------------

template <typename E, int P, bool DBG>
static KernelFn pick_algo(int algo)
{
    switch (algo) {
        case SYMAR_ONESHOT: return oneshot_kernel<E, P, DBG>;
        case SYMAR_TWOSHOT: return twoshot_kernel<E, P, DBG>;
        case SYMAR_LL:      return ll_kernel<E, P, DBG>;
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

cudaError_t launch_kernel(KernelFn fn, int P, int ctas_per_rank, int threads, const KArgs &args,
                          cudaStream_t stream)
{
    fn<<<dim3((unsigned)ctas_per_rank, (unsigned)P, 1), dim3((unsigned)threads, 1, 1), 0, stream>>>(args);
    return cudaGetLastError();
}

}  // namespace symar
