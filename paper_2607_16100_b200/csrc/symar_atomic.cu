// Two-shot AllReduce with atomic accumulation in the owner's scratch (paper Sec. IV,
// "LL128 Atomic AllReduce"; Table I, last row).
//
// Reduce-scatter: rank t owns chunk t of the message.  Every rank, the owner
// included, ADDS its part of chunk t into rank t's scratch with 16-byte vector
// atomics (red.global.add.v4.f32).  The scratch is an array of 128-byte lines of
// 32 binary32 words: word 0 counts contributions (every rank adds 1.0 to it),
// words 1..31 accumulate 31 consecutive elements of the chunk.  Eight threads
// serve one line, thread j words 4j..4j+3, so a warp issues whole lines.  There
// is no separate signal and no fence: the count rides with the data, as the
// flag does in the LL protocol, at 1/32 instead of 1/2 of the bytes.
//
// All-gather: the owner's CTAs poll their lines until the count equals P, read
// the sums, zero the line for its next use, narrow once, and store the result
// into every rank's output; then the usual "done" handoff of the two-shot kernel.
//
// Differences from the paper's kernel, and why:
//  * The paper keeps 16-byte aligned input vectors and moves the element that
//    the count displaces through shared memory to "extra" threads.  Here a line
//    simply takes 31 consecutive elements, read with scalar loads (coalesced:
//    a warp reads 4 x 124 contiguous bytes); same scratch format, no shared memory.
//  * bf16 inputs are widened and accumulated in binary32 (the paper adds bf16
//    vectors and accepts the larger error); the result is narrowed once, so it
//    differs from the rank-ordered sum only by the order of the binary32 adds.
//  * The paper relies on NVLink applying a 128-byte write atomically, so that
//    "count == N" proves the whole line complete.  One GPU's L2 documents no
//    such guarantee for the eight 16-byte atomics of a line.  A line whose
//    count has reached P is therefore read once more before it is used: the
//    second read is issued a full round trip after the last contribution's
//    count was seen, by which time the rest of that same 128-byte request has
//    been applied.  (Empirical, not architectural; variant bit 0 drops the
//    re-read for measurement.)
//  * The all-gather uses stores plus the flag handoff instead of polling a
//    sentinel-filled output buffer, so the output needs no preparation.
//
// The order of the atomic adds is not fixed: results are NOT bit-reproducible
// (Table I "Deterministic: no"); they obey the forward error bound
// gamma_{P-1} * sum|x_q| of Sec. IV.  Global binary32 atomics flush subnormal
// inputs and results to zero.  SYMAR_AUTO never picks this algorithm.
#include "symar_device.cuh"
#include "symar_internal.h"

namespace symar {

namespace {

__device__ __forceinline__ void red_add_v4_f32(void *p, float a, float b, float c, float d)
{
    p = SYMAR_PTR(p, 16, kRegAt);
    asm volatile("red.relaxed." SYMAR_SCOPE ".global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b),
                 "f"(c), "f"(d)
                 : "memory");
}

template <typename E> struct Elem;
template <> struct Elem<F32> {
    using T = float;
    __device__ static __forceinline__ float load(const char *p)
    {
        return __ldg(SYMAR_PTR(reinterpret_cast<const float *>(p), 4, kRegIn));
    }
    __device__ static __forceinline__ void store(char *p, float v) { *SYMAR_PTR(reinterpret_cast<float *>(p), 4, kRegOut) = v; }
};
template <> struct Elem<BF16> {
    using T = uint16_t;
    __device__ static __forceinline__ float load(const char *p)
    {
        return __uint_as_float((uint32_t)__ldg(SYMAR_PTR(reinterpret_cast<const unsigned short *>(p), 2, kRegIn)) << 16);
    }
    __device__ static __forceinline__ void store(char *p, float v)
    {
        __nv_bfloat16 h = __float2bfloat16_rn(v);
        *SYMAR_PTR(reinterpret_cast<uint16_t *>(p), 2, kRegOut) = *reinterpret_cast<uint16_t *>(&h);
    }
};

}  // namespace

template <typename E, int P, bool DBG>
__global__ void __launch_bounds__(kMaxThreads) twoshot_atomic_kernel(const KArgs a)
{
    using El = Elem<E>;
    constexpr uint32_t es = sizeof(typename El::T);
    SYMAR_CHECK_BEGIN(a, P, a.count * es, a.count * es);
    const int c = blockIdx.x, r = blockIdx.y, C = gridDim.x;
    const uint32_t t = threadIdx.x, T = blockDim.x;
    const uint32_t j = t & 7u;                       // position in the 8-thread group of a line
    const uint32_t g = t >> 3, G = T >> 3;           // group index, groups per CTA
    char *seg_r      = a.seg0 + (size_t)r * a.stride;
    const uint32_t *dcount = reinterpret_cast<const uint32_t *>(counters_near(a, r, c) + kCtrDone);
    if (a.pdl) {
        pdl_wait();                                  // the previous call has left the heap
        pdl_launch_dependents();
    }
    if (DBG) debug_delay(a, r, c);
    if (DBG && a.dbg_mute == r) return;              // test hook: this rank never joins

    // Which half of the scratch: the parity of this slot's handoff count, the same
    // on every rank (all ranks have made the same calls with the same launch shape).
    const uint32_t half = ld_relaxed_u32(dcount) & 1u;
    const uint64_t half_off = a.at_off + (uint64_t)half * (kAtHalfBytesPerRank * P);

    const uint64_t ch = (a.count + P - 1) / P;       // elements per chunk
    // lines of this CTA: L = c + C m; group g takes m = g, g + G, ...
    const uint64_t nl = (ch + kAtLinePayload - 1) / kAtLinePayload;           // lines per full chunk
    const uint64_t nm = nl > (uint64_t)c ? (nl - c + C - 1) / C : 0;          // values of m for this CTA

    // ---- reduce-scatter: add my part of every chunk into its owner's scratch ----
    const char *in = seg_r + a.in_off;
    for (uint64_t m = g; m < nm; m += G) {
        const uint64_t L  = (uint64_t)c + (uint64_t)C * m;
        const uint64_t e0 = L * kAtLinePayload + 4 * j;      // word 4j+i of the line holds chunk element e0 + i - 1
        float v[P][4];
#pragma unroll
        for (int k = 0; k < P; ++k) {
            const int tgt = (r + 1 + k) % P;                 // remote owners first, the own chunk last
            const uint64_t lo = (uint64_t)tgt * ch;
            const uint64_t len = lo < a.count ? (a.count - lo < ch ? a.count - lo : ch) : 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint64_t e = e0 + i - 1;               // (j == 0, i == 0) is the counter word
                const bool counter = (j == 0 && i == 0);
                v[k][i] = counter ? 1.0f : (e < len ? El::load(in + (lo + e) * es) : 0.0f);
            }
        }
#pragma unroll
        for (int k = 0; k < P; ++k) {
            const int tgt = (r + 1 + k) % P;
            char *line = a.seg0 + (size_t)tgt * a.stride + half_off + L * kAtLineBytes;
            red_add_v4_f32(line + 16 * j, v[k][0], v[k][1], v[k][2], v[k][3]);
        }
    }

    // ---- all-gather: my lines of my own chunk, once all P ranks have added to them ----
    bool ok = true;
    {
        const uint64_t lo  = (uint64_t)r * ch;
        const uint64_t len = lo < a.count ? (a.count - lo < ch ? a.count - lo : ch) : 0;
        const uint64_t mynl = (len + kAtLinePayload - 1) / kAtLinePayload;    // lines that carry payload
        const uint32_t lane = t & 31u;
        // a warp walks its four groups' lines together, so that every shuffle below is warp-uniform
        const uint64_t warp_g0 = g & ~3u;
        for (uint64_t mb = warp_g0; mb < nm && ok; mb += G) {
            const uint64_t m  = mb + (g & 3u);
            const uint64_t L  = (uint64_t)c + (uint64_t)C * m;
            const bool have   = m < nm;
            char *line        = seg_r + half_off + L * kAtLineBytes + 16 * j;
            uint4 x           = make_uint4(0, 0, 0, 0);
            Spin spin;
            for (;;) {
                if (have) x = ld_relaxed_v4(line);
                const uint32_t cnt = __shfl_sync(0xffffffffu, x.x, lane & ~7u);      // the group's counter word
                const unsigned late = __ballot_sync(0xffffffffu, have && __uint_as_float(cnt) != (float)P);
                if (late == 0) break;
                if (spin.due() && __any_sync(0xffffffffu, spin.expired(a.spin_ns))) {
                    if (lane == 0) report_timeout(a.ctl, r, -1, c);
                    ok = false;
                    break;
                }
            }
            if (!ok) break;
            if (have) {
                if (!(a.variant & 1u)) x = ld_relaxed_v4(line);                      // confirming re-read
                st_relaxed_v4(line, make_uint4(0, 0, 0, 0));                          // ready for the call after next
                if (L < mynl) {
                    const float f[4] = {__uint_as_float(x.x), __uint_as_float(x.y), __uint_as_float(x.z),
                                        __uint_as_float(x.w)};
                    const uint64_t e0 = L * kAtLinePayload + 4 * j;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint64_t e = e0 + i - 1;
                        if ((j != 0 || i != 0) && e < len) {
#pragma unroll
                            for (int q = 0; q < P; ++q)
                                El::store(a.seg0 + (size_t)q * a.stride + a.out_off + (lo + e) * es, f[i]);
                        }
                    }
                }
            }
        }
    }

    // handoff: my lines have landed in every output -> tell every peer; then wait
    // until every peer's CTA c has delivered its part here.
    uint32_t dwant;
    const bool all_ok = __syncthreads_and(ok);
    flag_exchange<P, true>(a, a.done_off, kPairDone, dcount, r, c, !all_ok, false, dwant);
    publish_u32(a, r, c, kCtrDone, dwant);
    if (DBG) debug_stamp_out(a);
}

using KernelFn = void (*)(const KArgs);

template <typename E, bool DBG>
static KernelFn pick_ranks(int P)
{
    switch (P) {
        case 1: return twoshot_atomic_kernel<E, 1, DBG>;
        case 2: return twoshot_atomic_kernel<E, 2, DBG>;
        case 4: return twoshot_atomic_kernel<E, 4, DBG>;
        case 8: return twoshot_atomic_kernel<E, 8, DBG>;
    }
    return nullptr;
}

KernelFn atomic_kernel_for(int dtype, int P, bool dbg)
{
    if (dtype == SYMAR_F32) return dbg ? pick_ranks<F32, true>(P) : pick_ranks<F32, false>(P);
    if (dtype == SYMAR_BF16) return dbg ? pick_ranks<BF16, true>(P) : pick_ranks<BF16, false>(P);
    return nullptr;
}

}  // namespace symar
