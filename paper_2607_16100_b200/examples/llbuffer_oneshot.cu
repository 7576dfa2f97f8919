// A one-shot AllReduce(sum) written ONLY with the public thread-level primitives of
// symar_llbuffer.cuh, after the example of the paper's Sec. V ("Example One-shot
// AllReduce"): wrap symmetric scratch memory in an LLBuffer with double buffering; every
// thread loads a 32-bit word of its rank's input, broadcasts it into its row of every
// peer's region, receives and reduces the P rows in rank order, stores the result, and
// advances the epoch.  Works for any message size (several epochs per launch).
//
// The P ranks are the rows of the grid (blockIdx.y), as everywhere in this library; all
// P * ctas CTAs wait for one another and must be co-resident, so keep the grid small.
// Not a tuned kernel: it shows that a collective is a dozen lines on top of the primitives,
// and it is the test vehicle of the header (tests/test_llbuffer_gpu.py).  A second kernel
// further down, an all-gather of 64-bit words, covers 8-byte elements and the single
// send / recv / reset calls on an undivided buffer.
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include "symar_llbuffer.cuh"

using namespace symar;

namespace {

struct F32Acc {
    float v;
    __device__ static F32Acc widen(uint32_t w) { return {__uint_as_float(w)}; }
    __device__ static F32Acc add(F32Acc a, F32Acc b) { return {__fadd_rn(a.v, b.v)}; }
    __device__ uint32_t narrow() const { return __float_as_uint(v); }
};
struct BF16x2Acc {                      // one word = two bf16 elements, accumulated in binary32
    float lo, hi;
    __device__ static BF16x2Acc widen(uint32_t w) { return {__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)}; }
    __device__ static BF16x2Acc add(BF16x2Acc a, BF16x2Acc b) { return {__fadd_rn(a.lo, b.lo), __fadd_rn(a.hi, b.hi)}; }
    __device__ uint32_t narrow() const
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&h);
    }
};

template <LLSync Mode, int P, typename Acc>
__global__ void oneshot_llbuffer_kernel(const char *in0, char *out0, size_t io_stride, char *scratch0,
                                        size_t scratch_stride, size_t nwords, uint64_t epoch, int slots_per_cta,
                                        unsigned *fail)
{
    const int cta = blockIdx.x, ctas = gridDim.x, rank = blockIdx.y;
    // region of a CTA and epoch: P rows (one per sender) of slots_per_cta slots
    LLBuffer<Mode> buf(scratch0, scratch_stride, rank, P, cta, ctas,
                       (size_t)P * slots_per_cta * LLBuffer<Mode>::template slotBytes<uint32_t>(), 2, epoch, 1u << 20);
    const uint32_t *in = reinterpret_cast<const uint32_t *>(in0 + (size_t)rank * io_stride);
    uint32_t *out      = reinterpret_cast<uint32_t *>(out0 + (size_t)rank * io_stride);
    const size_t per_epoch = (size_t)ctas * slots_per_cta;
    for (size_t first = (size_t)cta * slots_per_cta; first < nwords + (size_t)cta * slots_per_cta; first += per_epoch) {
        for (int k = threadIdx.x; k < slots_per_cta; k += blockDim.x) {
            const size_t i = first + k;
            if (i >= nwords) continue;
            uint32_t w = in[i];
            if (Mode == LLSync::Sentinel && w == 0xffffffffu) w = 0xfffffffeu;   // never send the sentinel (a NaN either way)
            buf.template bcast<uint32_t, P>((size_t)rank * slots_per_cta + k, w);        // my row, every rank's region
            Acc acc;
            const bool ok = buf.template recvReduce<Acc, uint32_t, P, P, Mode == LLSync::Sentinel>(
                (size_t)k, (size_t)slots_per_cta, P, [](uint32_t x) { return Acc::widen(x); },
                [](Acc a, Acc b) { return Acc::add(a, b); }, acc);
            if (!ok) {
                atomicExch(fail, 1u);
                return;
            }
            out[i] = acc.narrow();
        }
        // sentinel mode: the restored sentinels must be in place before this sub-buffer is used
        // again two epochs from now (Sec. V "reset": visibility needs a fence)
        if (Mode == LLSync::Sentinel) __threadfence();
        buf.advanceEpoch();
    }
}

template <LLSync Mode, typename Acc>
cudaError_t launch(int P, dim3 grid, dim3 block, cudaStream_t s, const char *in0, char *out0, size_t io_stride,
                   char *scratch0, size_t scratch_stride, size_t nwords, uint64_t epoch, int slots, unsigned *fail)
{
    switch (P) {
        case 1: oneshot_llbuffer_kernel<Mode, 1, Acc><<<grid, block, 0, s>>>(in0, out0, io_stride, scratch0, scratch_stride, nwords, epoch, slots, fail); break;
        case 2: oneshot_llbuffer_kernel<Mode, 2, Acc><<<grid, block, 0, s>>>(in0, out0, io_stride, scratch0, scratch_stride, nwords, epoch, slots, fail); break;
        case 4: oneshot_llbuffer_kernel<Mode, 4, Acc><<<grid, block, 0, s>>>(in0, out0, io_stride, scratch0, scratch_stride, nwords, epoch, slots, fail); break;
        case 8: oneshot_llbuffer_kernel<Mode, 8, Acc><<<grid, block, 0, s>>>(in0, out0, io_stride, scratch0, scratch_stride, nwords, epoch, slots, fail); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

// An all-gather of 64-bit words on the same primitives: exercises 8-byte elements (16-byte LL slots),
// send / recv / reset one at a time, and a buffer that is not subdivided (round_robin = 0: one fixed
// region per CTA, safe here because a launch is one epoch and a kernel boundary separates epochs).
template <LLSync Mode, int P>
__global__ void allgather_u64_kernel(const char *in0, char *out0, size_t io_stride, char *scratch0,
                                     size_t scratch_stride, size_t nwords, uint64_t epoch, unsigned *fail)
{
    const int cta = blockIdx.x, ctas = gridDim.x, rank = blockIdx.y;
    const size_t per_cta = (nwords + ctas - 1) / ctas;
    // a region holds P rows of per_cta slots; with round_robin = 0 the object applies no offset, so the
    // CTA's region is addressed through the slot index
    LLBuffer<Mode> buf(scratch0, scratch_stride, rank, P, cta, ctas, 0, 0, epoch, 1u << 20);
    const size_t region = (size_t)cta * P * per_cta;
    const uint64_t *in = reinterpret_cast<const uint64_t *>(in0 + (size_t)rank * io_stride);
    uint64_t *out      = reinterpret_cast<uint64_t *>(out0 + (size_t)rank * io_stride);
    for (size_t k = threadIdx.x; k < per_cta; k += blockDim.x) {
        const size_t i = (size_t)cta * per_cta + k;
        if (i >= nwords) continue;
        uint64_t w = in[i];
        if (Mode == LLSync::Sentinel && w == ~0ull) w = ~1ull;
        for (int q = 0; q < P; ++q) buf.template send<uint64_t>(q, region + (size_t)rank * per_cta + k, w);
        for (int q = 0; q < P; ++q) {
            uint64_t v;
            if (!buf.template recv<uint64_t>(region + (size_t)q * per_cta + k, v)) {
                atomicExch(fail, 1u);
                return;
            }
            if (Mode == LLSync::Sentinel) buf.template reset<uint64_t>(region + (size_t)q * per_cta + k);
            out[(size_t)q * nwords + i] = v;
        }
    }
}

// Stress of the 16-byte LL slot that an 8-byte element occupies ({payload64, flag64} in one vector
// store): for `epochs` epochs in one launch every thread sends a payload that spells out its epoch,
// sender and slot to all peers and receives the peers' payloads; a payload whose flag says "this
// epoch" while its own epoch field says otherwise would be a 16-byte store observed in two halves.
// Seeded idle times before every epoch vary which side is ahead.  counts[0]: a wait ran out;
// counts[1]: payloads that did not match their flag; counts[2]: payloads checked.
template <int P>
__global__ void slot_stress_u64_kernel(char *scratch0, size_t scratch_stride, int slots, uint64_t first_epoch,
                                       uint32_t epochs, uint32_t seed, uint32_t max_idle_ns, unsigned long long *counts)
{
    const int cta = blockIdx.x, ctas = gridDim.x, rank = blockIdx.y, t = threadIdx.x;
    LLBuffer<LLSync::LL> buf(scratch0, scratch_stride, rank, P, cta, ctas,
                             (size_t)P * slots * LLBuffer<LLSync::LL>::template slotBytes<uint64_t>(), 2, first_epoch,
                             1u << 22);
    unsigned long long bad = 0, seen = 0;
    for (uint32_t it = 0; it < epochs; ++it) {
        if (max_idle_ns != 0) {          // bounded pause, different per CTA, rank and epoch
            uint32_t h = seed ^ (uint32_t)(rank * 0x9E3779B1u) ^ (uint32_t)(cta * 0x85EBCA77u) ^ (it * 0xC2B2AE3Du);
            h ^= h >> 16; h *= 0x7feb352dU; h ^= h >> 15; h *= 0x846ca68bU; h ^= h >> 16;
            const uint64_t wait = h % max_idle_ns;
            uint64_t t0, now;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
            do { asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now)); } while (now - t0 < wait);
        }
        const uint64_t e = buf.epoch();
        if (t < slots) {
            const uint64_t mine = (e << 32) | ((uint64_t)rank << 16) | (uint64_t)t;
            for (int q = 0; q < P; ++q)
                if (q != rank) buf.template send<uint64_t>(q, (size_t)rank * slots + t, mine);
            for (int q = 0; q < P; ++q) {
                if (q == rank) continue;
                uint64_t v;
                if (!buf.template recv<uint64_t>((size_t)q * slots + t, v)) {
                    atomicAdd(&counts[0], 1ull);
                    return;
                }
                ++seen;
                if (v != ((e << 32) | ((uint64_t)q << 16) | (uint64_t)t)) ++bad;
            }
        }
        buf.advanceEpoch();
    }
    if (bad) atomicAdd(&counts[1], bad);
    atomicAdd(&counts[2], seen);
}

}  // namespace

extern "C" {

// Runs the slot stress above: P ranks x ctas CTAs x `slots` threads, `epochs` epochs from `first_epoch`
// (epochs below 2^32 so that the payload's epoch field is the flag).  Scratch per rank:
// symar_llbuffer_bytes(0, 8, P * slots, ctas, 2), zeroed before the first launch.  device_counts: three
// zeroed 64-bit counters (waits that ran out, mismatching payloads, payloads checked).
int llbuffer_slot_stress_u64(int P, void *scratch0, size_t scratch_stride, int ctas, int slots, unsigned long long first_epoch,
                             unsigned epochs, unsigned seed, unsigned max_idle_ns, unsigned long long *device_counts,
                             void *cuda_stream)
{
    if (!scratch0 || !device_counts || ctas < 1 || slots < 1 || slots > 1024 || first_epoch == 0 || max_idle_ns > 100000u ||
        first_epoch + epochs >= (1ull << 32))
        return -1;
    const dim3 grid(ctas, P), block((slots + 31) / 32 * 32);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    char *s0 = (char *)scratch0;
    if (P == 2) slot_stress_u64_kernel<2><<<grid, block, 0, s>>>(s0, scratch_stride, slots, first_epoch, epochs, seed, max_idle_ns, device_counts);
    else if (P == 4) slot_stress_u64_kernel<4><<<grid, block, 0, s>>>(s0, scratch_stride, slots, first_epoch, epochs, seed, max_idle_ns, device_counts);
    else if (P == 8) slot_stress_u64_kernel<8><<<grid, block, 0, s>>>(s0, scratch_stride, slots, first_epoch, epochs, seed, max_idle_ns, device_counts);
    else return -1;
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

// All-gather of nwords 64-bit words per rank: out[r] = in[0] | in[1] | ... | in[P-1] for every rank r.
// Scratch per rank: symar_llbuffer_bytes(mode, 8, P * ceil(nwords / ctas), ctas, 0).  mode / epoch /
// device_fail as for llbuffer_oneshot_allreduce; one epoch per launch.
int llbuffer_allgather_u64(int mode, int P, const void *in0, void *out0, size_t io_stride, void *scratch0,
                           size_t scratch_stride, size_t nwords, unsigned long long epoch, int ctas, int threads,
                           unsigned *device_fail, void *cuda_stream)
{
    if (!in0 || !out0 || !scratch0 || !device_fail || ctas < 1 || threads < 1 || threads > 1024 || epoch == 0)
        return -1;
    const dim3 grid(ctas, P), block(threads);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const char *i0 = (const char *)in0;
    char *o0 = (char *)out0, *s0 = (char *)scratch0;
#define SYMAR_EX_LAUNCH(M, N) allgather_u64_kernel<M, N><<<grid, block, 0, s>>>(i0, o0, io_stride, s0, scratch_stride, nwords, epoch, device_fail)
    if (mode == 0) {
        if (P == 1) SYMAR_EX_LAUNCH(LLSync::LL, 1); else if (P == 2) SYMAR_EX_LAUNCH(LLSync::LL, 2);
        else if (P == 4) SYMAR_EX_LAUNCH(LLSync::LL, 4); else if (P == 8) SYMAR_EX_LAUNCH(LLSync::LL, 8); else return -1;
    } else if (mode == 1) {
        if (P == 1) SYMAR_EX_LAUNCH(LLSync::Sentinel, 1); else if (P == 2) SYMAR_EX_LAUNCH(LLSync::Sentinel, 2);
        else if (P == 4) SYMAR_EX_LAUNCH(LLSync::Sentinel, 4); else if (P == 8) SYMAR_EX_LAUNCH(LLSync::Sentinel, 8); else return -1;
    } else {
        return -1;
    }
#undef SYMAR_EX_LAUNCH
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

// mode 0 = LL, 1 = sentinel; bf16 0 = fp32 words, 1 = bf16 pairs.  in0 / out0 / scratch0 are rank 0's
// device addresses, the strides the byte distance to the next rank's copy.  `epoch` is the first
// epoch this launch may use; *host_epochs_used (may be NULL) receives how many it consumes, so
// the next launch passes epoch + that.  device_fail: one zeroed u32 that becomes 1 if a wait ran
// out.  Returns 0 or a negative number for bad arguments / launch failure.
int llbuffer_oneshot_allreduce(int mode, int P, int bf16, const void *in0, void *out0, size_t io_stride,
                               void *scratch0, size_t scratch_stride, size_t nwords, unsigned long long epoch,
                               int ctas, int threads, int slots_per_cta, unsigned *device_fail, void *cuda_stream,
                               unsigned long long *host_epochs_used)
{
    if (!in0 || !out0 || !scratch0 || !device_fail || ctas < 1 || threads < 1 || threads > 1024 || slots_per_cta < 1)
        return -1;
    if (epoch == 0) return -1;
    const size_t per_epoch = (size_t)ctas * slots_per_cta;
    if (host_epochs_used) *host_epochs_used = (nwords + per_epoch - 1) / per_epoch + 1;   // + 1: a skipped flag value
    const dim3 grid(ctas, P), block(threads);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e;
    const char *i0 = (const char *)in0;
    char *o0 = (char *)out0, *s0 = (char *)scratch0;
    if (mode == 0)
        e = bf16 ? launch<LLSync::LL, BF16x2Acc>(P, grid, block, s, i0, o0, io_stride, s0, scratch_stride, nwords, epoch, slots_per_cta, device_fail)
                 : launch<LLSync::LL, F32Acc>(P, grid, block, s, i0, o0, io_stride, s0, scratch_stride, nwords, epoch, slots_per_cta, device_fail);
    else if (mode == 1)
        e = bf16 ? launch<LLSync::Sentinel, BF16x2Acc>(P, grid, block, s, i0, o0, io_stride, s0, scratch_stride, nwords, epoch, slots_per_cta, device_fail)
                 : launch<LLSync::Sentinel, F32Acc>(P, grid, block, s, i0, o0, io_stride, s0, scratch_stride, nwords, epoch, slots_per_cta, device_fail);
    else
        return -1;
    return e == cudaSuccess ? 0 : -3;
}

}  // extern "C"
