/* symar_llbuffer.cuh -- thread-level low-latency buffer primitives for custom collective
 * kernels on symmetric memory (paper Sec. V, "Low-Latency API Design": the buffer-centric
 * device object with send / recv / recvUnrolled / recvReduce / bcast / reset / advanceEpoch
 * and the two synchronisation modes of Sec. IV, LL and sentinel).
 *
 * Public and self-contained: CUDA only, no other header of this library.  Device code for
 * sm_70 and later; every primitive acts for ONE thread (Sec. V "Constraints": thread-level
 * primitives only).  The library's own AllReduce kernels do not use this header; it is the
 * building block for kernels the library does not ship (example: llbuffer_oneshot.cu in the
 * package's examples folder).
 *
 * Memory model of the object
 *   A buffer is symmetric memory: every rank owns a copy with the same layout, rank q's copy
 *   starts at base + q * rank_stride (bytes).  With round_robin R > 0 a copy is R sub-buffers
 *   of ctas * bytes_per_cta_per_epoch bytes each; the region of CTA c in epoch e starts at
 *       ((e mod R) * ctas + c) * bytes_per_cta_per_epoch,
 *   so consecutive epochs use disjoint memory (double buffering for R = 2) and a rank may run
 *   ahead of a peer by R - 1 epochs without overwriting what the peer still reads.  With
 *   R = 0 the copy is not subdivided, offsets are the caller's business and advanceEpoch()
 *   only advances the flag value.
 *   A slot holds one element of type T (4 or 8 bytes, trivially copyable):
 *       LL        2 * sizeof(T) bytes {payload, flag}, the flag as large as T and equal to the
 *                 buffer's epoch; payload and flag travel in ONE store (8 bytes for 4-byte T,
 *                 a 16-byte vector store for 8-byte T, which the device performs as one
 *                 access -- the assumption the paper's 16-byte LL stores make as well);
 *                 memory must be zero before first use (flag 0 = never written);
 *       Sentinel  sizeof(T) bytes; the slot holds the all-ones pattern until data arrives, so
 *                 a payload must not be all ones; memory is prepared with
 *                 symar_llbuffer_init_sentinel() and every slot is reset after it is read.
 *   Slot indices are relative to the CTA's region of the current epoch.
 *
 * Waiting is bounded: recv* poll at most `max_polls` times and then return false, leaving the
 * output unspecified; nothing in this header can spin forever.
 *
 * Epochs: the object does not persist its epoch.  A kernel receives the epoch of its first
 * iteration from its caller (a kernel argument, or a counter in memory when launches are
 * replayed from a CUDA graph) and every rank must pass the same value.  Epoch values whose
 * flag would be 0 are skipped by advanceEpoch().
 */
#ifndef SYMAR_LLBUFFER_CUH
#define SYMAR_LLBUFFER_CUH

#include <cstddef>
#include <cstdint>

namespace symar {

enum class LLSync { LL, Sentinel };

/* Bytes of ONE rank's copy for the given shape (host or device):
 * slots_per_cta elements of elem_bytes (4 or 8) per CTA and epoch.  (The host-side
 * counterpart of the paper's scratch-size helper; also exported from the library as
 * symar_llbuffer_bytes.) */
__host__ __device__ constexpr size_t llbuffer_bytes(LLSync mode, size_t elem_bytes, size_t slots_per_cta, int ctas,
                                                    int round_robin)
{
    return (mode == LLSync::LL ? 2 : 1) * elem_bytes * slots_per_cta * (size_t)ctas *
           (size_t)(round_robin > 0 ? round_robin : 1);
}

namespace llb_detail {

template <int Bytes> struct Word;
template <> struct Word<4> { using type = uint32_t; };
template <> struct Word<8> { using type = uint64_t; };

template <typename T> __device__ __forceinline__ typename Word<sizeof(T)>::type to_bits(const T &v)
{
    typename Word<sizeof(T)>::type b;
    __builtin_memcpy(&b, &v, sizeof(T));
    return b;
}
template <typename T> __device__ __forceinline__ T from_bits(typename Word<sizeof(T)>::type b)
{
    T v;
    __builtin_memcpy(&v, &b, sizeof(T));
    return v;
}

/* {payload, flag} as one store / one load */
__device__ __forceinline__ void st_pair(void *p, uint32_t payload, uint32_t flag)
{
    const uint64_t w = ((uint64_t)flag << 32) | payload;
    asm volatile("st.relaxed.sys.global.u64 [%0], %1;" ::"l"(p), "l"(w) : "memory");
}
__device__ __forceinline__ void st_pair(void *p, uint64_t payload, uint64_t flag)
{
    asm volatile("st.relaxed.sys.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(payload), "l"(flag) : "memory");
}
__device__ __forceinline__ void ld_pair(const void *p, uint32_t &payload, uint32_t &flag)
{
    uint64_t w;
    asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(w) : "l"(p) : "memory");
    payload = (uint32_t)w;
    flag    = (uint32_t)(w >> 32);
}
__device__ __forceinline__ void ld_pair(const void *p, uint64_t &payload, uint64_t &flag)
{
    asm volatile("ld.relaxed.sys.global.v2.u64 {%0, %1}, [%2];" : "=l"(payload), "=l"(flag) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_word(void *p, uint32_t v)
{
    asm volatile("st.relaxed.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_word(void *p, uint64_t v)
{
    asm volatile("st.relaxed.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void ld_word(const void *p, uint32_t &v)
{
    asm volatile("ld.relaxed.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
}
__device__ __forceinline__ void ld_word(const void *p, uint64_t &v)
{
    asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
}

}  // namespace llb_detail

template <LLSync Mode>
class LLBuffer {
public:
    /* base: rank 0's copy; rank_stride: bytes between two ranks' copies; rank / nranks: this
     * thread's rank and the number of ranks; cta / ctas: this thread's CTA index among the
     * CTAs of its rank that share the buffer; bytes_per_cta_per_epoch and round_robin as
     * described above; epoch: the first iteration's epoch (>= 1, the same on every rank);
     * max_polls: bound of every wait. */
    __device__ LLBuffer(void *base, size_t rank_stride, int rank, int nranks, int cta, int ctas,
                        size_t bytes_per_cta_per_epoch, int round_robin, uint64_t epoch,
                        uint32_t max_polls = 1u << 22)
        : base_(static_cast<char *>(base)), stride_(rank_stride), rank_(rank), nranks_(nranks), cta_(cta),
          ctas_(ctas), region_bytes_(bytes_per_cta_per_epoch), rr_(round_robin), epoch_(epoch ? epoch : 1),
          max_polls_(max_polls)
    {
        if (flag32() == 0) ++epoch_;
        update_offset();
    }

    __device__ __forceinline__ uint64_t epoch() const { return epoch_; }
    __device__ __forceinline__ int rank() const { return rank_; }
    __device__ __forceinline__ int nranks() const { return nranks_; }

    /* bytes one element of type T occupies in this mode */
    template <typename T> __host__ __device__ static constexpr size_t slotBytes()
    {
        return (Mode == LLSync::LL ? 2 : 1) * sizeof(T);
    }

    /* Next iteration: the other sub-buffer (if round_robin > 0) and the next flag value. */
    __device__ __forceinline__ void advanceEpoch()
    {
        ++epoch_;
        if (flag32() == 0) ++epoch_;          // 0 means "never written"
        update_offset();
    }

    /* Writes `value` into slot `slot` of peer `peer`'s copy (of this CTA's region, this epoch). */
    template <typename T> __device__ __forceinline__ void send(int peer, size_t slot, const T &value) const
    {
        using W = typename llb_detail::Word<sizeof(T)>::type;
        char *p = base_ + (size_t)peer * stride_ + offset_ + slot * slotBytes<T>();
        if (Mode == LLSync::LL) llb_detail::st_pair(p, llb_detail::to_bits(value), (W)flag<W>());
        else llb_detail::st_word(p, llb_detail::to_bits(value));
    }

    /* The same to every rank, this one included (no multicast on one device: a loop over peers,
     * unrolled Unroll times). */
    template <typename T, int Unroll = 8> __device__ __forceinline__ void bcast(size_t slot, const T &value) const
    {
#pragma unroll(Unroll)
        for (int q = 0; q < nranks_; ++q) send<T>(q, slot, value);
    }

    /* Clears slot `slot` of this rank's own copy: zero in LL mode, the sentinel in sentinel mode.
     * Visibility to other threads is not ordered; fence if the slot is reused within the kernel. */
    template <typename T> __device__ __forceinline__ void reset(size_t slot) const
    {
        using W = typename llb_detail::Word<sizeof(T)>::type;
        char *p = base_ + (size_t)rank_ * stride_ + offset_ + slot * slotBytes<T>();
        if (Mode == LLSync::LL) llb_detail::st_pair(p, (W)0, (W)0);
        else llb_detail::st_word(p, (W)~(W)0);
    }
    template <typename T> __device__ __forceinline__ void resetRange(size_t first_slot, size_t count) const
    {
        for (size_t i = 0; i < count; ++i) reset<T>(first_slot + i);
    }

    /* Polls slot `slot` of this rank's own copy until it holds data of the current epoch (LL) or
     * differs from the sentinel; false if max_polls ran out. */
    template <typename T, bool Reset = false> __device__ __forceinline__ bool recv(size_t slot, T &value) const
    {
        T v[1];
        const bool ok = recvUnrolled<T, 1, 1, Reset>(slot, 1, 1, v);
        value = v[0];
        return ok;
    }

    /* Receives elt_count elements from slots first_slot + i * slot_step, i < elt_count, polling
     * all of them together.  Elements [0, MinEltCount) are always accessed, [MinEltCount,
     * MaxEltCount) only if i < elt_count (compile-time unrolling; MinEltCount <= elt_count <=
     * MaxEltCount). */
    template <typename T, int MinEltCount, int MaxEltCount, bool Reset = false>
    __device__ __forceinline__ bool recvUnrolled(size_t first_slot, size_t slot_step, int elt_count,
                                                 T (&out)[MaxEltCount]) const
    {
        using W = typename llb_detail::Word<sizeof(T)>::type;
        const char *p0 = base_ + (size_t)rank_ * stride_ + offset_ + first_slot * slotBytes<T>();
        const size_t step = slot_step * slotBytes<T>();
        W bits[MaxEltCount];
        unsigned pending = 0;
#pragma unroll
        for (int i = 0; i < MaxEltCount; ++i)
            if (i < MinEltCount || i < elt_count) pending |= 1u << i;
        for (uint32_t polls = 0; pending != 0; ++polls) {
            if (polls >= max_polls_) return false;
#pragma unroll
            for (int i = 0; i < MaxEltCount; ++i) {
                if (!(pending >> i & 1u)) continue;
                if (Mode == LLSync::LL) {
                    W f;
                    llb_detail::ld_pair(p0 + (size_t)i * step, bits[i], f);
                    if (f == (W)flag<W>()) pending &= ~(1u << i);
                } else {
                    llb_detail::ld_word(p0 + (size_t)i * step, bits[i]);
                    if (bits[i] != (W)~(W)0) pending &= ~(1u << i);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < MaxEltCount; ++i)
            if (i < MinEltCount || i < elt_count) {
                out[i] = llb_detail::from_bits<T>(bits[i]);
                if (Reset) reset<T>(first_slot + (size_t)i * slot_step);
            }
        return true;
    }

    /* Receives one element from each of elt_count slots (typically one per peer) and folds them
     * IN SLOT ORDER: acc = cvt(x0); acc = op(acc, cvt(x1)); ...  (fixed order, so the result is
     * reproducible).  Cvt converts T to the accumulator type. */
    template <typename Acc, typename T, int MinEltCount, int MaxEltCount, bool Reset = false, typename Cvt,
              typename Op>
    __device__ __forceinline__ bool recvReduce(size_t first_slot, size_t slot_step, int elt_count, Cvt cvt, Op op,
                                               Acc &acc) const
    {
        T x[MaxEltCount];
        if (!recvUnrolled<T, MinEltCount, MaxEltCount, Reset>(first_slot, slot_step, elt_count, x)) return false;
        acc = cvt(x[0]);
#pragma unroll
        for (int i = 1; i < MaxEltCount; ++i)
            if (i < MinEltCount || i < elt_count) acc = op(acc, cvt(x[i]));
        return true;
    }

private:
    __device__ __forceinline__ uint32_t flag32() const { return (uint32_t)epoch_; }
    template <typename W> __device__ __forceinline__ W flag() const
    {
        return sizeof(W) == 4 ? (W)flag32() : (W)epoch_;
    }
    __device__ __forceinline__ void update_offset()
    {
        // iteration index = epoch minus the flag values skipped so far (multiples of 2^32), so that
        // consecutive epochs always land in consecutive sub-buffers
        const uint64_t iter = epoch_ - (epoch_ >> 32);
        offset_ = rr_ > 0 ? ((size_t)(iter % (uint64_t)rr_) * ctas_ + cta_) * region_bytes_ : 0;
    }

    char    *base_;
    size_t   stride_;
    int      rank_, nranks_, cta_, ctas_;
    size_t   region_bytes_;
    int      rr_;
    uint64_t epoch_;
    uint32_t max_polls_;
    size_t   offset_;
};

}  // namespace symar
#endif /* SYMAR_LLBUFFER_CUH */
