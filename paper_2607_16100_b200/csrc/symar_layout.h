// Internal layout of a symmetric heap, shared by the host code and the kernels
// of libsymar (never by the CPU oracle).
//
// heap memory:  [ control block | segment 0 | segment 1 | ... | segment P-1 ]
// segment q  :  [ user region | LL scratch | ready flags | done flags | epochs | pad ]
//
// Every rank segment has the same layout (symmetric objects: same offset + rank
// id addresses a peer's copy), every region starts on a 256-byte boundary.
//
// LL scratch of the RECEIVING rank, indexed [parity][slot c][sender q][half][k]:
//   parity  alternates with the slot's iteration counter (double buffering: a
//           rank may run one iteration ahead of a peer without overwriting
//           scratch the peer still reads);
//   slot c  the CTA slot; only CTA c of each rank ever touches region c, so the
//           flag values seen in a region are that slot's own increasing sequence;
//   half    0 holds {w0,flag,w1,flag} of payload vector k, 1 holds {w2,flag,w3,flag};
//           two planes so that a warp's 16-byte stores are contiguous.
#pragma once
#include <cstddef>
#include <cstdint>

#include "symar.h"

namespace symar {

constexpr int      kMaxRanks    = SYMAR_MAX_RANKS;
constexpr int      kMaxCtas     = SYMAR_MAX_CTAS;
constexpr int      kLLSlots     = SYMAR_LL_SLOTS;
constexpr uint32_t kLLSlotVecs  = SYMAR_LL_SLOT_VECS;
constexpr size_t   kAlign       = SYMAR_ALIGN;
constexpr size_t   kCtlBytes    = 256;              // control block at the heap base
constexpr size_t   kFlagGroup   = 32;               // kMaxRanks x u32: one L2 sector per (rank, slot)
constexpr size_t   kMaxThreads  = 512;

// control block words (u32)
enum : int { kCtlCode = 0, kCtlRank = 1, kCtlPeer = 2, kCtlCta = 3 };

__host__ __device__ constexpr size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
    int      P;
    size_t   user_bytes;     // rounded up
    size_t   ll_off;         // segment offset of the LL scratch
    size_t   ll_bytes;
    size_t   ready_off;      // kMaxCtas groups of kFlagGroup bytes
    size_t   done_off;
    size_t   epoch_off;      // kMaxCtas x u64 iteration counters
    size_t   seg_bytes;      // used bytes of a segment
    size_t   stride;         // segment pitch
    size_t   total;          // control block + P * stride
};

// bytes one sender occupies in one (parity, slot) region: vecs x 2 halves x 16 B
constexpr size_t kLLSenderBytes = (size_t)kLLSlotVecs * 32;

inline Layout make_layout(int P, size_t bytes_per_rank)
{
    Layout L{};
    L.P          = P;
    L.user_bytes = round_up(bytes_per_rank ? bytes_per_rank : 1, kAlign);
    L.ll_off     = L.user_bytes;
    L.ll_bytes   = (size_t)2 * kLLSlots * P * kLLSenderBytes;
    L.ready_off  = L.ll_off + L.ll_bytes;
    L.done_off   = L.ready_off + (size_t)kMaxCtas * kFlagGroup;
    L.epoch_off  = L.done_off + (size_t)kMaxCtas * kFlagGroup;
    L.seg_bytes  = round_up(L.epoch_off + (size_t)kMaxCtas * sizeof(uint64_t), kAlign);
    // Pitch: pad by an odd number of 256-byte units so that equal offsets of
    // different ranks do not all start on the same DRAM channel/bank set.
    L.stride     = L.seg_bytes + 9 * kAlign;
    L.total      = kCtlBytes + (size_t)P * L.stride;
    return L;
}

// What every kernel receives (by value, in the constant bank).
struct KArgs {
    char     *seg0;          // rank 0's segment
    uint64_t  stride;
    uint64_t  in_off;        // byte offsets inside the user region
    uint64_t  out_off;
    uint64_t  count;         // elements per rank
    uint64_t  nvec;          // 16-byte vectors per rank, ceil(count * elem / 16)
    uint64_t  ll_off;
    uint64_t  ready_off;
    uint64_t  done_off;
    uint64_t  epoch_off;
    uint32_t *ctl;           // control block
    uint64_t  spin_ns;       // bound of any wait
    uint32_t  tail_bytes;    // valid bytes of the last vector, 0 = the last vector is full
    uint32_t  cv;            // LL: vectors per CTA per iteration (<= kLLSlotVecs)
    uint32_t  iters;         // LL: iterations
    int32_t   dbg_mute;      // test hook: rank that stays silent, -1 = none
    uint32_t  dbg_seed;
    uint32_t  dbg_delay_ns;
};

}  // namespace symar
