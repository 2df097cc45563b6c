// Work distribution for the persistent attention kernels: one CTA per SM takes (tile, head) items
// from a global counter until none are left.
//
// Item order.  A causal tile's work grows with its position, so items are handed out longest first.
// Keeping one head's items together lets that head's streamed operands stay in L2, but then the last
// head's long tiles start late and set the length of the kernel's tail; sweeping tile positions
// across all heads ("banded") balances the tail but widens the L2 working set.  The order used here
// does both: the first h - banded_heads heads go head by head, the remaining banded_heads heads are
// swept position by position.  The host picks banded_heads so that those heads' operands fit in L2.
#pragma once
#include "sm100_ptx.cuh"

namespace laga {

struct WorkSchedule {
    int n_tiles;          // tiles per head (rank 0 = the longest)
    int h;                // heads
    int banded_heads;     // 1 <= banded_heads <= h
    int total_items;      // n_tiles * h
    unsigned int* counter;   // global, zero when the kernel starts
    const int4* tiles;    // packed sequences: one entry per tile rank (below); nullptr = one sequence of S tokens
};

// Packed variable-length sequences.  The tokens of all sequences are stacked along the row axis; a tile never
// spans two sequences.  The host lists every sequence's tiles, longest work first, as
// (seq_start, seq_len, tile index within the sequence, start of the sequence in the padded statistics arrays);
// rank r of the schedule is entry r.  Rows a tile reads past its sequence's end belong to the next sequence
// (or are TMA zero fill at the very end): the kernels mask them by the sequence length exactly as they mask
// the rows past S for a single sequence.
struct SeqTile {
    int seq_start;   // first row of the sequence in the packed tensors
    int seq_len;
    int tile;        // tile index within the sequence
    int pad_start;   // first entry of the sequence in the per-head statistics arrays (a multiple of 128)
};
__device__ __forceinline__ SeqTile seq_tile(const WorkSchedule& ws, int rank, int S, bool longest_is_last) {
    if (ws.tiles == nullptr) return SeqTile{0, S, longest_is_last ? ws.n_tiles - 1 - rank : rank, 0};
    const int4 t = __ldg(ws.tiles + rank);
    return SeqTile{t.x, t.y, t.z, t.w};
}

// item -> (rank of the tile within its head, longest first; head)
__device__ __forceinline__ void decode_item(const WorkSchedule& ws, int item, int& rank, int& head) {
    const int plain = (ws.h - ws.banded_heads) * ws.n_tiles;
    if (item < plain) {
        head = item / ws.n_tiles;
        rank = item - head * ws.n_tiles;
    } else {
        const int r = item - plain;
        rank = r / ws.banded_heads;
        head = (ws.h - ws.banded_heads) + (r - rank * ws.banded_heads);
    }
}

// The item ring inside a CTA: the producer lane fetches the next item and publishes it; the MMA lane
// and one lane of every consumer warp acknowledge having read it.  Two slots let the producer run
// one item ahead, which is what hides the next item's first loads behind the current item's tail.
struct ItemRing {
    uint64_t* full;     // [2] count 1
    uint64_t* empty;    // [2] count = number of acknowledging lanes
    volatile int* item; // [2]
};

// Producer lane: fetch and publish item number n of this CTA.  Returns the item or -1 (no more work,
// also published so every role leaves its loop).  false in `ok` after a timeout.
__device__ __forceinline__ int ring_publish(const ItemRing& ring, const WorkSchedule& ws, uint32_t n, AbortFlag* abort_flag,
                                            unsigned int* status, bool& ok) {
    const uint32_t slot = n & 1u;
    ok = mbar_wait(&ring.empty[slot], ((n >> 1) & 1u) ^ 1u, abort_flag, status, 0xA0);
    if (!ok) return -1;
    int it = static_cast<int>(atomicAdd(ws.counter, 1u));
    if (it >= ws.total_items) it = -1;
    ring.item[slot] = it;
    mbar_arrive(&ring.full[slot]);
    return it;
}

// Any other lane: read item number n.  Every lane of the calling warp (or the single MMA lane) gets the
// value; `ack` lanes then release the slot.
__device__ __forceinline__ int ring_read(const ItemRing& ring, uint32_t n, bool ack, AbortFlag* abort_flag,
                                         unsigned int* status, bool& ok) {
    const uint32_t slot = n & 1u;
    ok = mbar_wait(&ring.full[slot], (n >> 1) & 1u, abort_flag, status, 0xA1);
    if (!ok) return -1;
    const int it = ring.item[slot];
    if (ack) mbar_arrive(&ring.empty[slot]);
    return it;
}

// SM clock actually delivered during a kernel: CTA 0 stamps the cycle counter and the nanosecond timer
// when it starts and when it ends (a persistent CTA lives as long as the kernel).
struct ClockProbe {
    unsigned long long cycles_begin, ns_begin, cycles_end, ns_end;
};
__device__ __forceinline__ void clock_probe_begin(ClockProbe* p) {
    if (p != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
        p->cycles_begin = static_cast<unsigned long long>(clock64());
        p->ns_begin = global_timer_ns();
    }
}
__device__ __forceinline__ void clock_probe_end(ClockProbe* p) {
    if (p != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
        p->cycles_end = static_cast<unsigned long long>(clock64());
        p->ns_end = global_timer_ns();
    }
}

}  // namespace laga
