// Bookkeeping of the weight ring of the persistent pass kernel, in plain C++ so that a host program can
// exercise it (tests/test_ring_model.py compiles this header with g++ and checks, over sequences of stage
// sizes, that a stage is never written while an older stage that shares its bytes or its barrier pair may
// still be unread).
//
// The ring is kRingBytes of shared memory.  Stage j of the static schedule takes exactly the bytes of its
// boxes (a multiple of 1 KB), at the head of the ring, or at offset 0 if it would run past the end, and uses
// barrier pair j % kSlots in its (j / kSlots)-th phase.  The walk depends on the schedule only, so producers
// and issuer compute the same offsets without talking to each other.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define ADA_HD __host__ __device__ __forceinline__
#else
#define ADA_HD inline
#endif

namespace ada {

constexpr int kRingBytes = 128 * 1024;           // weight ring; stages take exactly the bytes of their boxes
constexpr int kFlight = 16;                      // most stages in flight
constexpr int kSlots = 32;                       // barrier pairs of the ring: twice kFlight, so that a pair is not
                                                 // reused before both producers have passed its previous use

struct RingCursor {
  uint32_t head;
  unsigned n;     // stages taken so far
  ADA_HD bool wraps(uint32_t bytes) const { return head + bytes > (uint32_t)kRingBytes; }
  ADA_HD uint32_t take(uint32_t bytes) {
    if (head + bytes > (uint32_t)kRingBytes) head = 0;
    const uint32_t off = head;
    head += bytes;
    ++n;
    return off;
  }
};

// What a producer keeps about the stages in flight.  Stages are read (and so released) in order, because one
// thread issues all products; `retire` is called for EVERY stage of the schedule, in order, by every producer,
// whether the stage is its own or not, and returns in `pending` the newest stage that must have been read
// before the stages placed so far may be written (kNone: none).  A producer waits for `pending` only before
// a stage of its own and then clears it.
//
// st_off / st_end: records of the last kFlight stages (caller's storage, e.g. shared memory).
struct RingRetire {
  static constexpr unsigned kNone = 0xffffffffu;
  RingCursor cur;
  unsigned tail;       // oldest stage the ring may still hold unread
  unsigned lap0;       // first stage of the current lap around the ring
  unsigned pending;    // newest retired stage not yet waited for
  uint32_t t_off, t_end;   // record of stage `tail`, read ahead of its use

  ADA_HD void init() { cur.head = 0; cur.n = 0; tail = 0; lap0 = 0; pending = kNone; t_off = t_end = 0; }

  // places stage j = cur.n of `bytes` bytes; returns its offset
  ADA_HD uint32_t place(uint32_t bytes, uint32_t *st_off, uint32_t *st_end) {
    const bool wraps = cur.wraps(bytes);
    const uint32_t off = cur.take(bytes);
    const unsigned j = cur.n - 1;
    if (wraps) {
      // A stage that starts a new lap retires everything older than the previous lap's first stage: stages
      // left near the end of the ring overlap nothing new and would otherwise stay "oldest" for ever, hiding
      // the younger stages at the start of the ring that the new lap does run into.
      if (tail < lap0) {
        pending = lap0 - 1;
        tail = lap0;
        t_off = st_off[tail % kFlight];
        t_end = st_end[tail % kFlight];
      }
      lap0 = j;
    }
    st_off[j % kFlight] = off;
    st_end[j % kFlight] = off + bytes;
    if (tail == j) { t_off = off; t_end = off + bytes; }
    // With at most one wrap among the stages in flight, the oldest ones are the first a new stage can run
    // into: retire them until a barrier pair is free and no unread stage overlaps the new one.
    while (tail < j && (j - tail >= (unsigned)kFlight || (t_off < off + bytes && off < t_end))) {
      pending = tail;
      ++tail;
      t_off = st_off[tail % kFlight];
      t_end = st_end[tail % kFlight];
    }
    return off;
  }
};

}  // namespace ada
