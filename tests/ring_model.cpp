// Host model of the weight ring of the pass kernel: drives RingRetire (csrc/ada_ring.h, the code the kernel's
// producers run) over a sequence of stage sizes and checks the property the kernel relies on: when a producer
// is about to write one of its stages, every older stage that shares bytes or the barrier pair with it is
// covered by a wait the producer has made (stages are read in order, so waiting for stage w covers all <= w).
// usage: ring_model size:count[,size:count...] repeats   -> prints "ok" or the first violations; exit code 1 on error
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>
#include "ada_ring.h"
using namespace ada;

int main(int argc, char **argv) {
  if (argc < 3) return 2;
  std::vector<uint32_t> pat;
  for (char *tok = strtok(argv[1], ","); tok; tok = strtok(nullptr, ",")) {
    unsigned sz = 0, cnt = 0;
    if (sscanf(tok, "%u:%u", &sz, &cnt) != 2 || sz == 0 || sz % 1024 || sz > 32768) return 2;
    for (unsigned i = 0; i < cnt; ++i) pat.push_back(sz);
  }
  const int repeats = atoi(argv[2]);
  std::vector<uint32_t> sizes;
  for (int r = 0; r < repeats; ++r) sizes.insert(sizes.end(), pat.begin(), pat.end());
  std::vector<uint32_t> offs(sizes.size()), ends(sizes.size());
  {
    RingCursor c{0, 0};
    for (size_t j = 0; j < sizes.size(); ++j) { offs[j] = c.take(sizes[j]); ends[j] = offs[j] + sizes[j]; }
  }
  int bad = 0;
  for (unsigned pidx = 0; pidx < 2; ++pidx) {
    RingRetire rr;
    rr.init();
    uint32_t st_off[kFlight], st_end[kFlight];
    long waited = -1;   // newest stage this producer has waited for
    for (size_t jj = 0; jj < sizes.size(); ++jj) {
      const uint32_t off = rr.place(sizes[jj], st_off, st_end);
      const unsigned j = rr.cur.n - 1;
      if (off != offs[j] || off + sizes[jj] > (uint32_t)kRingBytes) { printf("stage %u: offset %u\n", j, off); ++bad; }
      if ((j & 1u) != pidx) continue;
      if (rr.pending != RingRetire::kNone) {
        if ((long)rr.pending >= (long)j) { printf("stage %u waits for itself or later (%u)\n", j, rr.pending); ++bad; }
        if ((long)rr.pending > waited) waited = rr.pending;
        rr.pending = RingRetire::kNone;
      }
      for (long i = (long)j - 1; i >= 0 && i > (long)j - 4 * kSlots; --i) {
        const bool ov = offs[i] < off + sizes[jj] && off < ends[i];
        const bool pair = (i % kSlots) == (long)(j % kSlots);
        const bool rec = (i % kFlight) == (long)(j % kFlight);   // the record slot is reused as well
        if ((ov || pair || rec) && i > waited) {
          if (bad < 10) printf("producer %u stage %u: older stage %ld not covered (bytes %d pair %d record %d, waited %ld)\n", pidx, j, i, ov, pair, rec, waited);
          ++bad;
        }
      }
    }
  }
  if (bad) { printf("%d violations\n", bad); return 1; }
  printf("ok %zu stages\n", sizes.size());
  return 0;
}
