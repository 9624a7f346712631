// Host side of the inter-replica ring all-reduce: the membership descriptor the CPU control plane edits and the
// per-member schedule of copy / reduce steps derived from it (Section 6, "Decoupled communication domains"; appendix
// "Decoupled Communication Domain": the CPU keeps the active replica set, recomputes the ring order when a replica
// leaves or joins - a metadata edit - and the data plane derives its peers from that metadata at launch time, so it
// never addresses a dead endpoint).  No GPU code here; libra_ring_all_reduce_local (libra_api.cu) runs a schedule
// over buffers of one device.  C ABI in include/libra.h.
#include <algorithm>
#include <cstdint>

#include "libra.h"

namespace {

int position_of(const libra_ring_t* ring, int32_t id) {
  for (int32_t i = 0; i < ring->n_members; ++i)
    if (ring->members[i] == id) return i;
  return -1;
}

bool valid_ring(const libra_ring_t* ring) {
  return ring && ring->n_members >= 0 && ring->n_members <= LIBRA_RING_MAX_MEMBERS;
}

// Segment c of a vector of n16 16-byte units cut into m equal parts, the first n16 % m one unit longer.
void segment_range(int64_t n16, int32_t m, int32_t c, int64_t* begin, int64_t* end) {
  const int64_t base = n16 / m, extra = n16 % m;
  *begin = base * c + std::min<int64_t>(c, extra);
  *end = *begin + base + (c < extra ? 1 : 0);
}

inline int32_t wrap(int32_t x, int32_t m) { return ((x % m) + m) % m; }

}  // namespace

extern "C" {

int libra_ring_init(libra_ring_t* ring, const int32_t* ids, int32_t n) {
  if (!ring || n < 0 || n > LIBRA_RING_MAX_MEMBERS || (n > 0 && !ids)) return LIBRA_INVALID_ARGUMENT;
  for (int32_t i = 0; i < n; ++i)
    for (int32_t j = 0; j < i; ++j)
      if (ids[i] == ids[j]) return LIBRA_INVALID_ARGUMENT;
  ring->n_members = n;
  ring->epoch = 0;
  for (int32_t i = 0; i < LIBRA_RING_MAX_MEMBERS; ++i) ring->members[i] = (i < n) ? ids[i] : -1;
  return LIBRA_OK;
}

int libra_ring_remove(libra_ring_t* ring, int32_t id) {
  if (!valid_ring(ring)) return LIBRA_INVALID_ARGUMENT;
  const int pos = position_of(ring, id);
  if (pos < 0) return LIBRA_INVALID_ARGUMENT;
  for (int32_t i = pos; i + 1 < ring->n_members; ++i) ring->members[i] = ring->members[i + 1];
  ring->members[--ring->n_members] = -1;
  ++ring->epoch;
  return LIBRA_OK;
}

int libra_ring_insert(libra_ring_t* ring, int32_t id, int32_t position) {
  if (!valid_ring(ring) || ring->n_members >= LIBRA_RING_MAX_MEMBERS) return LIBRA_INVALID_ARGUMENT;
  if (position < 0 || position > ring->n_members || position_of(ring, id) >= 0) return LIBRA_INVALID_ARGUMENT;
  for (int32_t i = ring->n_members; i > position; --i) ring->members[i] = ring->members[i - 1];
  ring->members[position] = id;
  ++ring->n_members;
  ++ring->epoch;
  return LIBRA_OK;
}

int libra_ring_neighbors(const libra_ring_t* ring, int32_t id, int32_t* predecessor, int32_t* successor) {
  if (!valid_ring(ring) || !predecessor || !successor) return LIBRA_INVALID_ARGUMENT;
  const int pos = position_of(ring, id);
  if (pos < 0) return LIBRA_INVALID_ARGUMENT;
  const int32_t m = ring->n_members;
  *predecessor = ring->members[wrap(pos - 1, m)];
  *successor = ring->members[wrap(pos + 1, m)];
  return LIBRA_OK;
}

int libra_ring_schedule(const libra_ring_t* ring, int32_t id, int64_t bytes, int64_t piece_bytes, libra_ring_op_t* ops,
                        int32_t capacity, int32_t* n_ops) {
  if (!valid_ring(ring) || !n_ops || bytes < 0 || bytes % 16 != 0 || piece_bytes < 16 || piece_bytes % 16 != 0 ||
      capacity < 0 || (capacity > 0 && !ops)) {
    return LIBRA_INVALID_ARGUMENT;
  }
  const int pos = position_of(ring, id);
  if (pos < 0) return LIBRA_INVALID_ARGUMENT;
  const int32_t m = ring->n_members;
  const int64_t n16 = bytes / 16;
  const int32_t pred = ring->members[wrap(pos - 1, m)], succ = ring->members[wrap(pos + 1, m)];
  int64_t count = 0;
  auto emit = [&](int32_t kind, int32_t phase, int32_t step, int32_t segment, int32_t peer) {
    int64_t b16, e16;
    segment_range(n16, m, segment, &b16, &e16);
    int32_t piece = 0;
    for (int64_t off = b16 * 16; off < e16 * 16; off += piece_bytes, ++piece) {
      if (count < capacity) {
        libra_ring_op_t& op = ops[count];
        op.kind = kind;
        op.phase = phase;
        op.step = step;
        op.segment = segment;
        op.piece = piece;
        op.peer = peer;
        op.offset = off;
        op.bytes = std::min<int64_t>(piece_bytes, e16 * 16 - off);
      }
      ++count;
    }
  };
  // ReduceScatter: in step s the member at position p sends segment p - s and adds what arrives into segment p - 1 - s;
  // after m - 1 steps it holds the complete sum of segment p + 1.  AllGather: it sends segment p + 1 - s and overwrites
  // segment p - s with what arrives.
  for (int32_t s = 0; s + 1 < m; ++s) {
    emit(LIBRA_RING_OP_SEND, 0, s, wrap(pos - s, m), succ);
    emit(LIBRA_RING_OP_RECV_REDUCE, 0, s, wrap(pos - 1 - s, m), pred);
  }
  for (int32_t s = 0; s + 1 < m; ++s) {
    emit(LIBRA_RING_OP_SEND, 1, s, wrap(pos + 1 - s, m), succ);
    emit(LIBRA_RING_OP_RECV_COPY, 1, s, wrap(pos - s, m), pred);
  }
  *n_ops = int32_t(std::min<int64_t>(count, INT32_MAX));
  return count > capacity ? LIBRA_WORKSPACE_TOO_SMALL : LIBRA_OK;
}

}  // extern "C"
