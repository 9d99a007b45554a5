// Flat-buffer layout planner (host, integers only).
//
// The paper splits every layer equally over the S ranks of a sharding group in shards of size M and
// requires all federation groups to use the same sharding policy.  Here a unit u of n_u elements gets
// M_u = roundup(ceil(n_u / S), Q) elements per rank and is zero-padded to S * M_u.  Gradients and the
// bf16 copy keep the unsharded order (units back to back); master, m and v use the rank-major shard
// order: rank s holds its slice of every unit, one after the other.
#include "fls_internal.h"

namespace fls {

std::string build_layout(const std::vector<uint64_t>& unit_numel, uint32_t S, uint32_t Q, uint32_t scratch_slots,
                         uint32_t ring_replicas, uint32_t groups, Layout* out) {
  if (unit_numel.empty()) return "empty unit table";
  if (S == 0 || Q == 0) return "shard_dim and align_elems must be >= 1";
  Layout& L = *out;
  L = Layout();
  L.unit_numel = unit_numel;
  const size_t n_units = unit_numel.size();
  uint64_t off = 0, soff = 0, total = 0;
  for (size_t u = 0; u < n_units; ++u) {
    const uint64_t n = unit_numel[u];
    if (n == 0) return "unit with zero elements";
    if (n > (1ull << 46)) return "unit too large";
    const uint64_t per_rank = (n + S - 1) / S;
    const uint64_t m = (per_rank + Q - 1) / Q * Q;
    L.unit_offset.push_back(off);
    L.unit_shard_numel.push_back(m);
    L.unit_shard_offset.push_back(soff);
    off += m * S;
    soff += m;
    total += n;
    if (off > (1ull << 47)) return "plan too large";
  }
  L.n_params = total;
  L.n_padded = off;
  L.shard_numel = soff;

  // Segments in shard-address order: for each rank, for each unit.  Neighbours that are adjacent in
  // both orders are merged (a single unit collapses to one segment covering the whole buffer), except for
  // ring-order plans, whose kernels need to know the rank and the position inside the rank's slice.
  for (uint32_t s = 0; s < S; ++s) {
    for (size_t u = 0; u < n_units; ++u) {
      Segment g{};
      g.j0 = L.unit_offset[u] + uint64_t(s) * L.unit_shard_numel[u];
      g.a0 = uint64_t(s) * L.shard_numel + L.unit_shard_offset[u];
      g.len = L.unit_shard_numel[u];
      g.shard = s;
      g.sub_len = ring_replicas ? (g.len + ring_replicas - 1) / ring_replicas : g.len;
      if (!L.segments.empty() && !ring_replicas) {
        Segment& p = L.segments.back();
        if (p.j0 + p.len == g.j0 && p.a0 + p.len == g.a0) {
          p.len += g.len;
          continue;
        }
      }
      L.segments.push_back(g);
    }
  }
  uint64_t tile = 0;
  for (Segment& g : L.segments) {
    g.aligned = (g.j0 % kVec == 0 && g.a0 % kVec == 0) ? 1 : 0;
    if (!g.aligned) L.vector_path = false;
    g.tile_begin = tile;
    tile += (g.len + kTile - 1) / kTile;
    g.tile_end = tile;
  }
  // an aligned segment whose length is not a multiple of kVec still takes the vector path except for
  // its last few elements; report the plan as "vector" only if nothing at all falls off it
  for (const Segment& g : L.segments)
    if (g.len % kVec != 0) L.vector_path = false;
  L.n_tiles = tile;
  const uint64_t seg_bytes = L.segments.size() * sizeof(Segment);
  if (L.n_tiles >= (1ull << 32)) return "plan too large";
  L.ws_partials_offset = (kWsSegments + seg_bytes + 255) / 256 * 256;
  // norm tree: at most one partial per tile, then one sum and one arrival counter per chunk of kNormChunkCtas partials
  // (per group: group g's arrays start g * n_tiles, g * n_chunks entries in)
  const uint64_t n_chunks = (L.n_tiles + kNormChunkCtas - 1) / kNormChunkCtas;
  const uint64_t G = groups ? groups : 1;
  L.n_chunks = n_chunks;
  L.ws_chunk_partials_offset = (L.ws_partials_offset + 8 * L.n_tiles * G + 255) / 256 * 256;
  L.ws_chunk_count_offset = (L.ws_chunk_partials_offset + 8 * n_chunks * G + 255) / 256 * 256;
  L.ws_chunk_count_bytes = 4 * n_chunks * G;
  L.ws_scratch_offset = (L.ws_chunk_count_offset + L.ws_chunk_count_bytes + 255) / 256 * 256;
  L.scratch_slots = scratch_slots ? scratch_slots : 1;
  L.scratch_stride = (4ull * L.n_padded + 255) / 256 * 256;
  L.workspace_bytes = L.ws_scratch_offset + L.scratch_stride * L.scratch_slots;
  return "";
}

}  // namespace fls
