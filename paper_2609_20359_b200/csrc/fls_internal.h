// Internal declarations shared by the host code and the kernels of libfls.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "fls.h"

namespace fls {

constexpr int kThreads = 256;            // threads per CTA, all kernels
constexpr int kVec = 8;                  // elements per thread per tile
constexpr int kTile = kThreads * kVec;   // 2048 elements per tile
constexpr int kParamSegs = 512;          // segment tables up to this size also travel in the kernel parameters
constexpr int kNormChunkCtas = 256;      // CTA partials of the squared norm are first added up in chunks of this many

// A run of elements that is contiguous in both the unsharded order (index j) and the shard order
// (address a): one rank's slice of one unit, or several merged when they are adjacent in both.
struct Segment {
  uint64_t tile_begin;  // first tile of this segment
  uint64_t tile_end;    // one past its last tile
  uint64_t j0;          // start in the unsharded order (gradients, bf16 copy)
  uint64_t a0;          // start in the shard order (master, m, v, reduced gradient)
  uint64_t len;         // elements
  uint64_t aligned;     // 1 if j0 and a0 are multiples of kVec: 128/256-bit accesses allowed
  // ring-order plans only (their segments are never merged: one rank's slice of one unit each)
  uint64_t shard;       // the rank s that owns this slice after the reduce-scatter
  uint64_t sub_len;     // ceil(M_u / R_rep): length of one sub-chunk of the all-reduce across replicas
};

// Workspace layout (byte offsets); the head is fixed, the segment table and the scratch follow.
constexpr uint64_t kWsStatus = 0;        // uint32 status, uint32 (unused), uint32[2] speculative commits / redos
constexpr uint64_t kWsNorms = 256;       // float[64]
constexpr uint64_t kWsCoefs = 512;       // float[64]
constexpr uint64_t kWsNormSq = 768;      // double[64]
constexpr uint64_t kWsTickets = 1280;    // uint32[64]: one ticket counter per group
constexpr uint64_t kWsReady = 1536;      // uint32[64]: resident step, id of the last launch whose coefficient is published
constexpr uint64_t kWsSegments = 1792;   // Segment[n_segments], then per group the norm tree (double[n_tiles] CTA partials,
                                         // chunk sums, chunk arrival counters), then the reduced-gradient scratch

struct Layout {
  std::vector<uint64_t> unit_numel, unit_offset, unit_shard_numel, unit_shard_offset;
  std::vector<Segment> segments;
  uint64_t n_params = 0, n_padded = 0, shard_numel = 0, n_tiles = 0;
  uint64_t ws_partials_offset = 0, ws_chunk_partials_offset = 0, ws_chunk_count_offset = 0, ws_chunk_count_bytes = 0;
  uint64_t n_chunks = 0;                   // chunks of CTA partials per group; every group has its own tree arrays
  uint64_t ws_scratch_offset = 0, workspace_bytes = 0;
  bool vector_path = true;
  uint32_t scratch_slots = 1;              // reduced-gradient buffers in the workspace, each 4*n_padded bytes (256-byte aligned)
  uint64_t scratch_stride = 0;             // bytes between two of them
};

// Host planner: fills `out` from the unit table; returns an error message or "" on success.
// scratch_slots: how many reduced-gradient buffers the workspace holds (1, or G for the fused aggregation).
// ring_replicas: 0 for the ascending reduction order; R_rep for the ring order, whose segments stay unmerged and
// carry the owning rank and the all-reduce sub-chunk length.
// groups: G (every group gets its own norm-tree arrays, so that the groups' kernels may run in one grid).
std::string build_layout(const std::vector<uint64_t>& unit_numel, uint32_t S, uint32_t Q, uint32_t scratch_slots,
                         uint32_t ring_replicas, uint32_t groups, Layout* out);

// Sets the calling thread's message returned by fls_last_error() (defined beside it).
void set_last_error(const char* msg);

// route: how fls_sync_step currently runs (0 store-and-reread, 1 recompute, 2 single pass), for the HBM byte count
void comm_report(const Layout& lay, const fls_plan_desc& d, int route, const double* bw, fls_comm_costs* out);

}  // namespace fls
