// Hooks through which the tcgen05 / TMA kernels replace stages of the portable pipeline.
// Each hook returns false when it did not take the stage, in which case the caller emits the
// portable kernels.
#pragma once

namespace {

inline void fast_carve(Bump &, std::vector<CellWork> &, bool) {}
inline void fast_carve_decode(Bump &, std::vector<CellWork> &, bool) {}
inline bool fast_decode_ok(const CellDesc &, const jolt_layout *, bool) { return false; }
inline bool fast_residual(Program &, std::vector<CellWork> &, const std::vector<BackboneRef> &, std::vector<RowJob> &,
                          jolt_handle *, uint64_t, bool) { return false; }
inline bool fast_decode(Program &, std::vector<CellWork> &, const std::vector<BackboneRef> &, std::vector<RowJob> &,
                        const jolt_handle *, const jolt_layout *, bool) { return false; }

}  // namespace
