// Seeded exclusive scans (the flag ACC_FLAG_SCAN_EXCLUSIVE): alone, fed by a fused map, from
// the right, and per row of a rank-2 array.
#include "../device/launch.cuh"

namespace acc {

constexpr PNode exclusive(PNode p) { return fixed(p, 1, kRunTime); }

constexpr CProgram make_exclusive_scans() {
  CProgram p{5, (1ull << 3) | (1ull << 4), {}};
  p.nodes[0] = pnode(ACC_INPUT, ACC_I32, 1, 0, 0, 0);
  p.nodes[1] = pnode(ACC_INPUT, ACC_F32, 1, 0, 0, 0);
  p.nodes[2] = pnode(ACC_MAP, ACC_I32, 1, ACC_FN_AND_MASK, 0, 1, 0);                  // counts
  p.nodes[3] = exclusive(pnode(ACC_SCANL, ACC_I32, 1, ACC_FN_ADD, 0, 1, 2));          // offsets
  p.nodes[4] = exclusive(pnode(ACC_SCANR, ACC_F32, 1, ACC_FN_ADD, 0, 1, 1));          // after
  return p;
}
inline constexpr CProgram k_exclusive_scans = make_exclusive_scans();
ACC_CLUSTER(k_exclusive_scans, 0x8, exclusive_scans__offsets)
ACC_CLUSTER(k_exclusive_scans, 0xC, exclusive_scans__counts_offsets)
ACC_CLUSTER(k_exclusive_scans, 0x10, exclusive_scans__after)

constexpr CProgram make_exclusive_row_scans() {
  CProgram p{2, (1ull << 1), {}};
  p.nodes[0] = pnode(ACC_INPUT, ACC_F32, 2, 0, 0, 0);
  p.nodes[1] = exclusive(pnode(ACC_SCANL, ACC_F32, 2, ACC_FN_MAX, 0, 1, 0));          // best_before
  return p;
}
inline constexpr CProgram k_exclusive_row_scans = make_exclusive_row_scans();
ACC_CLUSTER(k_exclusive_row_scans, 0x2, exclusive_row_scans__best_before)

}  // namespace acc
