// Host-side launcher of a cluster instantiation: picks the skeleton from the cluster's
// roots, the vector width from the shapes, sizes the grid to the machine and the scratch
// region to the grid.
#pragma once
#include <algorithm>

#include "../graph.h"
#include "../registry.h"
#include "hist.cuh"
#include "segfold.cuh"
#include "skeletons.cuh"
#include "slabgather.cuh"
#include "stencil.cuh"
#include "tile.cuh"

namespace acc {

// Opt-in to `smem` bytes of dynamic shared memory for a kernel, asked of the driver once per device
// and size: `granted` (one per kernel, 64 zeroed words) remembers the largest size already granted.
template <class K>
inline bool opt_in_shared_memory(K kern, size_t smem, int* granted) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) {
    cudaGetLastError();
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess;
  }
  if (granted[device] >= (int)smem + 1) return true;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
  granted[device] = (int)smem + 1;
  return true;
}

// Blocks of `kern` (no dynamic shared memory) that are resident at once on the current device, 0 if the device
// cannot launch a grid cooperatively; asked of the driver once per kernel and device (`fit_on`: 64 zeroed words).
inline int resident_grid(const void* kern, int block, int* fit_on) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) { cudaGetLastError(); return 0; }
  if (fit_on[device] == 0) {
    int fit = 0;
    if (!cooperative_launch_ok() || cudaOccupancyMaxActiveBlocksPerMultiprocessor(&fit, kern, block, 0) != cudaSuccess) {
      cudaGetLastError();
      fit = 0;
    }
    fit_on[device] = fit + 1;
  }
  return (fit_on[device] - 1) * sm_count();
}

template <class CL>
struct Launcher {
  static constexpr int N = CL::c.n;
  static constexpr bool kHasScan = dev::count_if<CL>(dev::is_scan_root) > 0;
  static constexpr bool kHasRowFold = dev::count_if<CL>(dev::is_row_fold) > 0;
  static constexpr int kScalarFolds = dev::count_if<CL>(dev::is_scalar_fold);
  static constexpr int kScanBlock = dev::scan_block<CL>();
  static constexpr int kScanTile = kScanBlock * dev::scan_rows<CL>() * 4;
  static constexpr bool kHasSegFold = dev::count_if<CL>(dev::is_segfold_root) > 0;
  // exactly one scatter, fp32 '+': its bins can live in shared memory (k_hist)
  static constexpr bool kHistShape = !kHasScan && !kHasRowFold && dev::count_if<CL>(dev::is_permute_root) == 1 &&
                                     dev::count_if<CL>(dev::is_f32_add_permute) == 1;

  // Local id of the array whose index space root `i` iterates over, -1 if i is no root.
  static int domain_of(int i) {
    const CNode& n = CL::c.nodes[i];
    if (dev::is_store_root(n) || dev::is_scan_root(n) || dev::is_segfold_root(n)) return i;
    if (dev::is_fold_root(n)) return n.in[0];
    if (dev::is_permute_root(n)) return n.in[1];
    return -1;
  }

  // Iteration domain: shape of the first root's index space.
  static bool domain(const ClusterLaunch& L, int& R, int& C) {
    for (int i = 0; i < N; ++i) {
      const int at = domain_of(i);
      if (at >= 0) { R = L.nodes[at].R; C = L.nodes[at].C; return true; }
    }
    return false;
  }

  // Every root must iterate over the same domain (a legal cluster has one iteration size).
  static bool domains_agree(const ClusterLaunch& L, int R, int C) {
    for (int i = 0; i < N; ++i) {
      const int at = domain_of(i);
      if (at >= 0 && (L.nodes[at].R != R || L.nodes[at].C != C)) return false;
    }
    return true;
  }

  // 128-bit accesses need every array's innermost extent and base address to allow them.
  static bool vec_ok(const ClusterLaunch& L, int C) {
    if (C % 4) return false;
    for (int i = 0; i < N; ++i) {
      const CNode& n = CL::c.nodes[i];
      if (!n.member) {
        bool as_array = false;                         // free variables are scalar reads
        for (int j = 0; j < N; ++j)
          for (int s = 0; s < CL::c.nodes[j].narr; ++s)
            if (CL::c.nodes[j].member && CL::c.nodes[j].in[s] == i) as_array = true;
        if (!as_array) continue;
      } else if (!dev::is_store_root(n) && !dev::is_scan_root(n)) {
        continue;                                      // never written with a vector store
      }
      if (L.nodes[i].C % 4 || (reinterpret_cast<uintptr_t>(L.nodes[i].ptr) & 15)) return false;
    }
    return true;
  }

  static int stream_grid(int R, int C, bool vec) {
    const int64_t per_row = C / (vec ? 4 : 1);
    const int64_t trips = dev::domain_rank<CL>() <= 1
                              ? (per_row + dev::kBlock - 1) / dev::kBlock
                              : ((per_row + 31) / 32) * ((R + dev::kStreamTileRows - 1) / dev::kStreamTileRows);
    return (int)std::max<int64_t>(1, std::min<int64_t>(trips, (int64_t)sm_count() * 8));
  }

  // transposes staged through shared-memory tile pairs (k_tile_pair)
  static constexpr bool kTileShape = dev::tile_eligible<CL>();
  static constexpr int kRowFolds = dev::count_if<CL>(dev::is_row_fold);

  // The tile-pair kernel wants a square domain of at least one tile, and every staged
  // external of that same shape.
  static bool use_tiles(const ClusterLaunch& L, int R, int C) {
    if constexpr (kTileShape) {
      if (R != C || R < dev::kTile) return false;
      for (int i = 0; i < N; ++i)
        if (dev::is_staged_external<CL>(i) && (L.nodes[i].R != R || L.nodes[i].C != C)) return false;
      return true;
    } else {
      return false;
    }
  }

  // blocks of k_segfold: one per run of kSegTilesPerBlock tiles of the folds' source (its records are laid out for them)
  static int seg_grid(const ClusterLaunch& L) {
    if constexpr (kHasSegFold) {
      const int src = CL::c.nodes[dev::first_segfold<CL>()].in[0];
      const int64_t n_src = (int64_t)L.nodes[src].R * L.nodes[src].C;
      const int64_t tiles = std::max<int64_t>(1, (n_src + dev::kSegTile - 1) / dev::kSegTile);
      return (int)((tiles + dev::kSegTilesPerBlock - 1) / dev::kSegTilesPerBlock);
    } else {
      return 0;
    }
  }

  // 128-bit reads of a segmented fold's operands: every array read as an array has 16-byte rows and base
  static bool seg_vec_ok(const ClusterLaunch& L) {
    for (int i = 0; i < N; ++i) {
      if (CL::c.nodes[i].member) continue;
      bool as_array = false;
      for (int j = 0; j < N; ++j)
        for (int s = 0; s < CL::c.nodes[j].narr; ++s)
          if (CL::c.nodes[j].member && CL::c.nodes[j].in[s] == i) as_array = true;
      if (as_array && (L.nodes[i].C % 4 || (reinterpret_cast<uintptr_t>(L.nodes[i].ptr) & 15))) return false;
    }
    return true;
  }

  // Whether the gather below the scan runs as slab passes: decided by shapes alone, so that the scratch
  // layout (which is fixed before any pointer is known) and the launch agree.
  static constexpr bool kSlabShape = dev::slab_gather_eligible<CL>();
  static bool slab_shapes_ok(const ClusterLaunch& L, int R, int C) {
    if constexpr (kSlabShape) {
      const int src = CL::c.nodes[dev::the_gather<CL>()].in[1];
      const int64_t src_bytes = (int64_t)L.nodes[src].R * L.nodes[src].C * 4;
      return R == 1 && C >= dev::kSlabMinElements && C % 4 == 0 && src_bytes >= dev::kSlabMinSourceBytes && src_bytes <= dev::kSlabMaxSourceBytes;
    } else {
      return false;
    }
  }

  // The same for a cluster of element-wise roots only (k_stream_merge): every root a rank-1 array of the domain's length.
  static constexpr bool kStreamSlabShape = dev::slab_stream_eligible<CL>();
  static bool stream_slab_shapes_ok(const ClusterLaunch& L, int R, int C) {
    if constexpr (kStreamSlabShape) {
      const int src = CL::c.nodes[dev::the_gather<CL>()].in[1];
      const int64_t src_bytes = (int64_t)L.nodes[src].R * L.nodes[src].C * 4;
      for (int i = 0; i < N; ++i)
        if (dev::is_store_root(CL::c.nodes[i]) && (L.nodes[i].R != 1 || L.nodes[i].C != C)) return false;
      return R == 1 && C >= dev::kSlabMinElements && C % 4 == 0 && src_bytes >= dev::kSlabMinSourceBytes && src_bytes <= dev::kSlabMaxSourceBytes;
    } else {
      return false;
    }
  }
  // bytes of the group sizes and slab codes of the slab passes, which lie behind `base` bytes of other scratch
  static int64_t with_slab_area(int64_t base, int C) {
    const int64_t full = C / dev::kSlabWarpTile;
    return ((base + 15) & ~int64_t(15)) + full * 4 + full * 32 * 4;
  }

  static int64_t scratch_bytes(const ClusterLaunch& L) {
    int R, C;
    if (!domain(L, R, C)) return ACC_ERR_NO_KERNEL;
    if (use_tiles(L, R, C)) {
      const int blocks = (R + dev::kTile - 1) / dev::kTile;
      return (dev::tile_partials_off(blocks) + (int64_t)kRowFolds * blocks * R) * 4;
    }
    if (kHasScan) {
      int64_t bytes = 16 + (int64_t)R * ((C + kScanTile - 1) / kScanTile) * 8;
      if (slab_shapes_ok(L, R, C)) {                      // + group sizes and slab codes of the slab passes (slabgather.cuh)
        const int64_t full = C / dev::kSlabWarpTile;
        bytes = ((bytes + 15) & ~int64_t(15)) + full * 4 + full * 32 * 4;
      }
      return bytes;
    }
    if (kHasSegFold) return dev::seg_scratch_words(dev::count_if<CL>(dev::is_segfold_root), seg_grid(L)) * 4;
    if (kHasRowFold) return 0;
    int64_t words = dev::stream_acc64_off(kScalarFolds, sm_count() * 8);
    for (int i = 0; i < N; ++i)
      if (dev::is_f32_add_permute(CL::c.nodes[i])) words += 2 * (int64_t)L.nodes[i].R * L.nodes[i].C;
    dev::HistPlan plan;
    if (use_hist(L, R, C, plan)) words += (int64_t)sm_count() * plan.overflow;   // private overflow bins per CTA
    if (stream_slab_shapes_ok(L, R, C)) return with_slab_area(words * 4, C);
    return words * 4;
  }

  // Counters, tickets, tile states and accumulators start from zero; what a kernel writes before it reads
  // (partial sums per tile, the codes and group sizes of the slab passes) need not be cleared, and lies last.
  static int64_t zeroed_bytes(const ClusterLaunch& L) {
    int R, C;
    if (!domain(L, R, C)) return 0;
    if (use_tiles(L, R, C)) return dev::tile_partials_off((R + dev::kTile - 1) / dev::kTile) * 4;
    if (kHasScan && slab_shapes_ok(L, R, C)) return ((16 + (int64_t)R * ((C + kScanTile - 1) / kScanTile) * 8) + 15) & ~int64_t(15);
    if (stream_slab_shapes_ok(L, R, C)) return (((int64_t)dev::stream_acc64_off(kScalarFolds, sm_count() * 8) * 4) + 15) & ~int64_t(15);
    return scratch_bytes(L);
  }

  static void fill(const ClusterLaunch& L, dev::Args<N>& a, int R, int C) {
    for (int i = 0; i < N; ++i) a.n[i] = L.nodes[i];
    a.R = R;
    a.C = C;
    a.scratch = L.scratch;
    a.status = L.status;
    a.spin_limit = L.spin_limit;
    a.grid = sm_count() * 8;             // the partials' layout is sized for the largest grid
  }

  static int launch_hist(const ClusterLaunch& L, dev::Args<N>& a, int R, int C, bool vec);

  // clamped shifts served from halo tiles copied by cp.async.bulk.tensor (k_stencil)
  static constexpr bool kStencilShape = dev::stencil_eligible<CL>();

  // Returns ACC_OK after a launch, an error, or 1 when k_stream should run instead: no
  // 128-bit rows, an external of another shape, a shift by more than one, or a domain too
  // small to fill the machine with tiles.
  static int launch_stencil(const ClusterLaunch& L, dev::Args<N>& a, int R, int C, bool vec) {
    if constexpr (kStencilShape) {
      if (!vec || R < 1 || (int64_t)R * C < (int64_t)dev::kStRows * dev::kStCols * 64) return 1;
      constexpr int depth = dev::max_shift_depth<CL>();
      dev::StencilMaps maps;
      for (int i = 0; i < N; ++i) {
        const CNode& n = CL::c.nodes[i];
        if (n.member && n.kind == ACC_BACKPERMUTE && n.idxfn == ACC_IDX_SHIFT_CLAMP &&
            (L.nodes[i].ip0 < -1 || L.nodes[i].ip0 > 1 || L.nodes[i].ip1 < -1 || L.nodes[i].ip1 > 1))
          return 1;
        if (dev::is_staged_external<CL>(i)) {
          if (L.nodes[i].R != R || L.nodes[i].C != C) return 1;
          if (!make_tensor_map_2d(&maps.m[dev::tile_slot<CL>(i)], L.nodes[i].ptr, R, C, dev::st_box_rows(depth), dev::kStBoxCols)) return 1;
        }
      }
      auto kern = dev::k_stencil<CL>;
      // two stages of every external's box, one box per member kept on chip
      const size_t smem = (size_t)(dev::kStStages * dev::staged_externals<CL>() + dev::staged_members<CL>()) * dev::st_box_stride(depth) * 4;
      static int granted[64];
      if (!opt_in_shared_memory(kern, smem, granted))
        return set_error(ACC_ERR_CUDA, "shared-memory opt-in failed: %s", cudaGetErrorString(cudaGetLastError()));
      const int64_t tiles = (int64_t)((C + dev::kStCols - 1) / dev::kStCols) * ((R + dev::kStRows - 1) / dev::kStRows);
      const int per_sm = std::max(1, std::min(3, (int)((size_t)220 * 1024 / (smem + 1024))));
      const int grid = (int)std::min<int64_t>(tiles, (int64_t)sm_count() * per_sm);
      kern<<<grid, dev::kBlock, smem, L.stream>>>(a, maps);
      const cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
      return ACC_OK;
    } else {
      return 1;
    }
  }

  // Tile pairs staged by tensor copies (k_tile_pair_tma): clusters whose roots are row folds, rows
  // 16-byte friendly.
  // Returns ACC_OK after a launch, an error, or 1 when k_tile_pair should run instead.
  static int launch_tiles_tma(const ClusterLaunch& L, dev::Args<N>& a, int n, bool vec) {
    if constexpr (dev::tile_tma_eligible<CL>()) {
      if (!vec || !cooperative_launch_ok()) return 1;
      dev::TileMaps maps;
      for (int i = 0; i < N; ++i)
        if (dev::is_staged_external<CL>(i) &&
            !make_tensor_map_2d(&maps.m[dev::tile_slot<CL>(i)], L.nodes[i].ptr, n, n, dev::kTile, dev::kTile))
          return 1;
      auto kern = dev::k_tile_pair_tma<CL>;
      constexpr int E = dev::staged_externals<CL>();
      const size_t smem = (size_t)dev::tp_stages<E>() * E * dev::kTpSlotWords * 4 + 128;   // + room to align the copies
      static int fit_on[64];                               // blocks of this kernel per SM, + 1, by device (asked once each)
      int device = 0;
      if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) { cudaGetLastError(); return 1; }
      int per_sm = fit_on[device] - 1;
      if (per_sm < 0) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
          return set_error(ACC_ERR_CUDA, "shared-memory opt-in failed: %s", cudaGetErrorString(cudaGetLastError()));
        int fit = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&fit, kern, dev::kTpThreads, smem) != cudaSuccess) {
          cudaGetLastError();
          fit = 0;
        }
        per_sm = fit;
        fit_on[device] = fit + 1;
      }
      if (per_sm < 1) return 1;
      const int64_t blocks = (n + dev::kTile - 1) / dev::kTile;
      const int64_t pairs = blocks * (blocks + 1) / 2;
      const int grid = (int)std::min<int64_t>(pairs, (int64_t)sm_count() * per_sm);
      void* params[] = {&a, &maps};                        // all blocks resident: they meet at a counter after their walk
      cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kern), dim3(grid), dim3(dev::kTpThreads), params, smem, L.stream);
      const cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
      return ACC_OK;
    } else {
      return 1;
    }
  }

  // Whether the scatter's bins go on chip: they must fit (see hist_plan) and there must be
  // enough elements per bin to repay clearing and flushing them.
  static bool use_hist(const ClusterLaunch& L, int R, int C, dev::HistPlan& plan) {
    if constexpr (kHistShape) {
      constexpr int P = dev::the_f32_add_permute<CL>();
      const int64_t bins = (int64_t)L.nodes[P].R * L.nodes[P].C;
      if (bins <= 0 || (int64_t)R * C < 8 * bins) return false;
      return dev::hist_plan(bins, sm_count(), plan);
    } else {
      return false;
    }
  }

  static int launch(const ClusterLaunch& L) {
    int R, C;
    if (!domain(L, R, C)) return set_error(ACC_ERR_NO_KERNEL, "cluster without a root");
    if (!domains_agree(L, R, C)) return set_error(ACC_ERR_SHAPE, "members of one cluster iterate over different sizes");
    const bool vec = vec_ok(L, C);
    // scatters on integers work in place on a copy of the defaults
    for (int i = 0; i < N; ++i) {
      const CNode& n = CL::c.nodes[i];
      if (dev::is_permute_root(n) && !dev::is_f32_add_permute(n)) {
        const size_t bytes = (size_t)L.nodes[i].R * L.nodes[i].C * 4;
        if (bytes && cudaMemcpyAsync(const_cast<void*>(L.nodes[i].ptr), L.nodes[n.in[0]].ptr, bytes,
                                     cudaMemcpyDeviceToDevice, L.stream) != cudaSuccess)
          return set_error(ACC_ERR_CUDA, "copy of scatter defaults failed: %s", cudaGetErrorString(cudaGetLastError()));
      }
    }
    dev::Args<N> a;
    fill(L, a, R, C);
    if constexpr (dev::rowfold_then_eligible<CL>()) {
      // row folds consumed by element-wise members: the block walks the folds' source rows
      int src = -1;
      for (int i = 0; i < N && src < 0; ++i)
        if (dev::is_inner_row_fold(CL::c.nodes[i])) src = CL::c.nodes[i].in[0];
      bool same = true;                                  // every fold reduces an array of one shape
      for (int i = 0; i < N; ++i)
        if (dev::is_inner_row_fold(CL::c.nodes[i]))
          same = same && L.nodes[CL::c.nodes[i].in[0]].R == L.nodes[src].R && L.nodes[CL::c.nodes[i].in[0]].C == L.nodes[src].C;
      if (same && L.nodes[src].C >= 64) {                // short rows are as well off pulled through
        a.R = L.nodes[src].R;
        a.C = L.nodes[src].C;
        if (a.R == 0) return ACC_OK;
        const int grid = std::min(a.R, sm_count() * 16);
        const bool v4 = vec_ok(L, a.C);
        if (v4) dev::k_rowfold_then<CL, true><<<grid, dev::kBlock, 0, L.stream>>>(a);
        else dev::k_rowfold_then<CL, false><<<grid, dev::kBlock, 0, L.stream>>>(a);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
        return ACC_OK;
      }
    }
    if (use_tiles(L, R, C)) {
      if constexpr (kTileShape) {
        const int rc = launch_tiles_tma(L, a, R, vec);
        if (rc != 1) return rc;                          // 1 = no tensor copies here: the threads stage the tiles
        auto kern = vec ? dev::k_tile_pair<CL, true> : dev::k_tile_pair<CL, false>;
        const size_t smem = (size_t)dev::staged_externals<CL>() * 2 * dev::kTileWords * 4;
        static int granted[2][64];
        if (!opt_in_shared_memory(kern, smem, granted[vec ? 1 : 0]))
          return set_error(ACC_ERR_CUDA, "shared-memory opt-in failed: %s", cudaGetErrorString(cudaGetLastError()));
        const int blocks = (R + dev::kTile - 1) / dev::kTile;
        kern<<<blocks * (blocks + 1) / 2, dev::kBlock, smem, L.stream>>>(a);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
      }
      return ACC_OK;
    }
    if constexpr (kHasSegFold) {
      if constexpr (dev::segfold_eligible<CL>()) {
        if (C == 0) return ACC_OK;
        constexpr int NFOLD = dev::count_if<CL>(dev::is_segfold_root);
        const int grid = seg_grid(L);
        const int per_block = dev::kSegTilesPerBlock;
        const bool v4 = seg_vec_ok(L);
        const size_t smem = v4 ? 0 : (size_t)NFOLD * dev::kSegTile * 4;    // operands are staged only where rows are not 128-bit friendly
        auto kern = v4 ? dev::k_segfold<CL, true> : dev::k_segfold<CL, false>;
        static int granted[2][64];
        if (smem > 48 * 1024 && !opt_in_shared_memory(kern, smem, granted[v4 ? 1 : 0]))
          return set_error(ACC_ERR_CUDA, "shared-memory opt-in failed: %s", cudaGetErrorString(cudaGetLastError()));
        kern<<<grid, dev::kBlock, smem, L.stream>>>(a, per_block);
        dev::k_segfold_across<CL><<<(grid + dev::kBlock / 32 - 1) / (dev::kBlock / 32), dev::kBlock, 0, L.stream>>>(a, grid);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
        return ACC_OK;
      } else {
        return set_error(ACC_ERR_NO_KERNEL, "segmented folds share a kernel only with each other and over one offsets array");
      }
    }
    if constexpr (kStencilShape) {
      const int rc = launch_stencil(L, a, R, C, vec);
      if (rc != 1) return rc;                            // 1 = shapes or shifts it does not cover: stream instead
    }
    if constexpr (kHasScan) {
      if ((int64_t)R * C == 0) return ACC_OK;
      const int per_row = (C + kScanTile - 1) / kScanTile;
      const int64_t tiles = (int64_t)R * per_row;
      if (tiles >= (int64_t(1) << 31)) return set_error(ACC_ERR_SHAPE, "too many rows to scan in one launch");
      const int grid = (int)std::min<int64_t>(tiles, (int64_t)sm_count() * (1536 / kScanBlock));
      if constexpr (kSlabShape) {
        if (vec && slab_shapes_ok(L, R, C)) {
          // partition the indices by slab, gather slab by slab from L2, merge and scan (slabgather.cuh)
          const int src = CL::c.nodes[dev::the_gather<CL>()].in[1];
          const int64_t n_src = (int64_t)L.nodes[src].R * L.nodes[src].C;
          const uint32_t mul = (uint32_t)(((uint64_t)dev::kSlabs << 32) / (uint64_t)n_src);
          const int full = C / dev::kSlabWarpTile;
          const int64_t states = ((16 + tiles * 8) + 15) & ~int64_t(15);
          uint32_t* counts = L.scratch + states / 4;
          uint32_t* codes = counts + full;
          const int warps = dev::kBlock / 32;
          const int pgrid = (int)std::min<int64_t>((full + warps - 1) / warps, (int64_t)sm_count() * 4);
          const int ggrid = (int)std::min<int64_t>((full + warps - 1) / warps, (int64_t)sm_count() * 8);
          // (word 1 of the scratch, cleared with the tile states: how many sampled warp tiles have local indices)
          const int probes = (int)std::min<int64_t>((full + warps - 1) / warps, (int64_t)sm_count());
          const dev::SlabIn slab{codes, counts, full, L.scratch + 1, (uint32_t)(probes * warps)};
          dev::k_slab_probe<CL><<<probes, dev::kBlock, 0, L.stream>>>(a, full, L.scratch + 1);
          dev::k_slab_partition<CL><<<pgrid, dev::kBlock, 0, L.stream>>>(a, codes, counts, full, mul, slab);
          for (int k = 0; k < dev::kSlabs; ++k) dev::k_slab_gather<CL><<<ggrid, dev::kBlock, 0, L.stream>>>(a, counts, full, (uint32_t)k, slab);
          {
            int per_row_arg = per_row, tiles_arg = (int)tiles;
            dev::SlabIn slab_arg = slab;
            void* params[] = {&a, &per_row_arg, &tiles_arg, &slab_arg};
            static int fit_on[64];
            const int resident = resident_grid(reinterpret_cast<const void*>(dev::k_scan_merge_pipelined<CL>), kScanBlock + 32, fit_on);
            if (resident > 0)
              cudaLaunchCooperativeKernel(reinterpret_cast<void*>(dev::k_scan_merge_pipelined<CL>), dim3((unsigned)std::min<int64_t>(tiles, resident)),
                                          dim3(kScanBlock + 32), params, 0, L.stream);
            else
              dev::k_scan_merge<CL><<<grid, kScanBlock, 0, L.stream>>>(a, per_row, (int)tiles, slab);
          }
          L.extra_launches = 2 + dev::kSlabs;
          const cudaError_t e = cudaGetLastError();
          if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
          return ACC_OK;
        }
      }
      {
        // all blocks resident at once where the device can promise it (then tiles need no ticket), else ticketed tiles
        int per_row_arg = per_row, tiles_arg = (int)tiles;
        void* params[] = {&a, &per_row_arg, &tiles_arg};
        static int fit_on[2][64];
        // (small tiles: with a warp of its own for the look-back, see scan_tiles_pipelined)
        constexpr bool kPipelined = dev::scan_pipelines<CL>();
        constexpr int kThreads = kScanBlock + (kPipelined ? 32 : 0);
        const void* kern;
        if constexpr (kPipelined)
          kern = vec ? reinterpret_cast<const void*>(dev::k_scan_pipelined<CL, true>) : reinterpret_cast<const void*>(dev::k_scan_pipelined<CL, false>);
        else
          kern = vec ? reinterpret_cast<const void*>(dev::k_scan<CL, true, true>) : reinterpret_cast<const void*>(dev::k_scan<CL, false, true>);
        const int resident = resident_grid(kern, kThreads, fit_on[vec ? 1 : 0]);
        if (resident > 0)
          cudaLaunchCooperativeKernel(const_cast<void*>(kern), dim3((unsigned)std::min<int64_t>(tiles, resident)), dim3(kThreads), params, 0, L.stream);
        else if (vec) dev::k_scan<CL, true><<<grid, kScanBlock, 0, L.stream>>>(a, per_row, (int)tiles);
        else dev::k_scan<CL, false><<<grid, kScanBlock, 0, L.stream>>>(a, per_row, (int)tiles);
      }
    } else if constexpr (kHasRowFold) {
      if (R == 0) return ACC_OK;
      const int grid = std::min(R, sm_count() * 16);
      if (vec) dev::k_rowfold<CL, true><<<grid, dev::kBlock, 0, L.stream>>>(a);
      else dev::k_rowfold<CL, false><<<grid, dev::kBlock, 0, L.stream>>>(a);
    } else {
      if constexpr (kHistShape) {
        const int rc = launch_hist(L, a, R, C, vec);
        if (rc != 1) return rc;                        // 1 = not worth it or does not fit: stream instead
      }
      if constexpr (kStreamSlabShape) {
        if (vec && stream_slab_shapes_ok(L, R, C)) {
          // the gather's source does not fit L2: partition the indices by slab, gather slab by slab, store from the merged values
          const int src = CL::c.nodes[dev::the_gather<CL>()].in[1];
          const int64_t n_src = (int64_t)L.nodes[src].R * L.nodes[src].C;
          const uint32_t mul = (uint32_t)(((uint64_t)dev::kSlabs << 32) / (uint64_t)n_src);
          const int full = C / dev::kSlabWarpTile;
          const int64_t base = (((int64_t)dev::stream_acc64_off(kScalarFolds, sm_count() * 8) * 4) + 15) & ~int64_t(15);
          uint32_t* counts = L.scratch + base / 4;
          uint32_t* codes = counts + full;
          const int warps = dev::kBlock / 32;
          const int pgrid = (int)std::min<int64_t>((full + warps - 1) / warps, (int64_t)sm_count() * 4);
          const int ggrid = (int)std::min<int64_t>((full + warps - 1) / warps, (int64_t)sm_count() * 8);
          const int probes = (int)std::min<int64_t>((full + warps - 1) / warps, (int64_t)sm_count());
          const dev::SlabIn slab{codes, counts, full, L.scratch + 1, (uint32_t)(probes * warps)};
          dev::k_slab_probe<CL><<<probes, dev::kBlock, 0, L.stream>>>(a, full, L.scratch + 1);
          dev::k_slab_partition<CL><<<pgrid, dev::kBlock, 0, L.stream>>>(a, codes, counts, full, mul, slab);
          for (int k = 0; k < dev::kSlabs; ++k) dev::k_slab_gather<CL><<<ggrid, dev::kBlock, 0, L.stream>>>(a, counts, full, (uint32_t)k, slab);
          dev::k_stream_merge<CL><<<pgrid, dev::kBlock, 0, L.stream>>>(a, slab);
          L.extra_launches = 2 + dev::kSlabs;
          const cudaError_t e = cudaGetLastError();
          if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
          return ACC_OK;
        }
      }
      // an empty domain still runs one block: a scatter must copy its defaults out
      const int grid = stream_grid(R, C, vec);
      if (vec) dev::k_stream<CL, true><<<grid, dev::kBlock, 0, L.stream>>>(a);
      else dev::k_stream<CL, false><<<grid, dev::kBlock, 0, L.stream>>>(a);
    }
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    return ACC_OK;
  }
};

// On-chip histogram path.  Returns ACC_OK after a launch, an error, or 1 when the generic
// streaming kernel should run instead.
template <class CL>
int Launcher<CL>::launch_hist(const ClusterLaunch& L, dev::Args<N>& a, int R, int C, bool vec) {
  if constexpr (kHistShape) {
    dev::HistPlan plan;
    if (!use_hist(L, R, C, plan)) return 1;
    constexpr int P = dev::the_f32_add_permute<CL>();
    const int64_t bins = (int64_t)L.nodes[P].R * L.nodes[P].C;
    auto kern = vec ? dev::k_hist<CL, true> : dev::k_hist<CL, false>;
    const size_t smem = (size_t)plan.per_cta * 4;
    static int granted[2][64];
    if (!opt_in_shared_memory(kern, smem, granted[vec ? 1 : 0]))
      return set_error(ACC_ERR_CUDA, "shared-memory opt-in failed: %s", cudaGetErrorString(cudaGetLastError()));
    const int64_t chunks = (int64_t)R * C / (vec ? 4 : 1);
    const int64_t per_team = (int64_t)dev::kHistBlock * dev::kHistUnroll;
    const int64_t want = (chunks + per_team - 1) / per_team;
    const int teams = (int)std::max<int64_t>(1, std::min<int64_t>(want, sm_count() / plan.group));
    const int grid = teams * plan.group;                  // one CTA per SM: all of them are resident together
    int* overflow = reinterpret_cast<int*>(L.scratch + dev::stream_acc64_off(kScalarFolds, a.grid) + 2 * bins);
    kern<<<grid, dev::kHistBlock, smem, L.stream>>>(a, plan, overflow);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(ACC_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    return ACC_OK;
  } else {
    return 1;
  }
}

// A cluster whose accumulating roots no single skeleton walks together (two scans; a scan beside a
// fold or a scatter; row folds beside a scatter) runs as several passes over the same description.
// Each pass keeps one group of those roots and treats the others as absent; only the first pass writes
// the element-wise roots.  Producers that the groups share are evaluated again in every pass, from
// the cluster's inputs: nothing beyond the cluster's own manifest arrays reaches memory.
constexpr int kMaxPasses = 6;
struct PassPlan {
  int n = 0;
  uint64_t keep[kMaxPasses] = {};     // bit i: accumulating root i runs in this pass
};

constexpr bool is_accumulating_root(const CNode& n) {
  return dev::is_fold_root(n) || dev::is_scan_root(n) || dev::is_permute_root(n);
}

template <class CL> constexpr PassPlan pass_plan() {
  PassPlan p;
  uint64_t folds = 0, permutes = 0;
  for (int i = 0; i < CL::c.n; ++i) {
    const CNode& n = CL::c.nodes[i];
    if (dev::is_scan_root(n)) p.keep[p.n++] = 1ull << i;             // a scan walks alone
    else if (dev::is_fold_root(n)) folds |= 1ull << i;
    else if (dev::is_permute_root(n)) permutes |= 1ull << i;
  }
  // whole-array folds and scatters share the streaming kernel; row folds have a kernel of their own
  const bool together = dev::domain_rank<CL>() <= 1 || !folds || !permutes;
  if (together) {
    if (p.n == 0 || (folds | permutes)) p.keep[p.n++] = folds | permutes;
  } else {
    p.keep[p.n++] = folds;
    p.keep[p.n++] = permutes;
  }
  return p;
}

// The scan whose values element-wise member i consumes inside the cluster, -1 if none.
constexpr int scan_needed_by(const CCluster& c, int i) {
  for (int s = 0; s < c.n; ++s)
    if (dev::is_scan_root(c.nodes[s]) && dev::needs_scan(c, i, s)) return s;
  return -1;
}

constexpr CNode unread_array(const CNode& n) {
  return CNode{ACC_INPUT, n.dtype, n.rank, 0, 0, 0, 0, {-1, -1, -1, -1, -1, -1}, false, true};
}

// The description of one pass: the accumulating roots in `keep` stay; element-wise roots that consume a
// scan are written by that scan's pass, the other element-wise roots by the first pass; members that no
// root of the pass reaches any more, and the roots of other passes, become arrays nobody reads.
constexpr CCluster pass_cluster(CCluster c, uint64_t keep, bool first) {
  const CCluster whole = c;
  int scan = -1;
  for (int i = 0; i < c.n; ++i)
    if (((keep >> i) & 1) && dev::is_scan_root(whole.nodes[i])) scan = i;
  for (int i = 0; i < c.n; ++i) {
    if (is_accumulating_root(whole.nodes[i]) && !((keep >> i) & 1)) {
      c.nodes[i] = unread_array(whole.nodes[i]);
    } else if (dev::is_store_root(whole.nodes[i])) {
      const int needs = scan_needed_by(whole, i);
      if (needs >= 0 ? needs != scan : !first) c.nodes[i].manifest = false;
    }
  }
  bool live[kMaxCluster] = {};
  for (int i = c.n - 1; i >= 0; --i) {
    const CNode& n = c.nodes[i];
    if (!n.member) continue;
    if (is_accumulating_root(n) || dev::is_store_root(n) || dev::is_segfold_root(n)) live[i] = true;
    if (live[i])
      for (int k = 0; k < n.nin; ++k) live[n.in[k]] = true;
  }
  for (int i = 0; i < c.n; ++i)
    if (c.nodes[i].member && !live[i]) c.nodes[i] = unread_array(c.nodes[i]);
  return c;
}

template <class CL, int P>
struct PassOf {
  static constexpr CCluster c = pass_cluster(CL::c, pass_plan<CL>().keep[P], P == 0);
};

template <class CL>
struct Passes {
  static constexpr PassPlan plan = pass_plan<CL>();

  template <int P>
  static int64_t scratch_from(const ClusterLaunch& L) {
    if constexpr (P < plan.n) {
      const int64_t here = Launcher<PassOf<CL, P>>::scratch_bytes(L);
      if (here < 0) return here;
      const int64_t rest = scratch_from<P + 1>(L);
      return rest < 0 ? rest : ((here + 255) & ~int64_t(255)) + rest;
    } else {
      return 0;
    }
  }
  static int64_t scratch_bytes(const ClusterLaunch& L) {
    if constexpr (plan.n <= 1) return Launcher<CL>::scratch_bytes(L);
    else return scratch_from<0>(L);
  }
  static int64_t zeroed_bytes(const ClusterLaunch& L) {
    if constexpr (plan.n <= 1) return Launcher<CL>::zeroed_bytes(L);
    else return scratch_from<0>(L);                   // the passes' regions follow one another: all of it
  }

  template <int P>
  static int launch_from(ClusterLaunch& L) {
    if constexpr (P < plan.n) {
      const int64_t here = Launcher<PassOf<CL, P>>::scratch_bytes(L);
      if (here < 0) return (int)here;
      const int rc = Launcher<PassOf<CL, P>>::launch(L);
      if (rc != ACC_OK) return rc;
      L.scratch += ((here + 255) & ~int64_t(255)) / 4;
      return launch_from<P + 1>(L);
    } else {
      return ACC_OK;
    }
  }
  static int launch(const ClusterLaunch& L) {
    if constexpr (plan.n <= 1) {
      return Launcher<CL>::launch(L);
    } else {
      ClusterLaunch pass = L;
      return launch_from<0>(pass);
    }
  }
};

template <class CL>
struct Registrar {
  explicit Registrar(const char* name) {
    // (a cluster of segmented folds is a walk over the elements and a small second launch for the segments that
    // cross its blocks)
    register_kernel(KernelEntry{signature(CL::c), name, &Passes<CL>::scratch_bytes, &Passes<CL>::zeroed_bytes, &Passes<CL>::launch,
                                Passes<CL>::plan.n > 1 ? Passes<CL>::plan.n : (dev::count_if<CL>(dev::is_segfold_root) > 0 ? 2 : 1)});
  }
};

#define ACC_CAT2(a, b) a##b
#define ACC_CAT(a, b) ACC_CAT2(a, b)
// Instantiates the kernels of cluster MASK of program PROG and registers them under NAME.
#define ACC_CLUSTER(PROG, MASK, NAME)                                              \
  struct ACC_CAT(Cl_, NAME) { static constexpr CCluster c = extract(PROG, MASK); }; \
  static Registrar<ACC_CAT(Cl_, NAME)> ACC_CAT(reg_, NAME)(#NAME);

}  // namespace acc
