// Shared device helpers: kernel arguments, cp.async wrappers, tile rasterisation.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace b2 {

// Arguments of one real GEMM launch, C := alpha*op(A)*op(B) + beta*C (column-major).
// op() is folded into the kernel's template parameters; m, n, k are the BLAS sizes.
template <typename T>
struct GemmArgs {
  int64_t m, n, k;
  T alpha, beta;
  const T* A;
  int64_t lda;
  const T* B;
  int64_t ldb;
  T* C;
  int64_t ldc;
  int tiles_m, tiles_n;  // CTA-tile counts along m and n
  int group_m;           // rasterisation: tile rows per group
  int tri;               // 0: all of C;  1: only i >= j (lower triangle);  2: only i <= j (upper triangle)
  int batch;             // number of problems of a strided batch (grid.y), at most 65535 per launch
  // k split over a thread-block cluster (grid.z = cluster size = ksplit, 1: off): CTA z of a cluster multiplies
  // the z-th share of the k-slabs of its tile; the shares are summed in rank order by CTA 0 through
  // distributed shared memory, which then runs the epilogue.
  int ksplit;
  int64_t batch_a, batch_b, batch_c;  // element offsets between the operands of consecutive problems
};

// ---- thread-block cluster helpers ---------------------------------------------------------
// All threads of all CTAs of the cluster arrive and wait (no thread of a split launch leaves before both
// barriers of the reduction, so the barrier always completes).
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of `local_smem_addr` (a shared::cta address) in the shared memory of CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cluster_map_shared(uint32_t local_smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ unsigned long long ld_cluster_b64(uint32_t addr) {
  unsigned long long v;
  asm volatile("ld.shared::cluster.b64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
  return v;
}

// Does the BM x BN tile at (m0, n0) lie entirely outside the stored triangle?
__device__ __forceinline__ bool tile_outside_triangle(int tri, int64_t m0, int64_t n0, int bm, int bn) {
  return (tri == 1 && n0 > m0 + bm - 1) || (tri == 2 && m0 > n0 + bn - 1);
}
// Does it cross the diagonal (so that single elements have to be masked)?
__device__ __forceinline__ bool tile_crosses_diagonal(int tri, int64_t m0, int64_t n0, int bm, int bn) {
  return tri != 0 && !((tri == 1 && m0 >= n0 + bn - 1) || (tri == 2 && n0 >= m0 + bm - 1));
}
__device__ __forceinline__ bool in_triangle(int tri, int64_t row, int64_t col) {
  return tri == 0 || (tri == 1 ? row >= col : row <= col);
}

// ---- cp.async (global -> shared, asynchronous, zero-filling past src_bytes) -------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- bulk reductions: shared -> global with an addition at the destination ------------------------------
// Every element of the block (both addresses 16-byte aligned, size a multiple of 16 bytes) is ADDED to the
// element in global memory, one IEEE addition each, done by the memory system; the copy is tracked by the issuing
// thread's bulk async-groups like a bulk store.
__device__ __forceinline__ void bulk_reduce_add(double* gmem_dst, const double* smem_src, uint32_t bytes) {
  asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f64 [%0], [%1], %2;" ::"l"(gmem_dst),
               "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_reduce_add(float* gmem_dst, const float* smem_src, uint32_t bytes) {
  asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(gmem_dst),
               "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
}
// shared -> global, tracked by the issuing thread's bulk async-groups
__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst), "r"(smem_u32(smem_src)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all of this thread's bulk copies have read their shared-memory source
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

template <int BYTES>
__device__ __forceinline__ void cp_async_zfill(void* smem_dst, const void* gmem_src, int src_bytes) {
  static_assert(BYTES == 4 || BYTES == 8 || BYTES == 16, "cp.async copies 4, 8 or 16 bytes");
  if constexpr (BYTES == 16) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_u32(smem_dst)), "l"(gmem_src),
                 "r"(src_bytes)
                 : "memory");
  } else {
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;\n" ::"r"(smem_u32(smem_dst)), "l"(gmem_src),
                 "n"(BYTES), "r"(src_bytes)
                 : "memory");
  }
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }

template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// ---- tile rasterisation ---------------------------------------------------------------
// Linear CTA index -> (tile row, tile column).  Tiles are visited in groups of `group_m` tile
// rows, column by column inside a group, so that the CTAs resident at one time cover a
// compact block of C and share their A row-panels and B column-panels in L2 (the role the
// nc/mc loops play in the paper's Figure 1 loop nest).
__device__ __forceinline__ void tile_coords(int linear, int tiles_m, int tiles_n, int group_m, int& tm, int& tn) {
  const int per_group = group_m * tiles_n;
  const int group = linear / per_group;
  const int first_m = group * group_m;
  const int rows = min(group_m, tiles_m - first_m);
  const int in_group = linear - group * per_group;
  tn = in_group / rows;
  tm = first_m + (in_group - tn * rows);
}

}  // namespace b2
