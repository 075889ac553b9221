// Tensor-core micro-batch product of a forward row tile (sm_100a: tcgen05.mma with the accumulator in tensor memory).
//
//   D[m][n] = sum_k W[m][k] X[n][k]      m < 64 output rows of the tile, n < N messages of the micro-batch, bf16 x bf16 -> fp32
//
// Both operands live in shared memory as bfloat16 in the canonical K-major layout without swizzling: 8 rows x 16 bytes
// form a core matrix of 128 contiguous bytes; the core matrices of one 8-row group follow each other along k, the
// 8-row groups follow each other K * 16 bytes apart.  One instruction covers 16 values of k (two core matrices per row
// group), so the descriptors of step s start 256 bytes further on.  With M = 64 the accumulator row m sits in
// tensor-memory lane (m mod 16) + 32 (m / 16), column n; a warp reads the 32 lanes of its quadrant (warp index mod 4).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace tc {

constexpr int M = 64;                 // output rows per tile (the instruction's M)
constexpr int TMEM_COLS = 64;         // tensor-memory columns a tile allocates (fp32 accumulator columns = messages), power of two >= 32

__device__ __forceinline__ unsigned smem_addr(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
// byte offset of element (row r, column k) of an operand with K columns
__device__ __forceinline__ unsigned elem_off(const int r, const int k, const int K) {
  return (unsigned)(r >> 3) * (unsigned)(K * 16) + (unsigned)(k >> 3) * 128u + (unsigned)(r & 7) * 16u + (unsigned)(k & 7) * 2u;
}
// shared-memory matrix descriptor: start address, leading byte offset (between the two core matrices along k), stride byte
// offset (between 8-row groups), all in units of 16 bytes; descriptor version 1, no swizzle
__device__ __forceinline__ uint64_t smem_desc(const unsigned saddr, const unsigned lbo_bytes, const unsigned sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) | ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// instruction descriptor of kind::f16: D fp32, A and B bfloat16, both K-major, dense, no negation
__host__ __device__ constexpr uint32_t instr_desc(const int m, const int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ---- tensor memory: one warp allocates and frees; the address lands in shared memory --------------------------
__device__ __forceinline__ void tmem_alloc(unsigned* slot_in_smem) {            // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_addr(slot_in_smem)), "r"((unsigned)TMEM_COLS) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(const unsigned taddr) {               // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(taddr), "r"((unsigned)TMEM_COLS) : "memory");
}

// ---- operands ------------------------------------------------------------------------------------------------------
// Eight consecutive fp32 values of row r from k on, rounded to bfloat16 (exact for payloads that were rounded when they
// were emitted), into the operand at `base`.
__device__ __forceinline__ void store8(unsigned char* base, const int r, const int k, const int K, const float4 a, const float4 b) {
  const __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w), p2 = __floats2bfloat162_rn(b.x, b.y), p3 = __floats2bfloat162_rn(b.z, b.w);
  uint4 v;
  v.x = *reinterpret_cast<const unsigned*>(&p0); v.y = *reinterpret_cast<const unsigned*>(&p1);
  v.z = *reinterpret_cast<const unsigned*>(&p2); v.w = *reinterpret_cast<const unsigned*>(&p3);
  *reinterpret_cast<uint4*>(base + elem_off(r, k, K)) = v;
}
// Rows [0, n_rows) of an operand from fp32 rows in device memory (row b at src(b), K values, 16-byte aligned), all threads
// of the CTA.  Work items run over (8-row group, k chunk, row in group) with the row fastest: eight lanes fill one core
// matrix (128 contiguous bytes of shared memory).
template <class RowPtr>
__device__ __forceinline__ void fill_operand(unsigned char* base, const int n_rows, const int K, const RowPtr src, const int tid, const int n_threads) {
  const int K8 = K >> 3, items = ((n_rows + 7) >> 3) * K8 * 8;
  constexpr int U = 4;
  for (int i0 = tid; i0 < items; i0 += U * n_threads) {
    float4 a[U], b[U];
#pragma unroll
    for (int u = 0; u < U; u++) {
      const int i = i0 + u * n_threads, r = ((i >> 3) / K8) * 8 + (i & 7), k8 = (i >> 3) % K8;
      if (i < items && r < n_rows) {
        const float4* p = reinterpret_cast<const float4*>(src(r)) + 2 * k8;
        a[u] = __ldcg(p); b[u] = __ldcg(p + 1);
      } else a[u] = b[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < U; u++) {
      const int i = i0 + u * n_threads, r = ((i >> 3) / K8) * 8 + (i & 7), k8 = (i >> 3) % K8;
      if (i < items) store8(base, r, 8 * k8, K, a[u], b[u]);
    }
  }
}

// ---- the product ------------------------------------------------------------------------------------------------------
// One thread issues K / 16 instructions (the first overwrites the accumulator) and commits them to the mbarrier at `bar`
// (one arrival when they have all completed).  The operands must have been written, fenced for the asynchronous proxy
// (fence_operands by every writing thread) and the CTA synchronised before.
__device__ __forceinline__ void fence_operands() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void issue(const unsigned taddr, const void* Wb, const void* Xb, const int K, const int N, const unsigned bar) {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned wa = smem_addr(Wb), xa = smem_addr(Xb), sbo = (unsigned)K * 16u;
  const uint32_t idesc = instr_desc(M, N);
  for (int s = 0; s < (K >> 4); s++) {
    const uint64_t da = smem_desc(wa + 256u * s, 128u, sbo), db = smem_desc(xa + 256u * s, 128u, sbo);
    const unsigned acc = s > 0;
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 :: "r"(taddr), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
  }
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
// After the mbarrier has flipped: warps 0-3 read the accumulator.  Lane l < 16 of warp q holds row 16 q + l; out[n * ldo + row]
// receives column n for n < n_cols (n_cols <= N, a multiple of 16 columns is read).
__device__ __forceinline__ void read_accumulator(const unsigned taddr, const int N, const int n_cols, float* out, const int ldo, const int rows_valid) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp >= 4) return;
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const int row = 16 * warp + lane;
  for (int c0 = 0; c0 < N && c0 < n_cols; c0 += 16) {
    unsigned v[16];
    const unsigned a = taddr + ((unsigned)(32 * warp) << 16) + (unsigned)c0;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(a) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    if (lane < 16 && row < rows_valid) {
#pragma unroll
      for (int j = 0; j < 16; j++) if (c0 + j < n_cols) out[(c0 + j) * ldo + row] = __uint_as_float(v[j]);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

// ---- a handful of messages: the same product on the FMA units ------------------------------------------------------
// Below SMALL_ROWS + 1 messages the product is no dense contraction: 512 threads take (row, one of eight k-slices) and
// read the same bfloat16 operands (so a tile computes with the same weights whatever the size of the batch); the slices
// meet by shared-memory adds in out[n * ldo + row], which the caller has zeroed.
constexpr int SMALL_ROWS = 4;
__device__ __forceinline__ void small_product(const unsigned char* Wb, const unsigned char* Xb, const int K, const int count, float* out, const int ldo, const int tid) {
  const int r = tid & (M - 1), s = tid >> 6, K8 = K >> 3;
  float acc[SMALL_ROWS];
#pragma unroll
  for (int b = 0; b < SMALL_ROWS; b++) acc[b] = 0.f;
  for (int c = s; c < K8; c += 8) {
    const uint4 w = *reinterpret_cast<const uint4*>(Wb + elem_off(r, 8 * c, K));
    const unsigned wu[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int b = 0; b < SMALL_ROWS; b++) {
      if (b >= count) break;
      const uint4 x = *reinterpret_cast<const uint4*>(Xb + elem_off(b, 8 * c, K));
      const unsigned xu[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int q = 0; q < 4; q++) {
        acc[b] = fmaf(__uint_as_float(wu[q] << 16), __uint_as_float(xu[q] << 16), acc[b]);
        acc[b] = fmaf(__uint_as_float(wu[q] & 0xffff0000u), __uint_as_float(xu[q] & 0xffff0000u), acc[b]);
      }
    }
  }
#pragma unroll
  for (int b = 0; b < SMALL_ROWS; b++) if (b < count) atomicAdd(out + b * ldo + r, acc[b]);
}

}  // namespace tc
