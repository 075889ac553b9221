// Persistent message-driven training kernel (device code).
//
// One CTA per role: CTA 0 is the controller (admission under max_active_keys, retirement, Sec. 3 / Sec. 4
// "controller loop"); every other CTA owns one row tile of one parameterised (PPT) node and keeps that
// tile's weights and fp32 gradient accumulators in shared memory for the whole epoch.  Messages are headers
// in per-node ring queues; their payloads live in caches keyed by (key slot, iteration, position), which
// double as the activation caches of Sec. 4.  The parameter-free nodes (Cond, Phi, Isu, Concat, Bcast,
// Group, Ungroup, Flatmap, row sum, Loss, Sink) are executed by the warp that emits a message: it walks
// the IR graph until the message lands in the input cache and queue of the next PPT node.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "engine_types.h"

namespace amp {

// ------------------------------------------------------------------------------------------------
// memory-model helpers, bounded waits
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned ld_acq(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Several independent flags polled at once: relaxed loads overlap in flight where acquire loads would not; one fence
// after them orders everything read afterwards behind all of them.
__device__ __forceinline__ unsigned ld_rlx(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_acq() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
__device__ __forceinline__ void st_rel(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void fail(const Ctx& C, int code, int node, int detail) {
  if (atomicCAS(&C.g->status, 0, code) == 0) { C.g->err_node = node; C.g->err_detail = detail; }
  __threadfence();
  st_rel(&C.g->abort_flag, 1u);
}
__device__ __forceinline__ bool aborted(const Ctx& C) { return ld_acq(&C.g->abort_flag) != 0; }
// Warp-uniform reads: one lane reads, all lanes take its value, so that a value changing under the warp can never
// send lanes of one warp down different paths around a warp-synchronous primitive.
__device__ __forceinline__ unsigned warp_uniform(unsigned v) { return __shfl_sync(0xffffffffu, v, 0); }
__device__ __forceinline__ bool aborted_warp(const Ctx& C) {
  unsigned v = 0;
  if ((threadIdx.x & 31) == 0) v = *(volatile unsigned*)&C.g->abort_flag;
  return warp_uniform(v) != 0;
}

// Every wait in the kernel goes through this: it gives up when another CTA has raised the abort word or
// when the run's time budget is spent (status AMPNET_ETIMEOUT), so no wait can hang the GPU.
template <class Cond>
__device__ __forceinline__ bool spin_until(const Ctx& C, unsigned long long t0, Cond cond) {
  unsigned it = 0;
  while (!cond()) {
    if ((++it & 31u) == 0) {
      if (aborted(C)) return false;
      if (gtime() - t0 > C.timeout_ns) { fail(C, ST_TIMEOUT, -1, 0); return false; }
    }
    if (it > 32) __nanosleep(it < 256 ? 20 : 100);
  }
  return true;
}

// Barrier among `n` CTAs on a monotone counter; gen is the caller's local generation.  Returns false on abort.
__device__ __forceinline__ bool cta_barrier(const Ctx& C, unsigned long long t0, unsigned* ctr, unsigned n,
                                            unsigned& gen, int* s_ok) {
  __syncthreads();
  gen++;
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(ctr, 1u);
    unsigned target = gen * n;
    bool ok = spin_until(C, t0, [&] { return ld_acq(ctr) >= target; });
    __threadfence();
    *s_ok = ok ? 1 : 0;
  }
  __syncthreads();
  return *s_ok != 0;
}

__device__ __forceinline__ long long key_of(const Ctx& C, int node, int slot, int it, int u, int U) {
  if ((unsigned)slot >= (unsigned)C.mak || (unsigned)it >= (unsigned)C.IT || (unsigned)u >= (unsigned)U) {
    fail(C, ST_OVERFLOW, node, u);
    return -1;
  }
  return ((long long)slot * C.IT + it) * U + u;
}

__device__ __forceinline__ unsigned long long mix64(unsigned long long x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

// Per-CTA copies of the node and PPT tables (read on every step of a walk): shared memory instead of device memory.
__shared__ DevNode g_nodes[MAX_SMEM_NODES];
__shared__ DevPPT g_ppts[MAX_SMEM_PPTS];
__shared__ int g_bf16;      // payloads are rounded to bfloat16 (round to nearest even) where they are emitted

// What a node emits as a payload passes through here: identity for fp32 messages, bf16 rounding otherwise.
// Weights, accumulators and the arithmetic on cached activations stay fp32.
__device__ __forceinline__ float emit_round(float v) { return g_bf16 ? __bfloat162float(__float2bfloat16_rn(v)) : v; }

// ------------------------------------------------------------------------------------------------
// walking warp: executes the parameter-free nodes between two PPT nodes
// ------------------------------------------------------------------------------------------------
struct Frame {
  int node, aport, dir, iter;
  int inst, seq, slot, it, u, port, rows, flags;
  int dim, ld;
  int nsum, sstride;    // payload element (r, i) = sum over j < nsum of p[j * sstride + r * ld + i]
  long long ibase, ebase; // first position / first edge of the instance in the structure tables (loaded once per message)
  int part, nparts;     // nparts > 1: the rows of the first row-wise fork are shared among nparts CTAs; this walker takes
                        // rows j = part (mod nparts); until that fork only part 0 has side effects (the others are shadows)
  const float* p;       // payload rows (device memory); nullptr = zeros
};

// Frames offered by a walking warp to the other warps of its CTA (continuations of forks).
constexpr int POOL = 64;
struct WalkPool {
  Frame f[POOL];
  unsigned ready[POOL];      // ticket + 1 while the slot holds a frame, 0 when free
  unsigned head, tail;
  int outstanding;           // frames queued or being walked
};

struct WalkAcc { unsigned long long msgs, hash; };

__device__ __forceinline__ float ld_payload(const float* p, int nsum, int sstride, size_t off) {
  float s = __ldcg(p + off);
  for (int j = 1; j < nsum; j++) s += __ldcg(p + (size_t)j * sstride + off);     // addend order
  return nsum > 1 ? emit_round(s) : s;
}
// Copy payload rows into a cache; a lazy sum is evaluated on the way.  The rows are flattened so that every lane keeps
// four (vector) loads in flight whatever the row length.
template <int V>
__device__ __forceinline__ void warp_copy_v(float* dst, int dld, const float* src, int sld, int nsum, int sstride, int rows, int dim, int lane) {
  const int wv = dim / V, total = rows * wv;
  for (int base = lane; base < total; base += 128) {
    float v[4][V];
    size_t off[4], doff[4];
#pragma unroll
    for (int k = 0; k < 4; k++) {
      const int idx = base + 32 * k;
      int r = 0, c = idx;
      if (rows > 1) { r = idx / wv; c = idx - r * wv; }
      off[k] = (size_t)r * sld + (size_t)c * V;
      doff[k] = (size_t)r * dld + (size_t)c * V;
#pragma unroll
      for (int q = 0; q < V; q++) v[k][q] = 0.f;
    }
    for (int j = 0; j < nsum; j++) {                             // addend order; the four loads of one addend overlap
      const float* a = src + (size_t)j * sstride;
#pragma unroll
      for (int k = 0; k < 4; k++) {
        if (base + 32 * k < total) {
          if (V == 4) { const float4 t = __ldcg(reinterpret_cast<const float4*>(a + off[k])); v[k][0] += t.x; v[k][1 % V] += t.y; v[k][2 % V] += t.z; v[k][3 % V] += t.w; }
          else if (V == 2) { const float2 t = __ldcg(reinterpret_cast<const float2*>(a + off[k])); v[k][0] += t.x; v[k][1 % V] += t.y; }
          else v[k][0] += __ldcg(a + off[k]);
        }
      }
    }
#pragma unroll
    for (int k = 0; k < 4; k++) {
      if (base + 32 * k < total) {
        if (nsum > 1) {
#pragma unroll
          for (int q = 0; q < V; q++) v[k][q] = emit_round(v[k][q]);
        }
        float* d = dst + doff[k];
        if (V == 4) *reinterpret_cast<float4*>(d) = make_float4(v[k][0], v[k][1 % V], v[k][2 % V], v[k][3 % V]);
        else if (V == 2) *reinterpret_cast<float2*>(d) = make_float2(v[k][0], v[k][1 % V]);
        else d[0] = v[k][0];
      }
    }
  }
}
__device__ __noinline__ void warp_copy_p(float* dst, int dld, const float* src, int sld, int nsum, int sstride, int rows, int dim,
                                          int lane) {
  if (!src) {
    for (int r = 0; r < rows; r++) for (int i = lane; i < dim; i += 32) dst[(size_t)r * dld + i] = 0.f;
    return;
  }
  const unsigned long long al = (unsigned long long)dst | (unsigned long long)src;
  const int geo = dim | dld | (rows > 1 ? sld : 0) | (nsum > 1 ? sstride : 0);
  if (((geo & 3) == 0) && ((al & 15) == 0)) warp_copy_v<4>(dst, dld, src, sld, nsum, sstride, rows, dim, lane);
  else if (((geo & 1) == 0) && ((al & 7) == 0)) warp_copy_v<2>(dst, dld, src, sld, nsum, sstride, rows, dim, lane);
  else warp_copy_v<1>(dst, dld, src, sld, nsum, sstride, rows, dim, lane);
}

#define warp_copy(dst, dld, f, rows, dim, lane) warp_copy_p((dst), (dld), (f).p, (f).ld, (f).nsum, (f).sstride, (rows), (dim), (lane))

// A producer takes its ticket before it copies the payload (the two round trips overlap) and publishes afterwards.
__device__ __forceinline__ unsigned ring_ticket(Ring& r) { return atomicAdd(r.tail, 1u); }
__device__ __forceinline__ void ring_publish(Ring& r, unsigned t, const Frame& f) {   // one lane; the release store orders the payload
  unsigned s = t & r.mask;
  int4* d = reinterpret_cast<int4*>(&r.e[s]);
  d[0] = make_int4(f.inst, f.seq, f.slot, f.it);
  d[1] = make_int4(f.u, f.port, f.rows, f.flags);
  st_rel(&r.seq[s], t + 1u);
}

// A source message came home (or, in evaluation, reached a Loss / Sink): one lane.  The arrival that completes the
// instance tells the controller; the others only count down.
__device__ __forceinline__ int atom_add_acq_rel(int* p, int v);
__device__ __forceinline__ void retire_push(const Ctx& C, int slot) {
  if (atom_add_acq_rel(&C.outstanding[slot], -1) != 1) return;
  unsigned t = atomicAdd(&C.g->retire_tail, 1u);
  unsigned s = t & C.retire_mask;
  C.retire_e[s] = (unsigned)slot;
  st_rel(&C.retire_seq[s], t + 1u);
}

// Join on a keyed counter: every arriving warp has written its part; the one that completes the count
// continues.  Returns true for the completing arrival (and resets the counter for the key's next use).
__device__ __forceinline__ int atom_add_acq_rel(int* p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ bool join_arrive(int* cnt, int expected, int lane) {
  __syncwarp();                       // the lanes' writes of this part are ordered before lane 0's release
  int last = 0;
  if (lane == 0) {
    int old = atom_add_acq_rel(cnt, 1);
    last = (old + 1 == expected);
    if (last) { *cnt = 0; }
  }
  last = __shfl_sync(0xffffffffu, last, 0);
  return last != 0;
}

// ---- CTA-wide pool of frames: a warp that forks offers the rest of the fork to idle warps --------------
__device__ __forceinline__ bool pool_offer(const Ctx& C, WalkPool* Q, const Frame& c, int lane) {
  if (!Q) return false;
  int ok = 0;
  if (lane == 0) {
    unsigned t = *(volatile unsigned*)&Q->tail;
    for (;;) {
      const unsigned h = *(volatile unsigned*)&Q->head;
      if (t - h >= (unsigned)POOL) break;
      const unsigned old = atomicCAS(&Q->tail, t, t + 1u);
      if (old == t) { ok = 1; break; }
      t = old;
    }
    if (ok) {
      const unsigned idx = t % POOL;
      atomicAdd(&Q->outstanding, 1);
      int spins = 0;
      while (*(volatile unsigned*)&Q->ready[idx] != 0u && ++spins < (1 << 20)) {}
      if (*(volatile unsigned*)&Q->ready[idx] != 0u) fail(C, ST_TIMEOUT, -5, (int)idx);   // the slot never drained: report, the run is over
      Q->f[idx] = c;
      __threadfence_block();
      *(volatile unsigned*)&Q->ready[idx] = t + 1u;
    }
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ void to_succ(Frame& f, const DevNode& n, int k) {
  f.node = n.succ_node[k]; f.aport = n.succ_port[k]; f.dir = FWD; f.iter = 0;
}
__device__ __forceinline__ void to_pred(Frame& f, const DevNode& n, int j) {
  f.node = n.pred_node[j]; f.aport = n.pred_port[j]; f.dir = BWD; f.iter = 0;
}

__device__ __forceinline__ float sigm(float v) { return 1.f / (1.f + expf(-v)); }

// first position (token / tree node / graph node) of an instance
#define IBASE(inst) (I.offsets ? I.offsets[(inst)] : 0)
__device__ __noinline__ void walk(const Ctx& C, Frame f, Frame* stack, WalkAcc& acc, WalkPool* Q) {
  const int lane = threadIdx.x & 31;
  const DevInst& I = C.inst;
  int sp = 0;
  bool have = true;
  int steps = 0;
  while (have) {
    if (f.node < 0) { fail(C, ST_OVERFLOW, -2, 0); return; }
    // self-checks: no endless walk, no absurd fork width, stop early once the run is being aborted
    if (++steps > (1 << 20) || (unsigned)f.nsum > 64u || (unsigned)f.rows > 4096u || (unsigned)f.nparts > 64u) {
      fail(C, ST_OVERFLOW, -3, f.node * 100000 + (f.rows & 0xffff));
      return;
    }
    if ((steps & 63) == 0 && aborted_warp(C)) return;
    const DevNode& n = g_nodes[f.node];
    const long long tstep = (C.tune & 8) ? clock64() : 0;
    const int ptype = n.type * 2 + f.dir;
    bool cont = false;                       // true: f was rewritten and continues
    const bool shadow = f.nparts > 1 && f.part > 0;
    const bool dies_as_shadow = shadow && !(n.type == COND || n.type == PHI || n.type == ISU) && (n.type == LINEAR || n.type == LOOKUP || n.type == GRUCELL || n.type == LOSS_CE ||
                                           n.type == LOSS_MSE || n.type == SINK || n.type == SOURCE || n.type == NPT_SUMROWS ||
                                           (n.type == BCAST && f.dir == BWD) || (n.type == CONCAT && f.dir == FWD) || (n.type == SPLIT && f.dir == BWD) || n.type == NPT_LSTM ||
                                           (n.type == GROUP && f.dir == FWD) || (n.type == UNGROUP && f.dir == BWD) ||
                                           (n.type == FLATMAP && f.dir == BWD));
    if (dies_as_shadow) {
      // a shadow reached a node with side effects before any row-wise fork: the real walker handles it
    } else if (n.type == SOURCE) {           // a source message came home to the controller
      if (f.dir == BWD && lane == 0) retire_push(C, f.slot);
    } else {
      if (f.iter == 0 && !shadow) acc.msgs++;
      if (f.iter == 0 && !shadow && (C.det || (C.tune & 16))) {
        unsigned long long a = (unsigned long long)f.node | ((unsigned long long)f.dir << 16) |
                               ((unsigned long long)(f.aport & 0xff) << 20) | ((unsigned long long)(f.port & 0xff) << 28);
        unsigned long long b = ((unsigned long long)(unsigned)f.inst << 32) | ((unsigned long long)(f.it & 0xff) << 24) |
                               (unsigned long long)(f.u & 0xffffff);
        acc.hash += mix64(mix64(a) ^ (b * 0x9E3779B97F4A7C15ull));
        if (lane == 0 && !(C.tune & 4)) atomicAdd(&C.node_msgs[f.node * 2 + f.dir], 1ull);
      }
      switch (n.type) {
        case LINEAR: case LOOKUP: case GRUCELL: {
          DevPPT& P = g_ppts[n.ppt];
          long long key = key_of(C, f.node, f.slot, f.it, f.u, P.U);
          if (key < 0) return;
          if (f.rows > P.rows_max) { fail(C, ST_OVERFLOW, f.node, f.rows); return; }
          unsigned ticket = 0;
          const long long tq0 = (C.tune & 8) ? clock64() : 0;
          if (lane == 0) ticket = ring_ticket(P.ring[f.dir]);
          if (f.dir == FWD) {
            if (P.xcache) {
              float* dst = P.xcache + key * (long long)P.rows_max * P.xld;
              if (f.p != dst) warp_copy(dst, P.xld, f, f.rows, P.in_dim, lane);
            }
          } else if (n.type != LOOKUP || f.dim > 0) {
            warp_copy(P.gbuf + key * (long long)P.rows_max * P.out_dim, P.out_dim, f, f.rows, P.out_dim, lane);
          }
          __syncwarp();
          const long long tq1 = (C.tune & 8) ? clock64() : 0;
          if (lane == 0) ring_publish(P.ring[f.dir], ticket, f);
          if ((C.tune & 8) && lane == 0) {      // profile: SPLIT slots = copy (+ticket) / publish, SOURCE FWD slot = before
            const long long tq2 = clock64();
            atomicAdd(&C.g->walk_cycles[SPLIT * 2], (unsigned long long)(tq1 - tq0)); atomicAdd(&C.g->walk_steps[SPLIT * 2], 1ull);
            atomicAdd(&C.g->walk_cycles[SPLIT * 2 + 1], (unsigned long long)(tq2 - tq1)); atomicAdd(&C.g->walk_steps[SPLIT * 2 + 1], 1ull);
            atomicAdd(&C.g->walk_cycles[SOURCE * 2], (unsigned long long)(tq0 - tstep)); atomicAdd(&C.g->walk_steps[SOURCE * 2], 1ull);
          }
        } break;
        case LOSS_CE: case LOSS_MSE: {
          long long key = key_of(C, f.node, f.slot, f.it, f.u, n.U_in);
          if (key < 0) return;
          float* g = n.jbuf + key * n.jstride;
          if (n.type == LOSS_CE) {
            int label = I.labels_i[I.labels_per_node ? f.ibase + f.u : f.inst];
            float mx = -3.4e38f; int arg = 0x7fffffff;
            for (int j = lane; j < n.in_dim; j += 32) { float v = ld_payload(f.p, f.nsum, f.sstride, j); if (v > mx) { mx = v; arg = j; } }
            for (int o = 16; o; o >>= 1) {
              float om = __shfl_xor_sync(0xffffffffu, mx, o); int oa = __shfl_xor_sync(0xffffffffu, arg, o);
              if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
            }
            float s = 0.f;
            for (int j = lane; j < n.in_dim; j += 32) s += expf(ld_payload(f.p, f.nsum, f.sstride, j) - mx);
            for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            float lse = mx + logf(s);
            for (int j = lane; j < n.in_dim; j += 32) g[j] = emit_round(expf(ld_payload(f.p, f.nsum, f.sstride, j) - lse) - (j == label ? 1.f : 0.f));
            if (lane == 0) { n.lossval[key] = lse - ld_payload(f.p, f.nsum, f.sstride, label); n.predok[key] = (arg == label) ? 1 : 0; }
          } else {
            if (lane == 0) {
              float d = ld_payload(f.p, f.nsum, f.sstride, 0) - I.labels_f[f.inst];
              n.lossval[key] = d * d; g[0] = emit_round(2.f * d); n.predok[key] = 0;
            }
          }
          if (f.flags & HDR_EVAL) { __syncwarp(); if (lane == 0) retire_push(C, f.slot); }
          else { __syncwarp(); f.p = g; f.nsum = 1; f.dim = n.in_dim; f.ld = n.in_dim; to_pred(f, n, 0); cont = true; }
        } break;
        case SINK:
          if (f.flags & HDR_EVAL) { if (lane == 0) retire_push(C, f.slot); }
          else { f.p = nullptr; f.nsum = 1; to_pred(f, n, 0); cont = true; }
          break;
        case COND:
          if (f.dir == FWD) {
            int k = 0;
            switch (n.fn) {
              case 1: k = f.u < (int)(I.offsets[f.inst + 1] - f.ibase) ? 0 : 1; break;
              case 2: k = I.parent[f.ibase + f.u] < 0 ? 0 : 1; break;      // the root has no parent
              case 3: k = f.u; break;
              case 4: k = f.it < n.fn_arg ? 0 : 1; break;
              case 5: k = (f.inst + f.u) % n.n_succ; break;                  // replicas of a node (Sec. 5)
            }
            if ((unsigned)k >= (unsigned)n.n_succ) { fail(C, ST_OVERFLOW, f.node, k); return; }
            to_succ(f, n, k);
          } else to_pred(f, n, 0);
          cont = true;
          break;
        case PHI: {
          long long key = key_of(C, f.node, f.slot, f.it, f.u, n.U_in);
          if (key < 0) return;
          if (f.dir == FWD) {
            if (lane == 0 && !(f.flags & HDR_EVAL) && !shadow) n.origin[key] = (unsigned char)(f.aport + 1);
            to_succ(f, n, 0);
            cont = true;
          } else {
            int j = (int)*(volatile unsigned char*)&n.origin[key] - 1;
            if (shadow) { if (j >= 0 && j < n.n_pred) { to_pred(f, n, j); cont = true; } }   // the real walker may have cleared it
            else {
              if (j < 0 || j >= n.n_pred) { fail(C, ST_OVERFLOW, f.node, j); return; }
              __syncwarp();
              if (lane == 0) n.origin[key] = 0;
              to_pred(f, n, j);
              cont = true;
            }
          }
        } break;
        case ISU:
          if (f.dir == FWD) {
            if (n.fn == 1) f.u += 1;
            else if (n.fn == 2) { f.port = I.child_slot[f.ibase + f.u]; f.u = I.parent[f.ibase + f.u]; }
            else f.it += 1;
            to_succ(f, n, 0);
          } else {
            if (n.fn == 1) f.u -= 1;
            else if (n.fn == 2) { f.u = f.port == 0 ? I.left[f.ibase + f.u] : I.right[f.ibase + f.u]; f.port = 0; }
            else f.it -= 1;
            to_pred(f, n, 0);
          }
          cont = true;
          break;
        case BCAST:
          if (f.dir == FWD) {
            int k = f.iter;
            if (k + 1 < n.fn_arg) { Frame c = f; c.iter = k + 1;
              if (!pool_offer(C, Q, c, lane)) { if (sp >= WALK_STACK) { fail(C, ST_OVERFLOW, f.node, sp); return; }
                                             if (lane == 0) stack[sp] = c; sp++; __syncwarp(); } }
            to_succ(f, n, k);
            cont = true;
          } else {
            long long key = key_of(C, f.node, f.slot, f.it, f.u, n.U_in);
            if (key < 0) return;
            float* base = n.jbuf + key * n.jstride;
            const int blk = n.rows_in * n.in_dim;
            warp_copy(base + (size_t)f.aport * blk, n.in_dim, f, f.rows, n.in_dim, lane);
            if (join_arrive(&n.jcnt[key], n.fn_arg, lane)) {
              f.p = base; f.nsum = n.fn_arg; f.sstride = blk;      // summed in successor order by whoever reads it
              f.ld = n.in_dim; f.dim = n.in_dim;
              to_pred(f, n, 0);
              cont = true;
            }
          }
          break;
        case CONCAT:
          if (f.dir == FWD) {
            int port = n.fn == 2 ? f.port : f.aport;
            long long key = key_of(C, f.node, f.slot, f.it, f.u, n.U_out);
            if (key < 0) return;
            if ((unsigned)port >= (unsigned)n.fn_arg || f.rows > n.rows_in) { fail(C, ST_OVERFLOW, f.node, port); return; }
            float* base = n.jbuf + key * n.jstride;
            if (f.p != base + port * n.in_dim || f.nsum != 1) warp_copy(base + port * n.in_dim, n.out_dim, f, f.rows, n.in_dim, lane);
            if (join_arrive(&n.jcnt[key], n.fn_arg, lane)) {
              f.p = base; f.nsum = 1; f.dim = n.out_dim; f.ld = n.out_dim; f.port = 0;
              to_succ(f, n, 0);
              cont = true;
            }
          } else {
            int k = f.iter;
            if (k + 1 < n.fn_arg) { Frame c = f; c.iter = k + 1;
              if (!pool_offer(C, Q, c, lane)) { if (sp >= WALK_STACK) { fail(C, ST_OVERFLOW, f.node, sp); return; }
                                             if (lane == 0) stack[sp] = c; sp++; __syncwarp(); } }
            f.p = f.p ? f.p + k * n.in_dim : nullptr; f.dim = n.in_dim;
            if (n.fn == 2) { f.port = k; to_pred(f, n, 0); } else to_pred(f, n, k);
            cont = true;
          }
          break;
        case NPT_LSTM: {                          // LSTM gate combination; cache per key: [pre-activations | cells | output]
          const int H = n.out_dim / 2;
          long long key = key_of(C, f.node, f.slot, f.it, f.u, n.U_in);
          if (key < 0) return;
          if (f.rows != 1) { fail(C, ST_OVERFLOW, f.node, f.rows); return; }
          float* base = n.jbuf + key * n.jstride;
          float* cells = base + n.in_dim;
          if (f.dir == FWD) {
            if (f.aport == 0) warp_copy(base, n.in_dim, f, 1, n.in_dim, lane);
            else warp_copy(cells, n.out_dim, f, 1, n.out_dim, lane);
            if (n.fn == 2) { if (!join_arrive(&n.jcnt[key], 2, lane)) break; }       // the other port's message is still under way
            else __syncwarp();
            float* outp = cells + n.out_dim;
            for (int j = lane; j < H; j += 32) {
              float cj, oj;
              if (n.fn == 1) { cj = sigm(base[j]) * tanhf(base[2 * H + j]); oj = sigm(base[H + j]); }
              else {
                cj = sigm(base[j]) * tanhf(base[4 * H + j]) + sigm(base[H + j]) * cells[j] + sigm(base[2 * H + j]) * cells[H + j];
                oj = sigm(base[3 * H + j]);
              }
              outp[j] = emit_round(oj * tanhf(cj));
              outp[H + j] = emit_round(cj);
            }
            __syncwarp();
            f.p = outp; f.nsum = 1; f.sstride = 0; f.dim = n.out_dim; f.ld = n.out_dim;
            to_succ(f, n, 0);
            cont = true;
          } else if (f.iter == 0) {
            // gradients in place: d pre-activations over the cached pre-activations, [dcL; dcR] over the cached cells
            for (int j = lane; j < H; j += 32) {
              const float gh = ld_payload(f.p, f.nsum, f.sstride, j), gc = ld_payload(f.p, f.nsum, f.sstride, H + j);
              if (n.fn == 1) {
                const float i = sigm(base[j]), o = sigm(base[H + j]), u = tanhf(base[2 * H + j]);
                const float tc = tanhf(i * u), d = gc + gh * o * (1.f - tc * tc);
                base[j] = emit_round(d * u * i * (1.f - i));
                base[H + j] = emit_round(gh * tc * o * (1.f - o));
                base[2 * H + j] = emit_round(d * i * (1.f - u * u));
              } else {
                const float i = sigm(base[j]), fl = sigm(base[H + j]), fr = sigm(base[2 * H + j]),
                            o = sigm(base[3 * H + j]), u = tanhf(base[4 * H + j]);
                const float cl = cells[j], cr = cells[H + j];
                const float tc = tanhf(i * u + fl * cl + fr * cr), d = gc + gh * o * (1.f - tc * tc);
                base[j] = emit_round(d * u * i * (1.f - i));
                base[H + j] = emit_round(d * cl * fl * (1.f - fl));
                base[2 * H + j] = emit_round(d * cr * fr * (1.f - fr));
                base[3 * H + j] = emit_round(gh * tc * o * (1.f - o));
                base[4 * H + j] = emit_round(d * i * (1.f - u * u));
                cells[j] = emit_round(d * fl);
                cells[H + j] = emit_round(d * fr);
              }
            }
            __syncwarp();
            if (n.fn == 2) {                      // second message: the cells' gradient to port 1
              Frame c = f; c.iter = 1;
              if (!pool_offer(C, Q, c, lane)) { if (sp >= WALK_STACK) { fail(C, ST_OVERFLOW, f.node, sp); return; }
                                             if (lane == 0) stack[sp] = c; sp++; __syncwarp(); }
            }
            f.p = base; f.nsum = 1; f.sstride = 0; f.dim = n.in_dim; f.ld = n.in_dim;
            to_pred(f, n, 0);
            cont = true;
          } else {
            f.p = cells; f.nsum = 1; f.sstride = 0; f.dim = n.out_dim; f.ld = n.out_dim;
            to_pred(f, n, 1);
            cont = true;
          }
        } break;
        case SPLIT:                               // inverse of Concat: successor k gets the columns [k w, (k + 1) w)
          if (f.dir == FWD) {
            const int k = f.iter;
            if (k + 1 < n.fn_arg) { Frame c = f; c.iter = k + 1;
              if (!pool_offer(C, Q, c, lane)) { if (sp >= WALK_STACK) { fail(C, ST_OVERFLOW, f.node, sp); return; }
                                             if (lane == 0) stack[sp] = c; sp++; __syncwarp(); } }
            f.p = f.p ? f.p + k * n.out_dim : nullptr; f.dim = n.out_dim;
            to_succ(f, n, k);
            cont = true;
          } else {                                // the parts' gradients meet again, keyed on the state
            const int port = f.aport;
            long long key = key_of(C, f.node, f.slot, f.it, f.u, n.U_in);
            if (key < 0) return;
            if ((unsigned)port >= (unsigned)n.fn_arg || f.rows > n.rows_in) { fail(C, ST_OVERFLOW, f.node, port); return; }
            float* base = n.jbuf + key * n.jstride;
            warp_copy(base + port * n.out_dim, n.in_dim, f, f.rows, n.out_dim, lane);
            if (join_arrive(&n.jcnt[key], n.fn_arg, lane)) {
              f.p = base; f.nsum = 1; f.dim = n.in_dim; f.ld = n.in_dim;
              to_pred(f, n, 0);
              cont = true;
            }
          }
          break;
        case GROUP:
          if (f.dir == FWD) {
            int gkey = 0, member = 0, count = 1;
            const long long ebase = f.ebase;
            if (n.fn == 1) { int c = I.etype[ebase + f.u]; gkey = c; member = I.rank_type[ebase + f.u];
                             const long long* to = I.type_off + (long long)f.inst * I.NT + c; count = (int)(to[1] - to[0]); }
            else if (n.fn == 2) { int v = I.edst[ebase + f.u]; gkey = v; member = I.rank_in[ebase + f.u];
                                  count = (int)(I.in_off[f.ibase + v + 1] - I.in_off[f.ibase + v]); }
            else { gkey = 0; member = f.u; count = (int)(I.offsets[f.inst + 1] - f.ibase); }
            long long key = key_of(C, f.node, f.slot, f.it, gkey, n.U_out);
            if (key < 0) return;
            if (member >= n.rows_out || count > n.rows_out) { fail(C, ST_OVERFLOW, f.node, member); return; }
            float* base = n.jbuf + key * n.jstride;
            warp_copy(base + (size_t)member * n.jld, n.jld, f, 1, n.in_dim, lane);
            if (join_arrive(&n.jcnt[key], count, lane)) {
              f.u = gkey; f.rows = count; f.p = base; f.nsum = 1; f.ld = n.jld; f.dim = n.in_dim;
              to_succ(f, n, 0);
              cont = true;
            }
          } else {
            const int i = f.iter * f.nparts + f.part;       // this walker's share of the rows
            if (i >= f.rows) break;
            if (i + f.nparts < f.rows) { Frame c = f; c.iter = f.iter + 1;
              if (!pool_offer(C, Q, c, lane)) { if (sp >= WALK_STACK) { fail(C, ST_OVERFLOW, f.node, sp); return; }
                                             if (lane == 0) stack[sp] = c; sp++; __syncwarp(); } }
            f.nparts = 1; f.part = 0;
            const long long ebase = f.ebase;
            int mu;
            if (n.fn == 1) mu = I.type_list[I.type_off[(long long)f.inst * I.NT + f.u] + i];
            else if (n.fn == 2) mu = I.in_list[I.in_off[f.ibase + f.u] + i];
            else mu = i;
            (void)ebase;
            f.p = f.p ? f.p + (size_t)i * f.ld : nullptr; f.rows = 1; f.u = mu;
            to_pred(f, n, 0);
            cont = true;
          }
          break;
        case UNGROUP:
          if (f.dir == FWD) {
            const int i = f.iter * f.nparts + f.part;       // this walker's share of the rows
            if (i >= f.rows) break;
            if (i + f.nparts < f.rows) { Frame c = f; c.iter = f.iter + 1;
              if (!pool_offer(C, Q, c, lane)) { if (sp >= WALK_STACK) { fail(C, ST_OVERFLOW, f.node, sp); return; }
                                             if (lane == 0) stack[sp] = c; sp++; __syncwarp(); } }
            f.nparts = 1; f.part = 0;
            int mu = n.fn == 2 ? I.type_list[I.type_off[(long long)f.inst * I.NT + f.u] + i] : n.fn == 3 ? I.leaf_ids[I.leaf_off[f.inst] + i] : i;
            f.p = f.p ? f.p + (size_t)i * f.ld : nullptr; f.rows = 1; f.u = mu;
            to_succ(f, n, 0);
            cont = true;
          } else {
            int gkey, row, expected;
            if (n.fn == 2) { const long long ebase = f.ebase; gkey = I.etype[ebase + f.u]; row = I.rank_type[ebase + f.u];
                             const long long* to = I.type_off + (long long)f.inst * I.NT + gkey; expected = (int)(to[1] - to[0]); }
            else if (n.fn == 3) {                   // the leaf's rank among the leaves of its tree (their positions ascend)
              const long long l0 = I.leaf_off[f.inst];
              expected = (int)(I.leaf_off[f.inst + 1] - l0);
              int lo = 0, hi = expected - 1;
              while (lo < hi) { const int mid = (lo + hi) >> 1; if (I.leaf_ids[l0 + mid] < f.u) lo = mid + 1; else hi = mid; }
              if (expected < 1 || I.leaf_ids[l0 + lo] != f.u) { fail(C, ST_OVERFLOW, f.node, f.u); return; }
              gkey = 0; row = lo;
            }
            else { gkey = 0; row = f.u; expected = (int)(I.offsets[f.inst + 1] - f.ibase); }
            long long key = key_of(C, f.node, f.slot, f.it, gkey, n.U_in);
            if (key < 0) return;
            if (row >= n.rows_in) { fail(C, ST_OVERFLOW, f.node, row); return; }
            float* base = n.jbuf + key * n.jstride;
            warp_copy(base + (size_t)row * n.in_dim, n.in_dim, f, 1, n.in_dim, lane);
            if (join_arrive(&n.jcnt[key], expected, lane)) {
              f.u = gkey; f.rows = expected; f.p = base; f.nsum = 1; f.ld = n.in_dim; f.dim = n.in_dim;
              to_pred(f, n, 0);
              cont = true;
            }
          }
          break;
        case FLATMAP: {
          if (f.dir == FWD) {
            const long long* oo = I.out_off + f.ibase + f.u;
            int deg = (int)(oo[1] - oo[0]);
            int i = f.iter;
            if (deg > 0) {
              if (i + 1 < deg) { Frame c = f; c.iter = i + 1;
              if (!pool_offer(C, Q, c, lane)) { if (sp >= WALK_STACK) { fail(C, ST_OVERFLOW, f.node, sp); return; }
                                             if (lane == 0) stack[sp] = c; sp++; __syncwarp(); } }
              f.u = I.out_list[oo[0] + i];
              to_succ(f, n, 0);
              cont = true;
            }
          } else {
            const long long ebase = f.ebase;
            int v = I.esrc[ebase + f.u], member = I.rank_out[ebase + f.u];
            int deg = (int)(I.out_off[f.ibase + v + 1] - I.out_off[f.ibase + v]);
            long long key = key_of(C, f.node, f.slot, f.it, v, n.U_in);
            if (key < 0) return;
            const int maxdeg = (int)(n.jstride / n.in_dim) - 1;
            if (member >= maxdeg || deg > maxdeg) { fail(C, ST_OVERFLOW, f.node, member); return; }
            float* base = n.jbuf + key * n.jstride;
            warp_copy(base + (size_t)member * n.in_dim, n.in_dim, f, 1, n.in_dim, lane);
            if (join_arrive(&n.jcnt[key], deg, lane)) {
              f.u = v; f.rows = 1; f.p = base; f.nsum = deg; f.sstride = n.in_dim;   // summed in edge order when read
              f.ld = n.in_dim; f.dim = n.in_dim;
              to_pred(f, n, 0);
              cont = true;
            }
          }
        } break;
        case NPT_SUMROWS: {
          long long key = key_of(C, f.node, f.slot, f.it, f.u, n.U_in);
          if (key < 0) return;
          if (f.dir == FWD) {
            float* out = n.jbuf + key * n.jstride;
            for (int i = lane; i < n.in_dim; i += 32) {
              float s = 0.f;
              for (int r = 0; r < f.rows; r++) s += f.p ? ld_payload(f.p, f.nsum, f.sstride, (size_t)r * f.ld + i) : 0.f;   // row order
              out[i] = emit_round(s);
            }
            if (lane == 0 && !(f.flags & HDR_EVAL)) n.rowcnt[key] = f.rows;
            __syncwarp();
            f.rows = 1; f.p = out; f.nsum = 1; f.ld = n.in_dim; f.dim = n.in_dim;
            to_succ(f, n, 0);
          } else {
            int rows = *(volatile int*)&n.rowcnt[key];
            __syncwarp();
            if (lane == 0) n.rowcnt[key] = 0;
            f.rows = rows; f.ld = 0;         // the same gradient row for every summed row
            to_pred(f, n, 0);
          }
          cont = true;
        } break;
        default:
          fail(C, ST_OVERFLOW, f.node, n.type);
          return;
      }
    }
    if ((C.tune & 8) && lane == 0) { atomicAdd(&C.g->walk_cycles[ptype], (unsigned long long)(clock64() - tstep)); atomicAdd(&C.g->walk_steps[ptype], 1ull); }
    if (!cont) {
      if (sp > 0) { __syncwarp(); f = stack[--sp]; __syncwarp(); }
      else have = false;
    }
  }
}

__device__ __forceinline__ void flush_acc(const Ctx& C, WalkAcc& a, int lane) {
  if (lane == 0 && a.msgs) {
    atomicAdd(&C.g->node_messages, a.msgs);
    atomicAdd(&C.g->route_hash, a.hash);
  }
  a.msgs = 0; a.hash = 0;
}

// A warp that has walked its own frames helps with what the others offered, until nothing is outstanding.
__device__ __noinline__ void pool_steal(const Ctx& C, WalkPool* Q, Frame* stack, WalkAcc& acc) {
  const int lane = threadIdx.x & 31;
  unsigned idle = 0;
  for (;;) {
    int got = 0;
    unsigned h = 0;
    if (lane == 0) {
      h = *(volatile unsigned*)&Q->head;
      unsigned t = *(volatile unsigned*)&Q->tail;
      while (h != t) {
        const unsigned old = atomicCAS(&Q->head, h, h + 1u);
        if (old == h) { got = 1; break; }
        h = old;
        t = *(volatile unsigned*)&Q->tail;
      }
    }
    got = __shfl_sync(0xffffffffu, got, 0);
    if (got) {
      h = __shfl_sync(0xffffffffu, h, 0);
      const unsigned idx = h % POOL;
      unsigned lost = 0;
      if (lane == 0) {
        int spins = 0;
        while (*(volatile unsigned*)&Q->ready[idx] != h + 1u && ++spins < (1 << 20)) {}
        if (*(volatile unsigned*)&Q->ready[idx] != h + 1u) { fail(C, ST_TIMEOUT, -6, (int)idx); lost = 1; }   // never published
      }
      if (warp_uniform(lost)) { if (lane == 0) atomicSub(&Q->outstanding, 1); break; }
      __syncwarp();
      Frame f = Q->f[idx];
      __syncwarp();
      if (lane == 0) *(volatile unsigned*)&Q->ready[idx] = 0u;
      walk(C, f, stack, acc, Q);
      __syncwarp();
      if (lane == 0) atomicSub(&Q->outstanding, 1);
      idle = 0;
    } else {
      int left = 0;
      if (lane == 0) left = *(volatile int*)&Q->outstanding;
      if ((int)warp_uniform((unsigned)left) <= 0) break;
      if ((++idle & 1023u) == 0) {
        if (aborted_warp(C)) break;
        if (idle > (1u << 26)) { fail(C, ST_TIMEOUT, -4, 0); break; }
      }
      __nanosleep(20);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// tile arithmetic: lanes stride over the input dimension (column i = lane + 32 j)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float act_fwd(int a, float v) {
  switch (a) {
    case 1: return v > 0.f ? v : 0.f;
    case 2: return tanhf(v);
    case 3: return 1.f / (1.f + expf(-v));
    default: return v;
  }
}
__device__ __forceinline__ float act_grad(int a, float y) {
  switch (a) {
    case 1: return y > 0.f ? 1.f : 0.f;
    case 2: return 1.f - y * y;
    case 3: return y * (1.f - y);
    default: return 1.f;
  }
}

// Shared-memory layout of a tile's operands: weight / accumulator rows have a leading dimension of a multiple of 4 floats
// (ldw), staged input rows one that is 4 (mod 8) floats (ldx, so that a warp whose lanes read 16 bytes each from 32
// different rows meets no bank conflict), gradient rows D a multiple of 4 (ldd); all padding is kept at zero.
__host__ __device__ __forceinline__ int pad_ldw(int in) { return (in + 3) & ~3; }
__host__ __device__ __forceinline__ int pad_ldx(int in) { int l = (in + 3) & ~3; while ((l & 7) != 4) l += 4; return l; }
__host__ __device__ __forceinline__ int xwt_scratch_floats(int rb) { return WARPS * 32 * rb; }     // partial sums of the k-slices

// out[b][r] = sum_k X[b][k] * W[r][k]  for b < nb, r < R (whole CTA; ends with a block barrier).  Lanes own batch rows:
// warp (g, s) takes the 32 batch rows of group g and the k-slice s, keeps RB outputs per lane in registers, reads its row
// 16 bytes at a time and the weight rows as broadcasts; the slices' partial sums meet in `scratch` and are added in
// slice order.
template <int RB>
__device__ __forceinline__ void xwT_pass(const float* __restrict__ Xs, int ldx, int nb, const float* __restrict__ Ws, int ldw, int r0, int R,
                                         int K4, float* __restrict__ scratch, int G, int S) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = warp % G, s = warp / G;
  const int b = g * 32 + lane;
  const int k4_per = (K4 + S - 1) / S, k4a = s * k4_per, k4b = min(K4, k4a + k4_per);
  float acc[RB];
#pragma unroll
  for (int q = 0; q < RB; q++) acc[q] = 0.f;
  const float4* xrow = reinterpret_cast<const float4*>(Xs + (size_t)min(b, nb - 1) * ldx);
#pragma unroll 2
  for (int k4 = k4a; k4 < k4b; k4++) {
    const float4 x = xrow[k4];
#pragma unroll
    for (int q = 0; q < RB; q++) {
      const float4 w = *reinterpret_cast<const float4*>(Ws + (size_t)min(r0 + q, R - 1) * ldw + 4 * k4);
      acc[q] = fmaf(x.x, w.x, acc[q]); acc[q] = fmaf(x.y, w.y, acc[q]); acc[q] = fmaf(x.z, w.z, acc[q]); acc[q] = fmaf(x.w, w.w, acc[q]);
    }
  }
  if (b < nb) {
#pragma unroll
    for (int q = 0; q < RB; q++) scratch[((size_t)s * 32 * G + b) * RB + q] = acc[q];
  }
}
__device__ __noinline__ void tile_xwT(const float* __restrict__ Xs, int ldx, int nb, const float* __restrict__ Ws, int ldw, int R,
                                      int in_dim, float* __restrict__ out, int ldo, float* __restrict__ scratch, int rb_max) {
  const int G = nb > 32 ? 2 : 1, S = WARPS / G, K4 = (in_dim + 3) >> 2;
  for (int r0 = 0; r0 < R; r0 += rb_max) {                 // up to rb_max (8 or 16) output rows per pass over the staged inputs
    const int rb = min(rb_max, R - r0), RBs = rb > 12 ? 16 : rb > 10 ? 12 : rb > 8 ? 10 : rb > 4 ? 8 : 4;
    if (RBs == 16) xwT_pass<16>(Xs, ldx, nb, Ws, ldw, r0, R, K4, scratch, G, S);
    else if (RBs == 12) xwT_pass<12>(Xs, ldx, nb, Ws, ldw, r0, R, K4, scratch, G, S);
    else if (RBs == 10) xwT_pass<10>(Xs, ldx, nb, Ws, ldw, r0, R, K4, scratch, G, S);
    else if (RBs == 8) xwT_pass<8>(Xs, ldx, nb, Ws, ldw, r0, R, K4, scratch, G, S);
    else xwT_pass<4>(Xs, ldx, nb, Ws, ldw, r0, R, K4, scratch, G, S);
    __syncthreads();
    for (int idx = threadIdx.x; idx < nb * rb; idx += THREADS) {
      const int b = idx / rb, q = idx - b * rb;
      float v = 0.f;
      for (int s = 0; s < S; s++) v += scratch[((size_t)s * 32 * G + b) * RBs + q];
      out[b * ldo + r0 + q] = v;
    }
    __syncthreads();
  }
}

// dx[b][i] = sum_r D[b][r] * W[r][i], written to dst (device memory, ld = in_dim).  The gradient rows are read four
// outputs at a time as 16-byte broadcasts (their stride ldd is a multiple of four and the padding beyond R is zero) and
// the loop carries no predicate: weight rows beyond R, columns beyond in_dim and batch rows beyond nb are read from
// whatever follows in shared memory, multiplied by zero or never stored.  INVARIANT this relies on: what follows Ws in
// the tile's carve-up (accumulators, biases, staging rows; all zero-filled at start) holds finite numbers.  A run whose
// accumulators have overflowed to Inf / NaN has diverged already (its parameters are Inf / NaN after the next update),
// so the 0 x Inf = NaN this could add to an input gradient changes nothing that was still meaningful.
template <int J, bool ACCUM = false>
__device__ __noinline__ void tile_dW(const float* __restrict__ Ds, int ldd, int nb, const float* __restrict__ Ws, int ldw, int R,
                        int in_dim, float* __restrict__ dst) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int R4 = (R + 3) >> 2, ld4 = ldd >> 2;
  for (int b0 = warp * 4; b0 < nb; b0 += WARPS * 4) {
    float acc[4][J];
#pragma unroll
    for (int m = 0; m < 4; m++)
#pragma unroll
      for (int j = 0; j < J; j++) acc[m][j] = 0.f;
    const float4* dp = reinterpret_cast<const float4*>(Ds + (size_t)b0 * ldd);
    const float* wp = Ws + lane;
    for (int c = 0; c < R4; c++, wp += 4 * ldw) {
      float4 d[4];
#pragma unroll
      for (int m = 0; m < 4; m++) d[m] = dp[m * ld4 + c];
#pragma unroll
      for (int j = 0; j < J; j++) {
        const float w0 = wp[32 * j], w1 = wp[ldw + 32 * j], w2 = wp[2 * ldw + 32 * j], w3 = wp[3 * ldw + 32 * j];
#pragma unroll
        for (int m = 0; m < 4; m++) {
          acc[m][j] = fmaf(d[m].x, w0, acc[m][j]); acc[m][j] = fmaf(d[m].y, w1, acc[m][j]);
          acc[m][j] = fmaf(d[m].z, w2, acc[m][j]); acc[m][j] = fmaf(d[m].w, w3, acc[m][j]);
        }
      }
    }
#pragma unroll
    for (int m = 0; m < 4; m++)
      if (b0 + m < nb)
#pragma unroll
        for (int j = 0; j < J; j++) {
          const int i = lane + 32 * j;
          if (i < in_dim) {
            float* o = dst + (size_t)(b0 + m) * in_dim + i;
            *o = ACCUM ? *o + acc[m][j] : acc[m][j];
          }
        }
  }
}

// dst[b][i] = (i < nbase ? base[b][i] : 0) + sum_r D1[b][r] * W1[r][i] + sum_r D2[b][r] * W2[r][i]: the second backward
// stage of the GRU cell in one pass with one store per element (dst and base in device memory, ld = in_dim).
template <int J>
__device__ __noinline__ void tile_dW2(const float* __restrict__ D1, const float* __restrict__ D2, int ldd, int nb,
                                      const float* __restrict__ W1, const float* __restrict__ W2, int ldw, int R, int in_dim,
                                      const float* __restrict__ base, int nbase, float* __restrict__ dst) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b0 = warp * 4; b0 < nb; b0 += WARPS * 4) {
    float acc[4][J];
#pragma unroll
    for (int m = 0; m < 4; m++)
#pragma unroll
      for (int j = 0; j < J; j++) {
        const int i = lane + 32 * j;
        acc[m][j] = (b0 + m < nb && i < nbase) ? __ldcg(base + (size_t)(b0 + m) * in_dim + i) : 0.f;
      }
#pragma unroll
    for (int pass = 0; pass < 2; pass++) {
      const float* __restrict__ Ds = pass ? D2 : D1;
      const float* __restrict__ Ws = pass ? W2 : W1;
      for (int r = 0; r < R; r++) {
        float d[4];
#pragma unroll
        for (int m = 0; m < 4; m++) d[m] = (b0 + m < nb) ? Ds[(b0 + m) * ldd + r] : 0.f;
#pragma unroll
        for (int j = 0; j < J; j++) {
          const int i = lane + 32 * j;
          const float w = i < in_dim ? Ws[r * ldw + i] : 0.f;
#pragma unroll
          for (int m = 0; m < 4; m++) acc[m][j] = fmaf(d[m], w, acc[m][j]);
        }
      }
    }
#pragma unroll
    for (int m = 0; m < 4; m++)
      if (b0 + m < nb)
#pragma unroll
        for (int j = 0; j < J; j++) {
          const int i = lane + 32 * j;
          if (i < in_dim) dst[(size_t)(b0 + m) * in_dim + i] = acc[m][j];
        }
  }
}

// A[r][k] += sum_b D[b][r] * X[b][k];  a warp's unit is 4 accumulator rows x 64 columns (a lane owns two), the four
// gradient entries of a batch row come as one 16-byte broadcast (D rows are padded to a multiple of 4 with zeros).
__device__ __noinline__ void tile_accum(const float* __restrict__ Ds, int ldd, int nb, const float* __restrict__ Xs, int ldx,
                                        float* __restrict__ As, int lda, int R, int in_dim) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int K = (in_dim + 1) & ~1;
  const int nrg = (R + 3) >> 2, ncg = (K + 63) >> 6;
  for (int unit = warp; unit < nrg * ncg; unit += WARPS) {
    const int r0 = (unit / ncg) * 4, k = (unit % ncg) * 64 + 2 * lane;
    if (k >= K) continue;
    float2 a[4];
#pragma unroll
    for (int q = 0; q < 4; q++) a[q] = r0 + q < R ? *reinterpret_cast<const float2*>(As + (size_t)(r0 + q) * lda + k) : make_float2(0.f, 0.f);
#pragma unroll 4
    for (int b = 0; b < nb; b++) {
      const float4 d = *reinterpret_cast<const float4*>(Ds + (size_t)b * ldd + r0);
      const float2 x = *reinterpret_cast<const float2*>(Xs + (size_t)b * ldx + k);
      a[0].x = fmaf(d.x, x.x, a[0].x); a[0].y = fmaf(d.x, x.y, a[0].y);
      a[1].x = fmaf(d.y, x.x, a[1].x); a[1].y = fmaf(d.y, x.y, a[1].y);
      a[2].x = fmaf(d.z, x.x, a[2].x); a[2].y = fmaf(d.z, x.y, a[2].y);
      a[3].x = fmaf(d.w, x.x, a[3].x); a[3].y = fmaf(d.w, x.y, a[3].y);
    }
#pragma unroll
    for (int q = 0; q < 4; q++) if (r0 + q < R) *reinterpret_cast<float2*>(As + (size_t)(r0 + q) * lda + k) = a[q];
  }
}

#define AMP_DISPATCH_J(Jv, CALL)                                  \
  switch (Jv) {                                                   \
    case 4: { constexpr int J = 4; CALL; } break;                 \
    case 7: { constexpr int J = 7; CALL; } break;                 \
    case 10: { constexpr int J = 10; CALL; } break;               \
    case 16: { constexpr int J = 16; CALL; } break;               \
    case 25: { constexpr int J = 25; CALL; } break;               \
    default: { constexpr int J = 32; CALL; } break;               \
  }

// ------------------------------------------------------------------------------------------------
// PPT tile: batch bookkeeping in shared memory
// ------------------------------------------------------------------------------------------------
struct LeaderState {
  unsigned head[2], sched_w, batch_w;
  int n_acc, version, log_n;
  unsigned long long n_updates, n_grads_applied, msgs, batches, batch_rows;
};

struct TileShared : BatchCtx {
  LeaderState ls;
  int ok;
  unsigned tail_snap[2];
  unsigned long long stale_hist[64];
  int max_stale;
  unsigned long long phase[16];
  unsigned long long step[16];
  long long step_t;
  unsigned long long mbar;             // transaction barrier of the bulk copies that stage a batch's input rows
  int mylist[MAX_BATCH_ROWS], mycount; // embedding node: the batch rows this tile handles
  unsigned mbar_parity;
  Frame stack[WARPS][WALK_STACK];
  WalkPool pool;
};
// Scheduler CTA: a batch formed by warp 0 waits here for warp 1, which assembles and publishes its context while warp 0
// polls for the next one.  full = batch number + 1 while occupied (shared memory, written behind a block-level fence).
struct SchedSlot {
  BatchDesc desc;
  int ver_form;
  unsigned full;
  int pad[2];
  Hdr hdr[MAX_BATCH_MSGS];
};
static_assert(2 * sizeof(SchedSlot) <= 2048 * sizeof(float), "the launch reserves 2048 floats of dynamic shared memory at least");
#define AMP_STEP(k) do { if (threadIdx.x == 0) { const long long n_ = clock64(); S.step[k] += (unsigned long long)(n_ - S.step_t); S.step_t = n_; } } while (0)

__device__ __forceinline__ int node_muf(const Ctx& C, const DevPPT& P) {
  return P.muf_override > 0 ? P.muf_override : C.muf;
}

// Inclusive prefix sums over 64 values held two per lane (v[0]: index lane, v[1]: index lane + 32).
__device__ __forceinline__ void scan64(int (&v)[2], const int lane) {
#pragma unroll
  for (int j = 0; j < 2; j++)
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, v[j], o); if (lane >= o) v[j] += t; }
  v[1] += __shfl_sync(0xffffffffu, v[0], 31);
}
__device__ __forceinline__ unsigned long long ballot64(const bool p0, const bool p1) {
  return (unsigned long long)__ballot_sync(0xffffffffu, p0) | ((unsigned long long)__ballot_sync(0xffffffffu, p1) << 32);
}

// Warp 0 of the leader: take up to 64 candidate messages (two ring slots per lane, in processing order: candidate
// lane and candidate lane + 32), cut the batch at the row capacity and at the message that triggers an update (Sec. 3),
// publish it.  Returns the number of messages taken.
__device__ __noinline__ int form_batch(const Ctx& C, DevPPT& P, TileShared& S, int dir, const unsigned (&slot)[2], int ncand,
                                       SchedSlot* q = nullptr) {
  const int lane = threadIdx.x & 31;
  Ring& R = P.ring[dir];
  Hdr h[2];
  int cum[2];
#pragma unroll
  for (int j = 0; j < 2; j++) {
    h[j] = Hdr{0, 0, 0, 0, 0, 0, 0, 0};
    if (lane + 32 * j < ncand) {
      const int4* e = reinterpret_cast<const int4*>(&R.e[slot[j]]);
      int4 a = __ldcg(e), b = __ldcg(e + 1);
      h[j].inst = a.x; h[j].seq = a.y; h[j].slot = a.z; h[j].it = a.w; h[j].u = b.x; h[j].port = b.y; h[j].rows = b.z; h[j].flags = b.w;
    }
    cum[j] = lane + 32 * j < ncand ? (h[j].rows > 0 ? h[j].rows : 1) : 0;
  }
  const int rows0 = cum[0];
  scan64(cum, lane);
  // a batch is all training or all forward-only messages (concurrent inference): cut where the flag changes
  const int eval0 = __shfl_sync(0xffffffffu, (int)((h[0].flags & HDR_EVAL) != 0), 0);
  const bool ok0 = lane < ncand && cum[0] <= P.BM && (int)((h[0].flags & HDR_EVAL) != 0) == eval0,
             ok1 = lane + 32 < ncand && cum[1] <= P.BM && (int)((h[1].flags & HDR_EVAL) != 0) == eval0;
  const unsigned long long okm = ballot64(ok0, ok1);
  int take = okm == ~0ull ? 64 : __ffsll((long long)~okm) - 1;
  if (take == 0) { fail(C, ST_OVERFLOW, P.node, rows0); return 0; }     // a single message larger than a batch
  bool upd = false;
  if (dir == BWD && !eval0) {
    const int muf = node_muf(C, P);
    const unsigned long long tm = ballot64(ok0 && lane < take && S.ls.n_acc + cum[0] >= muf,
                                           ok1 && lane + 32 < take && S.ls.n_acc + cum[1] >= muf);
    if (tm) { take = __ffsll((long long)tm); upd = true; }
  }
  const int t0v = __shfl_sync(0xffffffffu, cum[0], (take - 1) & 31), t1v = __shfl_sync(0xffffffffu, cum[1], (take - 1) & 31);
  const int total = take > 32 ? t1v : t0v;
#pragma unroll
  for (int j = 0; j < 2; j++) {
    const int i = lane + 32 * j;
    if (i >= take) continue;
    P.sched[(S.ls.sched_w + i) & P.sched_mask] = slot[j];
    if (q) q->hdr[i] = h[j];                           // the scheduler CTA assembles the batch context from its own copy
    else if (!C.det) {
      int4* b = reinterpret_cast<int4*>(&P.bhdr[(S.ls.batch_w & (BATCH_BLOCKS - 1)) * MAX_BATCH_MSGS + i]);
      b[0] = make_int4(h[j].inst, h[j].seq, h[j].slot, h[j].it);
      b[1] = make_int4(h[j].u, h[j].port, h[j].rows, h[j].flags);
    }
    if (!eval0) {
      long long key = key_of(C, P.node, h[j].slot, h[j].it, h[j].u, P.U);
      if (key >= 0) {
        if (dir == FWD) P.vcache[key] = S.ls.version;
        else if (!q) {                        // a scheduler CTA accounts staleness after it has published the batch
          int s = S.ls.version - P.vcache[key];
          if (s < 0) s = 0;
          atomicAdd(&S.stale_hist[s > 63 ? 63 : s], 1ull);
          atomicMax(&S.max_stale, s);
        }
      }
    }
  }
  __syncwarp();
  if (lane == 0) {
    BatchDesc d;
    d.sched_start = S.ls.sched_w; d.count = take; d.dir = dir; d.flags = upd ? BATCH_UPDATE : 0;
    d.n_upd = upd ? S.ls.n_acc + total : 0; d.nrows = total; d.upd_t = upd ? (int)S.ls.n_updates + 1 : 0; d.pad1 = 0;
    if (q) {                                              // a scheduler CTA: hand the batch to the warp that assembles and publishes
      q->desc = d; q->ver_form = S.ls.version;            // its context before the bookkeeping below (that warp is waiting)
      __threadfence_block();
      *reinterpret_cast<volatile unsigned*>(&q->full) = S.ls.batch_w + 1u;
    } else { P.batches[S.ls.batch_w & P.batch_mask] = d; __threadfence(); st_rel(P.batch_pub, S.ls.batch_w + 1u); }
    S.ls.batch_w++;
    S.ls.sched_w += take;
    LeaderState& st = S.ls;
    st.msgs += take; st.batches++; st.batch_rows += total;
    if (upd) {
      if (st.log_n < P.update_log_cap) P.update_log[st.log_n] = d.n_upd;
      st.log_n++; st.n_updates++; st.n_grads_applied += d.n_upd;
      S.ls.n_acc = 0; S.ls.version++;
    } else if (dir == BWD && !eval0) S.ls.n_acc += total;
  }
  __syncwarp();
  return take;
}

__device__ void publish_marker(const Ctx& C, DevPPT& P, TileShared& S, int flags, SchedSlot* q = nullptr) {   // one thread
  BatchDesc d;
  d.sched_start = S.ls.sched_w; d.count = 0; d.dir = BWD; d.flags = flags; d.n_upd = 0; d.nrows = 0; d.upd_t = d.pad1 = 0;
  if ((flags & BATCH_TERMINATE) && S.ls.n_acc > 0 && !C.eval) {      // epoch-end flush of the leftover gradients
    d.flags |= BATCH_UPDATE; d.n_upd = S.ls.n_acc; d.upd_t = (int)S.ls.n_updates + 1;
    LeaderState& st = S.ls;
    if (st.log_n < P.update_log_cap) P.update_log[st.log_n] = d.n_upd;
    st.log_n++; st.n_updates++; st.n_grads_applied += d.n_upd;
    S.ls.n_acc = 0; S.ls.version++;
  }
  if (q) { q->desc = d; q->ver_form = S.ls.version; __threadfence_block(); *reinterpret_cast<volatile unsigned*>(&q->full) = S.ls.batch_w + 1u; }
  else { P.batches[S.ls.batch_w & P.batch_mask] = d; __threadfence(); st_rel(P.batch_pub, S.ls.batch_w + 1u); }
  S.ls.batch_w++;
}

// Asynchronous mode, warp 0 of the leader: whatever is pending, backward first (App. A).
// gate (optional): a counter read together with the ring polls; the call does nothing and returns false with *open = 0
// while gate + 1 < gate_min (the scheduler's look-ahead limit).
__device__ __noinline__ bool leader_try_schedule(const Ctx& C, DevPPT& P, TileShared& S, const unsigned* gate = nullptr,
                                                 unsigned gate_min = 0, bool* open = nullptr, SchedSlot* q = nullptr) {
  const int lane = threadIdx.x & 31;
  unsigned slot[2][2];
  bool mready[2][2];
  unsigned gv = 0;
  if (gate && lane == 0) gv = ld_rlx(gate);
#pragma unroll
  for (int dir = 0; dir < 2; dir++)               // both rings are polled before either result is needed
#pragma unroll
    for (int j = 0; j < 2; j++) {
      const unsigned t = S.ls.head[dir] + lane + 32 * j;
      slot[dir][j] = t & P.ring[dir].mask;
      mready[dir][j] = ld_rlx(&P.ring[dir].seq[slot[dir][j]]) == t + 1u;
    }
  fence_acq();
  if (gate) {
    const bool go = warp_uniform(gv) + 1u >= gate_min;
    *open = go;
    if (!go) return false;
  }
  int nready[2];
#pragma unroll
  for (int dir = 0; dir < 2; dir++) {
    const unsigned long long m = ballot64(mready[dir][0], mready[dir][1]);
    nready[dir] = m == ~0ull ? 64 : __ffsll((long long)~m) - 1;
  }
  // Backward first (App. A), but a cycle costs the same whether the batch holds 2 messages or 64: a short backward
  // queue gives way to a longer forward queue and is taken once it has grown to half a batch, has caught up with the
  // forward queue, or the forward queue has run dry (max_active_keys bounds the forward supply, so it always does).
  const bool fwd_first = !(C.tune & 128) && nready[BWD] < MAX_BATCH_MSGS / 2 && nready[FWD] > nready[BWD];
  for (int k = 0; k < 2; k++) {
    const int dir = (k == 0) == fwd_first ? FWD : BWD;
    const int n = nready[dir];
    if (n == 0) continue;
    int take = dir == FWD ? form_batch(C, P, S, FWD, slot[FWD], n, q) : form_batch(C, P, S, BWD, slot[BWD], n, q);
    if (lane == 0) S.ls.head[dir] += take;
    __syncwarp();
    return true;
  }
  unsigned fin = 0;
  if (lane == 0) fin = ld_acq(&C.g->done);
  if (warp_uniform(fin)) {
    if (lane == 0) publish_marker(C, P, S, BATCH_TERMINATE, q);
    __syncwarp();
    return true;
  }
  return false;
}

// Deterministic mode, whole leader CTA: this round's inbox = tickets [head, tail) of each ring, sorted by
// (admission seq, it, u, port), backward ring first; cut into batches; then the end-of-round marker.
__device__ __noinline__ void leader_schedule_round(const Ctx& C, DevPPT& P, TileShared& S, unsigned long long t0) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (ld_acq(&C.g->done)) {
    if (tid == 0) publish_marker(C, P, S, BATCH_TERMINATE);
    __syncthreads();
    return;
  }
  for (int dir = BWD; dir >= FWD; dir--) {
    Ring& R = P.ring[dir];
    const unsigned head = S.ls.head[dir];
    const unsigned n = S.tail_snap[dir] - head;
    if (n == 0) { __syncthreads(); continue; }
    if (n > R.mask + 1u) { if (tid == 0) fail(C, ST_OVERFLOW, P.node, (int)n); __syncthreads(); return; }
    unsigned np2 = 1;
    while (np2 < n) np2 <<= 1;
    for (unsigned i = tid; i < np2; i += THREADS) {
      unsigned long long k = ~0ull;
      if (i < n) {
        const unsigned slot = (head + i) & R.mask;
        spin_until(C, t0, [&] { return ld_acq(&R.seq[slot]) == head + i + 1u; });
        const int4* e = reinterpret_cast<const int4*>(&R.e[slot]);
        int4 a = __ldcg(e), b = __ldcg(e + 1);
        k = ((unsigned long long)(a.y & 0xffffff) << 40) | ((unsigned long long)(a.w & 0xf) << 36) |
            ((unsigned long long)(b.x & 0x3fff) << 22) | ((unsigned long long)(b.y & 0x3) << 20) | (unsigned long long)i;
      }
      P.sortbuf[i] = k;
    }
    __syncthreads();
    for (unsigned k2 = 2; k2 <= np2; k2 <<= 1)
      for (unsigned j = k2 >> 1; j > 0; j >>= 1) {
        for (unsigned i = tid; i < np2; i += THREADS) {
          unsigned ixj = i ^ j;
          if (ixj > i) {
            unsigned long long a = P.sortbuf[i], b = P.sortbuf[ixj];
            bool asc = (i & k2) == 0;
            if ((a > b) == asc) { P.sortbuf[i] = b; P.sortbuf[ixj] = a; }
          }
        }
        __syncthreads();
      }
    if (warp == 0) {
      unsigned pos = 0;
      while (pos < n) {
        int nc = (int)min((unsigned)MAX_BATCH_MSGS, n - pos);
        unsigned slot[2] = {0, 0};
#pragma unroll
        for (int j = 0; j < 2; j++)
          if (lane + 32 * j < nc) slot[j] = (head + (unsigned)(P.sortbuf[pos + lane + 32 * j] & 0xfffffull)) & R.mask;
        int take = form_batch(C, P, S, dir, slot, nc);
        if (take <= 0) break;
        pos += take;
      }
      if (lane == 0) S.ls.head[dir] = head + n;
    }
    __syncthreads();
  }
  if (tid == 0) publish_marker(C, P, S, BATCH_END_ROUND);
  __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// PPT tile main loop
// ------------------------------------------------------------------------------------------------
// Copy the cached input rows of a batch into shared memory with several loads in flight per thread.
// rowptr[b] points at row b's `width` floats in device memory; V = 4, 2 or 1 floats per load.
template <int V>
__device__ __forceinline__ void stage_rows_v(float* __restrict__ Xs, int ldx, const float* const* rowptr, int nb, int width) {
  const int wv = width / V, total = nb * wv;
  for (int base = threadIdx.x; base < total; base += THREADS * 4) {
    float v[4][V];
#pragma unroll
    for (int k = 0; k < 4; k++) {
      const int idx = base + k * THREADS;
      if (idx < total) {
        const int b = idx / wv, c = idx - b * wv;
        const float* src = rowptr[b] + c * V;
        if (V == 4) { float4 t = __ldcg(reinterpret_cast<const float4*>(src)); v[k][0] = t.x; v[k][1] = t.y; v[k][2 % V] = t.z; v[k][3 % V] = t.w; }
        else if (V == 2) { float2 t = __ldcg(reinterpret_cast<const float2*>(src)); v[k][0] = t.x; v[k][1 % V] = t.y; }
        else v[k][0] = __ldcg(src);
      }
    }
#pragma unroll
    for (int k = 0; k < 4; k++) {
      const int idx = base + k * THREADS;
      if (idx < total) {
        const int b = idx / wv, c = idx - b * wv;
#pragma unroll
        for (int q = 0; q < V; q++) Xs[b * ldx + c * V + q] = v[k][q];
      }
    }
  }
}
// Bulk-copy staging (TMA, untiled): one cp.async.bulk per input row, issued by the row's thread, completion counted in
// bytes on a shared-memory transaction barrier that every thread then waits for (bounded).  Needs rows that start on 16
// bytes and are a multiple of 16 bytes long in device memory.  The proxy fence orders the issuing thread's view of the
// rows (written by other SMs with ordinary stores and acquired through the queues) before the asynchronous read.
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __noinline__ void stage_rows_bulk(const Ctx& C, TileShared& S, float* Xs, int ldx, const float* const* rowptr, int nb, int width,
                                             int node, unsigned long long t0) {
  const int tid = threadIdx.x;
  const unsigned bar = smem_u32(&S.mbar), parity = S.mbar_parity;
  if (tid == 0) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"((unsigned)(nb * width * 4)) : "memory");
  __syncthreads();
  if (tid < nb) {
    asm volatile("fence.proxy.async;" ::: "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(Xs + (size_t)tid * ldx)), "l"(rowptr[tid]), "r"((unsigned)(width * 4)), "r"(bar) : "memory");
  }
  unsigned done = 0, spins = 0;
  for (;;) {
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) break;
    if ((++spins & 1023u) == 0 && (aborted(C) || gtime() - t0 > C.timeout_ns)) {
      if (tid == 0) fail(C, ST_TIMEOUT, node, 7);
      for (unsigned extra = 0; extra < (1u << 16) && !done; extra++)      // copies already issued still land in this CTA's shared memory
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
      break;
    }
  }
  __syncthreads();
  if (tid == 0) S.mbar_parity = parity ^ 1u;
}
__device__ __noinline__ void stage_rows(float* Xs, int ldx, const float* const* rowptr, int nb, int width, int align_floats) {
  if ((width & 3) == 0 && (align_floats & 3) == 0) stage_rows_v<4>(Xs, ldx, rowptr, nb, width);
  else if ((width & 1) == 0 && (align_floats & 1) == 0) stage_rows_v<2>(Xs, ldx, rowptr, nb, width);
  else stage_rows_v<1>(Xs, ldx, rowptr, nb, width);
}

struct TileMem {           // carve-up of the dynamic shared memory of a tile (floats)
  float *Ws, *As, *bs, *Abs, *Xs, *Ds, *Ys, *XC, *scratch;
  int LW, LX, RP;          // leading dimensions: weight / accumulator rows, staged input rows, gradient rows
};

__device__ __forceinline__ const float* msg_x(const Ctx& C, const DevPPT& P, const Hdr& h, long long key) {
  if (P.xcache) return P.xcache + key * (long long)P.rows_max * P.xld;
  return C.inst.dense + (long long)h.inst * C.inst.dense_dim;         // fed directly by a dense-row source
}

__device__ __forceinline__ void write_leader_stats(DevPPT& P, TileShared& S) {      // whole CTA
  const int tid = threadIdx.x;
  if (tid < 64) P.stats->stale_hist[tid] = S.stale_hist[tid];
  if (tid == 0) {
    PPTStats& st = *P.stats;
    st.max_staleness = S.max_stale; st.log_n = S.ls.log_n; st.n_updates = S.ls.n_updates;
    st.n_grads_applied = S.ls.n_grads_applied; st.msgs = S.ls.msgs; st.batches = S.ls.batches; st.batch_rows = S.ls.batch_rows;
  }
}

__device__ __forceinline__ void init_leader_state(TileShared& S) {                 // whole CTA, before a barrier
  const int tid = threadIdx.x;
  if (tid == 0) {
    S.ls.head[0] = S.ls.head[1] = 0; S.ls.sched_w = S.ls.batch_w = 0; S.ls.n_acc = 0; S.ls.version = 0; S.max_stale = 0;
    S.ls.log_n = 0; S.ls.n_updates = S.ls.n_grads_applied = S.ls.msgs = S.ls.batches = S.ls.batch_rows = 0;
  }
  if (tid < 64) S.stale_hist[tid] = 0;
}

// Warp 0 of a CTA: descriptor, headers, keys, row offsets and row pointers of batch `batch` into shared memory.
// q: descriptor and headers are already in this CTA's shared memory (the scheduler CTA that has just formed the batch).
__device__ __noinline__ void load_batch_ctx(const Ctx& C, DevPPT& P, TileShared& S, const unsigned my_batch, const SchedSlot* q = nullptr) {
  const bool local = q != nullptr;
  const int lane = threadIdx.x & 31;
  const int in = P.in_dim;
  int4 d0, d1;
  if (local) { const int4* dp = reinterpret_cast<const int4*>(&q->desc); d0 = dp[0]; d1 = dp[1]; }
  else { const int4* dp = reinterpret_cast<const int4*>(&P.batches[my_batch & P.batch_mask]); d0 = __ldcg(dp); d1 = __ldcg(dp + 1); }
  const int cnt = d0.y, ddir = d0.z;
  Hdr h[2];
  int cum[2], rows[2];
#pragma unroll
  for (int j = 0; j < 2; j++) {                             // message lane + 32 j
    const int i = lane + 32 * j;
    int4 ha = make_int4(0, 0, 0, 0), hb = make_int4(0, 0, 0, 0);
    if (local) {
      if (i < cnt) { const int4* e = reinterpret_cast<const int4*>(&q->hdr[i]); ha = e[0]; hb = e[1]; }
    } else if (!C.det) {                                    // headers travel with the descriptor: load both at once
      const int4* e = reinterpret_cast<const int4*>(&P.bhdr[(my_batch & (BATCH_BLOCKS - 1)) * MAX_BATCH_MSGS + i]);
      ha = __ldcg(e); hb = __ldcg(e + 1);
    } else if (i < cnt) {
      const unsigned slot = P.sched[((unsigned)d0.x + i) & P.sched_mask];
      const int4* e = reinterpret_cast<const int4*>(&P.ring[ddir].e[slot]);
      ha = __ldcg(e); hb = __ldcg(e + 1);
    }
    h[j].inst = ha.x; h[j].seq = ha.y; h[j].slot = ha.z; h[j].it = ha.w; h[j].u = hb.x; h[j].port = hb.y; h[j].rows = hb.z; h[j].flags = hb.w;
    if (h[j].rows <= 0) h[j].rows = 1;
    rows[j] = i < cnt ? h[j].rows : 0;
    cum[j] = rows[j];
  }
  scan64(cum, lane);
  const int total = __shfl_sync(0xffffffffu, cum[1], 31);
  bool badkey = false;
#pragma unroll
  for (int j = 0; j < 2; j++) {
    const int i = lane + 32 * j;
    if (i >= cnt) continue;
    const int off = cum[j] - rows[j];
    const long long key = key_of(C, P.node, h[j].slot, h[j].it, h[j].u, P.U);
    S.hdr[i] = h[j]; S.key[i] = key; S.rowoff[i] = off;
    if (key < 0) { badkey = true; continue; }
    if (total > P.BM) continue;
    if (P.kind != LOOKUP) {
      const float* x0 = msg_x(C, P, h[j], key);
      for (int r = 0; r < rows[j]; r++) { S.rowmsg[off + r] = i; S.rowptr[off + r] = x0 ? x0 + (size_t)r * P.xld : nullptr; }
    } else {                                                // table rows and the rows of the incoming gradient
      const DevInst& I = C.inst;
      const long long base = I.offsets[h[j].inst];
      const float* g0 = P.gbuf + (size_t)key * P.rows_max * P.out_dim;
      const DevNode& feeder = g_nodes[g_nodes[P.node].pred_node[0]];
      const bool by_leaf = feeder.type == SOURCE && feeder.fn == 6;      // row r is the tree's r-th leaf
      for (int r = 0; r < rows[j]; r++) {
        const int id = I.tokens[base + (I.kind == 3 ? r : by_leaf ? I.leaf_ids[I.leaf_off[h[j].inst] + r] : h[j].u)];
        S.rowmsg[off + r] = i; S.rowptr[off + r] = g0 + (size_t)r * P.out_dim;
        S.rowid[off + r] = (unsigned)id < (unsigned)in ? id : -1;
      }
    }
  }
  if (P.kind == LOOKUP && ddir == BWD && total <= P.BM) {   // chain the batch rows that hit the same table row
    __syncwarp();
    for (int b = lane; b < total; b += 32) {
      const int id = S.rowid[b];
      int nx = -1, first = 1;
      for (int k = b + 1; k < total; k++) if (S.rowid[k] == id) { nx = k; break; }
      for (int k = 0; k < b; k++) if (S.rowid[k] == id) { first = 0; break; }
      S.rownext[b] = nx; S.rowfirst[b] = id >= 0 ? first : 0;
    }
  }
  const unsigned bad = __ballot_sync(0xffffffffu, badkey);
  if (lane == 0) {
    S.rowoff[cnt] = total;
    BatchDesc dd; dd.sched_start = (unsigned)d0.x; dd.count = d0.y; dd.dir = d0.z; dd.flags = d0.w;
    dd.n_upd = d1.x; dd.nrows = d1.y; dd.upd_t = d1.z; dd.pad1 = 0;
    if (bad) { S.ok = 0; dd.pad1 = 1; }
    if (total > P.BM) { fail(C, ST_OVERFLOW, P.node, total); S.ok = 0; dd.pad1 = 1; }
    S.desc = dd;
  }
}

// With scheduler CTAs: the assembled context of batch `batch`, one 16-byte piece per thread (whole CTA, no barrier).
__device__ __forceinline__ void fetch_ctx_block(const DevPPT& P, TileShared& S, const unsigned batch) {
  const int4* src = reinterpret_cast<const int4*>(P.ctxblk + (batch & (BATCH_BLOCKS - 1)));
  int4* dst = reinterpret_cast<int4*>(static_cast<BatchCtx*>(&S));
  for (int i = threadIdx.x; i < (int)(sizeof(BatchCtx) / 16); i += THREADS) dst[i] = __ldcg(src + i);
}
// Scheduler CTA, one warp: assemble the context of the batch formed into slot q and publish it.
__device__ __noinline__ void publish_ctx_block(const Ctx& C, DevPPT& P, TileShared& S, const unsigned batch, const SchedSlot* q) {
  const int lane = threadIdx.x & 31;
  load_batch_ctx(C, P, S, batch, q);
  __syncwarp();
  const int4* src = reinterpret_cast<const int4*>(static_cast<BatchCtx*>(&S));
  int4* dst = reinterpret_cast<int4*>(P.ctxblk + (batch & (BATCH_BLOCKS - 1)));
  for (int i = lane; i < (int)(sizeof(BatchCtx) / 16); i += 32) dst[i] = src[i];
  __syncwarp();
  if (lane == 0) st_rel(P.batch_pub, batch + 1u);     // the release store is cumulative over the warp barrier above
  __syncwarp();
}

// Emission of a batch by one CTA: reduce the tiles' partial input gradients for the rows this CTA emits, then walk
// the messages through the parameter-free nodes.  `parity` selects the per-batch buffers, `stage` the staging rows.
// This CTA emits share `tile` of `NT` shares: message i belongs to share i % NT (row-wise forks: every share walks every
// message and takes the rows j = part (mod NT)).
__device__ __noinline__ void emit_batch(const Ctx& C, DevPPT& P, const int tile, const int NT, TileShared& S, const BatchDesc d,
                                        const unsigned parity, float* stage, WalkAcc& acc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const DevNode& N = g_nodes[P.node];
  const int in = P.in_dim, out = P.out_dim, count = d.count, dir = d.dir;
  const int nb = S.rowoff[count];
  const unsigned my_batch = parity;
    if (g_bf16 && dir == BWD && P.kind == LINEAR && P.T == 1 && !(P.flags & 1)) {
      for (int idx = tid; idx < nb * in; idx += THREADS) stage[idx] = emit_round(stage[idx]);
      __syncthreads();
    }
    const bool split = C.wide && NT > 1;           // share row-wise forks among the emitting CTAs
    if (dir == BWD && P.kind != LOOKUP && !(P.flags & 1) && (P.T > 1 || P.kind == GRUCELL)) {
      // Sum the tiles' partial input gradients (tile order) for the rows this tile emits; every thread keeps
      // all T loads of an element in flight.
      const size_t pstride = (size_t)P.BM * in;
      const float* pa = P.dxpart + (size_t)(my_batch % (unsigned)C.depth) * P.T * pstride;
      const float* pb = P.kind == GRUCELL ? P.part2 + (size_t)(my_batch % (unsigned)C.depth) * (P.T + 1) * pstride : nullptr;
      const float* dirb = pb ? pb + (size_t)P.T * pstride : nullptr;
      const int H = out;
      for (int i = split ? 0 : tile; i < count; i += split ? 1 : NT) {
        const int part = (tile - i % NT + NT) % NT;
        const int ro = S.rowoff[i], ne = S.hdr[i].rows * in;
        for (int k = tid; k < ne; k += THREADS) {
          const int row = k / in;
          if (part != 0 && row % NT != part) continue;
          const size_t e = (size_t)ro * in + k;
          const int c = k - row * in;
          float sum = 0.f;
          for (int t0 = 0; t0 < P.T; t0 += 16) {         // sixteen tiles' partials in flight, added in tile order
            float v[16];
#pragma unroll
            for (int t = 0; t < 16; t++) v[t] = t0 + t < P.T ? __ldcg(pa + (size_t)(t0 + t) * pstride + e) : 0.f;
#pragma unroll
            for (int t = 0; t < 16; t++) sum += v[t];
          }
          if (pb && c >= H) sum += __ldcg(dirb + (size_t)(ro + row) * H + (c - H));
          stage[e] = emit_round(sum);
        }
      }
      __syncthreads();
    }
    if (tid == 0) S.pool.outstanding = split ? count : (tile < count ? (count - tile + NT - 1) / NT : 0);
    __syncthreads();
    const long long tw0 = clock64();
    int mine = 0;
    for (int i = 0; i < count; i++) {
      const int part = (tile - i % NT + NT) % NT;
      if (!split && part != 0) continue;
      if ((mine++ % WARPS) != warp) continue;
      const Hdr& h = S.hdr[i];
      Frame f;
      f.iter = 0; f.inst = h.inst; f.seq = h.seq; f.slot = h.slot; f.it = h.it; f.u = h.u; f.port = h.port;
      f.rows = h.rows; f.flags = h.flags; f.nsum = 1; f.sstride = 0;
      f.part = split ? part : 0; f.nparts = split ? NT : 1;
      f.ibase = C.inst.offsets ? C.inst.offsets[h.inst] : 0; f.ebase = C.inst.edge_off ? C.inst.edge_off[h.inst] : 0;
      if (dir == FWD) {
        f.node = N.succ_node[0]; f.aport = N.succ_port[0]; f.dir = FWD; f.dim = out; f.ld = out;
        f.p = P.kind == LOOKUP ? stage + (size_t)S.rowoff[i] * out
                               : P.ycache + (size_t)S.key[i] * P.rows_max * out;
      } else {
        f.node = N.pred_node[0]; f.aport = N.pred_port[0]; f.dir = BWD; f.dim = in; f.ld = in;
        if (P.kind == LOOKUP || (P.flags & 1)) { f.p = nullptr; f.dim = 0; f.rows = 1; }
        else f.p = stage + (size_t)S.rowoff[i] * in;
      }
      walk(C, f, S.stack[warp], acc, &S.pool);
      __syncwarp();
      if (lane == 0) atomicSub(&S.pool.outstanding, 1);
    }
    const long long tw1 = clock64();
    pool_steal(C, &S.pool, S.stack[warp], acc);
    const long long tw2 = clock64();
    if (lane == 0 && warp < 2) { S.phase[10 + 2 * warp] += (unsigned long long)(tw1 - tw0); S.phase[11 + 2 * warp] += (unsigned long long)(tw2 - tw1); }
    flush_acc(C, acc, lane);
    __syncthreads();
    if (tid == 0) S.phase[14] += (unsigned long long)(clock64() - tw2);
}

// Local update of one parameter from its accumulated gradient (Sec. 3; the update rule is a run-time option, App. A):
// g = A / n, then SGD, momentum-SGD (v <- mu v + g, theta <- theta - lr v) or Adam with bias correction, where t counts
// the updates of this node.  The moments live in device memory and are touched only here.
struct OptStep {
  int opt; float lr, inv_n, mu, b1, b2, eps, c1, c2; float *om, *ov;
  __device__ OptStep(const Ctx& C, const DevPPT& P, const BatchDesc& d)
      : opt(C.opt), lr(C.lr), inv_n(1.f / (float)d.n_upd), mu(C.mu), b1(C.beta1), b2(C.beta2), eps(C.eps), c1(1.f), c2(1.f),
        om(P.om), ov(P.ov) {
    if (opt == 2) {
      const double t = (double)(P.opt_t0 + d.upd_t);
      c1 = (float)(1.0 / (1.0 - pow((double)b1, t)));
      c2 = (float)(1.0 / (1.0 - pow((double)b2, t)));
    }
  }
  __device__ __forceinline__ void apply(float& w, float& a, const size_t k) const {
    if (opt == 0) { w = fmaf(-(lr * inv_n), a, w); a = 0.f; return; }
    const float g = a * inv_n;
    a = 0.f;
    if (opt == 1) {
      const float v = fmaf(mu, om[k], g);
      om[k] = v;
      w = fmaf(-lr, v, w);
    } else {
      const float m = fmaf(b1, om[k], (1.f - b1) * g), v = fmaf(b2, ov[k], (1.f - b2) * g * g);
      om[k] = m; ov[k] = v;
      w -= lr * (m * c1) / (sqrtf(v * c2) + eps);
    }
  }
};

// Embedding table, one batch (whole CTA).  Forward: gather the table rows into the staging rows.  Backward: accumulate
// in message order, as if the rows arrived one by one: the first batch row of every table row adds the gradients of all
// batch rows that hit the same table row, in order.  A warp takes whole rows and keeps ten loads per lane in flight.
// The table rows are dealt to the node's tiles (row id belongs to tile id % T): every tile sees the whole batch and
// handles the batch rows whose table row it owns, with a list of touched rows of its own.
__device__ __noinline__ void lookup_batch(DevPPT& P, TileShared& S, const int dir, const int nb, float* stage_k, const int tile) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, out = P.out_dim, T = P.T;
  int* const tlist = P.touched_list + (size_t)tile * ((P.in_dim + T - 1) / T);
  constexpr int K = 10;                                     // column chunks of 32 per pass: a 320-wide row in one round trip
  // the batch rows this tile handles (forward: rows whose table row it owns; backward: the owned chain heads), compacted
  if (warp == 0) {
    int n = 0;
    for (int b0 = 0; b0 < nb; b0 += 32) {
      const int b = b0 + lane;
      bool m = false;
      if (b < nb) {
        const int id = S.rowid[b];
        m = dir == FWD ? (id >= 0 ? id % T == tile : tile == 0) : (S.rowfirst[b] && id % T == tile);     // rows outside the table read as zero
      }
      const unsigned bal = __ballot_sync(0xffffffffu, m);
      if (m) S.mylist[n + __popc(bal & ((1u << lane) - 1u))] = b;
      n += __popc(bal);
    }
    if (lane == 0) S.mycount = n;
  }
  __syncthreads();
  const int mine = S.mycount;
  if (dir == FWD) {
    for (int k0 = warp; k0 < mine; k0 += WARPS) {
      const int b = S.mylist[k0], id = S.rowid[b];
      for (int c0 = 0; c0 < out; c0 += 32 * K) {
        float v[K];
#pragma unroll
        for (int k = 0; k < K; k++) {
          const int c = c0 + k * 32 + lane;
          v[k] = (id >= 0 && c < out) ? P.W[(size_t)id * out + c] : 0.f;
        }
#pragma unroll
        for (int k = 0; k < K; k++) {
          const int c = c0 + k * 32 + lane;
          if (c < out) stage_k[(size_t)b * out + c] = emit_round(v[k]);
        }
      }
    }
  } else {
    for (int k0 = warp; k0 < mine; k0 += WARPS) {
      const int b = S.mylist[k0], id = S.rowid[b];
      int fresh = 0;
      if (lane == 0) fresh = !P.touched_flag[id];
      float* arow = P.A + (size_t)id * out;
      for (int c0 = 0; c0 < out; c0 += 32 * K) {
        float a[K], g0[K];
#pragma unroll
        for (int k = 0; k < K; k++) {
          const int c = c0 + k * 32 + lane;
          a[k] = c < out ? arow[c] : 0.f;
          g0[k] = c < out ? __ldcg(S.rowptr[b] + c) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < K; k++) a[k] += g0[k];
        for (int nx = S.rownext[b]; nx >= 0; nx = S.rownext[nx]) {
#pragma unroll
          for (int k = 0; k < K; k++) { const int c = c0 + k * 32 + lane; g0[k] = c < out ? __ldcg(S.rowptr[nx] + c) : 0.f; }
#pragma unroll
          for (int k = 0; k < K; k++) a[k] += g0[k];
        }
#pragma unroll
        for (int k = 0; k < K; k++) { const int c = c0 + k * 32 + lane; if (c < out) arow[c] = a[k]; }
      }
      if (lane == 0 && fresh) { P.touched_flag[id] = 1; tlist[atomicAdd(P.touched_n + tile, 1)] = id; }
    }
  }
}

// GRU cell: XC = [a; r * h] from X = [a; h] (shared memory) and the reset gates of all tiles (device memory), a batch
// row per warp pass with eight gate loads per lane in flight (whole CTA, no barrier).
__device__ __noinline__ void gru_gated_input(const DevPPT& P, const TileShared& S, const float* __restrict__ Xs, float* __restrict__ XC,
                                             const int ldx, const int nb) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, in = P.in_dim, H = P.out_dim;
  for (int idx = threadIdx.x; idx < nb * (in - H); idx += THREADS) {
    const int b = idx / (in - H), c = idx - b * (in - H);
    XC[b * ldx + c] = Xs[b * ldx + c];
  }
  for (int b0 = warp; b0 < nb; b0 += WARPS * 4)               // four batch rows per warp pass
    for (int c0 = 0; c0 < H; c0 += 32 * 4) {
      float rg[4][4];
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const int b = b0 + j * WARPS;
        const float* rrow = nullptr;
        if (b < nb) { const int m = S.rowmsg[b]; rrow = P.rc + (size_t)(S.key[m] * P.rows_max + (b - S.rowoff[m])) * H; }
#pragma unroll
        for (int k = 0; k < 4; k++) { const int c = c0 + k * 32 + lane; rg[j][k] = (rrow && c < H) ? __ldcg(rrow + c) : 0.f; }
      }
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const int b = b0 + j * WARPS;
        if (b >= nb) continue;
#pragma unroll
        for (int k = 0; k < 4; k++) { const int c = c0 + k * 32 + lane; if (c < H) XC[b * ldx + (in - H) + c] = Xs[b * ldx + (in - H) + c] * rg[j][k]; }
      }
    }
}

// Local update of a tile's share of the node's parameters (whole CTA; ends with a block barrier).
__device__ __noinline__ void tile_update(const Ctx& C, DevPPT& P, const TileMem& M, const BatchDesc& d, const int R,
                                         const int r_begin, const int tile) {
  const int tid = threadIdx.x, in = P.in_dim, out = P.out_dim;
  const int nmat = P.kind == GRUCELL ? 3 : 1;
  const OptStep os(C, P, d);
  if (P.kind == LOOKUP) {
    __threadfence_block();
    // this tile's touched table rows, a row per warp with ten elements per lane in flight
    int* const tlist = P.touched_list + (size_t)tile * ((P.in_dim + P.T - 1) / P.T);
    const int nt = P.touched_n[tile];
    const int lane = tid & 31, warp = tid >> 5;
    constexpr int K = 5;
    for (int k = warp; k < nt; k += WARPS) {
      const int id = tlist[k];
      const size_t o0 = (size_t)id * out;
      for (int c0 = 0; c0 < out; c0 += 32 * K) {
        float w[K], a[K];
#pragma unroll
        for (int j = 0; j < K; j++) { const int c = c0 + j * 32 + lane; if (c < out) { w[j] = P.W[o0 + c]; a[j] = P.A[o0 + c]; } }
#pragma unroll
        for (int j = 0; j < K; j++) { const int c = c0 + j * 32 + lane; if (c < out) { os.apply(w[j], a[j], o0 + c); P.W[o0 + c] = w[j]; P.A[o0 + c] = a[j]; } }
      }
      if (lane == 0) P.touched_flag[id] = 0;
    }
    __syncthreads();
    if (tid == 0) P.touched_n[tile] = 0;
  } else {
    const size_t nW = (size_t)nmat * out * in;
    for (int m = 0; m < nmat; m++) {
      for (int i = tid; i < R * in; i += THREADS) {
        const int r = i / in, o = (m * P.R + r) * M.LW + (i - r * in);
        os.apply(M.Ws[o], M.As[o], (size_t)m * out * in + (size_t)r_begin * in + i);
      }
      for (int i = tid; i < R; i += THREADS) {
        const int o = m * P.R + i;
        os.apply(M.bs[o], M.Abs[o], nW + (size_t)m * out + r_begin + i);
      }
    }
  }
  __syncthreads();
}

__device__ __noinline__ void ppt_main(const Ctx& C, DevPPT& P, const int tile, float* smem, TileShared& S,
                         const unsigned long long t0) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int in = P.in_dim, out = P.out_dim;
  const int r_begin = tile * P.R;
  const int R = P.kind == LOOKUP ? 0 : max(0, min(P.R, out - r_begin));
  const int nmat = P.kind == GRUCELL ? 3 : 1;
  TileMem M;
  {
    M.LW = pad_ldw(in); M.LX = pad_ldx(in); M.RP = (P.R + 3) & ~3;
    float* p = smem;                                 // every array starts on a 16-byte boundary
    M.Ws = p; p += (size_t)nmat * P.R * M.LW;
    if (P.a_global) M.As = P.A + (size_t)tile * nmat * P.R * M.LW;       // zeroed with the run state
    else { M.As = p; p += (size_t)nmat * P.R * M.LW; }
    M.bs = p; p += (nmat * P.R + 3) & ~3;
    M.Abs = p; p += (nmat * P.R + 3) & ~3;
    M.Xs = p; p += (size_t)P.BM * M.LX;
    M.Ds = p; p += (size_t)(nmat + 1) * P.BM * M.RP;
    M.Ys = p; p += ((size_t)nmat * P.BM * P.R + 3) & ~(size_t)3;
    M.scratch = p; p += xwt_scratch_floats(P.xwt_rb);
    M.XC = p; p += P.kind == GRUCELL ? (size_t)P.BM * M.LX : 0;
    if (P.kind != LOOKUP) for (float* q = smem + tid; q < p; q += THREADS) *q = 0.f;     // the padding stays zero
  }
  __syncthreads();
  const int LW = M.LW, LX = M.LX, RP = M.RP;
  if (P.kind != LOOKUP) {
    for (int m = 0; m < nmat; m++) {
      for (int i = tid; i < R * in; i += THREADS) {
        const int r = i / in, c = i - r * in;
        M.Ws[(m * P.R + r) * LW + c] = P.W[(size_t)m * out * in + (size_t)r_begin * in + i];
      }
      for (int i = tid; i < R; i += THREADS) M.bs[m * P.R + i] = P.b[m * out + r_begin + i];
    }
  }
  if (tid == 0) {
    S.ls.head[0] = S.ls.head[1] = 0; S.ls.sched_w = S.ls.batch_w = 0; S.ls.n_acc = 0; S.ls.version = 0; S.max_stale = 0;
    S.ls.log_n = 0; S.ls.n_updates = S.ls.n_grads_applied = S.ls.msgs = S.ls.batches = S.ls.batch_rows = 0;
  }
  if (tid < 64) S.stale_hist[tid] = 0;
  if (tid < 16) { S.phase[tid] = 0; S.step[tid] = 0; }
  if (tid < POOL) S.pool.ready[tid] = 0;
  if (tid == 0) { S.pool.head = S.pool.tail = 0; S.pool.outstanding = 0; }
  if (tid == 0) { asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&S.mbar)) : "memory"); S.mbar_parity = 0; }
  __syncthreads();
#define AMP_PHASE(k) do { if (tid == 0) { long long now_ = clock64(); S.phase[k] += (unsigned long long)(now_ - tph); tph = now_; } } while (0)
  long long tph = clock64();

  unsigned my_batch = 0, grid_gen = 0, node_gen = 0;
  WalkAcc acc = {0, 0};
  bool running = true;
  while (running) {
    if (C.det) {
      if (!cta_barrier(C, t0, &C.g->grid_bar, (unsigned)C.n_ctas, grid_gen, &S.ok)) break;     // barrier A
      // This round's inbox is what is queued now; nothing may be emitted before every leader has looked.
      if (tile == 0 && tid == 0) { S.tail_snap[FWD] = ld_acq(P.ring[FWD].tail); S.tail_snap[BWD] = ld_acq(P.ring[BWD].tail); }
      if (!cta_barrier(C, t0, &C.g->grid_bar, (unsigned)C.n_ctas, grid_gen, &S.ok)) break;     // barrier A2
      if (tile == 0) leader_schedule_round(C, P, S, t0);
    }
    bool round_open = true;
    while (round_open) {
      // ---- obtain the next batch ------------------------------------------------------------
      AMP_PHASE(7);
      if (tid == 0) S.ok = 1;
      __syncthreads();
      if (tile == 0 && !C.sched_ctas) {
        if (warp == 0) {
          unsigned it = 0;
          for (;;) {
            unsigned bw = 0;
            if (lane == 0) bw = S.ls.batch_w;
            if (warp_uniform(bw) != my_batch) break;
            if (C.det) { if (lane == 0) { fail(C, ST_OVERFLOW, P.node, -7); S.ok = 0; } break; }
            if (leader_try_schedule(C, P, S)) break;
            if ((++it & 15u) == 0) {
              if (aborted_warp(C)) { if (lane == 0) S.ok = 0; break; }
              unsigned late = 0;
              if (lane == 0) late = gtime() - t0 > C.timeout_ns;
              if (warp_uniform(late)) { if (lane == 0) { fail(C, ST_TIMEOUT, P.node, 1); S.ok = 0; } break; }
            }
            __nanosleep(it < 16 ? 20 : 200);
          }
          __syncwarp();
        }
      } else {
        if (tid == 0) { if (!spin_until(C, t0, [&] { return ld_acq(P.batch_pub) > my_batch; })) S.ok = 0; }
        // Meanwhile warp 1 makes sure that the per-batch buffers of this batch are free: they are reused every `depth`
        // batches and read by the emitters of every tile, all of which must be done with their previous user.
        if (warp == 1 && C.emit_ctas && my_batch >= (unsigned)C.depth) {
          const unsigned j = my_batch - (unsigned)C.depth;
          unsigned it = 0;
          for (;;) {
            bool ok = true;
            for (int e = lane; e < P.NE; e += 32)
              if ((unsigned)(e % P.G) == j % (unsigned)P.G) ok = ok && ld_acq(&P.emit_done[e]) >= j + 1u;
            if (__all_sync(0xffffffffu, ok)) break;
            if ((++it & 15u) == 0) {
              unsigned bad = 0;
              if (lane == 0) { bad = aborted(C); if (!bad && gtime() - t0 > C.timeout_ns) { fail(C, ST_TIMEOUT, P.node, 6); bad = 1; } }
              if (warp_uniform(bad)) { if (lane == 0) S.ok = 0; break; }
            }
            __nanosleep(it < 16 ? 20 : 100);
          }
        }
      }
      __syncthreads();
      if (!S.ok) { running = false; break; }
      if (C.sched_ctas) {
        if (tile == 0 && tid == 0) *reinterpret_cast<volatile unsigned*>(P.fetched) = my_batch + 1u;   // paces the scheduler: a hint, ordered with nothing
        fetch_ctx_block(P, S, my_batch);
      } else if (warp == 0) load_batch_ctx(C, P, S, my_batch);
      __syncthreads();
      const BatchDesc d = S.desc;
      my_batch++;
      AMP_PHASE(d.count > 0 ? 1 : 0);
      const int count = d.count, dir = d.dir;
      if (!S.ok || d.pad1) { running = false; break; }
      float* const stage_k = P.stage + (size_t)(my_batch % (unsigned)C.depth) * P.stage_floats;
      const int nb = S.rowoff[count];
      const bool eval = count > 0 && (S.hdr[0].flags & HDR_EVAL);
      AMP_PHASE(2);
      if (tid == 0 && count > 0) { S.phase[13 + dir] += 1ull; if (d.flags & BATCH_UPDATE) S.phase[15] += 1ull; }

      if (count > 0 && P.kind == LINEAR) {
        // stage the cached inputs of the batch
        if (P.xcache || (in & 3) == 0) stage_rows_bulk(C, S, M.Xs, LX, S.rowptr, nb, P.xcache ? P.xld : in, P.node, t0);
        else stage_rows(M.Xs, LX, S.rowptr, nb, in, P.xcache ? in : C.inst.dense_dim);
        if (dir == FWD) {
          __syncthreads();
          tile_xwT(M.Xs, LX, nb, M.Ws, LW, R, in, M.Ys, P.R, M.scratch, P.xwt_rb);
          __syncthreads();
          for (int idx = tid; idx < nb * R; idx += THREADS) {
            const int b = idx / R, r = idx - b * R, m = S.rowmsg[b];
            const float y = act_fwd(P.act, M.Ys[b * P.R + r] + M.bs[r]);
            P.ycache[(S.key[m] * P.rows_max + (b - S.rowoff[m])) * out + r_begin + r] = emit_round(y);
          }
        } else {
          for (int idx = tid; idx < nb * R; idx += THREADS) {
            const int b = idx / R, r = idx - b * R, m = S.rowmsg[b];
            const size_t o = (size_t)(S.key[m] * P.rows_max + (b - S.rowoff[m])) * out + r_begin + r;
            M.Ds[b * RP + r] = __ldcg(P.gbuf + o) * act_grad(P.act, __ldcg(P.ycache + o));
          }
          __syncthreads();
          if (!(P.flags & 1)) {
            float* dst = P.T > 1 ? P.dxpart + ((size_t)(my_batch % (unsigned)C.depth) * P.T + tile) * P.BM * in : stage_k;
            AMP_DISPATCH_J(P.J, (tile_dW<J>(M.Ds, RP, nb, M.Ws, LW, R, in, dst)));
          }
          tile_accum(M.Ds, RP, nb, M.Xs, LX, M.As, LW, R, in);
          for (int r = tid; r < R; r += THREADS) {
            float s = M.Abs[r];
            for (int b = 0; b < nb; b++) s += M.Ds[b * RP + r];
            M.Abs[r] = s;
          }
        }
      } else if (count > 0 && P.kind == GRUCELL) {
        // x = [a; h]; the tile owns rows [r_begin, r_begin + R) of Wz, Wr, Wc (matrix m at Ws + m * P.R * in)
        const int H = out, SR = P.R, BR = P.BM * P.R, BRD = P.BM * RP;      // Ys arrays: [BM][SR]; D arrays: [BM][RP]
        const float *Wz = M.Ws, *Wr = M.Ws + SR * LW, *Wc = M.Ws + 2 * SR * LW;
        if (tid == 0) S.step_t = clock64();
        if (P.xcache) stage_rows_bulk(C, S, M.Xs, LX, S.rowptr, nb, P.xld, P.node, t0);
        else stage_rows(M.Xs, LX, S.rowptr, nb, in, in);
        __syncthreads();
        AMP_STEP(0);
        if (dir == FWD) {
          // phase 1: gates z, r for the tile's rows
          tile_xwT(M.Xs, LX, nb, Wz, LW, R, in, M.Ys, SR, M.scratch, P.xwt_rb);
          tile_xwT(M.Xs, LX, nb, Wr, LW, R, in, M.Ys + BR, SR, M.scratch, P.xwt_rb);
          __syncthreads();
          for (int idx = tid; idx < nb * R; idx += THREADS) {
            const int b = idx / R, r = idx - b * R, m = S.rowmsg[b];
            const size_t o = (size_t)(S.key[m] * P.rows_max + (b - S.rowoff[m])) * H + r_begin + r;
            const float z = act_fwd(3, M.Ys[b * SR + r] + M.bs[r]);
            const float rg = act_fwd(3, M.Ys[BR + b * SR + r] + M.bs[SR + r]);
            M.Ys[b * SR + r] = z;
            P.zc[o] = z; P.rc[o] = rg;
          }
          AMP_STEP(1);
          __threadfence();
          if (P.T > 1) { if (!cta_barrier(C, t0, P.nbar, (unsigned)P.T, node_gen, &S.ok)) { running = false; break; } }
          else __syncthreads();
          AMP_STEP(2);
          // phase 2: candidate c = tanh(Wc [a; r*h] + bc) and the new state
          gru_gated_input(P, S, M.Xs, M.XC, LX, nb);
          __syncthreads();
          AMP_STEP(3);
          tile_xwT(M.XC, LX, nb, Wc, LW, R, in, M.Ys + 2 * BR, SR, M.scratch, P.xwt_rb);
          __syncthreads();
          AMP_STEP(4);
          for (int idx = tid; idx < nb * R; idx += THREADS) {
            const int b = idx / R, r = idx - b * R, m = S.rowmsg[b];
            const size_t o = (size_t)(S.key[m] * P.rows_max + (b - S.rowoff[m])) * H + r_begin + r;
            const float cnd = tanhf(M.Ys[2 * BR + b * SR + r] + M.bs[2 * SR + r]);
            const float z = M.Ys[b * SR + r];
            P.cc[o] = cnd;
            P.ycache[o] = emit_round((1.f - z) * M.Xs[b * LX + H + r_begin + r] + z * cnd);
          }
          AMP_STEP(5);
        } else {
          const size_t pstride = (size_t)P.BM * in;
          float* part1 = P.part2 + ((size_t)(my_batch % (unsigned)C.depth) * (P.T + 1) + tile) * pstride;
          const float* part1_all = P.part2 + (size_t)(my_batch % (unsigned)C.depth) * (P.T + 1) * pstride;
          float* dirbuf = P.part2 + ((size_t)(my_batch % (unsigned)C.depth) * (P.T + 1) + P.T) * pstride;     // [BM][H]
          float* part2 = P.dxpart + ((size_t)(my_batch % (unsigned)C.depth) * P.T + tile) * pstride;
          float *dpz = M.Ds, *dpr = M.Ds + BRD, *dpc = M.Ds + 2 * BRD, *dirp = M.Ds + 3 * BRD;
          for (int idx = tid; idx < nb * R; idx += THREADS) {
            const int b = idx / R, r = idx - b * R, m = S.rowmsg[b];
            const size_t o = (size_t)(S.key[m] * P.rows_max + (b - S.rowoff[m])) * H + r_begin + r;
            const float g = __ldcg(P.gbuf + o), z = __ldcg(P.zc + o), rg = __ldcg(P.rc + o), cnd = __ldcg(P.cc + o);
            const float h = M.Xs[b * LX + H + r_begin + r];
            dpc[b * RP + r] = g * z * (1.f - cnd * cnd);
            dpz[b * RP + r] = g * (cnd - h) * z * (1.f - z);
            dirp[b * RP + r] = g * (1.f - z);
            M.Ys[b * SR + r] = rg;
          }
          gru_gated_input(P, S, M.Xs, M.XC, LX, nb);
          __syncthreads();
          AMP_STEP(6);
          AMP_DISPATCH_J(P.J, (tile_dW<J>(dpc, RP, nb, Wc, LW, R, in, part1)));      // [da_c; dq] partial
          AMP_STEP(7);
          __threadfence();
          if (P.T > 1) { if (!cta_barrier(C, t0, P.nbar, (unsigned)P.T, node_gen, &S.ok)) { running = false; break; } }
          else __syncthreads();
          AMP_STEP(8);
          for (int idx = tid; idx < nb * R; idx += THREADS) {
            const int b = idx / R, r = idx - b * R;
            float dq = 0.f;
            for (int tb = 0; tb < P.T; tb += 8) {        // eight tiles' partials in flight, added in tile order
              float v[8];
#pragma unroll
              for (int t = 0; t < 8; t++) v[t] = tb + t < P.T ? __ldcg(part1_all + (size_t)(tb + t) * pstride + (size_t)b * in + H + r_begin + r) : 0.f;
#pragma unroll
              for (int t = 0; t < 8; t++) dq += v[t];
            }
            const float rg = M.Ys[b * SR + r], h = M.Xs[b * LX + H + r_begin + r];
            dpr[b * RP + r] = dq * h * rg * (1.f - rg);
            dirbuf[(size_t)b * H + r_begin + r] = dirp[b * RP + r] + dq * rg;
          }
          __syncthreads();
          AMP_STEP(9);
          // this tile's share of da_c joins its second partial here, so that emission sums one partial array per tile
          AMP_DISPATCH_J(P.J, (tile_dW2<J>(dpz, dpr, RP, nb, Wz, Wr, LW, R, in, part1, H, part2)));
          AMP_STEP(10);
          tile_accum(dpz, RP, nb, M.Xs, LX, M.As, LW, R, in);
          tile_accum(dpr, RP, nb, M.Xs, LX, M.As + SR * LW, LW, R, in);
          tile_accum(dpc, RP, nb, M.XC, LX, M.As + 2 * SR * LW, LW, R, in);
          AMP_STEP(11);
          for (int k = tid; k < 3 * R; k += THREADS) {
            const int m = k / R, r = k - m * R;
            float sacc = M.Abs[m * SR + r];
            for (int b = 0; b < nb; b++) sacc += M.Ds[m * BRD + b * RP + r];
            M.Abs[m * SR + r] = sacc;
          }
        }
      } else if (count > 0 && P.kind == LOOKUP) {
        const long long tl0 = clock64();
        lookup_batch(P, S, dir, nb, stage_k, tile);
        __syncthreads();
        if (tid == 0) { S.phase[9 + 2 * dir] += (unsigned long long)(clock64() - tl0); S.phase[10 + 2 * dir] += (unsigned long long)nb; }
      }
      __syncthreads();
      AMP_PHASE(3);
      // ---- local update (Sec. 3): theta -= lr * A / n, accumulator cleared --------------------------
      if (d.flags & BATCH_UPDATE) tile_update(C, P, M, d, R, r_begin, tile);
      AMP_PHASE(4);
      // ---- all tiles of the node done with the batch, then emit ------------------------------------
      if (count > 0) {
        // With emitter CTAs the block barrier below orders every thread's writes before thread 0's release store of
        // the hand-over counter (a release is cumulative over the barrier); only the barrier among tiles needs the fence.
        if (!C.emit_ctas) __threadfence();
        // tiles that emit themselves wait for each other here; emitter CTAs wait for all tiles instead
        if (P.T > 1 && !C.emit_ctas) { if (!cta_barrier(C, t0, P.nbar, (unsigned)P.T, node_gen, &S.ok)) { running = false; break; } }
        else __syncthreads();
        AMP_PHASE(5);
        if (tile == 0 && warp == 0 && !C.det && !C.sched_ctas && !(C.tune & 2)) {   // look ahead: form the next batch now
          unsigned bw = 0;
          if (lane == 0) bw = S.ls.batch_w;
          const long long tq = clock64();
          if (warp_uniform(bw) == my_batch) leader_try_schedule(C, P, S);
          if (lane == 0) S.phase[8] += (unsigned long long)(clock64() - tq);
        }
        if (!C.emit_ctas) emit_batch(C, P, tile, P.T, S, d, my_batch, stage_k, acc);
        AMP_PHASE(6);
      }
      if (C.emit_ctas && tid == 0) {                                        // hand the batch to this tile's emitter CTAs
        st_rel(&P.emit_pub[tile], my_batch);
        if (d.flags & BATCH_TERMINATE) st_rel(&P.emit_fin[tile], 1u);
      }
      if (d.flags & BATCH_TERMINATE) { running = false; round_open = false; }
      if (d.flags & BATCH_END_ROUND) round_open = false;
      (void)eval;
    }
    if (!running) break;
    if (C.det) { if (!cta_barrier(C, t0, &C.g->grid_bar, (unsigned)C.n_ctas, grid_gen, &S.ok)) break; }   // barrier B
  }
  // ---- epilogue: parameters back to device memory, statistics ---------------------------------------
  __syncthreads();
  if (P.kind != LOOKUP)
    for (int m = 0; m < nmat; m++) {
      for (int i = tid; i < R * in; i += THREADS) { const int r = i / in; P.W[(size_t)m * out * in + (size_t)r_begin * in + i] = M.Ws[(m * P.R + r) * LW + (i - r * in)]; }
      for (int i = tid; i < R; i += THREADS) P.b[m * out + r_begin + i] = M.bs[m * P.R + i];
    }
  if (tile == 0) {
    if (!C.sched_ctas) write_leader_stats(P, S);
    if (tid < 16) P.stats->phase_cycles[tid] = S.phase[tid];
    if (tid < 16) C.g->step_cycles[(int)(&P - g_ppts)][tid] = S.step[tid];
  }
}

// ------------------------------------------------------------------------------------------------
// emitter CTA (asynchronous mode): the partner of one tile.  It emits the tile's share of every batch while the tile
// already stages and computes the next one.
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void emitter_main(const Ctx& C, DevPPT& P, const int which, TileShared& S,
                                          const unsigned long long t0) {
  const int tile = 0;                                         // whose termination flag this emitter watches
  const int grp = which % P.G, member = which / P.G, members = (P.NE - grp + P.G - 1) / P.G;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid < POOL) S.pool.ready[tid] = 0;
  if (tid < 16) S.phase[tid] = 0;
  if (tid == 0) { S.pool.head = S.pool.tail = 0; S.pool.outstanding = 0; }
  __syncthreads();
  unsigned my_batch = (unsigned)grp;            // this emitter's group takes batches grp, grp + G, grp + 2G, ...
  WalkAcc acc = {0, 0};
  unsigned long long* const rc = C.g->role_cycles + 8 + 8 * (int)(&P - g_ppts);
  long long tp = clock64();
#define EMIT_PHASE(k) do { if (tid == 0) { const long long tn = clock64(); S.phase[k] += (unsigned long long)(tn - tp); tp = tn; } } while (0)
  for (;;) {
    // (1) As soon as the scheduler has published the batch its context is copied: that overlaps the tiles' work on it.
    // (2) The batch is emitted once every tile of the node has handed it over (the tiles do not wait for each other).
    // Both waits end when tile 0 has seen the terminating batch and nothing is left for this emitter.
    BatchDesc d;
    bool stop = false;
    for (int phase = 0; phase < 2 && !stop; phase++) {
      if (tid == 0) S.ok = 1;
      __syncthreads();
      if (warp == 0) {
        const int lane = tid & 31;
        unsigned it = 0;
        int state = 0;                                          // 1: ready, 2: finished, 3: give up
        while (state == 0) {
          bool ready;
          if (phase == 0) { unsigned pub = 0; if (lane == 0) pub = ld_acq(P.batch_pub); ready = warp_uniform(pub) > my_batch; }
          else { const unsigned pub = lane < P.T ? ld_acq(&P.emit_pub[lane]) : 0xffffffffu; ready = __all_sync(0xffffffffu, pub > my_batch); }
          if (ready) state = 1;
          else {
            unsigned fin = 0;
            if (lane == 0) fin = ld_acq(&P.emit_fin[tile]) != 0u && ld_acq(&P.emit_pub[tile]) <= my_batch;
            if (warp_uniform(fin)) state = 2;
            else if ((++it & 15u) == 0) {
              unsigned bad = 0;
              if (lane == 0) { bad = aborted(C); if (!bad && gtime() - t0 > C.timeout_ns) { fail(C, ST_TIMEOUT, P.node, 5); bad = 1; } }
              if (warp_uniform(bad)) state = 3;
            }
            if (state == 0) __nanosleep(it < 16 ? 20 : 100);
          }
        }
        if (lane == 0) S.tail_snap[0] = (unsigned)state;
      }
      __syncthreads();
      if (S.tail_snap[0] != 1u) { stop = true; break; }        // finished and nothing left for this emitter, or aborted
      if (phase == 0) {
        EMIT_PHASE(3);
        fetch_ctx_block(P, S, my_batch);
        __syncthreads();
        d = S.desc;
        if (!S.ok || d.pad1) stop = true;
      }
    }
    if (stop) break;
    EMIT_PHASE(4);
    if (d.count > 0) emit_batch(C, P, member, members, S, d, my_batch + 1u, P.stage + (size_t)((my_batch + 1u) % (unsigned)C.depth) * P.stage_floats, acc);
    __syncthreads();
    EMIT_PHASE(5);
    if (tid == 0) S.phase[6] += 1ull;
    if (tid == 0) st_rel(&P.emit_done[which], my_batch + 1u);          // after the block barrier above
    my_batch += (unsigned)P.G;
  }
  __syncthreads();
  if (which == 0 && tid >= 3 && tid < 7) rc[tid] = S.phase[tid];
}

// ------------------------------------------------------------------------------------------------
// scheduler CTA (asynchronous mode): the leader of one PPT node on an SM of its own.  It forms the next micro-batch
// as soon as tile 0 has fetched the previous one, so that batch formation overlaps the tiles' work.
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void scheduler_main(const Ctx& C, DevPPT& P, TileShared& S, float* smem, const unsigned long long t0) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  SchedSlot* const Q = reinterpret_cast<SchedSlot*>(smem);
  init_leader_state(S);
  if (tid < 2) Q[tid].full = 0u;
  __syncthreads();
  unsigned long long* const rc = C.g->role_cycles + 8 + 8 * (int)(&P - g_ppts);
  // Warp 0 polls the rings and forms batches, one ahead of the batch tile 0 is working on: the batch is formed as late
  // as still keeps the tile fed, so that messages arriving meanwhile join it (a second batch of look-ahead adds a tile
  // cycle to every hop; AMPNET_TUNE bit 256 restores it).
  if (warp == 0) {
    unsigned it = 0;
    long long tp = clock64();
    unsigned long long rcl[3] = {0, 0, 0};
    for (;;) {
      unsigned bw = 0, busy = 0;
      if (lane == 0) { bw = S.ls.batch_w; busy = *reinterpret_cast<volatile unsigned*>(&Q[bw & 1u].full); }
      bw = warp_uniform(bw);
      SchedSlot* const q = &Q[bw & 1u];
      bool gow = false, progressed = false;
      if (!warp_uniform(busy)) progressed = leader_try_schedule(C, P, S, P.fetched, bw + ((C.tune & 256) ? 0u : 1u), &gow, q);
      unsigned fin = 0;
      if (progressed) {                  // (the slot was handed to warp 1 as soon as its descriptor was written)
        __syncwarp();
        if (lane == 0) fin = q->desc.flags & BATCH_TERMINATE;
      }
      if (lane == 0) { const long long tn = clock64(); rcl[!gow ? 0 : progressed ? 2 : 1] += (unsigned long long)(tn - tp); tp = tn; }
      if (warp_uniform(fin)) break;
      if (progressed) { it = 0; continue; }
      if ((++it & 15u) == 0) {
        if (aborted_warp(C)) break;
        unsigned late = 0;
        if (lane == 0) late = gtime() - t0 > C.timeout_ns;
        if (warp_uniform(late)) { if (lane == 0) fail(C, ST_TIMEOUT, P.node, 3); break; }
      }
      __nanosleep(it < 16 ? 20 : 100);
    }
    if (lane == 0) { rc[0] = rcl[0]; rc[1] = rcl[1]; rc[2] = rcl[2]; }
  } else if (warp == 1) {                // assembles and publishes the contexts, in batch order
    unsigned long long busy_cycles = 0;
    for (unsigned b = 0;; b++) {
      SchedSlot* const q = &Q[b & 1u];
      unsigned it = 0, stop = 0;
      for (;;) {
        unsigned f = 0;
        if (lane == 0) f = *reinterpret_cast<volatile unsigned*>(&q->full) == b + 1u;
        if (warp_uniform(f)) break;
        if ((++it & 63u) == 0) {
          if (aborted_warp(C)) { stop = 1; break; }
          unsigned late = 0;
          if (lane == 0) late = gtime() - t0 > C.timeout_ns;
          if (warp_uniform(late)) { if (lane == 0) fail(C, ST_TIMEOUT, P.node, 8); stop = 1; break; }
        }
        __nanosleep(20);
      }
      if (stop) break;
      __threadfence_block();
      long long tf = 0;
      if (lane == 0) tf = clock64();
      publish_ctx_block(C, P, S, b, q);
      if (S.desc.dir == BWD && S.desc.count > 0 && !(S.hdr[0].flags & HDR_EVAL)) {     // staleness of the batch just published
        const int ver = q->ver_form;
        for (int i = lane; i < S.desc.count; i += 32) {
          int st = ver - P.vcache[S.key[i]];
          if (st < 0) st = 0;
          atomicAdd(&S.stale_hist[st > 63 ? 63 : st], 1ull);
          atomicMax(&S.max_stale, st);
        }
      }
      __syncwarp();
      unsigned fin = 0;
      if (lane == 0) {
        fin = q->desc.flags & BATCH_TERMINATE;
        __threadfence_block();
        *reinterpret_cast<volatile unsigned*>(&q->full) = 0u;
        busy_cycles += (unsigned long long)(clock64() - tf);
      }
      if (warp_uniform(fin)) break;
    }
    if (lane == 0) rc[7] = busy_cycles;
  }
  __syncthreads();
  write_leader_stats(P, S);
}

// ------------------------------------------------------------------------------------------------
// controller CTA: admission under max_active_keys, source messages, retirement (Sec. 3, Sec. 4)
// ------------------------------------------------------------------------------------------------
constexpr int OCC_SLOTS = 8192;
__device__ __forceinline__ bool source_is_bulk(const Ctx& C, const DevNode& sn) {
  if (C.det || (C.tune & 16) || !(sn.fn == 1 || sn.fn == 2 || sn.fn == 4)) return false;
  const DevNode& dn = g_nodes[sn.succ_node[0]];
  return (dn.type == LINEAR || dn.type == LOOKUP || dn.type == GRUCELL) && g_ppts[dn.ppt].xcache == nullptr && g_ppts[dn.ppt].rows_max >= 1;
}
struct CtrlShared {
  int ok;
  long long next, retired;
  int active;
  unsigned retire_head;
  int admit_slot, admit_inst, admit_seq, n_src_msgs, admit_eval;
  int src_count[4], src_base[5];
  unsigned long long prof[8];
  unsigned occ[OCC_SLOTS / 32];          // occupied key slots (slots beyond OCC_SLOTS are found by scanning slot_inst)
  Frame stack[WARPS][WALK_STACK];
  WalkPool pool;
};

__device__ __noinline__ void controller_main(const Ctx& C, CtrlShared& S, const unsigned long long t0) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const DevInst& I = C.inst;
  if (tid == 0) { S.next = 0; S.retired = 0; S.active = 0; S.retire_head = 0; S.ok = 1; S.pool.head = S.pool.tail = 0; S.pool.outstanding = 0; }
  if (tid < POOL) S.pool.ready[tid] = 0;
  for (int i = tid; i < OCC_SLOTS / 32; i += THREADS) S.occ[i] = 0u;
  if (tid < 8) S.prof[tid] = 0;
  __syncthreads();
  unsigned grid_gen = 0;
  WalkAcc acc = {0, 0};
  long long round = 0;
  unsigned idle = 0;
  long long tp = clock64();
#define CTRL_PHASE(k) do { if (tid == 0) { const long long tn = clock64(); S.prof[k] += (unsigned long long)(tn - tp); tp = tn; } } while (0)
  for (;; round++) {
    CTRL_PHASE(4);
    // ---- retirements ------------------------------------------------------------------------------
    if (warp == 0) {
      for (;;) {
        unsigned h = 0, ready = 0;
        if (lane == 0) { h = S.retire_head; ready = ld_acq(&C.retire_seq[h & C.retire_mask]) == h + 1u; }
        h = warp_uniform(h);
        if (!warp_uniform(ready)) break;
        const unsigned s = h & C.retire_mask;
        const int slot = (int)__ldcg(&C.retire_e[s]);
        __syncwarp();
        if (lane == 0) S.retire_head = h + 1u;
        {
          // instance finished: sum its loss cells in key order, free the slot
          const int inst = C.slot_inst[slot];
          double tot = 0.0; int okc = 0, np = 0;
          for (int li = 0; li < C.n_loss; li++) {
            const DevNode& L = g_nodes[C.loss_nodes[li]];
            const long long k0 = (long long)slot * C.IT * L.U_in, k1 = k0 + (long long)C.IT * L.U_in;
            double dpart = 0.0;   // lane partial over a strided subset, then a fixed-order warp sum
            for (long long k = k0 + lane; k < k1; k += 32) {
              const int pk = __ldcg(&L.predok[k]);
              if (pk >= 0) { dpart += (double)__ldcg(&L.lossval[k]); okc += pk; np += 1; }
            }
            for (int o = 16; o; o >>= 1) dpart += __shfl_xor_sync(0xffffffffu, dpart, o);
            tot += dpart;
          }
          for (int o = 16; o; o >>= 1) { okc += __shfl_xor_sync(0xffffffffu, okc, o); np += __shfl_xor_sync(0xffffffffu, np, o); }
          if (lane == 0) {
            C.loss_out[inst] = (float)tot;
            if (C.inference_only && C.inference_only[inst]) { C.g->inf_loss += tot; C.g->inf_instances += 1; C.g->inf_correct += okc; C.g->inf_pred += np; }
            else { C.g->total_loss += tot; C.g->correct += okc; C.g->n_pred += np; }
            C.slot_inst[slot] = -1;
            if (slot < OCC_SLOTS) S.occ[slot >> 5] &= ~(1u << (slot & 31));
            S.active--; S.retired++;
            if (C.det && C.keylog) C.keylog[C.slot_log[slot]].release = round;
          }
          __syncwarp();
        }
      }
    }
    __syncthreads();
    CTRL_PHASE(0);
    // ---- admission ----------------------------------------------------------------------------------
    for (;;) {
      if (tid == 0) {
        S.admit_slot = -1;
        if (S.active < C.mak && S.next < C.n_order) {
          int slot = 0;                                                   // lowest free slot
          const int nw = (min(C.mak, OCC_SLOTS) + 31) >> 5;
          int w = 0;
          while (w < nw && S.occ[w] == 0xffffffffu) w++;
          if (w < nw) slot = w * 32 + __ffs(~S.occ[w]) - 1;
          else { slot = OCC_SLOTS; while (slot < C.mak && C.slot_inst[slot] >= 0) slot++; }
          if (slot < OCC_SLOTS) S.occ[slot >> 5] |= 1u << (slot & 31);
          const int inst = (int)(C.order ? C.order[S.next] : S.next);
          S.admit_slot = slot; S.admit_inst = inst; S.admit_seq = (int)S.next;
          C.slot_inst[slot] = inst;
          S.active++;
          if (S.active > C.g->max_active) C.g->max_active = S.active;
          int total = 0;
          for (int s = 0; s < C.n_sources; s++) {
            const DevNode& sn = g_nodes[C.src_nodes[s]];
            int cnt = 1;
            if (sn.fn == 2) cnt = (int)(I.offsets[inst + 1] - I.offsets[inst]);
            else if (sn.fn == 4) cnt = (int)(I.leaf_off[inst + 1] - I.leaf_off[inst]);
            S.src_base[s] = total; S.src_count[s] = cnt; total += cnt;
          }
          S.src_base[C.n_sources] = total;
          S.n_src_msgs = total;
          S.admit_eval = C.eval || (C.inference_only && C.inference_only[inst]);
          if (S.admit_eval) {      // forward only: the instance is finished when every Loss / Sink has been reached
            int exp = C.ends_per_instance;
            if (C.ends_per_position) exp += C.ends_per_position * (int)(I.offsets[inst + 1] - I.offsets[inst]);
            C.outstanding[slot] = exp;
          } else C.outstanding[slot] = total;
          if (C.det && C.keylog) {
            const long long li = C.g->n_keylog++;
            C.slot_log[slot] = (int)li;
            KeyLog kl; kl.inst = inst; kl.slot = slot; kl.pad = 0; kl.admit = round; kl.release = -1;
            C.keylog[li] = kl;
          }
          S.next++;
        }
      }
      __syncthreads();
      const int slot = S.admit_slot;
      CTRL_PHASE(1);
      if (slot < 0) break;
      // clear the slot's loss cells (predok = -1 marks "no loss evaluated at this key")
      for (int li = 0; li < C.n_loss; li++) {
        const DevNode& L = g_nodes[C.loss_nodes[li]];
        const long long k0 = (long long)slot * C.IT * L.U_in, cnt = (long long)C.IT * L.U_in;
        for (long long k = tid; k < cnt; k += THREADS) { L.lossval[k0 + k] = 0.f; L.predok[k0 + k] = -1; }
      }
      __threadfence();
      __syncthreads();
      // pump the source messages (Sec. 4: tokens / leaves / graph nodes, initial hidden state, dense row)
      const int inst = S.admit_inst;
      if (tid == 0) { S.pool.outstanding = S.n_src_msgs; S.prof[5] += 1ull; }
      __syncthreads();
      CTRL_PHASE(2);
      // A source that feeds a parameterised node directly (token / leaf / dense-row messages carry no payload of their
      // own) is pumped 32 messages at a time: one ticket grab per warp, every lane publishes its own header.
      for (int s = 0; s < C.n_sources; s++) {
        const DevNode& sn = g_nodes[C.src_nodes[s]];
        if (!source_is_bulk(C, sn)) continue;
        const DevNode& dn = g_nodes[sn.succ_node[0]];
        DevPPT& P = g_ppts[dn.ppt];
        const int cnt = S.src_count[s];
        for (int c0 = warp * 32; c0 < cnt; c0 += WARPS * 32) {
          const int k = c0 + lane;
          int u = 0;
          if (k < cnt) u = sn.fn == 2 ? k : sn.fn == 4 ? I.leaf_ids[I.leaf_off[inst] + k] : 0;
          const bool okm = k < cnt && key_of(C, sn.succ_node[0], slot, 0, u, P.U) >= 0;
          const unsigned vm = __ballot_sync(0xffffffffu, okm);
          unsigned tk = 0;
          if (lane == 0 && vm) tk = atomicAdd(P.ring[FWD].tail, (unsigned)__popc(vm));
          tk = __shfl_sync(0xffffffffu, tk, 0) + (unsigned)__popc(vm & ((1u << lane) - 1u));
          if (okm) {
            const unsigned q = tk & P.ring[FWD].mask;
            int4* d = reinterpret_cast<int4*>(&P.ring[FWD].e[q]);
            d[0] = make_int4(inst, S.admit_seq, slot, 0);
            d[1] = make_int4(u, 0, 1, S.admit_eval ? HDR_EVAL : 0);
            st_rel(&P.ring[FWD].seq[q], tk + 1u);
          }
          const int n_here = min(32, cnt - c0);
          acc.msgs += (unsigned long long)__popc(vm);
          if (lane == 0) atomicSub(&S.pool.outstanding, n_here);
        }
      }
      for (int mi = warp; mi < S.n_src_msgs; mi += WARPS) {
        int s = 0;
        while (mi >= S.src_base[s + 1]) s++;
        const int k = mi - S.src_base[s];
        const DevNode& sn = g_nodes[C.src_nodes[s]];
        if (source_is_bulk(C, sn)) continue;
        Frame f;
        f.node = sn.succ_node[0]; f.aport = sn.succ_port[0]; f.dir = FWD; f.iter = 0;
        f.inst = inst; f.seq = S.admit_seq; f.slot = slot; f.it = 0; f.u = 0; f.port = 0; f.rows = 1;
        f.flags = S.admit_eval ? HDR_EVAL : 0; f.dim = 0; f.ld = 0; f.p = nullptr; f.nsum = 1; f.sstride = 0; f.part = 0; f.nparts = 1;
        f.ibase = I.offsets ? I.offsets[inst] : 0; f.ebase = I.edge_off ? I.edge_off[inst] : 0;
        switch (sn.fn) {
          case 1: f.p = I.dense + (long long)inst * I.dense_dim; f.dim = I.dense_dim; f.ld = I.dense_dim; break;
          case 2: f.u = k; break;
          case 3: f.dim = sn.out_dim; f.ld = sn.out_dim; break;
          case 4: f.u = I.leaf_ids[I.leaf_off[inst] + k]; break;
          case 5: f.rows = (int)(I.offsets[inst + 1] - I.offsets[inst]); break;
          case 6: f.rows = (int)(I.leaf_off[inst + 1] - I.leaf_off[inst]); break;      // the tree's leaves as the rows of one message
        }
        walk(C, f, S.stack[warp], acc, &S.pool);
        __syncwarp();
        if (lane == 0) atomicSub(&S.pool.outstanding, 1);
      }
      pool_steal(C, &S.pool, S.stack[warp], acc);
      flush_acc(C, acc, lane);
      __syncthreads();
      CTRL_PHASE(3);
    }
    // ---- termination / pacing -------------------------------------------------------------------------
    const bool finished = S.retired == C.n_order;
    if (finished && tid == 0) { C.g->rounds = (unsigned long long)(round + 1); __threadfence(); st_rel(&C.g->done, 1u); }
    if (C.det) {
      if (!cta_barrier(C, t0, &C.g->grid_bar, (unsigned)C.n_ctas, grid_gen, &S.ok)) break;   // barrier A
      if (!cta_barrier(C, t0, &C.g->grid_bar, (unsigned)C.n_ctas, grid_gen, &S.ok)) break;   // barrier A2
      if (finished) break;
      if (!cta_barrier(C, t0, &C.g->grid_bar, (unsigned)C.n_ctas, grid_gen, &S.ok)) break;   // barrier B
    } else {
      if (finished) break;
      if (tid == 0) {
        S.ok = 1;
        if ((++idle & 15u) == 0) {
          if (aborted(C)) S.ok = 0;
          else if (gtime() - t0 > C.timeout_ns) { fail(C, ST_TIMEOUT, -1, 2); S.ok = 0; }
        }
        // wait for the next retire notice instead of spinning through the whole loop
        const unsigned h = S.retire_head;
        unsigned spins = 0;
        while (ld_acq(&C.retire_seq[h & C.retire_mask]) != h + 1u && spins < 64) { __nanosleep(50); spins++; }
      }
      __syncthreads();
      if (!S.ok) break;
    }
  }
  __syncthreads();
  if (tid < 8) C.g->role_cycles[tid] = S.prof[tid];
}

union SharedUnion { TileShared t; CtrlShared c; };

__global__ void __launch_bounds__(THREADS, 1) ampnet_engine(const __grid_constant__ Ctx C) {
  extern __shared__ __align__(16) float dyn_smem[];
  __shared__ SharedUnion SU;
  const unsigned long long t0 = gtime();
  {
    const int* src = reinterpret_cast<const int*>(C.nodes);
    int* dst = reinterpret_cast<int*>(g_nodes);
    for (int i = threadIdx.x; i < C.n_nodes * (int)(sizeof(DevNode) / 4); i += THREADS) dst[i] = src[i];
    src = reinterpret_cast<const int*>(C.ppts);
    dst = reinterpret_cast<int*>(g_ppts);
    for (int i = threadIdx.x; i < C.n_ppts * (int)(sizeof(DevPPT) / 4); i += THREADS) dst[i] = src[i];
  }
  if (threadIdx.x == 0) g_bf16 = C.bf16;
  __syncthreads();
  const Role role = C.roles[blockIdx.x];
  if (role.ppt < 0) controller_main(C, SU.c, t0);
  else if (role.kind == 1) emitter_main(C, g_ppts[role.ppt], role.pad, SU.t, t0);
  else if (role.kind == 2) scheduler_main(C, g_ppts[role.ppt], SU.t, dyn_smem, t0);
  else ppt_main(C, g_ppts[role.ppt], role.tile, dyn_smem, SU.t, t0);
}

}  // namespace amp
