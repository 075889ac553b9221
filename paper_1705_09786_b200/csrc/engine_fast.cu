// Direct-delivery engine: the asynchronous (measured) mode for IR graphs whose messages are single rows.
//
// Roles: CTA 0 is the controller (admission under max_active_keys, retirement: Sec. 3, Sec. 4 "controller loop");
// every other CTA is a row tile of one parameterised node and keeps its rows of W resident in shared memory for the
// whole epoch.  There is no scheduler and no emitter between two nodes:
//   * every tile polls its node's two rings itself and forms its own micro-batches (backward first, App. A).  All tiles
//     of a node see the same messages in the same order (the ring is the order), so all of them cut their backward
//     batches at the same gradient counts and update at the same points (Sec. 3): a tile is a node of its own in the
//     sense of the tiling the paper describes in Sec. 5, forward and backward batches may interleave differently;
//   * the chain of parameter-free nodes behind a message (Cond, Phi, Isu, Bcast, Concat, Sink, Loss) is a function of
//     the message state and the instance's structure tables alone.  One thread per message resolves it ("route") while
//     the batch's input rows are still in flight, down to the buffers the payload finally lands in: the input cache of
//     the next parameterised node (a Concat assembles there), or its incoming-gradient buffer (a Bcast's backward sum
//     forms there);
//   * after the arithmetic every tile stores its slice of the outputs (forward) or adds its partial input gradient
//     (backward, red.global.add) straight into those buffers and arrives at the landing's join counter with its share
//     of JOIN_UNIT; the arrival that completes the count publishes the header in the consumer's ring.
// One hop is therefore: stores -> one acquire-release atomic -> ticket + release store -> the consumer's poll.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "engine_types.h"
#include "tc_tile.cuh"

namespace ampf {
using namespace amp;

constexpr int FT = 512;               // threads per CTA
constexpr int FW = FT / 32;
constexpr int FBM = 128;              // messages (= rows) per micro-batch
constexpr int MAXD = 2;               // landings per message
constexpr int RSTACK = 4;             // pending forks per routed message

// ------------------------------------------------------------------------------------------------
// memory-model helpers, bounded waits
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned ld_acq(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_rlx(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void fence_acq() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
__device__ __forceinline__ void st_rel(unsigned* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int atom_add_acq_rel(int* p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
// Ring entries of this engine carry their own ticket, so that one round trip brings a message: two 16-byte halves
// {inst, seq, slot, tag} and {u, base position, it | port << 16 | flags << 24, tag} with tag = ticket + 1 (16-byte stores
// are single transactions; an entry is taken when both tags match).  The second half is stored with release and loaded
// with acquire semantics: what the producer wrote before (payloads, the arrivals it has acquired) is visible to the
// thread that takes the message.  Entries are zeroed before every run (tickets start over).
__device__ __forceinline__ void entry_store(Hdr* e, int inst, int seq, int slot, int it, int u, int port, int rows, int flags, unsigned tag) {
  asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};" :: "l"(e), "r"(inst), "r"(seq), "r"(slot), "r"(tag) : "memory");
  asm volatile("st.release.gpu.global.v4.u32 [%0], {%1, %2, %3, %4};" :: "l"(reinterpret_cast<char*>(e) + 16), "r"(u), "r"(rows), "r"(it | (port << 16) | (flags << 24)), "r"(tag) : "memory");
}
__device__ __forceinline__ bool entry_load(const Hdr* e, unsigned tag, Hdr& h) {
  unsigned a0, a1, a2, a3, b0, b1, b2, b3;
  asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "l"(e) : "memory");
  asm volatile("ld.acquire.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(b0), "=r"(b1), "=r"(b2), "=r"(b3) : "l"(reinterpret_cast<const char*>(e) + 16) : "memory");
  h.inst = (int)a0; h.seq = (int)a1; h.slot = (int)a2; h.u = (int)b0; h.rows = (int)b1;
  h.it = (int)(b2 & 0xffffu); h.port = (int)((b2 >> 16) & 0xffu); h.flags = (int)(b2 >> 24);
  return a3 == tag && b3 == tag;
}
// Retire notices are one 8-byte word each: (ticket + 1) << 32 | key slot, stored with release and polled with acquire.
__device__ __forceinline__ void retire_push(const Ctx& C, const int slot) {
  const unsigned t = atomicAdd(&C.g->retire_tail, 1u);
  const unsigned long long v = ((unsigned long long)(t + 1u) << 32) | (unsigned)slot;
  asm volatile("st.release.gpu.global.u64 [%0], %1;" :: "l"(reinterpret_cast<unsigned long long*>(C.retire_seq) + (t & C.retire_mask)), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long retire_poll(const Ctx& C, const unsigned h) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(reinterpret_cast<const unsigned long long*>(C.retire_seq) + (h & C.retire_mask)) : "memory");
  return v;
}
__device__ __forceinline__ void red_add(float* p, float v) {
  asm volatile("red.relaxed.gpu.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __noinline__ void fail(const Ctx& C, int code, int node, int detail) {
  if (atomicCAS(&C.g->status, 0, code) == 0) { C.g->err_node = node; C.g->err_detail = detail; }
  __threadfence();
  st_rel(&C.g->abort_flag, 1u);
}
__device__ __forceinline__ bool aborted(const Ctx& C) { return ld_acq(&C.g->abort_flag) != 0; }
__device__ __forceinline__ unsigned warp_uniform(unsigned v) { return __shfl_sync(0xffffffffu, v, 0); }
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ long long key_of(const Ctx& C, int node, int slot, int it, int u, int U) {   // the failure path is a call
  if ((unsigned)slot >= (unsigned)C.mak || (unsigned)it >= (unsigned)C.IT || (unsigned)u >= (unsigned)U) {
    fail(C, ST_OVERFLOW, node, u);
    return -1;
  }
  return ((long long)slot * C.IT + it) * U + u;
}

// Pointers into shared memory that reach a function as arguments would be dereferenced as generic addresses; this tells
// the compiler their address space.
#define IN_SMEM(p) __builtin_assume(__isShared(p))

constexpr int DIRECT_MAX_NODES = 24, DIRECT_MAX_PPTS = 12;      // the graphs this engine takes are small (checked on the host)
__shared__ DevNode g_nodes[DIRECT_MAX_NODES];
__shared__ DevPPT g_ppts[DIRECT_MAX_PPTS];
__shared__ int g_bf16;
// What a node emits as a payload: identity for fp32 messages, rounded to bfloat16 (nearest even) otherwise.
__device__ __forceinline__ float emit_round(float v) { return g_bf16 ? __bfloat162float(__float2bfloat16_rn(v)) : v; }

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

// ------------------------------------------------------------------------------------------------
// routes: where the payload of one message lands
// ------------------------------------------------------------------------------------------------
enum { ACT_PUSH = 1, ACT_RETIRE = 2, ACT_LOSS = 3 };

// One landing of a message.  Columns [s0, s0 + w) of the payload go to dst[0 .. w) (dst == nullptr: nothing to
// deposit, the arrival alone counts).  The arrival that brings *jcnt to `expected` (ACT_RETIRE: down to zero) clears
// the recorded Phi origin, publishes the header (ACT_PUSH) or tells the controller (ACT_RETIRE).
struct __align__(16) Deliv {
  float* dst;
  int* jcnt;
  unsigned char *clear, *clear2;  // recorded Phi origins the completing arrival clears
  int expected, s0, w, act;
  int ppt, dir, u, it;
  int port, post, node, zero, pad[2];   // post: logical node-messages the completing arrival accounts for; node: the Loss;
                                  // zero: the payload is a zero vector (deposit zeros of width w)
};

// The same, as it is kept per message in shared memory (48 bytes): counters and origins live in the control arena and
// are addressed by their byte offsets from its start (0: none).
struct __align__(16) Landing {
  float* dst;
  unsigned jcnt_off, clear_off, clear2_off;
  int expected;
  unsigned short s0, w;
  int u;
  unsigned char act, dir, ppt, port, zero, post, it, pad0;
  short node, pad1;
};
__device__ __forceinline__ Landing pack_landing(const Ctx& C, const Deliv& d) {
  Landing L;
  L.dst = d.dst;
  L.jcnt_off = d.jcnt ? (unsigned)((char*)d.jcnt - C.ctl_base) : 0u;
  L.clear_off = d.clear ? (unsigned)((char*)d.clear - C.ctl_base) : 0u;
  L.clear2_off = d.clear2 ? (unsigned)((char*)d.clear2 - C.ctl_base) : 0u;
  L.expected = d.expected; L.s0 = (unsigned short)d.s0; L.w = (unsigned short)d.w; L.u = d.u;
  L.act = (unsigned char)d.act; L.dir = (unsigned char)d.dir; L.ppt = (unsigned char)d.ppt; L.port = (unsigned char)d.port;
  L.zero = (unsigned char)d.zero; L.post = (unsigned char)d.post; L.it = (unsigned char)d.it; L.pad0 = 0; L.node = (short)d.node; L.pad1 = 0;
  return L;
}

struct Route {                    // state of one message on its way through the parameter-free nodes
  int node, aport, dir, u, it, port, s0, w, null;
};

// The message `h` leaves parameterised node `P` in direction `dir`.  Follows the parameter-free nodes (Sec. 4: Cond
// queries the state, Phi records / recalls the origin, Isu updates the state and inverts the update, Bcast copies and
// sums, Concat joins and splits) and writes the landings to out[0 .. returned count).  pre: node-messages consumed on
// the way that every arrival sees (added once per message by the first row tile).  width: payload width at the start.
__device__ __noinline__ int route_message(const Ctx& C, const Hdr h, int start_node, int start_aport, const int dir0, const int width,
                                          Landing* out, int& pre) {
  IN_SMEM(out);
  const DevInst& I = C.inst;
  const long long ibase = h.rows;          // every message is one row here: the field carries the instance's first position instead
  // the tree tables of the message's own position, fetched together (one round trip instead of one per node on the way)
  int own_parent = 0, own_slot = 0, own_left = 0, own_right = 0;
  if (I.parent) { const long long o = ibase + h.u; own_parent = I.parent[o]; own_slot = I.child_slot[o]; own_left = I.left[o]; own_right = I.right[o]; }
  Route stack[RSTACK];
  int sp = 0, nout = 0;
  Route f;
  f.node = start_node; f.aport = start_aport; f.dir = dir0; f.u = h.u; f.it = h.it; f.port = h.port; f.s0 = 0; f.w = width; f.null = 0;
  pre = 0;
  bool have = true;
  // a pending join: the backward sum of a Bcast forms in the buffer the message lands in
  int* pend = nullptr; int pend_exp = 0, pend_slot = 0; int post = 0; unsigned char *clear = nullptr, *clear2 = nullptr;
  int* phi_cnt = nullptr;         // arrival counter of the last Phi passed backward (joins the tiles' arrivals of one message at a Source)
  int steps = 0;
  while (have) {
    if (f.node < 0 || ++steps > 256) { fail(C, ST_OVERFLOW, -2, f.node); return nout; }
    const DevNode& n = g_nodes[f.node];
    bool cont = false;
    auto count = [&] { if (pend) post++; else pre++; };
    auto to_succ = [&](int k) { f.aport = n.succ_port[k]; f.node = n.succ_node[k]; f.dir = FWD; cont = true; };
    auto to_pred = [&](int j) { f.aport = n.pred_port[j]; f.node = n.pred_node[j]; f.dir = BWD; cont = true; };
    auto land = [&](Deliv d) {
      if (nout >= MAXD) { fail(C, ST_OVERFLOW, f.node, -9); return; }
      d.clear = clear; d.clear2 = clear2; d.zero = f.null ? 1 : 0;
      out[nout++] = pack_landing(C, d);
      pend = nullptr; pend_exp = 0; pend_slot = 0; post = 0; clear = clear2 = nullptr; phi_cnt = nullptr;
    };
    Deliv d;
    bool landed = false;
    switch (n.type) {
      case LINEAR: case LOOKUP: {
        DevPPT& Q = g_ppts[n.ppt];
        const long long key = key_of(C, f.node, h.slot, f.it, f.u, Q.U);
        if (key < 0) return nout;
        if (f.dir == FWD) {
          if (!Q.xcache) { fail(C, ST_OVERFLOW, f.node, -10); return nout; }
          d.dst = Q.xcache + key * (long long)Q.xld;
        } else {
          // gradients land in slots: one per successor of the Bcast whose backward sum forms here, so that nothing is added
          // in memory (no atomics on payloads, nothing to clear); the reader adds the slots in successor order
          if (!pend && Q.NS != 1) { fail(C, ST_OVERFLOW, f.node, -15); return nout; }
          d.dst = Q.gbuf + (key * Q.NS + pend_slot) * (long long)Q.out_dim;
        }
        d.jcnt = pend ? pend : Q.injoin[f.dir] + key;
        d.expected = pend ? pend_exp : JOIN_UNIT;
        d.s0 = f.s0; d.w = f.w; d.act = ACT_PUSH; d.ppt = n.ppt; d.dir = f.dir; d.u = f.u; d.it = f.it; d.port = f.port;
        d.post = post + 1; d.node = f.node;
        landed = true;
      } break;
      case LOSS_CE: case LOSS_MSE: {
        pre++;
        d.dst = nullptr; d.jcnt = nullptr; d.expected = 0; d.s0 = f.s0; d.w = f.w; d.act = ACT_LOSS; d.ppt = -1; d.dir = FWD;
        d.u = f.u; d.it = f.it; d.port = f.port; d.post = 0; d.node = f.node;
        landed = true;
      } break;
      case SOURCE: {                                        // a source message came home
        if (pend) { fail(C, ST_OVERFLOW, f.node, -14); return nout; }
        d.dst = nullptr; d.jcnt = &C.outstanding[h.slot]; d.expected = 0; d.s0 = 0; d.w = 0; d.act = ACT_RETIRE; d.ppt = -1;
        d.dir = BWD; d.u = f.u; d.it = f.it; d.port = f.port; d.post = post; d.node = f.node;
        // a recorded origin may be cleared only when every tile has read it: the tiles' arrivals of this message meet at the
        // Phi's counter first, and the one that completes it retires the whole source message
        if (clear && phi_cnt) { d.jcnt = phi_cnt; d.expected = JOIN_UNIT; }
        landed = true;
      } break;
      case SINK:
        count();
        if (h.flags & HDR_EVAL) {
            d.dst = nullptr; d.jcnt = &C.outstanding[h.slot]; d.expected = 0; d.s0 = 0; d.w = 0; d.act = ACT_RETIRE; d.ppt = -1;
          d.dir = FWD; d.u = f.u; d.it = f.it; d.port = f.port; d.post = post; d.node = f.node;
          landed = true;
        } else { f.null = 1; to_pred(0); }                   // answers with a zero gradient
        break;
      case COND:
        count();
        if (f.dir == FWD) {
          int k = 0;
          switch (n.fn) {
            case 1: k = f.u < (int)(I.offsets[h.inst + 1] - ibase) ? 0 : 1; break;
            case 2: k = (f.u == h.u ? own_parent : I.parent[ibase + f.u]) < 0 ? 0 : 1; break;
            case 3: k = f.u; break;
            case 4: k = f.it < n.fn_arg ? 0 : 1; break;
            case 5: k = (h.inst + f.u) % n.n_succ; break;
          }
          if ((unsigned)k >= (unsigned)n.n_succ) { fail(C, ST_OVERFLOW, f.node, k); return nout; }
          to_succ(k);
        } else to_pred(0);
        break;
      case PHI: {
        count();
        const long long key = key_of(C, f.node, h.slot, f.it, f.u, n.U_in);
        if (key < 0) return nout;
        if (f.dir == FWD) {
          if (!(h.flags & HDR_EVAL)) n.origin[key] = (unsigned char)(f.aport + 1);   // every tile writes the same value
          to_succ(0);
        } else {
          const int j = (int)*(volatile unsigned char*)&n.origin[key] - 1;
          if (j < 0 || j >= n.n_pred) { fail(C, ST_OVERFLOW, f.node, -20); return nout; }
          if (clear2) { fail(C, ST_OVERFLOW, f.node, -11); return nout; }
          if (clear) clear2 = &n.origin[key]; else clear = &n.origin[key];   // cleared by the arrival that completes the landing
          phi_cnt = n.jcnt ? &n.jcnt[key] : nullptr;
          to_pred(j);
        }
      } break;
      case ISU:
        count();
        if (f.dir == FWD) {
          if (n.fn == 1) f.u += 1;
          else if (n.fn == 2) { const bool own = f.u == h.u; f.port = own ? own_slot : I.child_slot[ibase + f.u]; f.u = own ? own_parent : I.parent[ibase + f.u]; }
          else f.it += 1;
          to_succ(0);
        } else {
          if (n.fn == 1) f.u -= 1;
          else if (n.fn == 2) { const bool own = f.u == h.u; f.u = f.port == 0 ? (own ? own_left : I.left[ibase + f.u]) : (own ? own_right : I.right[ibase + f.u]); f.port = 0; }
          else f.it -= 1;
          to_pred(0);
        }
        break;
      case BCAST:
        if (f.dir == FWD) {
          count();
          for (int k = n.fn_arg - 1; k >= 1; k--) {
            if (sp >= RSTACK) { fail(C, ST_OVERFLOW, f.node, sp); return nout; }
            Route c = f; c.node = n.succ_node[k]; c.aport = n.succ_port[k]; c.dir = FWD;
            stack[sp++] = c;
          }
          to_succ(0);
        } else {
          count();
          const long long key = key_of(C, f.node, h.slot, f.it, f.u, n.U_in);
          if (key < 0) return nout;
          if (pend) { fail(C, ST_OVERFLOW, f.node, -12); return nout; }      // nested sums are not resolved here
          pend = &n.jcnt[key]; pend_exp = n.fn_arg * JOIN_UNIT; pend_slot = f.aport;
          if ((unsigned)pend_slot >= (unsigned)n.fn_arg) { fail(C, ST_OVERFLOW, f.node, -16); return nout; }
          to_pred(0);
        }
        break;
      case CONCAT:
        if (f.dir == FWD) {
          count();
          const int port = n.fn == 2 ? f.port : f.aport;
          const long long key = key_of(C, f.node, h.slot, f.it, f.u, n.U_out);
          if (key < 0) return nout;
          const DevNode& s = g_nodes[n.succ_node[0]];
          if ((unsigned)port >= (unsigned)n.fn_arg || !n.jalias || pend) { fail(C, ST_OVERFLOW, f.node, port); return nout; }
            d.dst = n.jbuf + key * n.jstride + port * n.in_dim;
          d.jcnt = &n.jcnt[key]; d.expected = n.fn_arg * JOIN_UNIT;
          d.s0 = f.s0; d.w = f.w; d.act = ACT_PUSH; d.ppt = s.ppt; d.dir = FWD; d.u = f.u; d.it = f.it; d.port = 0;
          d.post = 1; d.node = n.succ_node[0];
          landed = true;
        } else {
          count();
          for (int k = n.fn_arg - 1; k >= 0; k--) {
            Route c = f; c.s0 = f.s0 + k * n.in_dim; c.w = n.in_dim; c.dir = BWD;
            if (n.fn == 2) { c.port = k; c.node = n.pred_node[0]; c.aport = n.pred_port[0]; }
            else { c.node = n.pred_node[k]; c.aport = n.pred_port[k]; }
            if (k == 0) { f = c; cont = true; }
            else { if (sp >= RSTACK) { fail(C, ST_OVERFLOW, f.node, sp); return nout; } stack[sp++] = c; }
          }
        }
        break;
      default:
        fail(C, ST_OVERFLOW, f.node, n.type);
        return nout;
    }
    if (landed) land(d);                                 // (one copy of the code that packs a landing)
    if (!cont) {
      if (pend) { fail(C, ST_OVERFLOW, f.node, -13); return nout; }          // a sum that found no landing
      if (sp > 0) f = stack[--sp];
      else have = false;
    }
  }
  return nout;
}

// ------------------------------------------------------------------------------------------------
// tile state and arithmetic
// ------------------------------------------------------------------------------------------------
struct TileS {
  // Two batches are in flight in a tile: while most warps arrive for batch n, four warps already form batch n + 1 and
  // resolve its routes.  Headers, landings and counts are kept per batch parity.
  Hdr hdr[2][FBM];
  Landing dl[2][FBM][MAXD];
  unsigned char nd[2][FBM];
  short pre[2][FBM];
  long long key[FBM];
  const float* rowptr[FBM];
  int rowid[FBM];
  int fpb;                          // parity of the batch being formed
  unsigned arr_done;                // arrival warps that have finished, summed over the batches
  unsigned qmax[2];                 // most messages waiting in each ring when a batch was taken (queue occupancy)
  int count, dir, flags, n_upd, upd_t, eval, ok, term;
  unsigned head[2];
  int n_acc, version, log_n, max_stale;
  unsigned long long n_updates, n_grads_applied, msgs, batches, batch_rows, node_msgs;
  unsigned long long stale_hist[64];
  unsigned long long phase[16];
  unsigned long long mbar;
  unsigned mbar_parity;
  unsigned wver_seen;               // forward tile: the node's published-columns counter as last polled
  // tensor-core forward tile: address of its tensor-memory columns, the mbarrier its products are committed to (and the
  // parity to wait for next), micro-batches run this way
  unsigned tmem, tc_parity;
  unsigned long long tc_mbar, tc_batches;
};

__host__ __device__ __forceinline__ int pad4(int v) { return (v + 3) & ~3; }
// n / d for 0 <= n < 200000 and 1 <= d <= 2048 by one multiply-high (M = floor((2^32 - 1) / d) + 1; checked exhaustively
// for 2 <= d; d = 1 would need M = 2^32 and is handled apart)
struct FastDiv {
  unsigned d, M;
  __device__ explicit FastDiv(int d_) : d((unsigned)d_), M(d_ > 1 ? 0xFFFFFFFFu / (unsigned)d_ + 1u : 0u) {}
  __device__ __forceinline__ int div(int n) const { return d > 1 ? (int)__umulhi((unsigned)n, M) : n; }
};
__host__ __device__ __forceinline__ int pad_ldx(int in) { int l = (in + 3) & ~3; while ((l & 7) != 4) l += 4; return l; }
// out[b][o] = sum_k A[b][k] B[o][k] for b < nA, o < nB: both operands in shared memory with k contiguous, rows padded
// with zeros to K4 groups of four and strides of 4 (mod 8) floats.  A thread owns a 4 x 4 block of outputs (eight 16-byte
// loads feed 64 multiply-adds: two bytes of shared-memory traffic per multiply-add instead of eight) and one of nsl
// interleaved k-slices, as many slices as keep every thread busy (a single message still spreads over the CTA); the
// slices meet by shuffles.  Whole CTA, no barrier inside.
template <int TA>
__device__ __forceinline__ void gemm_nt_t(const float* __restrict__ A, const int lda, const int nA, const float* __restrict__ B, const int ldb,
                                          const int nB, const int K4, float* __restrict__ out, const int ldo) {
  const int tid = threadIdx.x;
  const int tA = (nA + TA - 1) / TA, tB = (nB + 3) >> 2, n_tiles = tA * tB;
  int nsl = 1, sh = 0;
  while (nsl < 32 && n_tiles * nsl * 4 <= FT) { nsl <<= 1; sh++; }       // (measured: merging more slices by shuffles costs more than it spreads)
  const int per_pass = FT >> sh, ks = tid & (nsl - 1);
  const FastDiv dB(tB);
  for (int t0 = 0; t0 < n_tiles; t0 += per_pass) {
    const int ti = t0 + (tid >> sh);
    const bool valid = ti < n_tiles;
    const int bt = valid ? dB.div(ti) : 0, ot = valid ? ti - bt * tB : 0;
    const float4* const A4 = reinterpret_cast<const float4*>(A);
    const float4* const B4 = reinterpret_cast<const float4*>(B);
    const int lda4 = lda >> 2, ldb4 = ldb >> 2;
    const int a0 = min(TA * bt, nA - 1) * lda4, a1 = min(TA * bt + 1, nA - 1) * lda4, a2 = min(TA * bt + 2, nA - 1) * lda4, a3 = min(TA * bt + 3, nA - 1) * lda4;
    const int w0 = min(4 * ot, nB - 1) * ldb4, w1 = min(4 * ot + 1, nB - 1) * ldb4, w2 = min(4 * ot + 2, nB - 1) * ldb4, w3 = min(4 * ot + 3, nB - 1) * ldb4;
    float acc[TA][4];
#pragma unroll
    for (int m = 0; m < TA; m++)
#pragma unroll
      for (int j = 0; j < 4; j++) acc[m][j] = 0.f;
    // (threads past the last block take part in the shuffles only: their loads would cost shared-memory bandwidth)
#pragma unroll 2
    for (int k4 = valid ? ks : K4; k4 < K4; k4 += nsl) {
      float4 x[4];
      x[0] = A4[a0 + k4];
      if (TA > 1) { x[1] = A4[a1 + k4]; x[2] = A4[a2 + k4]; x[3] = A4[a3 + k4]; }
      const float4 y[4] = {B4[w0 + k4], B4[w1 + k4], B4[w2 + k4], B4[w3 + k4]};
#pragma unroll
      for (int m = 0; m < TA; m++)
#pragma unroll
        for (int j = 0; j < 4; j++) {
          acc[m][j] = fmaf(x[m].x, y[j].x, acc[m][j]); acc[m][j] = fmaf(x[m].y, y[j].y, acc[m][j]);
          acc[m][j] = fmaf(x[m].z, y[j].z, acc[m][j]); acc[m][j] = fmaf(x[m].w, y[j].w, acc[m][j]);
        }
    }
    for (int off = 1; off < nsl; off <<= 1)
#pragma unroll
      for (int m = 0; m < TA; m++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[m][j] += __shfl_xor_sync(0xffffffffu, acc[m][j], off);
    if (valid && ks == 0) {
#pragma unroll
      for (int m = 0; m < TA; m++)
#pragma unroll
        for (int j = 0; j < 4; j++)
          if (TA * bt + m < nA && 4 * ot + j < nB) out[(TA * bt + m) * ldo + 4 * ot + j] = acc[m][j];
    }
  }
}
// Up to four rows of A: a warp per row of B, the lanes take interleaved groups of four k and meet by shuffles (no blocks to
// set up: a single message costs 900-1,300 cycles instead of 1,600).
__device__ __forceinline__ void gemm_small(const float* __restrict__ A, const int lda, const int nA, const float* __restrict__ B, const int ldb,
                                           const int nB, const int K4, float* __restrict__ out, const int ldo) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float4* const A4 = reinterpret_cast<const float4*>(A);
  const float4* const B4 = reinterpret_cast<const float4*>(B);
  const int lda4 = lda >> 2, ldb4 = ldb >> 2;
  for (int o = warp; o < nB; o += FW) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k4 = lane; k4 < K4; k4 += 32) {
      const float4 w = B4[o * ldb4 + k4];
#pragma unroll
      for (int b = 0; b < 4; b++)
        if (b < nA) {
          const float4 x = A4[b * lda4 + k4];
          acc[b] = fmaf(x.x, w.x, acc[b]); acc[b] = fmaf(x.y, w.y, acc[b]); acc[b] = fmaf(x.z, w.z, acc[b]); acc[b] = fmaf(x.w, w.w, acc[b]);
        }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1)
#pragma unroll
      for (int b = 0; b < 4; b++) acc[b] += __shfl_xor_sync(0xffffffffu, acc[b], off);
    if (lane < nA) out[lane * ldo + o] = lane == 0 ? acc[0] : lane == 1 ? acc[1] : lane == 2 ? acc[2] : acc[3];
  }
}
// A handful of messages: one row of A per thread (nothing is spent on padding rows); otherwise 4 x 4 blocks.
__device__ __forceinline__ void gemm_nt(const float* __restrict__ A, const int lda, const int nA, const float* __restrict__ B, const int ldb,
                                        const int nB, const int K4, float* __restrict__ out, const int ldo) {
  if (nA <= 4 && K4 <= 128) gemm_small(A, lda, nA, B, ldb, nB, K4, out, ldo);
  else if (nA <= 8) gemm_nt_t<1>(A, lda, nA, B, ldb, nB, K4, out, ldo);
  else gemm_nt_t<4>(A, lda, nA, B, ldb, nB, K4, out, ldo);
}

// Columns [col0, col0 + ncols) of every message's payload are in M (shared memory, one row per message): a warp per
// message copies what falls into each landing's column range, rounded like every emitted payload.
__device__ __forceinline__ void deliver_cols(const TileS& S, const int pb, const float* __restrict__ M, const int ldm, const int count, const int col0, const int ncols) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b = warp; b < count; b += FW) {
    const int nd = S.nd[pb][b];
    for (int q = 0; q < nd; q++) {
      const Landing& L = S.dl[pb][b][q];
      if (L.act != ACT_PUSH || !L.dst) continue;
      const int lo = max(L.s0, col0), hi = min(L.s0 + L.w, col0 + ncols);
      for (int i = lo + lane; i < hi; i += 32) L.dst[i - L.s0] = emit_round(M[b * ldm + (i - col0)]);
    }
  }
}

// Local update of one parameter from its accumulated gradient (Sec. 3; the rule is a run-time option, App. A):
// g = A / n, then SGD, momentum-SGD (v <- mu v + g, theta <- theta - lr v) or Adam with bias correction, where t counts
// the updates of this node.
struct OptStep {
  int opt; float lr, inv_n, mu, b1, b2, eps, c1, c2; float *om, *ov;
  __device__ OptStep(const Ctx& C, const DevPPT& P, int n_upd, int upd_t)
      : opt(C.opt), lr(C.lr), inv_n(1.f / (float)n_upd), mu(C.mu), b1(C.beta1), b2(C.beta2), eps(C.eps), c1(1.f), c2(1.f),
        om(P.om), ov(P.ov) {
    if (opt == 2) {
      const double t = (double)(P.opt_t0 + upd_t);
      c1 = (float)(1.0 / (1.0 - pow((double)b1, t)));
      c2 = (float)(1.0 / (1.0 - pow((double)b2, t)));
    }
  }
  __device__ __forceinline__ void apply(float& w, float& a, const size_t k) const {
    if (opt == 0) { w = fmaf(-(lr * inv_n), a, w); a = 0.f; return; }
    apply_moments(w, a, k);
  }
  __device__ __noinline__ void apply_moments(float& w, float& a, const size_t k) const {
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

__device__ __forceinline__ int node_muf(const Ctx& C, const DevPPT& P) { return P.muf_override > 0 ? P.muf_override : C.muf; }

// ------------------------------------------------------------------------------------------------
// arrivals
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void ring_push(Ring& r, const Hdr& h, int it, int u, int port) {     // one thread
  const unsigned t = atomicAdd(r.tail, 1u);
  entry_store(&r.e[t & r.mask], h.inst, h.seq, h.slot, it, u, port, h.rows, h.flags, t + 1u);
}
// The instance in key slot `slot` loses `wgt` of its outstanding source messages (JOIN_UNIT each); the arrival that
// brings the count to zero tells the controller.
__device__ __noinline__ void retire_arrive(const Ctx& C, int slot, int wgt) {
  const int old = atom_add_acq_rel(&C.outstanding[slot], -wgt);
  if (old < wgt) fail(C, ST_OVERFLOW, -30, slot);                // more source messages came home than were pumped
  if (old != wgt) return;
  retire_push(C, slot);
}
// One thread, after the barrier behind the deposits of its CTA: arrive at landing L of message h with weight wgt.
__device__ __noinline__ void arrive(const Ctx& C, const int inst, const int seq, const int slot, const int flags, const int ibase, const Landing& L, int wgt,
                                    unsigned long long* node_msgs) {
  IN_SMEM(&L); IN_SMEM(node_msgs);
  int* const jcnt = reinterpret_cast<int*>(C.ctl_base + L.jcnt_off);
  Hdr h; h.inst = inst; h.seq = seq; h.slot = slot; h.it = 0; h.u = 0; h.port = 0; h.rows = ibase; h.flags = flags;
  if (L.act == ACT_RETIRE && L.expected) {                       // the message's arrivals meet first, then it retires whole
    if (atom_add_acq_rel(jcnt, wgt) + wgt != L.expected) return;
    *(volatile int*)jcnt = 0;
    if (L.clear_off) *reinterpret_cast<unsigned char*>(C.ctl_base + L.clear_off) = 0;
    if (L.clear2_off) *reinterpret_cast<unsigned char*>(C.ctl_base + L.clear2_off) = 0;
    if (L.post) atomicAdd(node_msgs, (unsigned long long)L.post);
    retire_arrive(C, slot, JOIN_UNIT);
    return;
  }
  if (L.act == ACT_RETIRE) {
    const int old = atom_add_acq_rel(jcnt, -wgt);
    if (old < wgt) fail(C, ST_OVERFLOW, -30, slot);
    if (old != wgt) return;
    if (L.post) atomicAdd(node_msgs, (unsigned long long)L.post);
    retire_push(C, slot);
    return;
  }
  if (L.act != ACT_PUSH) return;
  const int sum = atom_add_acq_rel(jcnt, wgt) + wgt;
  if (sum > L.expected) fail(C, ST_OVERFLOW, L.node, -31);       // more arrivals than the landing expects
  if (sum != L.expected) return;
  *(volatile int*)jcnt = 0;                                     // the key's next use finds the counter at zero
  if (L.clear_off) *reinterpret_cast<unsigned char*>(C.ctl_base + L.clear_off) = 0;
  if (L.clear2_off) *reinterpret_cast<unsigned char*>(C.ctl_base + L.clear2_off) = 0;
  atomicAdd(node_msgs, (unsigned long long)L.post);
  ring_push(g_ppts[L.ppt].ring[L.dir], h, L.it, L.u, L.port);
}

__device__ __forceinline__ unsigned long long ballot64(const bool p0, const bool p1) {
  return (unsigned long long)__ballot_sync(0xffffffffu, p0) | ((unsigned long long)__ballot_sync(0xffffffffu, p1) << 32);
}

// Warp 0 of a tile: take the next micro-batch from the node's rings, backward first (App. A) unless the backward queue is
// short and the forward queue longer (a cycle costs the same for 2 messages as for 64; max_active_keys bounds the
// forward supply, so the backward queue is always reached).  The batch is cut at the tile's row capacity, where
// training and forward-only messages meet, and exactly at the gradient that triggers the update (Sec. 3).
// dirs: bit 0 forward ring, bit 1 backward ring.  Returns 1 with the batch in S, 2 when the epoch is over, 0 when
// nothing is pending.
__device__ __noinline__ int form_batch(const Ctx& C, DevPPT& P, TileS& S, const bool leader, const bool fused, const int dirs, const bool light, const int min_take) {
  IN_SMEM(&P); IN_SMEM(&S);
  const int lane = threadIdx.x & 31;
  if (dirs == 1 && lane == 0) S.wver_seen = ld_acq(P.wver);          // (acquire: the published columns are read after this)
  // queue occupancy (first tile of the node): tickets handed out and not yet taken, read along with the ring polls
  unsigned pending = 0;
  if (leader && lane < 2 && (dirs & (1 << lane))) pending = ld_rlx(P.ring[lane].tail) - S.head[lane];
  constexpr int NPL = FBM / 32;                                      // ring slots per lane
  auto leading = [](const unsigned (&m)[NPL]) {                      // length of the run of set bits from candidate 0 on
    int n = 0;
#pragma unroll
    for (int j = 0; j < NPL; j++) { if (m[j] == 0xffffffffu) n += 32; else { n += __ffs((int)~m[j]) - 1; break; } }
    return n;
  };
  // First wave: the W entries at the head of each ring, one per lane (a tile that found nothing a moment ago watches
  // eight; the end of the epoch is polled along).  One round trip brings the messages themselves.
  const int W = light ? 8 : 32;
  Hdr hh[2];
  int nready[2];
  unsigned fin0 = 0;
  if (light && lane == 31) fin0 = ld_rlx(&C.g->done);
#pragma unroll
  for (int dir = 0; dir < 2; dir++) {
    bool ready = false;
    if ((dirs & (1 << dir)) && lane < W) {
      const unsigned t = S.head[dir] + (unsigned)lane;
      ready = entry_load(&P.ring[dir].e[t & P.ring[dir].mask], t + 1u, hh[dir]);
    }
    const unsigned m = __ballot_sync(0xffffffffu, ready);
    nready[dir] = m == 0xffffffffu ? 32 : __ffs((int)~m) - 1;
  }
  if (light && nready[0] == 0 && nready[1] == 0 && !__shfl_sync(0xffffffffu, fin0, 31)) return 0;
  if (leader && lane < 2 && pending > S.qmax[lane] && pending < (1u << 30)) S.qmax[lane] = pending;
  (void)min_take;
  if (nready[0] == 0 && nready[1] == 0) {
    unsigned fin = 0;
    if (lane == 0) fin = ld_acq(&C.g->done);
    if (!warp_uniform(fin)) return 0;
    // (the rings are empty for good only if nothing arrived between the polls and the flag: look once more)
    bool late = false;
    if (lane < 2 && (dirs & (1 << lane))) { Hdr x; const unsigned t = S.head[lane]; late = entry_load(&P.ring[lane].e[t & P.ring[lane].mask], t + 1u, x); }
    if (__any_sync(0xffffffffu, late)) return 0;
    if (lane == 0) {
      S.count = 0; S.dir = BWD; S.flags = BATCH_TERMINATE; S.n_upd = 0; S.upd_t = 0; S.eval = 0;
      if (S.n_acc > 0 && !C.eval) {                            // epoch-end flush of the leftover gradients
        S.flags |= BATCH_UPDATE; S.n_upd = S.n_acc; S.upd_t = (int)S.n_updates + 1;
        if (leader && S.log_n < P.update_log_cap) P.update_log[S.log_n] = S.n_upd;
        S.log_n++; S.n_updates++; S.n_grads_applied += S.n_upd; S.n_acc = 0; S.version++;
      }
    }
    __syncwarp();
    return 2;
  }
  const bool fwd_first = !(C.tune & 128) && nready[BWD] < 32 && nready[FWD] > nready[BWD];
  const int dir = (nready[BWD] == 0 || (fwd_first && nready[FWD] > 0)) ? FWD : BWD;
  const int cap = min(P.BM, FBM);
  int take = min(nready[dir], cap);
  Hdr* const out = S.hdr[S.fpb];
  if (lane < take) out[lane] = dir == FWD ? hh[FWD] : hh[BWD];
  if (nready[dir] == W && W < cap) {                             // the window was full: the entries behind it, straight into the batch
    unsigned m[NPL];
#pragma unroll
    for (int j = 0; j < NPL; j++) {
      const int idx = W + lane + 32 * j;
      bool ready = false;
      if (idx < cap) {
        Hdr x;
        const unsigned t = S.head[dir] + (unsigned)idx;
        ready = entry_load(&P.ring[dir].e[t & P.ring[dir].mask], t + 1u, x);
        if (ready) out[idx] = x;
      }
      m[j] = __ballot_sync(0xffffffffu, ready);
    }
    take = min(W + leading(m), cap);
  }
  __syncwarp();
  // the batch ends where training and forward-only messages meet
  const int eval0 = (out[0].flags & HDR_EVAL) != 0;
  {
    unsigned em[NPL];
#pragma unroll
    for (int j = 0; j < NPL; j++) em[j] = __ballot_sync(0xffffffffu, lane + 32 * j < take && (int)((out[lane + 32 * j].flags & HDR_EVAL) != 0) == eval0);
    take = leading(em);
  }
  bool upd = false;
  const bool grads = (dir == BWD || fused) && !eval0;          // a fused loss head turns every forward message into a gradient at once
  if (grads) {
    const int muf = node_muf(C, P);
    if (S.n_acc + take >= muf) { take = max(1, muf - S.n_acc); upd = true; }
  }
  if (lane == 0) {
    S.count = take; S.dir = dir; S.flags = upd ? BATCH_UPDATE : 0; S.eval = eval0;
    S.n_upd = upd ? S.n_acc + take : 0; S.upd_t = upd ? (int)S.n_updates + 1 : 0;
    S.head[dir] += take;
    S.msgs += grads && fused ? 2 * take : take; S.batches++; S.batch_rows += take;
    if (upd) {
      if (leader && S.log_n < P.update_log_cap) P.update_log[S.log_n] = S.n_upd;
      S.log_n++; S.n_updates++; S.n_grads_applied += S.n_upd; S.n_acc = 0; S.version++;
    } else if (grads) S.n_acc += take;
  }
  __syncwarp();
  return 1;
}

// Loss head shared by LT tiles: tile t takes the tickets t, t + LT, t + 2 LT, ... of the node's forward ring (a message is
// handled by exactly one tile), so S.head[FWD] counts own tickets.  Every ticket is one gradient (no forward-only message
// travels in such a run), so update number k falls due exactly when the tickets below k x muf have been handled (Sec. 3);
// a tile that has handled its own takes part in the exchange of the partial sums as soon as that ticket has been handed
// out, or, at the end of the epoch, in the flush of what is left.  Returns like form_batch; a batch may be empty
// (update only).
__device__ __noinline__ int form_batch_split(const Ctx& C, DevPPT& P, TileS& S, const bool leader, const int LT, const int t, const bool light) {
  IN_SMEM(&P); IN_SMEM(&S);
  const int lane = threadIdx.x & 31;
  const Ring& rg = P.ring[FWD];
  const bool training = !C.eval;
  const unsigned k0 = S.head[FWD], own_next = k0 * (unsigned)LT + (unsigned)t;
  const unsigned muf = (unsigned)node_muf(C, P);
  const unsigned long long done_grads = S.n_updates * (unsigned long long)muf, bnd = done_grads + muf;     // tickets below bnd belong to the next update
  // one round trip: the ring's tail, the end of the epoch, and the first W own entries themselves
  const int W = light ? 8 : 32;
  unsigned probe = 0;
  if (lane == 30) probe = ld_rlx(rg.tail);
  if (lane == 31) probe = ld_rlx(&C.g->done);
  Hdr h0;
  bool ready0 = false;
  if (lane < W) {
    const unsigned tk = (k0 + (unsigned)lane) * (unsigned)LT + (unsigned)t;
    if (!training || tk < bnd) ready0 = entry_load(&rg.e[tk & rg.mask], tk + 1u, h0);
  }
  const unsigned m0 = __ballot_sync(0xffffffffu, ready0);
  int nready = m0 == 0xffffffffu ? 32 : __ffs((int)~m0) - 1;
  const unsigned tail = __shfl_sync(0xffffffffu, probe, 30), fin0 = __shfl_sync(0xffffffffu, probe, 31);
  const bool at_boundary = training && own_next >= bnd;
  if (light && !fin0 && !(at_boundary ? tail >= bnd : nready > 0)) return 0;
  if (leader && lane == 0 && tail - own_next < (1u << 30) && tail - own_next > S.qmax[FWD]) S.qmax[FWD] = tail - own_next;
  auto close_epoch = [&]() {                       // after `done`: the ring's tail is final
    unsigned fin_tail = 0;
    if (lane == 0) { fence_acq(); fin_tail = ld_rlx(rg.tail); }
    fin_tail = __shfl_sync(0xffffffffu, fin_tail, 0);
    if (training && (long long)fin_tail - (long long)done_grads >= (long long)muf) return 0;      // (the tail read above was stale: a whole update is still due)
    if (lane == 0) {
      S.count = 0; S.dir = FWD; S.flags = BATCH_TERMINATE; S.n_upd = 0; S.upd_t = 0; S.eval = 0;
      const long long left = training ? (long long)fin_tail - (long long)done_grads : 0;
      if (left > 0) {                                          // epoch-end flush of the leftover gradients
        S.flags |= BATCH_UPDATE; S.n_upd = (int)left; S.upd_t = (int)S.n_updates + 1;
        if (leader && S.log_n < P.update_log_cap) P.update_log[S.log_n] = S.n_upd;
        S.log_n++; S.n_updates++; S.n_grads_applied += S.n_upd; S.version++;
      }
    }
    __syncwarp();
    return 2;
  };
  auto count_update = [&]() {                      // lane 0: the update that closes the period
    S.flags = BATCH_UPDATE; S.n_upd = (int)muf; S.upd_t = (int)S.n_updates + 1;
    if (leader && S.log_n < P.update_log_cap) P.update_log[S.log_n] = S.n_upd;
    S.log_n++; S.n_updates++; S.n_grads_applied += S.n_upd; S.version++;
  };
  if (at_boundary) {
    if (tail >= bnd) {
      if (lane == 0) { S.count = 0; S.dir = FWD; S.eval = 0; count_update(); }
      __syncwarp();
      return 1;
    }
    unsigned fin = 0;
    if (lane == 0) fin = ld_acq(&C.g->done);
    if (!warp_uniform(fin)) return 0;
    return close_epoch();
  }
  if (nready == 0) {
    unsigned fin = 0;
    if (lane == 0) fin = ld_acq(&C.g->done);
    if (!warp_uniform(fin)) return 0;
    return close_epoch();
  }
  constexpr int NPL = FBM / 32;
  const int cap = min(P.BM, FBM);
  Hdr* const out = S.hdr[S.fpb];
  if (lane < nready) out[lane] = h0;
  if (nready == W && W < cap) {                                  // the window was full: the own entries behind it
    unsigned m[NPL];
#pragma unroll
    for (int j = 0; j < NPL; j++) {
      const int idx = W + lane + 32 * j;
      bool ready = false;
      if (idx < cap) {
        Hdr x;
        const unsigned tk = (k0 + (unsigned)idx) * (unsigned)LT + (unsigned)t;
        if (!training || tk < bnd) ready = entry_load(&rg.e[tk & rg.mask], tk + 1u, x);
        if (ready) out[idx] = x;
      }
      m[j] = __ballot_sync(0xffffffffu, ready);
    }
    int more = 0;
#pragma unroll
    for (int j = 0; j < NPL; j++) { if (m[j] == 0xffffffffu) more += 32; else { more += __ffs((int)~m[j]) - 1; break; } }
    nready += more;
  }
  const int take = min(nready, cap);
  __syncwarp();
  if (lane == 0) {
    const int eval0 = (S.hdr[S.fpb][0].flags & HDR_EVAL) != 0;
    S.count = take; S.dir = FWD; S.flags = 0; S.eval = eval0; S.n_upd = 0; S.upd_t = 0;
    S.head[FWD] = k0 + (unsigned)take;
    S.msgs += training ? 2 * take : take; S.batches++; S.batch_rows += take;
    if (training && (k0 + (unsigned)take) * (unsigned)LT + (unsigned)t >= bnd && tail >= bnd) count_update();   // this tile's last tickets of the period
  }
  __syncwarp();
  return 1;
}

// ------------------------------------------------------------------------------------------------
// row tile
// ------------------------------------------------------------------------------------------------
#define TPHASE(k) do { if (tid == 0) { const long long n_ = clock64(); S.phase[k] += (unsigned long long)(n_ - tph); tph = n_; } } while (0)

// Softmax cross-entropy / squared error on the full output row y (this tile owns the whole node), as the Loss node
// defines it: records the loss and the arg-max hit under the Loss's key and writes the gradient the Loss sends back
// (rounded like every emitted payload) to g (training messages only).
__device__ __forceinline__ void loss_row(const Ctx& C, const int loss_node, const Hdr& h, const float* y, float* g, const int label_bits) {
  const DevNode& n = g_nodes[loss_node];
  const long long key = key_of(C, loss_node, h.slot, h.it, h.u, n.U_in);
  if (key < 0) return;
  const bool train = !(h.flags & HDR_EVAL);
  if (n.type == LOSS_CE) {
    const int label = label_bits;
    float mx = -3.4e38f; int arg = 0;
    for (int j = 0; j < n.in_dim; j++) if (y[j] > mx) { mx = y[j]; arg = j; }
    float s = 0.f;
    for (int j = 0; j < n.in_dim; j++) s += expf(y[j] - mx);
    const float lse = mx + logf(s);
    if (train) for (int j = 0; j < n.in_dim; j++) g[j] = emit_round(expf(y[j] - lse) - (j == label ? 1.f : 0.f));
    n.lossval[key] = lse - y[label]; n.predok[key] = (arg == label) ? 1 : 0;
  } else {
    const float d = y[0] - __int_as_float(label_bits);
    n.lossval[key] = d * d; n.predok[key] = 0;
    if (train) g[0] = emit_round(2.f * d);
  }
}

__device__ __noinline__ void tile_main(const Ctx& C, DevPPT& P, const int tile, float* smem, TileS& S, const unsigned long long t0) {
  IN_SMEM(&P); IN_SMEM(smem); IN_SMEM(&S);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int in = P.in_dim, out = P.out_dim;
  const bool lookup = P.kind == LOOKUP, leader = tile == 0;
  const DevNode& N = g_nodes[P.node];
  // A node that feeds a Loss is one tile and runs the whole exchange in one pass: forward, Loss, and the backward message
  // the Loss answers with (which App. A's backward-first rule would take next anyway), so its forward messages count
  // as gradients where the batch is cut.
  const int loss_node = (!lookup && (g_nodes[N.succ_node[0]].type == LOSS_CE || g_nodes[N.succ_node[0]].type == LOSS_MSE)) ? N.succ_node[0] : -1;
  const bool fused = loss_node >= 0;
  // Several tiles may share a loss head: each takes every LT-th message and owns it whole (all rows, the Loss, the way
  // back); the partial gradient sums meet at every update.  Runs with forward-only instances among the training ones
  // (whose messages are no gradients, so tickets do not count them) leave the node to its first tile.
  const int LT = fused ? max(1, P.LT) : 1;
  const bool split = LT > 1 && C.inference_only == nullptr;
  const int r_begin = fused ? 0 : tile * P.R;
  const int R = lookup ? 0 : max(0, min(P.R, out - r_begin));
  const int LW = pad_ldx(in), LX = pad_ldx(in), RP = pad_ldx(max(P.R, 1)), DXL = LX;
  const int wgt = fused ? JOIN_UNIT : tile == P.T - 1 ? JOIN_UNIT - (P.T - 1) * (JOIN_UNIT / P.T) : JOIN_UNIT / P.T;
  if (fused && LT > 1 && !split && tile > 0) {                 // nothing to do in this run: wait for its end
    if (tid == 0) {
      for (unsigned it = 0; !ld_acq(&C.g->done); it++) {
        if ((it & 63u) == 63u && (aborted(C) || gtime() - t0 > C.timeout_ns)) break;
        __nanosleep(500);
      }
    }
    __syncthreads();
    return;
  }
  // Every other Linear node is split by direction: row tiles (this function) take the forward ring, column tiles
  // (bwd_tile_main) the backward ring.  The column tiles own the master weights and accumulators; after an update they
  // publish their columns and the row tiles reload their rows before their next batch.
  const bool fwd_only = !lookup && !fused;
  const int dirs = fwd_only ? 1 : 3;
  // A tensor-core tile (bf16 runs, 64 rows, in_dim a multiple of 16) keeps its rows and the staged batch as bfloat16 in
  // the operand layout of the tensor cores; the master weights stay fp32 in the column tiles and in device memory.
  const bool tcm = fwd_only && P.tc;
  const int NT = (P.BM + 15) & ~15;                          // accumulator columns of a tensor-core product
  const size_t ws_floats = tcm ? (size_t)tc::M * in / 2 : (size_t)P.R * LW, xs_floats = tcm ? (size_t)NT * in / 2 : (size_t)P.BM * LX;
  float *Ws = smem, *bs = Ws + ws_floats, *Abs = bs + RP, *Xs = Abs + RP, *Ys = Xs + xs_floats, *Ds = Ys + (size_t)P.BM * RP,
        *As = Ds + (fused ? (size_t)P.BM * RP : 0), *Wt = As + (fused ? (size_t)P.R * LW : 0), *Dx = Xs,
        *smem_end = Wt + (fused ? (size_t)in * RP : 0);      // gradients, accumulators, transposed weights: loss head only; its input
                                                             // gradients take the place of the staged rows once those are used up
  unsigned char *const Wb = reinterpret_cast<unsigned char*>(Ws), *const Xb = reinterpret_cast<unsigned char*>(Xs);
  if (tcm) {
    for (float* q = smem + tid; q < smem_end; q += FT) *q = 0.f;
    __syncthreads();
    tc::fill_operand(Wb, R, in, [&](const int r) { return P.W + (size_t)(r_begin + r) * in; }, tid, FT);
    for (int i = tid; i < R; i += FT) bs[i] = P.b[r_begin + i];
    tc::fence_operands();
  } else if (!lookup) {
    for (float* q = smem + tid; q < smem_end; q += FT) *q = 0.f;
    __syncthreads();
    for (int i = tid; i < R * in; i += FT) { const int r = i / in, c = i - r * in; Ws[r * LW + c] = P.W[(size_t)r_begin * in + i]; }
    for (int i = tid; i < R; i += FT) bs[i] = P.b[r_begin + i];
    if (fused) {
      __syncthreads();
      for (int i = tid; i < R * in; i += FT) { const int r = i / in, c = i - r * in; Wt[c * RP + r] = Ws[r * LW + c]; }
    }
  }
  if (split && tile > 0 && P.om) {                               // private copy of the optimiser moments (all tiles step alike)
    const size_t PS = (size_t)out * in + out;
    float* const m = P.lh_mom + (size_t)(tile - 1) * 2 * PS;
    for (size_t i = tid; i < PS; i += FT) { m[i] = P.om[i]; m[PS + i] = P.ov ? P.ov[i] : 0.f; }
  }
  if (tid == 0) {
    S.head[0] = S.head[1] = 0; S.n_acc = 0; S.version = 0; S.log_n = 0; S.max_stale = 0; S.ok = 1; S.term = 0; S.arr_done = 0; S.qmax[0] = S.qmax[1] = 0;
    S.n_updates = S.n_grads_applied = S.msgs = S.batches = S.batch_rows = S.node_msgs = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&S.mbar)) : "memory");
    S.mbar_parity = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&S.tc_mbar)) : "memory");
    S.tc_parity = 0; S.tc_batches = 0;
  }
  if (tid < 64) S.stale_hist[tid] = 0;
  if (tid < 16) S.phase[tid] = 0;
  __syncthreads();
  long long tph = clock64();
  const FastDiv dR(max(R, 1)), dIn(in);
  const bool bulk_ok = !tcm && !lookup && (P.xcache != nullptr || ((in & 3) == 0 && (C.inst.dense_dim & 3) == 0));
  const int xwidth = P.xcache ? P.xld : in;

  // Front end of a batch (warps 0-3, 128 threads = one per message): warp 0 takes the batch from the rings, then every
  // message gets its key, its staging copy is issued and its route resolved.  It runs for batch n + 1 while the other warps
  // arrive for batch n.
  unsigned arr_target = 0;          // value of S.arr_done once the arrivals of every batch so far are done
  auto front = [&](const int pbn, const unsigned done_when) {
    if (warp == 0) {
      if (lane == 0) S.fpb = pbn;
      __syncwarp();
      unsigned it = 0;
      for (;;) {
        const bool arrivals_pending = false;       // the next batch is taken as soon as the arithmetic of this one is done
        (void)done_when;
        const int r = split ? form_batch_split(C, P, S, leader, LT, tile, it > 0)
                            : form_batch(C, P, S, leader, fused, dirs, it > 0 && !arrivals_pending, 1);
        if (r) break;
        if ((++it & 15u) == 0) {
          unsigned bad = 0;
          if (lane == 0) { bad = aborted(C); if (!bad && gtime() - t0 > C.timeout_ns) { fail(C, ST_TIMEOUT, P.node, 1); bad = 1; } }
          if (warp_uniform(bad)) { if (lane == 0) S.ok = 0; break; }
        }
        __nanosleep(it < 16 ? 20 : 100);
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    TPHASE(0);
    if (!S.ok) return;
    const int count = S.count, dir = S.dir;
    if (count == 0) return;                         // (uniform over the front warps: nobody reaches the staging barrier)
    // The cached input row of every message is staged by a bulk asynchronous copy (TMA, untiled) issued by the message's
    // thread and counted in bytes on a transaction barrier that all threads wait on before the arithmetic; the proxy fence
    // orders the issuing thread's view of the row (ordinary stores of other SMs, acquired through the ring) before the copy.
    const unsigned bar = smem_u32(&S.mbar);
    if (tid == 0 && bulk_ok) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"((unsigned)(count * xwidth * 4)) : "memory");
    // Two jobs per message, on different warps so that they run side by side: its key, staging copy and bookkeeping
    // (message m on thread m), and its route (message m on thread m + 64, spread over two warps; a batch of more than 64
    // messages wraps around, each thread then doing one job after the other).
    auto stage_job = [&](const int m) {
      const Hdr h = S.hdr[pbn][m];
      const long long key = key_of(C, P.node, h.slot, h.it, h.u, P.U);
      S.key[m] = key;
      if (key < 0) { S.ok = 0; return; }
      if (!lookup) {
        const float* x = P.xcache ? P.xcache + key * (long long)P.xld : C.inst.dense + (long long)h.inst * C.inst.dense_dim;
        S.rowptr[m] = x;
        if (bulk_ok) {
          asm volatile("fence.proxy.async;" ::: "memory");
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                       :: "r"(smem_u32(Xs + (size_t)m * LX)), "l"(x), "r"((unsigned)(xwidth * 4)), "r"(bar) : "memory");
        }
      }
      if (lookup) {
        const int id = C.inst.tokens[(long long)h.rows + h.u];
        S.rowid[m] = (unsigned)id < (unsigned)in ? id : -1;
      }
      if ((leader || split) && !S.eval && fused) atomicAdd(&S.stale_hist[0], 1ull);
      else if (leader && !S.eval && fwd_only) P.vcache[key] = max(S.version, (int)(S.wver_seen / (unsigned)P.TB));   // the version this forward pass uses (Sec. 3: staleness)
      if (fused) {                                     // the label, fetched while the input rows are in flight
        const DevInst& I = C.inst;
        if (g_nodes[loss_node].type == LOSS_CE) S.rowid[m] = I.labels_i[I.labels_per_node ? (long long)h.rows + h.u : h.inst];
        else S.rowid[m] = __float_as_int(I.labels_f[h.inst]);
      }
    };
    auto route_job = [&](const int m) {
      const Hdr h = S.hdr[pbn][m];
      int pre = 0, nd = 0;
      if (fused) {                                     // the Loss and this node's own backward arrival, then the way back
        if (!S.eval) nd = route_message(C, h, N.pred_node[0], N.pred_port[0], BWD, in, S.dl[pbn][m], pre);
        pre += S.eval ? 1 : 2;
      } else if (dir == FWD) nd = route_message(C, h, N.succ_node[0], N.succ_port[0], FWD, out, S.dl[pbn][m], pre);
      else nd = route_message(C, h, N.pred_node[0], N.pred_port[0], BWD, in, S.dl[pbn][m], pre);
      S.nd[pbn][m] = (unsigned char)nd; S.pre[pbn][m] = (short)pre;
    };
    {
      const int mr = tid >= 64 ? 2 * (tid & 31) + ((tid >> 5) & 1) : 64 + tid;        // message whose route this thread resolves
#pragma unroll 1
      for (int step = 0; step < 2; step++) {
        if ((tid >= 64) == (step == 0)) { if (mr < count) route_job(mr); }
        else if (tid < count) stage_job(tid);
      }
    }
    __syncwarp();
    TPHASE(1);
  };

  int pb = 0;
  if (warp < 4) front(0, 0u);
  __syncthreads();
  for (;;) {
    if (!S.ok) break;
    TPHASE(4);
    const int count = S.count, dir = S.dir, flags = S.flags, eval_n = S.eval, n_upd = S.n_upd, upd_t = S.upd_t;
    if (tcm && (int)(S.wver_seen / (unsigned)P.TB) > S.version) {
      tc::fill_operand(Wb, R, in, [&](const int r) { return P.W + (size_t)(r_begin + r) * in; }, tid, FT);
      for (int i = tid; i < R; i += FT) bs[i] = __ldcg(P.b + r_begin + i);
      tc::fence_operands();
      __syncthreads();
      if (tid == 0) S.version = (int)(S.wver_seen / (unsigned)P.TB);
      TPHASE(3);
    } else if (fwd_only && (int)(S.wver_seen / (unsigned)P.TB) > S.version) {      // every column tile has published a newer version
      for (int i = tid; i < R * in; i += FT) { const int r = dIn.div(i), c = i - r * in; Ws[r * LW + c] = __ldcg(P.W + (size_t)r_begin * in + i); }
      for (int i = tid; i < R; i += FT) bs[i] = __ldcg(P.b + r_begin + i);
      __syncthreads();
      if (tid == 0) S.version = (int)(S.wver_seen / (unsigned)P.TB);
      TPHASE(3);
    }
    // ---- the staged input rows of this batch ---------------------------------------------------------------
    if (count > 0) {
      if (bulk_ok && S.ok) {
        const unsigned bar = smem_u32(&S.mbar), parity = S.mbar_parity;
        unsigned done = 0, spins = 0;
        for (;;) {
          asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
          if (done) break;
          if ((++spins & 1023u) == 0 && (aborted(C) || gtime() - t0 > C.timeout_ns)) {
            if (tid == 0) fail(C, ST_TIMEOUT, P.node, 7);
            for (unsigned extra = 0; extra < (1u << 16) && !done; extra++)      // copies already issued still land in this CTA's shared memory
              asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
            break;
          }
        }
        __syncthreads();
        if (tid == 0) S.mbar_parity ^= 1u;
      }
      if (tcm) {                                              // the batch as the second operand: fp32 rows from the cache, stored as bfloat16
        tc::fill_operand(Xb, count, in, [&](const int b) { return S.rowptr[b]; }, tid, FT);
        tc::fence_operands();
        __syncthreads();
      } else if (!lookup && !bulk_ok) {
        for (int idx = tid; idx < count * in; idx += FT) { const int b = dIn.div(idx), c = idx - b * in; Xs[b * LX + c] = __ldcg(S.rowptr[b] + c); }
        __syncthreads();
      }
      if (!S.ok) break;
    }
    TPHASE(1);
    // ---- arithmetic and deposits -------------------------------------------------------------------------
    if (count > 0 && fused) {
      gemm_nt(Xs, LX, count, Ws, LW, R, pad4(in) >> 2, Ys, RP);
      __syncthreads();
      TPHASE(5);
      if (R <= 32) {
        // the Loss on G = 8, 16 or 32 lanes per message (lane j holds output j): maximum and arg-max (lowest index on ties),
        // sum of exponentials and the label's output by shuffles inside the group
        const int G = R <= 8 ? 8 : R <= 16 ? 16 : 32, per_pass = FT / G, j = tid & (G - 1);
        const DevNode& ln = g_nodes[loss_node];
        for (int m0 = 0; m0 < count; m0 += per_pass) {
          const int m = m0 + tid / G;
          const bool live = m < count, mine = live && j < R;
          const float y = mine ? emit_round(act_fwd(P.act, Ys[m * RP + j] + bs[j])) : -3.4e38f;
          float gj = 0.f;
          if (ln.type == LOSS_CE) {
            float mx = y; int arg = mine ? j : 0x7fffffff;
            for (int o = G >> 1; o; o >>= 1) {
              const float om = __shfl_xor_sync(0xffffffffu, mx, o, G); const int oa = __shfl_xor_sync(0xffffffffu, arg, o, G);
              if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
            }
            const float e = mine ? expf(y - mx) : 0.f;
            float sum = e;
            for (int o = G >> 1; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o, G);
            const float lse = mx + logf(sum);
            const int label = live ? S.rowid[m] : 0;
            const float ylab = __shfl_sync(0xffffffffu, y, label & (G - 1), G);
            gj = expf(y - lse) - (j == label ? 1.f : 0.f);
            if (live && j == 0) {
              const Hdr& h = S.hdr[pb][m];
              const long long lkey = key_of(C, loss_node, h.slot, h.it, h.u, ln.U_in);
              if (lkey >= 0) { ln.lossval[lkey] = lse - ylab; ln.predok[lkey] = (arg == label) ? 1 : 0; }
            }
          } else {
            const float d = y - __int_as_float(live ? S.rowid[m] : 0);
            gj = 2.f * d;
            if (live && j == 0) {
              const Hdr& h = S.hdr[pb][m];
              const long long lkey = key_of(C, loss_node, h.slot, h.it, h.u, ln.U_in);
              if (lkey >= 0) { ln.lossval[lkey] = d * d; ln.predok[lkey] = 0; }
            }
          }
          if (mine && !eval_n) Ds[m * RP + j] = emit_round(gj) * act_grad(P.act, y);
        }
      } else if (tid < count) {
        float* y = Ys + tid * RP;
        for (int r = 0; r < R; r++) y[r] = emit_round(act_fwd(P.act, y[r] + bs[r]));
        float* g = Ds + tid * RP;
        loss_row(C, loss_node, S.hdr[pb][tid], y, g, S.rowid[tid]);
        if (!eval_n) for (int r = 0; r < R; r++) g[r] *= act_grad(P.act, y[r]);
      }
      __syncthreads();
      TPHASE(6);
      if (!eval_n) {
        // A[r][k] += sum_b D[b][r] X[b][k]: a thread per (row, four columns) and slice of the batch; the slices meet in A
        {
          const int K4 = pad4(in) >> 2, units = R * K4;
          const int nsl = max(1, min(8, FT / max(units, 1)));
          for (int u0 = 0; u0 < units; u0 += FT / nsl) {
            const int u = u0 + tid / nsl, sl = tid % nsl;
            if (u < units && tid / nsl < FT / nsl) {
              const int r = u / K4, k4 = u - r * K4;
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 2
              for (int b = sl; b < count; b += nsl) {
                const float d = Ds[b * RP + r];
                const float4 x = *reinterpret_cast<const float4*>(Xs + b * LX + 4 * k4);
                a0 = fmaf(d, x.x, a0); a1 = fmaf(d, x.y, a1); a2 = fmaf(d, x.z, a2); a3 = fmaf(d, x.w, a3);
              }
              float* arow = As + r * LW + 4 * k4;
              atomicAdd(arow, a0); atomicAdd(arow + 1, a1); atomicAdd(arow + 2, a2); atomicAdd(arow + 3, a3);
            }
          }
        }
        __syncthreads();                                    // the staged rows are used up: dx takes their place
        TPHASE(15);
        // dx = D W (complete sums: the node is one tile), stored into the slots it lands in.  With a handful of rows a thread
        // keeps its column of W in registers and walks a strip of the batch: one 16-byte broadcast of D per four rows, one
        // coalesced store per message.  Wider heads go through the transposed weights and the staging rows.
        if (!(P.flags & 1) && R <= 16) {
          if (tid < count) {                                // the common landing: the whole row to one place
            const Landing& L = S.dl[pb][tid][0];
            const bool simple = S.nd[pb][tid] == 1 && L.act == ACT_PUSH && L.dst && L.s0 == 0 && L.w == in;
            S.rowptr[tid] = simple ? L.dst : nullptr;
          }
          __syncthreads();
          const int nstr = in < FT ? FT / in : 1;
          for (int ib = 0; ib < in; ib += FT) {
            const int st = in < FT ? dIn.div(tid) : 0, i = in < FT ? tid - st * in : ib + tid;
            if (st >= nstr || i >= in) continue;
            float w[16];
#pragma unroll
            for (int r = 0; r < 16; r++) w[r] = r < R ? Ws[r * LW + i] : 0.f;
            for (int b = st; b < count; b += nstr) {
              const float4* d4 = reinterpret_cast<const float4*>(Ds + b * RP);
              float v = 0.f;
#pragma unroll
              for (int q = 0; q < 4; q++)
                if (4 * q < R) {
                  const float4 d = d4[q];
                  v = fmaf(d.x, w[4 * q], v); v = fmaf(d.y, w[4 * q + 1], v); v = fmaf(d.z, w[4 * q + 2], v); v = fmaf(d.w, w[4 * q + 3], v);
                }
              v = emit_round(v);
              float* const row = const_cast<float*>(S.rowptr[b]);
              if (row) row[i] = v;
              else
                for (int q = 0; q < S.nd[pb][b]; q++) {
                  const Landing& L = S.dl[pb][b][q];
                  if (L.act == ACT_PUSH && L.dst && i >= L.s0 && i < L.s0 + L.w) L.dst[i - L.s0] = v;
                }
            }
          }
        } else if (!(P.flags & 1)) {
          gemm_nt(Ds, RP, count, Wt, RP, in, RP >> 2, Dx, DXL);
          __syncthreads();
          deliver_cols(S, pb, Dx, DXL, count, 0, in);
        }
        TPHASE(7);
        for (int r = warp; r < R; r += FW) {
          float a = 0.f;
          for (int b = lane; b < count; b += 32) a += Ds[b * RP + r];
          for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
          if (lane == 0) Abs[r] += a;
        }
      }
    } else if (count > 0 && !lookup) {
      if (dir == FWD) {
        if (tcm && count <= tc::SMALL_ROWS) {
          // a handful of messages is no dense contraction: FMA units, same bfloat16 operands
          for (int i = tid; i < count * RP; i += FT) Ys[i] = 0.f;
          __syncthreads();
          tc::small_product(Wb, Xb, in, count, Ys, RP, tid);
          __syncthreads();
        } else if (tcm) {
          // Y^T = W X^T on the tensor cores: one thread issues in_dim / 16 instructions, everybody waits for the commit
          // (bounded like every wait here), warps 0-3 move the accumulator from tensor memory to Ys[message][row].
          const unsigned bar = smem_u32(&S.tc_mbar), parity = S.tc_parity;
          if (tid == 0) { tc::issue(S.tmem, Wb, Xb, in, NT, bar); S.tc_batches++; }
          unsigned done = 0, spins = 0;
          for (;;) {
            asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
            if (done) break;
            if ((++spins & 1023u) == 0 && (aborted(C) || gtime() - t0 > C.timeout_ns)) {
              if (tid == 0) { fail(C, ST_TIMEOUT, P.node, 8); S.ok = 0; }
              for (unsigned extra = 0; extra < (1u << 16) && !done; extra++)        // instructions already issued still write the accumulator
                asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
              break;
            }
          }
          if (__all_sync(0xffffffffu, done != 0)) tc::read_accumulator(S.tmem, NT, count, Ys, RP, R);
          __syncthreads();
          if (tid == 0) S.tc_parity ^= 1u;
          if (!S.ok) break;
        } else {
          gemm_nt(Xs, LX, count, Ws, LW, R, pad4(in) >> 2, Ys, RP);
          __syncthreads();
        }
        TPHASE(5);
        for (int idx = tid; idx < count * R; idx += FT) {
          const int b = dR.div(idx), r = idx - b * R;
          const float y = emit_round(act_fwd(P.act, Ys[b * RP + r] + bs[r]));
          Ys[b * RP + r] = y;
          if (!eval_n) P.ycache[S.key[b] * out + r_begin + r] = y;
        }
        __syncthreads();
        TPHASE(6);
        // this tile's slice of every output row, straight into the buffers it lands in
        for (int idx = tid; idx < count * MAXD * R; idx += FT) {
          const int bq = dR.div(idx), r = idx - bq * R, q = bq % MAXD, b = bq / MAXD;
          if (q >= S.nd[pb][b]) continue;
          const Landing& L = S.dl[pb][b][q];
          const int c = r_begin + r;
          if (L.act == ACT_PUSH && L.dst && c >= L.s0 && c < L.s0 + L.w) __stcg(L.dst + (c - L.s0), L.zero ? 0.f : Ys[b * RP + r]);
        }
      }
    } else if (count > 0) {
      // Embedding table: its rows are dealt to the node's tiles (row id belongs to tile id % T).  Every tile sees every
      // message and arrives for it; the owner of the table row moves the data.
      __syncthreads();
      for (int b = warp; b < count; b += FW) {
        const int id = S.rowid[b];
        const bool mine = id >= 0 ? id % P.T == tile : leader;
        if (!mine) continue;
        constexpr int K = 5;                                // column chunks of 32 in flight per lane
        if (dir == FWD) {
          for (int q = 0; q < S.nd[pb][b]; q++) {
            const Landing& L = S.dl[pb][b][q];
            if (L.act != ACT_PUSH || !L.dst) continue;
            for (int cc = 0; cc < L.w; cc += 32 * K) {
              float v[K];
#pragma unroll
              for (int k = 0; k < K; k++) { const int c = cc + 32 * k + lane; v[k] = (id >= 0 && c < L.w) ? P.W[(size_t)id * out + L.s0 + c] : 0.f; }
#pragma unroll
              for (int k = 0; k < K; k++) { const int c = cc + 32 * k + lane; if (c < L.w) L.dst[c] = emit_round(v[k]); }
            }
          }
        } else {
          const float* g = P.gbuf + S.key[b] * (long long)P.NS * out;
          if (id >= 0) {
            float* arow = P.A + (size_t)id * out;
            for (int cc = 0; cc < out; cc += 32 * K) {
              float v[K];
#pragma unroll
              for (int k = 0; k < K; k++) { const int c = cc + 32 * k + lane; v[k] = c < out ? __ldcg(g + c) : 0.f; }
#pragma unroll
              for (int k = 0; k < K; k++) { const int c = cc + 32 * k + lane; if (c < out) atomicAdd(arow + c, emit_round(v[k])); }
            }
            if (lane == 0 && atomicExch(&P.touched_flag[id], 1) == 0)
              P.touched_list[(size_t)tile * ((in + P.T - 1) / P.T) + atomicAdd(P.touched_n + tile, 1)] = id;
          }
        }
      }
    }
    __syncthreads();
    TPHASE(2);
    // ---- local update (Sec. 3): theta <- theta - lr A / n, accumulator cleared ------------------------------
    if (flags & BATCH_UPDATE) {
      OptStep os(C, P, n_upd, upd_t);
      if (split && tile > 0 && P.om) {                       // tiles 1.. of a shared loss head keep their own (identical) moments
        os.om = P.lh_mom + (size_t)(tile - 1) * 2 * ((size_t)out * in + out);
        os.ov = os.om + ((size_t)out * in + out);
      }
      if (lookup) {
        __threadfence();
        int* const tlist = P.touched_list + (size_t)tile * ((in + P.T - 1) / P.T);
        const int nt = *(volatile int*)&P.touched_n[tile];
        for (int k = warp; k < nt; k += FW) {
          const int id = tlist[k];
          const size_t o0 = (size_t)id * out;
          constexpr int K = 5;
          for (int cc = 0; cc < out; cc += 32 * K) {
            float w[K], a[K];
#pragma unroll
            for (int j = 0; j < K; j++) { const int c = cc + 32 * j + lane; if (c < out) { w[j] = P.W[o0 + c]; a[j] = __ldcg(P.A + o0 + c); } }
#pragma unroll
            for (int j = 0; j < K; j++) { const int c = cc + 32 * j + lane; if (c < out) { os.apply(w[j], a[j], o0 + c); P.W[o0 + c] = w[j]; P.A[o0 + c] = a[j]; } }
          }
          if (lane == 0) P.touched_flag[id] = 0;
        }
        __syncthreads();
        if (tid == 0) P.touched_n[tile] = 0;
      } else {
        const size_t nW = (size_t)out * in;
        if (split) {
          // The tiles of a shared loss head put their partial sums side by side (two sets of buffers, by update parity: a
          // tile can be at most one exchange ahead of the slowest), count themselves, wait for the others and add the
          // partials in tile order, so that every tile applies the same update to its copy of the weights.
          const size_t PS = nW + (size_t)out;
          float* const mine = P.lh_part + ((size_t)(upd_t & 1) * LT + tile) * PS;
          for (int i = tid; i < R * in; i += FT) { const int r = dIn.div(i); mine[i] = As[r * LW + (i - r * in)]; }
          for (int i = tid; i < R; i += FT) mine[nW + i] = Abs[i];
          __syncthreads();
          if (tid == 0) {
            __threadfence();
            atom_add_acq_rel(P.lh_count, 1);
            const unsigned target = (unsigned)LT * (unsigned)upd_t;
            for (unsigned it = 0; ld_acq(reinterpret_cast<const unsigned*>(P.lh_count)) < target; it++) {
              if ((it & 63u) == 63u && (aborted(C) || gtime() - t0 > C.timeout_ns)) { fail(C, ST_TIMEOUT, P.node, 9); S.ok = 0; break; }
              __nanosleep(40);
            }
          }
          __syncthreads();
          if (!S.ok) break;
          const float* const all = P.lh_part + (size_t)(upd_t & 1) * LT * PS;
          for (int i = tid; i < R * in; i += FT) {
            float a = 0.f;
            for (int tt = 0; tt < LT; tt++) a += __ldcg(all + tt * PS + i);
            const int r = dIn.div(i);
            As[r * LW + (i - r * in)] = a;
          }
          for (int i = tid; i < R; i += FT) {
            float a = 0.f;
            for (int tt = 0; tt < LT; tt++) a += __ldcg(all + tt * PS + nW + i);
            Abs[i] = a;
          }
          __syncthreads();
        }
        for (int i = tid; i < R * in; i += FT) { const int r = dIn.div(i), o = r * LW + (i - r * in); os.apply(Ws[o], As[o], (size_t)r_begin * in + i); }
        for (int i = tid; i < R; i += FT) os.apply(bs[i], Abs[i], nW + r_begin + i);
        if (fused) {
          __syncthreads();
          for (int i = tid; i < R * in; i += FT) { const int r = dIn.div(i), c = i - r * in; Wt[c * RP + r] = Ws[r * LW + c]; }
        }
      }
      __syncthreads();
    }
    TPHASE(3);
    // ---- arrivals of this batch (warps 4-15) while warps 0-3 take the next batch and resolve its routes -------------------
    if (flags & BATCH_TERMINATE) break;
    if (warp < 4) front(pb ^ 1, arr_target + (unsigned)(FW - 4));
    else if (count > 0) {
      for (int idx = tid - 128; idx < count * MAXD; idx += FT - 128) {
        const int b = idx / MAXD, q = idx - b * MAXD;
        if (q == 0 && (leader || split) && S.pre[pb][b]) atomicAdd(&S.node_msgs, (unsigned long long)S.pre[pb][b]);
        if (q == 0 && fused && eval_n) retire_arrive(C, S.hdr[pb][b].slot, JOIN_UNIT);   // a forward-only instance ends at its Losses
        if (q >= S.nd[pb][b]) continue;
        const Hdr& h = S.hdr[pb][b];
        arrive(C, h.inst, h.seq, h.slot, h.flags, h.rows, S.dl[pb][b][q], wgt, &S.node_msgs);
      }
    }
    if (warp >= 4) { __syncwarp(); if (lane == 0) atomicAdd(&S.arr_done, 1u); }
    __syncthreads();
    TPHASE(4);
    arr_target += FW - 4;
    pb ^= 1;
  }
  // ---- epilogue: parameters back to device memory, statistics ----------------------------------------------
  __syncthreads();
  if (fused && leader) {
    for (int i = tid; i < R * in; i += FT) { const int r = i / in; P.W[(size_t)r_begin * in + i] = Ws[r * LW + (i - r * in)]; }
    for (int i = tid; i < R; i += FT) P.b[r_begin + i] = bs[i];
  }
  if (tid == 0 && S.node_msgs) atomicAdd(&C.g->node_messages, S.node_msgs);
  if (split && !leader && tid == 0) {                          // the node's counts are the sums over its tiles
    PPTStats& st = *P.stats;
    atomicAdd(&st.stale_hist[0], S.stale_hist[0]);
    atomicAdd(&st.msgs, S.msgs); atomicAdd(&st.batches, S.batches); atomicAdd(&st.batch_rows, S.batch_rows);
  }
  if (leader) {
    if (split) { if (tid == 0) atomicAdd(&P.stats->stale_hist[0], S.stale_hist[0]); }
    else if (!fwd_only && tid < 64) P.stats->stale_hist[tid] = S.stale_hist[tid];
    if (tid < (fwd_only ? 8 : 16)) P.stats->phase_cycles[tid] = S.phase[tid];
    if (tid == 0) {
      PPTStats& st = *P.stats;
      if (!fwd_only) { st.max_staleness = S.max_stale; st.log_n = S.log_n; st.n_updates = S.n_updates; st.n_grads_applied = S.n_grads_applied; }
      atomicAdd(&st.msgs, S.msgs); atomicAdd(&st.batches, S.batches); atomicAdd(&st.batch_rows, S.batch_rows);
      st.tc_batches = tcm ? S.tc_batches : 0;
      st.max_pending[0] = S.qmax[0];
      if (!fwd_only) st.max_pending[1] = S.qmax[1];
    }
  }
}

// ------------------------------------------------------------------------------------------------
// backward column tile of a Linear node
// ------------------------------------------------------------------------------------------------
// The tile owns input columns [c0, c0 + CB) of W for all output rows: the master copy of those weights in shared memory
// and their gradient accumulators in registers.  For a backward message it needs the whole pre-activation gradient
// dpre = g * act'(y) (g: the sum of the gradient slots under the key, y: the cached output) and its own columns of the
// cached input x.  Its columns of the input gradient dx = W^T dpre are complete sums: they are stored, not added, into
// the slot they land in.  A[:, cols] += dpre x[cols]^T.  After the update (Sec. 3) the tile writes its columns to the
// parameter array in device memory and counts itself in the node's version counter; the forward row tiles reload.

__device__ __noinline__ void bwd_tile_main(const Ctx& C, DevPPT& P, const int tile, float* smem, TileS& S, const unsigned long long t0) {
  IN_SMEM(&P); IN_SMEM(smem); IN_SMEM(&S);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int in = P.in_dim, out = P.out_dim, CB = P.CB, c4n = CB >> 2;
  const bool leader = tile == 0;
  const int c0 = tile * CB;
  const int GL = pad_ldx(out), WL = GL;          // row strides of dpre [batch][out] and of the transposed weights [column][out]
  const int wgt = tile == P.TB - 1 ? JOIN_UNIT - (P.TB - 1) * (JOIN_UNIT / P.TB) : JOIN_UNIT / P.TB;
  const DevNode& N = g_nodes[P.node];
  float *Wt = smem, *G = Wt + (size_t)CB * WL, *Xc = G + (size_t)P.BM * GL, *Dx = Xc + (size_t)P.BM * CB, *bsv = Dx + (size_t)P.BM * CB, *Abs = bsv + GL,
        *smem_end = Abs + GL;
  for (float* q = smem + tid; q < smem_end; q += FT) *q = 0.f;
  __syncthreads();
  for (int i = tid; i < out * CB; i += FT) { const int r = i / CB, c = i - r * CB; if (c0 + c < in) Wt[c * WL + r] = P.W[(size_t)r * in + c0 + c]; }
  if (leader) for (int i = tid; i < out; i += FT) bsv[i] = P.b[i];
  float A[4][4];                          // this thread's accumulators: rows 4 r4 .. 4 r4 + 3, columns 4 c4 .. 4 c4 + 3 of the tile
#pragma unroll
  for (int k = 0; k < 4; k++)
#pragma unroll
    for (int j = 0; j < 4; j++) A[k][j] = 0.f;
  const int n_units = ((out + 3) >> 2) * c4n;
  const int ur4 = tid >> (31 - __clz(c4n)), uc4 = tid & (c4n - 1);
  const FastDiv dOut(out);
  const int cb_shift = 31 - __clz(CB);
  if (tid == 0) {
    S.head[0] = S.head[1] = 0; S.n_acc = 0; S.version = 0; S.log_n = 0; S.max_stale = 0; S.ok = 1; S.term = 0; S.arr_done = 0; S.qmax[0] = S.qmax[1] = 0;
    S.n_updates = S.n_grads_applied = S.msgs = S.batches = S.batch_rows = S.node_msgs = 0;
  }
  if (tid < 64) S.stale_hist[tid] = 0;
  if (tid < 16) S.phase[tid] = 0;
  __syncthreads();
  long long tph = clock64();

  // Front end of a batch (warps 0-3): warp 0 takes the batch from the backward ring, then every message gets its key and
  // its route.  It runs for batch n + 1 while the other warps arrive for batch n.
  unsigned arr_target = 0;          // value of S.arr_done once the arrivals of every batch so far are done
  auto front = [&](const int pbn, const unsigned done_when) {
    if (warp == 0) {
      if (lane == 0) S.fpb = pbn;
      __syncwarp();
      unsigned it = 0;
      for (;;) {
        const bool arrivals_pending = false;       // the next batch is taken as soon as the arithmetic of this one is done
        (void)done_when;
        const int r = form_batch(C, P, S, leader, false, 2, it > 0 && !arrivals_pending, 1);
        if (r) break;
        if ((++it & 15u) == 0) {
          unsigned bad = 0;
          if (lane == 0) { bad = aborted(C); if (!bad && gtime() - t0 > C.timeout_ns) { fail(C, ST_TIMEOUT, P.node, 11); bad = 1; } }
          if (warp_uniform(bad)) { if (lane == 0) S.ok = 0; break; }
        }
        __nanosleep(it < 16 ? 20 : 100);
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    TPHASE(0);
    if (!S.ok) return;
    const int count = S.count, flags = S.flags;
    // key and bookkeeping of message m on thread m, its route on thread m + 64 (two warps side by side; see tile_main)
    {
      const int mr = tid >= 64 ? 2 * (tid & 31) + ((tid >> 5) & 1) : 64 + tid;
#pragma unroll 1
      for (int step = 0; step < 2; step++) {
        if ((tid >= 64) == (step == 0)) {
          if (mr < count) {
            int pre = 0;
            S.nd[pbn][mr] = (unsigned char)route_message(C, S.hdr[pbn][mr], N.pred_node[0], N.pred_port[0], BWD, in, S.dl[pbn][mr], pre);
            S.pre[pbn][mr] = (short)pre;
          }
        } else if (tid < count) {
          const Hdr h = S.hdr[pbn][tid];
          const long long key = key_of(C, P.node, h.slot, h.it, h.u, P.U);
          S.key[tid] = key;
          if (key < 0) S.ok = 0;
          else {
            S.rowptr[tid] = P.xcache ? P.xcache + key * (long long)P.xld : C.inst.dense + (long long)h.inst * C.inst.dense_dim;
            if (leader) {                                  // staleness: updates of this node between forward and backward (Sec. 3)
              int st = S.version - ((flags & BATCH_UPDATE) ? 1 : 0) - P.vcache[key];
              if (st < 0) st = 0;
              atomicAdd(&S.stale_hist[st > 63 ? 63 : st], 1ull);
              atomicMax(&S.max_stale, st);
            }
          }
        }
      }
    }
    __syncwarp();
    TPHASE(1);
  };

  int pb = 0;
  if (warp < 4) front(0, 0u);
  __syncthreads();
  for (;;) {
    if (!S.ok) break;
    TPHASE(6);
    const int count = S.count, flags = S.flags, n_upd = S.n_upd, upd_t = S.upd_t;
    if (count > 0) {
      TPHASE(1);
      // ---- operands: dpre for all rows, this tile's columns of x -------------------------------------------------
      {
        constexpr int U = 4;                              // elements per thread whose loads are in flight together
        const int total = count * out;
        for (int base = tid; base < total; base += FT * U) {
          float gv[U], g2[U], yv[U];
#pragma unroll
          for (int u = 0; u < U; u++) {
            const int idx = base + u * FT;
            gv[u] = g2[u] = yv[u] = 0.f;
            if (idx < total) {
              const int b = dOut.div(idx), r = idx - b * out;
              const float* g = P.gbuf + S.key[b] * (long long)P.NS * out + r;
              gv[u] = __ldcg(g);
              if (P.NS > 1) g2[u] = __ldcg(g + out);
              yv[u] = __ldcg(P.ycache + S.key[b] * (long long)out + r);
            }
          }
#pragma unroll
          for (int u = 0; u < U; u++) {
            const int idx = base + u * FT;
            if (idx < total) {
              const int b = dOut.div(idx), r = idx - b * out;
              float v = gv[u];
              if (P.NS > 1) {                             // successor order
                v += g2[u];
                for (int sl = 2; sl < P.NS; sl++) v += __ldcg(P.gbuf + (S.key[b] * (long long)P.NS + sl) * out + r);
                v = emit_round(v);
              }
              G[b * GL + r] = v * act_grad(P.act, yv[u]);
            }
          }
        }
      }
      for (int idx = tid; idx < count * CB; idx += FT) {
        const int b = idx >> cb_shift, c = idx - (b << cb_shift);
        Xc[idx] = c0 + c < in ? __ldcg(S.rowptr[b] + c0 + c) : 0.f;
      }
      __syncthreads();
      TPHASE(2);
      // ---- dx[b][cols] = sum_r dpre[b][r] W[r][cols], then straight into the slots the gradient lands in ----------------
      if (!(P.flags & 1)) {
        gemm_nt(G, GL, count, Wt, WL, CB, pad4(out) >> 2, Dx, CB);
        __syncthreads();
        deliver_cols(S, pb, Dx, CB, count, c0, min(CB, in - c0));
      }
      TPHASE(3);
      // ---- A[r][cols] += sum_b dpre[b][r] x[b][cols]: accumulators in registers --------------------------------------
      if (tid < n_units) {
#pragma unroll 2
        for (int b = 0; b < count; b++) {
          const float4 g = *reinterpret_cast<const float4*>(G + b * GL + 4 * ur4);      // columns beyond `out` are zero
          const float4 x = *reinterpret_cast<const float4*>(Xc + b * CB + 4 * uc4);
          A[0][0] = fmaf(g.x, x.x, A[0][0]); A[0][1] = fmaf(g.x, x.y, A[0][1]); A[0][2] = fmaf(g.x, x.z, A[0][2]); A[0][3] = fmaf(g.x, x.w, A[0][3]);
          A[1][0] = fmaf(g.y, x.x, A[1][0]); A[1][1] = fmaf(g.y, x.y, A[1][1]); A[1][2] = fmaf(g.y, x.z, A[1][2]); A[1][3] = fmaf(g.y, x.w, A[1][3]);
          A[2][0] = fmaf(g.z, x.x, A[2][0]); A[2][1] = fmaf(g.z, x.y, A[2][1]); A[2][2] = fmaf(g.z, x.z, A[2][2]); A[2][3] = fmaf(g.z, x.w, A[2][3]);
          A[3][0] = fmaf(g.w, x.x, A[3][0]); A[3][1] = fmaf(g.w, x.y, A[3][1]); A[3][2] = fmaf(g.w, x.z, A[3][2]); A[3][3] = fmaf(g.w, x.w, A[3][3]);
        }
      }
      if (leader) for (int r = tid; r < out; r += FT) { float a = Abs[r];
#pragma unroll 4
        for (int b = 0; b < count; b++) a += G[b * GL + r]; Abs[r] = a; }
      TPHASE(4);
    }
    // ---- local update (Sec. 3), then the columns go to device memory for the forward tiles ---------------------------
    if (flags & BATCH_UPDATE) {
      const OptStep os(C, P, n_upd, upd_t);
      if (tid < n_units) {
#pragma unroll
        for (int k = 0; k < 4; k++)
#pragma unroll
          for (int j = 0; j < 4; j++) {
            const int r = 4 * ur4 + k, c = c0 + 4 * uc4 + j;
            if (r < out && c < in) {
              float w = Wt[(4 * uc4 + j) * WL + r];
              os.apply(w, A[k][j], (size_t)r * in + c);
              Wt[(4 * uc4 + j) * WL + r] = w;
              P.W[(size_t)r * in + c] = w;
            } else A[k][j] = 0.f;
          }
      }
      if (leader) for (int r = tid; r < out; r += FT) { os.apply(bsv[r], Abs[r], (size_t)out * in + r); P.b[r] = bsv[r]; }
      __syncthreads();
      if (tid == 0) { __threadfence(); atomicAdd(P.wver, 1u); }
      TPHASE(5);
    }
    // ---- arrivals of this batch (warps 4-15) while warps 0-3 take the next batch and resolve its routes -------------------
    __syncthreads();
    if (flags & BATCH_TERMINATE) break;
    if (warp < 4) front(pb ^ 1, arr_target + (unsigned)(FW - 4));
    else if (count > 0) {
      for (int idx = tid - 128; idx < count * MAXD; idx += FT - 128) {
        const int b = idx / MAXD, q = idx - b * MAXD;
        if (q == 0 && leader && S.pre[pb][b]) atomicAdd(&S.node_msgs, (unsigned long long)S.pre[pb][b]);
        if (q >= S.nd[pb][b]) continue;
        const Hdr& h = S.hdr[pb][b];
        arrive(C, h.inst, h.seq, h.slot, h.flags, h.rows, S.dl[pb][b][q], wgt, &S.node_msgs);
      }
    }
    if (warp >= 4) { __syncwarp(); if (lane == 0) atomicAdd(&S.arr_done, 1u); }
    __syncthreads();
    TPHASE(6);
    arr_target += FW - 4;
    pb ^= 1;
  }
  __syncthreads();
  if (tid == 0 && S.node_msgs) atomicAdd(&C.g->node_messages, S.node_msgs);
  if (leader) {
    if (tid < 64) P.stats->stale_hist[tid] = S.stale_hist[tid];
    if (tid < 8) P.stats->phase_cycles[8 + tid] = S.phase[tid];
    if (tid == 0) {
      PPTStats& st = *P.stats;
      st.max_staleness = S.max_stale; st.log_n = S.log_n; st.n_updates = S.n_updates; st.n_grads_applied = S.n_grads_applied;
      atomicAdd(&st.msgs, S.msgs); atomicAdd(&st.batches, S.batches); atomicAdd(&st.batch_rows, S.batch_rows);
      st.max_pending[1] = S.qmax[1];
    }
  }
}

// ------------------------------------------------------------------------------------------------
// controller CTA: admission under max_active_keys, source messages, retirement (Sec. 3, Sec. 4)
// ------------------------------------------------------------------------------------------------
constexpr int OCC_SLOTS = 8192;
struct CtrlS {
  int ok;
  long long next, retired;
  int active;
  unsigned retire_head;
  int admit_slot, admit_inst, admit_seq, admit_eval, admit_rows;
  int src_count[4];
  unsigned long long node_msgs;
  unsigned occ[OCC_SLOTS / 32];
  Landing dl[MAXD];
  // kept on chip so that a retirement and the admission behind it wait for no load of the controller's own state
  int slot_inst[OCC_SLOTS];           // instance in each key slot (slots beyond this live in device memory only)
  int max_active;
  double total_loss, inf_loss;
  unsigned long long correct, n_pred, inf_instances, inf_correct, inf_pred;
  unsigned src_tail[4];               // tickets handed out in the ring each direct source feeds (the controller is its only producer)
  // the next instance to admit, looked up ahead of time
  int pf_valid, pf_inst, pf_rows, pf_eval, pf_outstanding, pf_count[4];
};

// A source whose messages carry no payload of their own and feed a parameterised node directly (token ids, leaf ids,
// the dense feature row): its headers go straight into that node's forward ring.
__device__ __forceinline__ bool source_is_direct(const DevNode& sn) {
  if (!(sn.fn == 1 || sn.fn == 2 || sn.fn == 4)) return false;
  const DevNode& dn = g_nodes[sn.succ_node[0]];
  return (dn.type == LINEAR || dn.type == LOOKUP) && g_ppts[dn.ppt].xcache == nullptr;
}

__device__ __noinline__ void controller_main(const Ctx& C, CtrlS& S, const unsigned long long t0) {
  IN_SMEM(&S);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const DevInst& I = C.inst;
  if (tid == 0) {
    S.next = 0; S.retired = 0; S.active = 0; S.retire_head = 0; S.ok = 1; S.node_msgs = 0; S.max_active = 0; S.pf_valid = 0;
    S.total_loss = S.inf_loss = 0.0; S.correct = S.n_pred = S.inf_instances = S.inf_correct = S.inf_pred = 0;
  }
  if (tid < 4) S.src_tail[tid] = 0;
  for (int i = tid; i < OCC_SLOTS / 32; i += FT) S.occ[i] = 0u;
  for (int i = tid; i < min(C.mak, OCC_SLOTS); i += FT) S.slot_inst[i] = -1;
  // every loss cell starts empty (predok = -1 marks "no loss evaluated at this key"); a retirement leaves its cells empty again
  for (int li = 0; li < C.n_loss; li++) {
    const DevNode& L = g_nodes[C.loss_nodes[li]];
    const long long cnt = (long long)C.mak * C.IT * L.U_in;
    for (long long k = tid; k < cnt; k += FT) { L.lossval[k] = 0.f; L.predok[k] = -1; }
  }
  __syncthreads();
  // Look up the next instance of the order: what it pumps and what finishes it (thread 0, while nothing waits for it).
  auto prefetch = [&]() {
    S.pf_valid = 0;
    if (S.next >= C.n_order) return;
    const int inst = (int)(C.order ? C.order[S.next] : S.next);
    int total = 0;
    for (int s = 0; s < C.n_sources; s++) {
      const DevNode& sn = g_nodes[C.src_nodes[s]];
      int cnt = 1;
      if (sn.fn == 2) cnt = (int)(I.offsets[inst + 1] - I.offsets[inst]);
      else if (sn.fn == 4) cnt = (int)(I.leaf_off[inst + 1] - I.leaf_off[inst]);
      S.pf_count[s] = cnt; total += cnt;
    }
    S.pf_eval = C.eval || (C.inference_only && C.inference_only[inst]);
    if (S.pf_eval) {      // forward only: the instance is finished when every Loss / Sink has been reached
      int exp = C.ends_per_instance;
      if (C.ends_per_position) exp += C.ends_per_position * (int)(I.offsets[inst + 1] - I.offsets[inst]);
      S.pf_outstanding = exp * JOIN_UNIT;
    } else S.pf_outstanding = total * JOIN_UNIT;
    S.pf_rows = (int)(I.offsets ? I.offsets[inst] : 0);
    S.pf_inst = inst; S.pf_valid = 1;
  };
  if (tid == 0) prefetch();
  __syncthreads();
  unsigned idle = 0;
  for (;;) {
    // ---- retirements: sum the instance's loss cells in key order, free the slot ------------------------------
    if (warp == 0) {
      for (;;) {
        unsigned h = 0, ready = 0, rs = 0;
        if (lane == 0) { h = S.retire_head; const unsigned long long v = retire_poll(C, h); ready = (unsigned)(v >> 32) == h + 1u; rs = (unsigned)v; }
        h = warp_uniform(h);
        if (!warp_uniform(ready)) break;
        const int slot = (int)warp_uniform(rs);
        if ((unsigned)slot >= (unsigned)C.mak) { if (lane == 0) fail(C, ST_OVERFLOW, -33, slot); break; }
        __syncwarp();
        if (lane == 0) S.retire_head = h + 1u;
        const int inst = slot < OCC_SLOTS ? S.slot_inst[slot] : C.slot_inst[slot];
        double tot = 0.0; int okc = 0, np = 0;
        for (int li = 0; li < C.n_loss; li++) {
          const DevNode& L = g_nodes[C.loss_nodes[li]];
          const long long k0 = (long long)slot * C.IT * L.U_in, k1 = k0 + (long long)C.IT * L.U_in;
          double dpart = 0.0;
          for (long long k = k0 + lane; k < k1; k += 32) {
            const int pk = __ldcg(&L.predok[k]);
            const float lv = __ldcg(&L.lossval[k]);               // (both loads in flight together)
            if (pk >= 0) { dpart += (double)lv; okc += pk; np += 1; L.lossval[k] = 0.f; L.predok[k] = -1; }
          }
          for (int o = 16; o; o >>= 1) dpart += __shfl_xor_sync(0xffffffffu, dpart, o);
          tot += dpart;
        }
        for (int o = 16; o; o >>= 1) { okc += __shfl_xor_sync(0xffffffffu, okc, o); np += __shfl_xor_sync(0xffffffffu, np, o); }
        if (lane == 0) {
          C.loss_out[inst] = (float)tot;
          if (C.inference_only && C.inference_only[inst]) { S.inf_loss += tot; S.inf_instances += 1; S.inf_correct += okc; S.inf_pred += np; }
          else { S.total_loss += tot; S.correct += okc; S.n_pred += np; }
          C.slot_inst[slot] = -1;
          if (slot < OCC_SLOTS) { S.slot_inst[slot] = -1; S.occ[slot >> 5] &= ~(1u << (slot & 31)); }
          S.active--; S.retired++;
        }
        __syncwarp();
      }
    }
    __syncthreads();
    // ---- admission -------------------------------------------------------------------------------------------
    for (;;) {
      if (tid == 0) {
        S.admit_slot = -1;
        if (S.active < C.mak && S.pf_valid) {
          int slot = 0;                                                   // lowest free slot
          const int nw = (min(C.mak, OCC_SLOTS) + 31) >> 5;
          int w = 0;
          while (w < nw && S.occ[w] == 0xffffffffu) w++;
          if (w < nw) slot = w * 32 + __ffs(~S.occ[w]) - 1;
          else { slot = OCC_SLOTS; while (slot < C.mak && C.slot_inst[slot] >= 0) slot++; }
          if (slot < OCC_SLOTS) S.occ[slot >> 5] |= 1u << (slot & 31);
          const int inst = S.pf_inst;
          if ((slot < OCC_SLOTS ? S.slot_inst[slot] : C.slot_inst[slot]) >= 0) fail(C, ST_OVERFLOW, -32, slot);
          S.admit_slot = slot; S.admit_inst = inst; S.admit_seq = (int)S.next; S.admit_eval = S.pf_eval;
          for (int s = 0; s < C.n_sources; s++) S.src_count[s] = S.pf_count[s];
          C.slot_inst[slot] = inst;
          if (slot < OCC_SLOTS) S.slot_inst[slot] = inst;
          S.active++;
          if (S.active > S.max_active) S.max_active = S.active;
          C.outstanding[slot] = S.pf_outstanding;
          S.admit_rows = S.pf_rows;
          S.next++;
        }
      }
      __syncthreads();
      const int slot = S.admit_slot;
      if (slot < 0) break;
      // pump the source messages (Sec. 4: tokens / leaves, initial hidden state, dense row); the stores above (the slot's
      // bookkeeping, the emptied loss cells of its previous instance) are ordered before them by the entries' release
      const int inst = S.admit_inst;
      Hdr h; h.inst = inst; h.seq = S.admit_seq; h.slot = slot; h.it = 0; h.u = 0; h.port = 0; h.rows = S.admit_rows; h.flags = S.admit_eval ? HDR_EVAL : 0;
      for (int s = 0; s < C.n_sources; s++) {
        const DevNode& sn = g_nodes[C.src_nodes[s]];
        const int cnt = S.src_count[s];
        if (source_is_direct(sn)) {
          DevPPT& P = g_ppts[g_nodes[sn.succ_node[0]].ppt];
          for (int c0 = warp * 32; c0 < cnt; c0 += FW * 32) {
            const int k = c0 + lane;
            int u = 0;
            if (k < cnt) u = sn.fn == 2 ? k : sn.fn == 4 ? I.leaf_ids[I.leaf_off[inst] + k] : 0;
            const bool okm = k < cnt && key_of(C, sn.succ_node[0], slot, 0, u, P.U) >= 0;
            const unsigned vm = __ballot_sync(0xffffffffu, okm);
            unsigned tk = 0;
            if (lane == 0 && vm) tk = atomicAdd(&S.src_tail[s], (unsigned)__popc(vm));     // (shared memory: the only producer of this ring)
            tk = __shfl_sync(0xffffffffu, tk, 0) + (unsigned)__popc(vm & ((1u << lane) - 1u));
            if (okm) {
              entry_store(&P.ring[FWD].e[tk & P.ring[FWD].mask], inst, S.admit_seq, slot, 0, u, 0, h.rows, h.flags, tk + 1u);
            }
            if (lane == 0 && vm) atomicAdd(&S.node_msgs, (unsigned long long)__popc(vm));
          }
        } else if (warp == 0) {                     // a zero vector (initial hidden state) routed to where it lands
          int pre = 0, nd = 0;
          if (lane == 0) {
            nd = route_message(C, h, sn.succ_node[0], sn.succ_port[0], FWD, sn.out_dim, S.dl, pre);
            for (int q = 0; q < nd; q++) S.dl[q].zero = 1;
          }
          nd = (int)warp_uniform((unsigned)nd);
          __syncwarp();
          for (int q = 0; q < nd; q++) {
            const Landing& L = S.dl[q];
            if (L.act == ACT_PUSH && L.dst) for (int c = lane; c < L.w; c += 32) L.dst[c] = 0.f;
          }
          __syncwarp();
          if (lane == 0) {
            if (pre) atomicAdd(&S.node_msgs, (unsigned long long)pre);
            for (int q = 0; q < nd; q++) arrive(C, h.inst, h.seq, h.slot, h.flags, h.rows, S.dl[q], JOIN_UNIT, &S.node_msgs);
          }
          __syncwarp();
        }
      }
      __syncthreads();
      if (tid == 0) {
        for (int s = 0; s < C.n_sources; s++) {                 // the tickets handed out, for the tiles that read the ring's tail
          const DevNode& sn = g_nodes[C.src_nodes[s]];
          if (source_is_direct(sn)) *(volatile unsigned*)g_ppts[g_nodes[sn.succ_node[0]].ppt].ring[FWD].tail = S.src_tail[s];
        }
        prefetch();
      }
      __syncthreads();
    }
    // ---- termination / pacing ---------------------------------------------------------------------------------
    const bool finished = S.retired == C.n_order;
    if (finished) {
      if (tid == 0) {
        Globals& G = *C.g;
        G.max_active = S.max_active; G.total_loss = S.total_loss; G.correct = S.correct; G.n_pred = S.n_pred;
        G.inf_loss = S.inf_loss; G.inf_instances = S.inf_instances; G.inf_correct = S.inf_correct; G.inf_pred = S.inf_pred;
        G.rounds = 0; atomicAdd(&G.node_messages, S.node_msgs); __threadfence(); st_rel(&G.done, 1u);
      }
      break;
    }
    if (tid == 0) {
      S.ok = 1;
      if ((++idle & 15u) == 0) {
        if (aborted(C)) S.ok = 0;
        else if (gtime() - t0 > C.timeout_ns) { fail(C, ST_TIMEOUT, -1, 2); S.ok = 0; }
      }
      const unsigned hh = S.retire_head;
      unsigned spins = 0;
      while ((unsigned)(retire_poll(C, hh) >> 32) != hh + 1u && spins < 64) { __nanosleep(50); spins++; }
    }
    __syncthreads();
    if (!S.ok) break;
  }
}

union FastShared { TileS t; CtrlS c; };

}  // namespace ampf

__global__ void __launch_bounds__(ampf::FT, 1) ampnet_engine_direct(const __grid_constant__ amp::Ctx C) {
  using namespace ampf;
  extern __shared__ __align__(16) float dyn_smem[];
  __shared__ FastShared SU;
  const unsigned long long t0 = gtime();
  {
    const int* src = reinterpret_cast<const int*>(C.nodes);
    int* dst = reinterpret_cast<int*>(g_nodes);
    for (int i = threadIdx.x; i < C.n_nodes * (int)(sizeof(DevNode) / 4); i += FT) dst[i] = src[i];
    src = reinterpret_cast<const int*>(C.ppts);
    dst = reinterpret_cast<int*>(g_ppts);
    for (int i = threadIdx.x; i < C.n_ppts * (int)(sizeof(DevPPT) / 4); i += FT) dst[i] = src[i];
  }
  if (threadIdx.x == 0) g_bf16 = C.bf16;
  __syncthreads();
  const Role role = C.roles[blockIdx.x];
  if (role.ppt < 0) controller_main(C, SU.c, t0);
  else if (role.kind == 3) bwd_tile_main(C, g_ppts[role.ppt], role.tile, dyn_smem, SU.t, t0);
  else {
    // a tensor-core tile holds tensor-memory columns for its accumulator for the whole run; every way out of
    // tile_main comes back here, so they are always given back
    const bool tcm = g_ppts[role.ppt].tc != 0 && g_ppts[role.ppt].kind == LINEAR;
    if (tcm) {
      if (threadIdx.x < 32) tc::tmem_alloc(&SU.t.tmem);
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    tile_main(C, g_ppts[role.ppt], role.tile, dyn_smem, SU.t, t0);
    if (tcm) {
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();
      if (threadIdx.x < 32) tc::tmem_free(SU.t.tmem);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// host side: what the launch needs to know
// ------------------------------------------------------------------------------------------------
namespace ampf {
size_t tile_smem_floats(int in, int R, int BM, int loss_head) {
  const size_t LW = pad_ldx(in), LX = pad_ldx(in), RP = pad_ldx(R > 0 ? R : 1);
  return (size_t)R * LW + 2 * RP + (size_t)BM * LX + (size_t)BM * RP +
         (loss_head ? (size_t)BM * RP + (size_t)R * LW + (size_t)in * RP : 0);
}
}  // namespace ampf

namespace ampf {
size_t bwd_tile_smem_floats(int out, int cb, int BM) { const size_t GL = pad_ldx(out); return (size_t)cb * GL + (size_t)BM * GL + 2 * (size_t)BM * cb + 2 * GL; }
}  // namespace ampf
extern "C" size_t ampnet_direct_bwd_tile_smem_bytes(int out_dim, int cols, int batch_rows) { return ampf::bwd_tile_smem_floats(out_dim, cols, batch_rows) * sizeof(float) + 64; }
extern "C" int ampnet_direct_max_units() { return 4 * ampf::FT; }    // out_dim x (columns / 4) of a backward tile may not exceed this
extern "C" int ampnet_direct_threads() { return ampf::FT; }
extern "C" void ampnet_direct_limits(int* max_nodes, int* max_ppts, int* max_landings, int* batch_rows) {
  *max_nodes = ampf::DIRECT_MAX_NODES; *max_ppts = ampf::DIRECT_MAX_PPTS; *max_landings = ampf::MAXD; *batch_rows = ampf::FBM;
}
// shared memory of a tensor-core forward tile: 64 rows and the batch (rounded up to 16 messages) as bfloat16, bias, outputs
extern "C" size_t ampnet_direct_tc_tile_smem_bytes(int in_dim, int batch_rows) {
  const size_t RP = ampf::pad_ldx(tc::M), NT = (size_t)((batch_rows + 15) & ~15);
  return (size_t)tc::M * in_dim * 2 + 2 * RP * sizeof(float) + NT * in_dim * 2 + (size_t)batch_rows * RP * sizeof(float) + 64;
}
extern "C" void ampnet_direct_tc_limits(int* rows, int* max_batch_rows, int* k_multiple) { *rows = tc::M; *max_batch_rows = tc::TMEM_COLS; *k_multiple = 16; }
extern "C" size_t ampnet_direct_tile_smem_bytes(int in_dim, int rows, int batch_rows, int loss_head) {
  return ampf::tile_smem_floats(in_dim, rows, batch_rows, loss_head) * sizeof(float) + 64;
}
extern "C" cudaError_t ampnet_direct_static_smem(size_t* bytes) {
  cudaFuncAttributes fa{};
  const cudaError_t e = cudaFuncGetAttributes(&fa, ampnet_engine_direct);
  *bytes = fa.sharedSizeBytes;
  return e;
}
extern "C" cudaError_t ampnet_direct_launch(const amp::Ctx* ctx, int n_ctas, size_t smem_bytes, cudaStream_t stream, int n_sms) {
  cudaError_t e = cudaFuncSetAttribute(ampnet_engine_direct, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ampnet_engine_direct, ampf::FT, smem_bytes);
  if (e != cudaSuccess) return e;
  if (per_sm < 1 || (long long)per_sm * n_sms < n_ctas) return cudaErrorCooperativeLaunchTooLarge;
  void* args[] = {const_cast<amp::Ctx*>(ctx)};
  return cudaLaunchCooperativeKernel((void*)ampnet_engine_direct, dim3(n_ctas), dim3(ampf::FT), args, smem_bytes, stream);
}
