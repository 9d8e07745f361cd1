// Paired-row-block tensor-core attention kernel for sm_100a (head_dim 128,
// block 128): dense (pivot) and block-sparse (member) causal attention.
//
//   Section 5.1:  O = softmax(Q K^T / sqrt(d) - c (1 - M)) V,  c -> infinity,
//   causal.  A pivot walks every causal key-block and also emits the softmax
//   probability mass of each (query-block, key-block) tile; a member walks the
//   compacted list of key-blocks its cluster's pivot selected.
//
// Persistent CTAs, one per SM.  A work item is TWO tiles of 128 query rows that
// read the same KV head: two adjacent row-blocks of one head (tile A = row-block
// 2u, tile B = row-block 2u+1) or, where two heads of one KV head walk the same
// list (two members of a cluster, two dense heads), the same row-block of both.
// The items of a launch are ordered (the heads of one KV head together, the
// longest pairs first) and handed out through a device counter, so an SM that
// finishes early takes the next item; barriers and tensor memory are set up once
// per CTA, and the loads and the first QK^T of the next item are issued while the
// softmax warps still write out the item before.  The two tiles walk the UNION
// of their key-block lists in ascending order, so a K/V tile both of them need
// is brought into shared memory once and feeds four MMAs instead of two; a
// key-block only one of them selected is computed for that tile alone.  (Dense,
// one head: the union is 0..2u+1, the last key-block is B's diagonal tile only.
// Two heads on one list: the lists are equal and every K/V tile serves both.)
//
// Warp roles (320 threads):
//   warps 0-3   softmax of tile A: thread t owns query row t = TMEM lane t
//   warps 4-7   softmax of tile B
//   warp  8     MMA issuer, owner of the TMEM allocation (all 512 columns:
//               S_A, S_B, O_A, O_B, 128 fp32 columns each)
//   warp  9     producer: takes the next item from the counter, resolves it to
//               (head, pair, list, counts) and posts it in a two-slot ring of
//               shared memory that the other nine warps read (it runs ahead of
//               them by the depth of the K/V rings, so they find the item
//               waiting); merges the two lists; TMA loads of Q (once per item)
//               and of the K and V tiles into two-stage rings (128-byte swizzle)
//
// The kernel is sensitive to the size of its hot loops (an eleventh warp for the
// scheduling, bounded waits inlined at every site and the phase trace compiled
// into the loops cost 3 %, 3 % and 2 % of the layer): rare paths are kept out
// of line.
//
// Rings, barrier phases and named-barrier ids run on across items (every role
// counts key-blocks, tile steps and items for itself).
//
// Order of the MMAs, per merged key-block n:  PV_A(n), QK_A(n+1), PV_B(n),
// QK_B(n+1), all issued by one thread: while the softmax warps of A work on
// S_A(n) the tensor pipe runs PV_B(n-1) and QK_B(n); while those of B work on
// S_B(n) it runs PV_A(n) and QK_A(n+1).  (One issuer per tile was tried: the two
// tiles then fall into step, their softmax phases coincide and nothing overlaps
// the MMAs.)  P (bf16) overwrites the first half of the S columns it came from
// and is the TMEM A operand of PV; the next QK of that tile is issued after the
// PV that reads P, and the tensor pipe keeps issue order.
//
// What bounds the kernel: three things within a tenth of one another.  The issuing
// warp: the tensor pipe accepts an MMA only a couple of instructions ahead, and the
// issuing thread needs about twenty dependent instructions per tcgen05.mma
// (election, moves into uniform registers), on a scheduler it shares with two
// softmax warps; with the softmax arithmetic switched off (timing-only copy) a
// key-block still takes 3200 cycles against 2048 of tensor work, 3500 with it.
// Each tile's chain: S ready -> softmax -> P -> its sixteen MMAs -> S ready, 3400
// cycles, and TMEM holds two tiles.  The schedulers: each hosts one softmax warp of
// each tile, 2800 cycles of arithmetic per key-block.  So everything the issuing
// warp does per key-block is kept short: every shared-memory descriptor and barrier
// address is a compile-time constant (dynamic shared memory starts at offset
// 0x400 of the CTA's window and a whole-TMEM allocation at column 0; both are
// checked at kernel start, and the loop is unrolled over the two ring stages so
// that the stage is a constant too), and P is handed over once per tile and
// key-block (handing it over in two halves let the first PV start earlier but
// cost the issuing warp two more barrier syncs per key-block: 2 % slower).
//
// Hand-offs.  Completion of MMAs and of TMA copies arrives on mbarriers
// (tcgen05.commit, complete_tx).  What the issuing warp waits for comes through
// named barriers instead: a poll of an mbarrier is a shared-memory round trip,
// 150-250 cycles while the tensor pipe streams operands at the shared-memory
// limit (probing them one key-block ahead was tried: 1 % slower than the relay).
// The softmax warps `bar.arrive` when P is stored, the producer warp relays "K
// of the next key-block and V of this one have landed", the issuing warp
// `bar.sync`s.  The relay ids are taken in turn over four barriers: the producer
// makes the last relay of an item right after the one before it, so two arrivals
// can be pending before the issuing warp has taken the first.
//
// Block importance in one pass: as in the single-tile kernel, each softmax
// thread spills one float per visited tile, stat = m + log2(sum_c 2^(s_c - m))
// with m the row's reference max at that step; after the last tile the row's
// log-sum-exp L is known and the tile mass is (1/B) sum_rows 2^(stat - L).
// The statistics of an item live only until its epilogue, so each CTA owns one
// region of 2 * Nb * B floats that every item it runs writes and reads in turn.
//
// Every wait on an mbarrier is bounded: when it runs out the CTA raises an abort
// flag, records SP_ERR_TIMEOUT in the status word, and all roles fall through
// to the common teardown (TMEM is freed, the kernel returns).  The named-barrier
// syncs of the issuing warp have no limit of their own; they end because every
// arrival they count is reached through bounded waits only, and is made also
// when such a wait ran out (the warp that gave up arrives once more for the
// step it was in, on ids taken in turn so that an early arrival never lands in
// a phase the issuing warp has not left; the issuing warp looks at the abort
// flag after the last sync of every key-block).
#include <type_traits>

#include "tc_ptx.cuh"

namespace sp {
namespace {

using namespace tc;

constexpr int D = 128;      // head_dim
constexpr int BLK = 128;    // block
constexpr int kThreadsPair = 320;   // eight softmax warps, the issuing warp, the producer warp
constexpr int kItemReaders = 9;       // warps that take every posted item: all but the producer, which posts it
constexpr int kStages = 2;  // K ring and V ring depth

// shared-memory plan (bytes)
constexpr int kBox = 128 * 128;                 // one 64-column box of 128 rows
constexpr int kTile = 2 * kBox;                 // a 128 x 128 bf16 tile (two boxes)
constexpr int kQOff = 0;                        // [box][tile A|B][128 rows][128 B]
constexpr int kKOff = kQOff + 2 * kTile;        // [stage][box][128 rows][128 B]
constexpr int kVOff = kKOff + kStages * kTile;
constexpr int kMiscOff = kVOff + kStages * kTile;
constexpr int kMiscBytes = 2048;
constexpr int kSmemTotal = kMiscOff + kMiscBytes + 1024;   // + slack for 1024-byte alignment

// TMEM columns
constexpr uint32_t kSCol = 0;      // S_A at 0, S_B at 128 (P reuses the first 64 columns of each)
constexpr uint32_t kOCol = 256;    // O_A at 256, O_B at 384

enum {
  BAR_Q_FULL = 0,
  BAR_Q_EMPTY,
  BAR_K_FULL,                          // + stage
  BAR_K_EMPTY = BAR_K_FULL + kStages,  // + stage
  BAR_V_FULL = BAR_K_EMPTY + kStages,
  BAR_V_EMPTY = BAR_V_FULL + kStages,
  BAR_S_FULL = BAR_V_EMPTY + kStages,  // + tile (A = 0, B = 1)
  BAR_O_DONE = BAR_S_FULL + 2,
  BAR_ITEM_FULL = BAR_O_DONE + 2,      // + item slot
  BAR_ITEM_EMPTY = BAR_ITEM_FULL + 2,
  BAR_COUNT = BAR_ITEM_EMPTY + 2
};
static_assert(BAR_COUNT * 8 <= 256, "barriers overlap the TMEM slot");

enum { F_A = 1, F_B = 2, F_LAST = 4 };

// Named barriers (0 is __syncthreads, 1 and 2 the epilogues of the two tiles): P of tile x ready (the four softmax
// warps of the tile arrive, the issuing warp syncs), and K/V tiles of a merged key-block landed (the producer warp
// arrives, the issuing warp syncs).  Ids are taken in turn — two per tile for P, four for K/V — so that an arrival
// that comes early (the producer's last relay of an item, the release after a wait ran out) never lands in a phase
// the other side has not left yet.
enum { NB_P = 3, NB_KV = 11 };   // P: id NB_P + 4 * tile + 2 + (step & 1); K/V: id NB_KV + (relay & 3)

// ------------------------------------------------------------------ small PTX helpers of this kernel

__device__ __forceinline__ void tmem_ld32_async(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// Waits for this thread's outstanding tcgen05.ld and pins the 32 registers behind the wait,
// so that nothing that reads them can be scheduled ahead of it.
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void reg_fence32(uint32_t* r) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]),
                 "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]),
                 "+r"(r[30]), "+r"(r[31])::"memory");
}

// 16 consecutive 32-bit columns of this thread's TMEM lane <-> registers
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// The tile statistics are written once and read once by the same CTA about an item later; with the K/V tiles
// streaming through L2 they were evicted to DRAM in between (two thirds of K1's DRAM traffic).  Their lines are
// therefore stored with the evict-last priority and read with evict-first (dead after the read).
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_f32_hint(float* addr, float v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(addr), "f"(v), "l"(policy) : "memory");
}
__device__ __forceinline__ float4 ld_f32x4_hint(const float* addr, uint64_t policy) {
  float4 v;
  asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(addr), "l"(policy)
               : "memory");
  return v;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// bf16x2 with `lo` in the low half
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}


// Compile-time shared-memory addresses: dynamic shared memory starts at this offset of the CTA's shared window
// (checked at kernel start), so every descriptor and barrier address of the issuing warp is a constant.
constexpr uint32_t kSmemBase = 0x400;
constexpr uint64_t desc_c(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
constexpr uint32_t bar_c(int which) { return kSmemBase + kMiscOff + 8u * (uint32_t)which; }
template <int X, int ST>
__device__ __forceinline__ void issue_qk_c() {     // S_X = Q_X K^T from K stage ST
  constexpr uint64_t dq = desc_c(kSmemBase + kQOff + X * kBox, 16, 1024);
  constexpr uint64_t dk = desc_c(kSmemBase + kKOff + ST * kTile, 16, 1024);
  constexpr uint32_t idesc = instr_desc(128, BLK, 0, 0);
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
    const uint32_t qoff = ((kk >> 2) * kTile + (kk & 3) * 32) >> 4;
    const uint32_t koff = ((kk >> 2) * kBox + (kk & 3) * 32) >> 4;
    mma_ss(kSCol + X * 128, dq + qoff, dk + koff, idesc, kk > 0);
  }
  mma_commit(bar_c(BAR_S_FULL + X));
}
template <int X, int ST>
__device__ __forceinline__ void issue_pv_c(bool accumulate) {   // O_X (+)= P_X V from V stage ST
  constexpr uint64_t dv = desc_c(kSmemBase + kVOff + ST * kTile, kBox, 1024);
  constexpr uint32_t idesc = instr_desc(128, D, 0, 1);
#pragma unroll
  for (int kk = 0; kk < BLK / 16; ++kk)
    mma_ts(kOCol + X * 128, kSCol + X * 128 + kk * 8, dv + (uint32_t)((kk * 16 * 128) >> 4), idesc, (accumulate || kk > 0) ? 1u : 0u);
}

// One work item as the producer warp posts it to the other roles (shared memory, two slots of sixteen ints).
struct Item {
  int id;              // position in the work order, -1 = no more work
  int slotA, slotB;    // position of each tile's head in the call's head table
  int hA, hB;          // query head of each tile (both read the same KV head)
  int iA, iB;          // row-block of each tile (>= Nb: the tile does not exist)
  int listA, listB;    // list index of each tile, -1 = dense
  int cntA, cntB;      // key-blocks each tile visits
};
enum { ITEM_INTS = 16 };
// An entry of the work order: one head (tile A = row-block 2u, tile B = row-block 2u + 1 of that head), or two heads of
// one KV head that walk the same list (tile A = row-block i of the first, tile B = row-block i of the second; one entry
// for the even i, one for the odd i, so that every entry has ceil(Nb / 2) items).
enum { ENT_ONE_HEAD = 0, ENT_TWO_HEADS_EVEN = 1, ENT_TWO_HEADS_ODD = 2 };
// Position `raw` of the work order -> its two tiles.  Groups in turn; inside a group the longest pairs first, entries
// fastest.
struct WorkItemTiles { int slot_a, slot_b, rb_a, rb_b; };
__host__ __device__ inline WorkItemTiles resolve_item(const HeadTable& order, const GroupTable& group_start, int n_groups,
                                                      int n_pairs, int raw) {
  int rest = raw, g = 0;
  while (g + 1 < n_groups && rest >= (group_start.v[g + 1] - group_start.v[g]) * n_pairs) {
    rest -= (group_start.v[g + 1] - group_start.v[g]) * n_pairs;
    ++g;
  }
  const int ng = group_start.v[g + 1] - group_start.v[g];
  const int ent = order.v[group_start.v[g] + rest % ng];
  const int u = n_pairs - 1 - rest / ng;
  const int kind = ent >> 16;
  WorkItemTiles w;
  w.slot_a = ent & 0xff;
  w.slot_b = (ent >> 8) & 0xff;
  w.rb_a = kind == ENT_ONE_HEAD ? 2 * u : 2 * u + (kind - ENT_TWO_HEADS_EVEN);
  w.rb_b = kind == ENT_ONE_HEAD ? 2 * u + 1 : w.rb_a;
  return w;
}

// Rare path of the softmax, kept out of the hot loop: the row's reference max has moved, so O of the earlier
// steps (when there are any) and the P chunks of this key-block that are already stored are brought to the new
// reference.  alpha = 2^(old reference - new reference), 1 for a row whose reference stays.  Called by whole warps.
static __device__ __noinline__ void rescale_tmem(uint32_t tO, uint32_t tS, float alpha, int stored, bool with_o) {
  if (with_o) {
#pragma unroll 1
    for (int oc = 0; oc < D / 32; ++oc) {
      uint32_t o[32];
      tmem_ld32(tO + oc * 32, o);
#pragma unroll
      for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
      tmem_st32(tO + oc * 32, o);
    }
  }
#pragma unroll 1
  for (int pc = 0; pc < stored; ++pc) {
    uint32_t pp[16];
    tmem_ld16(tS + pc * 16, pp);
#pragma unroll
    for (int e = 0; e < 16; ++e)
      pp[e] = cvt_bf16x2(__uint_as_float(pp[e] << 16) * alpha, __uint_as_float(pp[e] & 0xffff0000u) * alpha);
    tmem_st16(tS + pc * 16, pp);
  }
}

// The diagonal tile, once per row-block and out of the hot loop: the scores of the keys after a row's own position
// are set to -infinity in TMEM before the common path reads them.  Called by whole warps.
static __device__ __noinline__ void mask_diag_tmem(uint32_t tS, int row) {
#pragma unroll 1
  for (int c = 0; c < BLK / 32; ++c) {
    uint32_t sc[32];
    tmem_ld32(tS + c * 32, sc);
#pragma unroll
    for (int e = 0; e < 32; ++e)
      if (c * 32 + e > row) sc[e] = __float_as_uint(-CUDART_INF_F);
    tmem_st32(tS + c * 32, sc);
  }
  tmem_wait_st();
}

// kTrace: the phase trace compiled in (a profiling aid; its code in the hot loops costs a few per cent).
template <bool kTrace>
__global__ void __launch_bounds__(kThreadsPair, 1)
attn_pair_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_u32(smem + kQOff), sK = smem_u32(smem + kKOff), sV = smem_u32(smem + kVOff);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kMiscOff);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kMiscOff + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kMiscOff + 260);
  volatile int* kflags = reinterpret_cast<volatile int*>(smem + kMiscOff + 264);   // [kStages]
  float* lse_smem = reinterpret_cast<float*>(smem + kMiscOff + 512);               // [2][128]
  volatile int* items = reinterpret_cast<volatile int*>(smem + kMiscOff + 1536);   // [2][ITEM_INTS]
  auto bar = [&](int which) { return smem_u32(bars + which); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_pairs = (a.Nb + 1) >> 1;
  const Abort ab{abort_flag, a.status};
  // Optional phase trace (one CTA, one thread per role): {(event << 32) | step, SM clock} pairs.
  const bool tracing = kTrace && a.trace != nullptr && blockIdx.x == 0;
  int trace_n = 0;
  auto trace = [&](int role, int event, int step) {
    if (tracing && trace_n < a.trace_cap) {
      long long* e = a.trace + ((size_t)role * a.trace_cap + trace_n) * 2;
      e[0] = ((long long)event << 32) | (unsigned)step;
      e[1] = clock64();
      ++trace_n;
    }
  };

  if (threadIdx.x == 0) {
    mbar_init(bar(BAR_Q_FULL), 1);
    mbar_init(bar(BAR_Q_EMPTY), 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(BAR_K_FULL + s), 1);
      mbar_init(bar(BAR_K_EMPTY + s), 1);
      mbar_init(bar(BAR_V_EMPTY + s), 1);
      mbar_init(bar(BAR_V_FULL + s), 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(BAR_S_FULL + x), 1);
      mbar_init(bar(BAR_O_DONE + x), 1);
      mbar_init(bar(BAR_ITEM_FULL + x), 1);
      mbar_init(bar(BAR_ITEM_EMPTY + x), kItemReaders);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) tmem_alloc(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const bool layout_ok = smem_u32(smem) == kSmemBase && tmem == 0u;
  if (!layout_ok && threadIdx.x == 0) { if (atomicCAS(a.status, 0, (int)SP_ERR_UNSUPPORTED) == 0) a.status[1] = 90; }

  // The k-th item of this CTA, taken by a whole warp.  False when the wait ran out or another role gave up.
  auto take_item = [&](int k, Item& it, int where) -> bool {
    const int sl = k & 1;
    if (!__all_sync(0xffffffffu, mbar_wait(bar(BAR_ITEM_FULL + sl), (uint32_t)(k >> 1) & 1u, ab, where))) return false;
    const volatile int* src = items + ITEM_INTS * sl;
    it.id = src[0];
    it.slotA = src[1]; it.slotB = src[2];
    it.hA = src[3]; it.hB = src[4];
    it.iA = src[5]; it.iB = src[6];
    it.listA = src[7]; it.listB = src[8];
    it.cntA = src[9]; it.cntB = src[10];
    __syncwarp();
    if (lane == 0) mbar_arrive(bar(BAR_ITEM_EMPTY + sl));
    return true;
  };

  if (warp >= 8) {
    if (warp == 9) {
      // ---------------------------------------------------------- producer
      const int n_items = a.n_heads * n_pairs;
      const bool poisoned = !layout_ok || *reinterpret_cast<volatile int*>(a.status) != 0;   // an earlier wait ran out: do no work
      int gk = 0;        // merged key-blocks of the finished items (ring position of the next item's first)
      int issued_k = 0, issued_v = 0;   // K and V loads issued so far
      int relays = 0;    // relays to the issuing warp so far
      int qn = 0;        // items with work so far (Q loads)
      bool ok = true;
      for (int k = 0; ok; ++k) {
        // Scheduling: the next position of the work order comes from the launch's counter; lane 0 resolves it to
        // (head, pair, list, counts) and posts it for the other roles.  Work order: the heads of one KV head together
        // (their K/V set, 64 MB at 128K, stays in L2 while they run), inside such a group the longest row-block pairs
        // first, heads fastest.  The slot is free once the nine reader warps have taken the item two before this one.
        Item it;
        {
          const int sl = k & 1;
          if (k >= 2) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_ITEM_EMPTY + sl), ((uint32_t)(k >> 1) & 1u) ^ 1u, ab, 40));
          if (!ok) break;
          it.id = -1; it.slotA = it.slotB = 0; it.hA = it.hB = 0; it.iA = it.iB = 0; it.listA = it.listB = -1; it.cntA = it.cntB = 0;
          if (lane == 0) {
            const int raw = poisoned ? n_items : atomicAdd(a.work_counter, 1);
            if (raw < n_items) {
              const WorkItemTiles w = resolve_item(a.order, a.group_start, a.n_groups, n_pairs, raw);
              it.id = raw;
              it.slotA = sp_in_range(w.slot_a, 0, a.n_heads - 1, a.status, 51);
              it.slotB = sp_in_range(w.slot_b, 0, a.n_heads - 1, a.status, 51);
              it.iA = w.rb_a;
              it.iB = w.rb_b;
              it.hA = sp_in_range(a.heads.v[it.slotA], 0, a.n_q_heads - 1, a.status, 51);
              it.hB = sp_in_range(a.heads.v[it.slotB], 0, a.n_q_heads - 1, a.status, 51);
              it.listA = a.lists_dev ? a.lists_dev[it.slotA] : a.lists.v[it.slotA];
              it.listB = a.lists_dev ? a.lists_dev[it.slotB] : a.lists.v[it.slotB];
              if (it.listA < 0) it.listA = -1;
              if (it.listB < 0) it.listB = -1;
              int cnt[2];
#pragma unroll
              for (int x = 0; x < 2; ++x) {
                const int i = x ? it.iB : it.iA, list = x ? it.listB : it.listA;
                int c = 0;
                if (i < a.Nb) {
                  c = list >= 0 ? a.counts[(size_t)list * a.Nb + i] : i + 1;
                  c = c < 0 ? 0 : (c > i + 1 ? i + 1 : c);
                }
                cnt[x] = c;
              }
              it.cntA = cnt[0];
              it.cntB = cnt[1];
            }
            volatile int* dst = items + ITEM_INTS * sl;
            dst[0] = it.id;
            dst[1] = it.slotA; dst[2] = it.slotB;
            dst[3] = it.hA; dst[4] = it.hB;
            dst[5] = it.iA; dst[6] = it.iB;
            dst[7] = it.listA; dst[8] = it.listB;
            dst[9] = it.cntA; dst[10] = it.cntB;
            mbar_arrive(bar(BAR_ITEM_FULL + sl));
          }
          it.id = __shfl_sync(0xffffffffu, it.id, 0);
          it.hA = __shfl_sync(0xffffffffu, it.hA, 0);
          it.hB = __shfl_sync(0xffffffffu, it.hB, 0);
          it.iA = __shfl_sync(0xffffffffu, it.iA, 0);
          it.iB = __shfl_sync(0xffffffffu, it.iB, 0);
          it.listA = __shfl_sync(0xffffffffu, it.listA, 0);
          it.listB = __shfl_sync(0xffffffffu, it.listB, 0);
          it.cntA = __shfl_sync(0xffffffffu, it.cntA, 0);
          it.cntB = __shfl_sync(0xffffffffu, it.cntB, 0);
        }
        if (it.id < 0) break;
        const int cntA = it.cntA, cntB = it.cntB;
        if (cntA + cntB == 0) continue;
        const int iA = it.iA, iB = it.iB;
        const int g = it.hA / a.group;     // tile B's head reads the same KV head
        // Q of the item before this one has been read by its last QK^T
        if (qn > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_Q_EMPTY), (uint32_t)(qn - 1) & 1u, ab, 15));
        if (!ok) break;
        if (lane == 0) {
          const int n_q = iB < a.Nb ? 2 : 1;     // tile A exists whenever the item has work
          mbar_expect_tx(bar(BAR_Q_FULL), n_q * kTile);
          for (int x = 0; x < n_q; ++x)
            for (int b = 0; b < 2; ++b)
              tma_load_3d(sQ + b * kTile + x * kBox, &tm_q, bar(BAR_Q_FULL), b * 64, (x ? iB : iA) * BLK, x ? it.hB : it.hA);
        }
        ++qn;
        // The two ascending lists are merged 32 entries at a time: lane l holds entry base + l.
        const int32_t* idxA = it.listA >= 0 && iA < a.Nb ? a.indices + ((size_t)it.listA * a.Nb + iA) * a.Nb : nullptr;
        const int32_t* idxB = it.listB >= 0 && iB < a.Nb ? a.indices + ((size_t)it.listB * a.Nb + iB) * a.Nb : nullptr;
        int pa = 0, pb = 0, n = 0;
        int chunkA = 0, chunkB = 0;
        if (idxA) chunkA = lane < cntA ? idxA[lane] : 0;
        if (idxB) chunkB = lane < cntB ? idxB[lane] : 0;
        const bool listedA = idxA != nullptr, listedB = idxB != nullptr;
        while ((pa < cntA || pb < cntB) && ok) {
          const int ja = pa < cntA ? (listedA ? __shfl_sync(0xffffffffu, chunkA, pa & 31) : pa) : 0x7fffffff;
          const int jb = pb < cntB ? (listedB ? __shfl_sync(0xffffffffu, chunkB, pb & 31) : pb) : 0x7fffffff;
          const int j_listed = ja < jb ? ja : jb;
          int f = (ja == j_listed ? F_A : 0) | (jb == j_listed ? F_B : 0);
          // a listed key-block lies on or before the diagonal of every tile that walks it
          const int j = sp_in_range(j_listed, 0, (f & F_A) ? ((f & F_B) && iB < iA ? iB : iA) : iB, a.status, 50);
          if (ja == j_listed) {
            ++pa;
            if (listedA && (pa & 31) == 0) chunkA = pa + lane < cntA ? idxA[pa + lane] : 0;
          }
          if (jb == j_listed) {
            ++pb;
            if (listedB && (pb & 31) == 0) chunkB = pb + lane < cntB ? idxB[pb + lane] : 0;
          }
          if (!(pa < cntA || pb < cntB)) f |= F_LAST;
          const int gn = gk + n;
          const int st = gn % kStages;
          const uint32_t ph = (uint32_t)(gn / kStages) & 1u;
          if (gn >= kStages) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_K_EMPTY + st), ph ^ 1u, ab, 10));
          if (!ok) break;
          if (lane == 0) {
            kflags[st] = f;
            mbar_expect_tx(bar(BAR_K_FULL + st), kTile);
            for (int b = 0; b < 2; ++b) tma_load_3d(sK + st * kTile + b * kBox, &tm_k, bar(BAR_K_FULL + st), b * 64, j * BLK, g);
            trace(0, 20, gn);
          }
          ++issued_k;
          if (gn >= kStages) ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_V_EMPTY + st), ph ^ 1u, ab, 11));
          if (!ok) break;
          if (lane == 0) {
            mbar_expect_tx(bar(BAR_V_FULL + st), kTile);
            for (int b = 0; b < 2; ++b) tma_load_3d(sV + st * kTile + b * kBox, &tm_v, bar(BAR_V_FULL + st), b * 64, j * BLK, g);
            trace(0, 21, gn);
          }
          ++issued_v;
          ++n;
          // relay for the issuing warp's iteration n - 2 of this item (key-block n - 2 computed, n - 1 multiplied
          // ahead): K of key-block n - 1 and V of key-block n - 2 have landed
          if (n >= 2) {
            const int mk = gk + n - 1, mv = gk + n - 2;
            ok = mbar_wait(bar(BAR_K_FULL + mk % kStages), (uint32_t)(mk / kStages) & 1u, ab, 12);
            if (ok) ok = mbar_wait(bar(BAR_V_FULL + mv % kStages), (uint32_t)(mv / kStages) & 1u, ab, 13);
            ok = __all_sync(0xffffffffu, ok);
            bar_arrive(NB_KV + (relays & 3), 64);     // also when a wait ran out: nobody may be left at a named barrier
            ++relays;
          }
        }
        if (__all_sync(0xffffffffu, ok) && n >= 1) {
          // the last key-block of the item: only its V is still awaited
          const int mv = gk + n - 1;
          ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_V_FULL + mv % kStages), (uint32_t)(mv / kStages) & 1u, ab, 13));
          bar_arrive(NB_KV + (relays & 3), 64);
          ++relays;
        } else if (n >= 1) {
          bar_arrive(NB_KV + (relays & 3), 64);       // a wait ran out above: release the issuing warp once more
        }
        gk += n;
      }
      if (*abort_flag && lane == 0) {
        // let the copies already in flight land before the CTA gives its shared memory back
        const long long t0 = clock64();
        while (clock64() - t0 < kWaitCycles / 8) {
          bool done = qn == 0 || mbar_try_wait(bar(BAR_Q_FULL), (uint32_t)(qn - 1) & 1u);
          for (int back = 1; back <= kStages; ++back) {   // at most the last kStages loads of a ring are in flight
            const int mk = issued_k - back, mv = issued_v - back;
            if (mk >= 0) done = done && mbar_try_wait(bar(BAR_K_FULL + mk % kStages), (uint32_t)(mk / kStages) & 1u);
            if (mv >= 0) done = done && mbar_try_wait(bar(BAR_V_FULL + mv % kStages), (uint32_t)(mv / kStages) & 1u);
          }
          if (done) break;
        }
      }
    } else if (warp == 8) {
      // ---------------------------------------------------------- MMA issuer
      int gk = 0;            // merged key-blocks so far, over all items (ring position)
      int relays = 0;        // relays taken from the producer warp so far
      int tA = 0, tB = 0;    // steps of each tile so far, over all items (parity of its P hand-offs)
      int qn = 0;            // items with work so far
      bool ok = true;
      for (int k = 0; ok; ++k) {
        Item it;
        if (!take_item(k, it, 22)) break;
        if (it.id < 0) break;
        const int cntA = it.cntA, cntB = it.cntB;
        if (cntA + cntB == 0) continue;
        ok = mbar_wait(bar(BAR_Q_FULL), (uint32_t)qn & 1u, ab, 20);
        if (ok) ok = mbar_wait(bar(BAR_K_FULL + gk % kStages), (uint32_t)(gk / kStages) & 1u, ab, 21);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        ++qn;
        tc_fence_after();
        int f = kflags[gk % kStages];
        if (lane == 0) {
          trace(1, 1, gk);
          if (gk & 1) {
            if (f & F_A) issue_qk_c<0, 1>();
            if (f & F_B) issue_qk_c<1, 1>();
          } else {
            if (f & F_A) issue_qk_c<0, 0>();
            if (f & F_B) issue_qk_c<1, 0>();
          }
          mma_commit(bar(BAR_K_EMPTY + gk % kStages));
          if (f & F_LAST) mma_commit(bar(BAR_Q_EMPTY));
          trace(1, 2, gk);
        }
        __syncwarp();
        // The loop's hand-offs come through named barriers (a poll of an mbarrier costs the issuing warp 150-250
        // cycles while the tensor pipe streams operands from shared memory; with five polls per key-block the
        // warp was waiting a quarter of the time with nothing queued): the producer warp relays "K of the next
        // key-block and V of this one have landed", the softmax warps "P of this tile is stored".  The flags of the
        // next key-block and the abort flag are read from shared memory ahead of the MMAs whose issue hides the trip.
        // The first PV of an item overwrites O of the item before: the softmax warps of the tile have read that O
        // out of TMEM before they produced the P this PV waits for.
        int tAl = 0, tBl = 0;  // steps of each tile inside this item
        auto body = [&](auto st_c) -> bool {       // one merged key-block read from ring stage ST; true: leave the loop
          constexpr int ST = decltype(st_c)::value, STN = ST ^ 1;
          const bool last = (f & F_LAST) != 0;
          bar_sync(NB_KV + (relays & 3), 64);
          ++relays;
          const int fn_early = last ? 0 : kflags[STN];
          if (f & F_A) bar_sync(NB_P + 2 + (tA & 1), 160);
          tc_fence_after();
          const int fn = fn_early;
          if (lane == 0) {
            if (f & F_A) {
              trace(1, 3, gk);
              issue_pv_c<0, ST>(tAl > 0);
              if (tAl + 1 == cntA) mma_commit(bar_c(BAR_O_DONE + 0));
            }
            if (fn & F_A) issue_qk_c<0, STN>();
            trace(1, 5, gk);
          }
          __syncwarp();
          if (f & F_A) { ++tA; ++tAl; }
          if (f & F_B) bar_sync(NB_P + 6 + (tB & 1), 160);
          const int abort_raw = *abort_flag;       // after all syncs of this key-block; looked at after the MMAs below
          tc_fence_after();
          if (lane == 0) {
            if (f & F_B) {
              trace(1, 6, gk);
              issue_pv_c<1, ST>(tBl > 0);
              if (tBl + 1 == cntB) mma_commit(bar_c(BAR_O_DONE + 1));
            }
            mma_commit(bar_c(BAR_V_EMPTY + ST));
            if (fn & F_B) issue_qk_c<1, STN>();
            if (!last) mma_commit(bar_c(BAR_K_EMPTY + STN));
            if (fn & F_LAST) mma_commit(bar_c(BAR_Q_EMPTY));   // Q of this item has been read for the last time
            trace(1, 4, gk);
          }
          __syncwarp();
          if (f & F_B) { ++tB; ++tBl; }
          ++gk;
          if (__any_sync(0xffffffffu, abort_raw != 0)) ok = false;
          if (last || !ok) return true;
          f = fn;
          return false;
        };
        bool done = false;
        if (gk & 1) done = body(std::integral_constant<int, 1>{});
        while (!done) {
          done = body(std::integral_constant<int, 0>{});
          if (!done) done = body(std::integral_constant<int, 1>{});
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue of tile x
    const int x = warp >> 2;
    const int row = threadIdx.x & 127;                 // TMEM lane == query row inside the tile
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t tS = tl + kSCol + x * 128, tO = tl + kOCol + x * 128;
    const float scale = a.scale_log2;
    const int trole = 2 + x;
    const bool tthread = row == 0;
    // per-CTA statistics region: [tile][step of the item][row]
    float* const stats = a.tile_stats ? a.tile_stats + ((size_t)blockIdx.x * 2 + x) * (size_t)a.Nb * BLK : nullptr;
    const uint64_t pol_keep = l2_policy_evict_last(), pol_done = l2_policy_evict_first();
    int ts = 0;          // steps of this tile so far, over all items (parity of S_FULL and of the P hand-offs)
    int on = 0;          // items in which this tile had work so far (parity of O_DONE)
    bool fail = false;   // a wait of this thread ran out
    for (int k = 0;; ++k) {
      Item it;
      it.id = -1;
      const bool got = !fail && take_item(k, it, 34 + x);
      // The four warps of the tile go on together or stop together (a warp whose wait ran out must not leave the
      // others at the barriers of the epilogue).  This barrier also separates the reads of the statistics region
      // by the epilogue of the item before from the writes of this item.
      if (!bar_and(1 + x, 128, got)) break;
      if (it.id < 0) break;
      const int i = x ? it.iB : it.iA, cnt = x ? it.cntB : it.cntA;
      const int h = x ? it.hB : it.hA, slot = x ? it.slotB : it.slotA, list = x ? it.listB : it.listA;
      const int32_t* idx = list >= 0 && i < a.Nb ? a.indices + ((size_t)list * a.Nb + i) * a.Nb : nullptr;
      const bool emit = a.importance != nullptr && list < 0;
      const int r = i * BLK + row;
      float m_ref = -CUDART_INF_F, l = 0.f;
      bool ok = cnt > 0;
      int j_next = cnt > 0 ? (idx ? idx[0] : 0) : 0;
      for (int t = 0; t < cnt && ok; ++t, ++ts) {
        const int j = j_next;
        if (t + 1 < cnt) j_next = idx ? idx[t + 1] : t + 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_S_FULL + x), (uint32_t)ts & 1u, ab, 30 + x));
        if (!ok) {
          fail = true;
          bar_arrive(NB_P + 4 * x + 2 + (ts & 1), 160);   // the issuing warp may be at this step's barrier: do not leave it there
          break;
        }
        tc_fence_after();
        if (tthread) trace(trole, 10, t);
        // The 128 columns are taken as four chunks of 32 (`tcgen05.ld.32x32b.x32`, the next chunk's load in flight),
        // each an online-softmax step of its own: chunk max, (rarely: only when the row max has grown by more than
        // 2^8) a move of the reference, exponentials, P chunk into columns the sweep has given up.  P is handed to
        // the issuing warp once, after the fourth chunk.
        float tile_sum = 0.f;
        uint32_t sa[32], sb[32];
        if (j == i) mask_diag_tmem(tS, row);
        tmem_ld32_async(tS, sa);
        auto chunk_max = [&](const uint32_t* sc) {
          float mx0 = max3(__uint_as_float(sc[0]), __uint_as_float(sc[1]), __uint_as_float(sc[2]));
          float mx1 = max3(__uint_as_float(sc[3]), __uint_as_float(sc[4]), __uint_as_float(sc[5]));
          float mx2 = max3(__uint_as_float(sc[6]), __uint_as_float(sc[7]), __uint_as_float(sc[8]));
          float mx3 = max3(__uint_as_float(sc[9]), __uint_as_float(sc[10]), __uint_as_float(sc[11]));
#pragma unroll
          for (int e = 12; e < 28; e += 8) {
            mx0 = max3(mx0, __uint_as_float(sc[e + 0]), __uint_as_float(sc[e + 1]));
            mx1 = max3(mx1, __uint_as_float(sc[e + 2]), __uint_as_float(sc[e + 3]));
            mx2 = max3(mx2, __uint_as_float(sc[e + 4]), __uint_as_float(sc[e + 5]));
            mx3 = max3(mx3, __uint_as_float(sc[e + 6]), __uint_as_float(sc[e + 7]));
          }
          mx0 = max3(mx0, __uint_as_float(sc[28]), __uint_as_float(sc[29]));
          mx1 = max3(mx1, __uint_as_float(sc[30]), __uint_as_float(sc[31]));
          return fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        };
        // mx: scaled max of the columns about to be exponentiated; stored: P chunks of this key-block already in TMEM
        auto move_reference = [&](const float mx, const int stored) {
          // the reference max only moves when the row max has grown by more than 2^8 (rare after the first chunk of
          // the first key-block; a fully masked chunk has mx = -inf and leaves it alone)
          if (__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
            const float m_new = (mx > m_ref + 8.f) ? mx : m_ref;
            const float alpha = ex2_approx(m_ref - m_new);
            // O of the previous steps is relative to the old reference (S of this step is complete, so the PV of
            // the previous step, issued before it, is too); none of the stored P chunks has been handed over yet
            rescale_tmem(tO, tS, alpha, stored, t > 0);
            l *= alpha;
            tile_sum *= alpha;
            m_ref = m_new;
          }
        };
        auto chunk_exps = [&](const uint32_t* sc, const int c) {   // exponentials, sums, P chunk c (columns 32c .. 32c+31)
          const float2 sc2 = make_float2(scale, scale), nm2 = make_float2(-m_ref, -m_ref);
          float2 sum01 = make_float2(0.f, 0.f), sum23 = make_float2(0.f, 0.f);
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            float2 x01 = __ffma2_rn(make_float2(__uint_as_float(sc[e]), __uint_as_float(sc[e + 1])), sc2, nm2);
            float2 x23 = __ffma2_rn(make_float2(__uint_as_float(sc[e + 2]), __uint_as_float(sc[e + 3])), sc2, nm2);
            x01.x = ex2_approx(x01.x);
            x01.y = ex2_approx(x01.y);
            x23.x = ex2_approx(x23.x);
            x23.y = ex2_approx(x23.y);
            sum01 = __fadd2_rn(sum01, x01);
            sum23 = __fadd2_rn(sum23, x23);
            pk[e / 2] = cvt_bf16x2(x01.x, x01.y);
            pk[e / 2 + 1] = cvt_bf16x2(x23.x, x23.y);
          }
          tile_sum += (sum01.x + sum01.y) + (sum23.x + sum23.y);
          tmem_st16(tS + c * 16, pk);
        };
        tmem_ld_wait();
        reg_fence32(sa);
        tmem_ld32_async(tS + 32, sb);
        move_reference(chunk_max(sa) * scale, 0);
        chunk_exps(sa, 0);
        tmem_ld_wait();
        reg_fence32(sb);
        tmem_ld32_async(tS + 64, sa);
        move_reference(chunk_max(sb) * scale, 1);
        chunk_exps(sb, 1);
        tmem_ld_wait();
        reg_fence32(sa);
        tmem_ld32_async(tS + 96, sb);
        move_reference(chunk_max(sa) * scale, 2);
        chunk_exps(sa, 2);
        tmem_ld_wait();
        reg_fence32(sb);
        if (tthread) trace(trole, 13, t);
        move_reference(chunk_max(sb) * scale, 3);
        chunk_exps(sb, 3);
        tmem_wait_st();
        tc_fence_before();
        bar_arrive(NB_P + 4 * x + 2 + (ts & 1), 160);
        if (tthread) trace(trole, 15, t);
        // off the critical path: running sum and the tile statistic
        l += tile_sum;
        if (emit) st_f32_hint(stats + (size_t)sp_in_range(t, 0, a.Nb - 1, a.status, 52) * BLK + row, m_ref + log2f(tile_sum), pol_keep);
      }
      if (ok) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar(BAR_O_DONE + x), (uint32_t)on & 1u, ab, 32 + x));
        if (!ok) fail = true;
      }
      if (cnt > 0) ++on;
      float lse2 = 0.f;
      if (ok) {
        tc_fence_after();
        const float inv_l = 1.f / l;
        __nv_bfloat16* orow = a.o + (size_t)h * a.o_sh + (size_t)r * a.o_sn;
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tO + c * 32, o);
          uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            uint4 w;
            w.x = cvt_bf16x2(__uint_as_float(o[8 * e + 0]) * inv_l, __uint_as_float(o[8 * e + 1]) * inv_l);
            w.y = cvt_bf16x2(__uint_as_float(o[8 * e + 2]) * inv_l, __uint_as_float(o[8 * e + 3]) * inv_l);
            w.z = cvt_bf16x2(__uint_as_float(o[8 * e + 4]) * inv_l, __uint_as_float(o[8 * e + 5]) * inv_l);
            w.w = cvt_bf16x2(__uint_as_float(o[8 * e + 6]) * inv_l, __uint_as_float(o[8 * e + 7]) * inv_l);
            dst[e] = w;
          }
        }
        // O has left TMEM: ordered before the P hand-off of the next item, after which its first PV overwrites O
        tc_fence_before();
        lse2 = m_ref + log2f(l);
        if (a.lse) a.lse[(size_t)slot * a.N + r] = lse2 * 0.6931471805599453f;
      }
      if (emit) {
        float* lse_x = lse_smem + x * 128;
        lse_x[row] = lse2;
        // the four softmax warps of this tile: statistics and lse visible to one another, and one
        // common decision (a thread whose wait ran out must not leave the others at a barrier)
        const bool all_ok = bar_and(1 + x, 128, ok);
        if (all_ok) {
          float* imp_row = a.importance + ((size_t)slot * a.Nb + i) * a.Nb;
          const float4 lse4 = *reinterpret_cast<const float4*>(lse_x + lane * 4);
          const int wq = warp & 3;
          // each warp takes tiles wq, wq + 4, ...; eight tiles in flight; lane l sums rows 4l..4l+3
          for (int t0 = wq; t0 < cnt; t0 += 32) {
            float4 v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int t = t0 + 4 * e;
              v[e] = t < cnt ? ld_f32x4_hint(stats + (size_t)t * BLK + lane * 4, pol_done)
                             : make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float acc = (ex2_approx(v[e].x - lse4.x) + ex2_approx(v[e].y - lse4.y)) +
                          (ex2_approx(v[e].z - lse4.z) + ex2_approx(v[e].w - lse4.w));
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
              const int t = t0 + 4 * e;
              if (lane == 0 && t < cnt) imp_row[t] = acc * (1.f / BLK);
            }
          }
          for (int jz = i + 1 + row; jz < a.Nb; jz += 128) imp_row[jz] = 0.f;
        }
      }
      if (!ok && !fail && cnt == 0 && i < a.Nb) {
        // an empty list is outside the contract; leave defined output (zeros) rather than garbage
        __nv_bfloat16* orow = a.o + (size_t)h * a.o_sh + (size_t)r * a.o_sn;
        for (int e = 0; e < D / 8; ++e) reinterpret_cast<uint4*>(orow)[e] = make_uint4(0, 0, 0, 0);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

bool attn_pair_supported(const AttnArgs& a) { return a.d == D && a.B == BLK; }

namespace {
int sm_count() {
  int n_sm = 148, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  return n_sm > 0 ? n_sm : 148;
}
}  // namespace

int attn_pair_ctas(int n_heads, int Nb) {
  const long items = (long)n_heads * ((Nb + 1) / 2);
  const int n_sm = sm_count();
  return (int)(items < n_sm ? items : n_sm);
}

size_t attn_pair_stats_bytes(int n_heads, int Nb) {
  return (size_t)attn_pair_ctas(n_heads, Nb) * 2 * (size_t)Nb * BLK * sizeof(float);
}

// Work order of a launch (host).  Many items (forty per SM or more): the slots sorted by KV head (stable), one group
// per KV head, so that a K/V set stays in L2 while its heads run.  Fewer: one group, i.e. the longest pairs of all
// heads first, because then the balance at the end matters more than L2.
// Two heads of one KV head that walk the same list (members of one cluster; two dense heads) share a work item
// row-block by row-block: their two tiles need exactly the same K/V tiles, so no K/V load serves one tile alone,
// as happens wherever two adjacent row-blocks of one head differ in their lists.  Such a pair takes two entries
// (even and odd row-blocks); a head without a partner keeps one entry and pairs its own adjacent row-blocks.
// Lists decided on the device are not known here: those heads stay single.
void attn_pair_work_order(AttnArgs& a, int n_sm) {
  const bool by_kv_head = (long)a.n_heads * ((a.Nb + 1) / 2) >= 40L * n_sm;
  int n = 0;
  a.n_groups = 0;
  bool taken[kMaxHeads];
  for (int t = 0; t < a.n_heads; ++t) taken[t] = false;
  auto add_head = [&](int t) {
    if (taken[t]) return;
    taken[t] = true;
    int partner = -1;
    if (!a.lists_dev && a.pair_heads) {
      const int lt = a.lists.v[t] < 0 ? -1 : a.lists.v[t];
      for (int t2 = t + 1; t2 < a.n_heads && partner < 0; ++t2) {
        const int l2 = a.lists.v[t2] < 0 ? -1 : a.lists.v[t2];
        if (!taken[t2] && a.heads.v[t2] / a.group == a.heads.v[t] / a.group && l2 == lt && a.heads.v[t2] != a.heads.v[t]) partner = t2;
      }
    }
    if (partner >= 0) {
      taken[partner] = true;
      a.order.v[n++] = t | (partner << 8) | (ENT_TWO_HEADS_EVEN << 16);
      a.order.v[n++] = t | (partner << 8) | (ENT_TWO_HEADS_ODD << 16);
    } else {
      a.order.v[n++] = t | (t << 8) | (ENT_ONE_HEAD << 16);
    }
  };
  if (by_kv_head) {
    for (int g = 0; g < a.n_kv_heads; ++g) {
      const int start = n;
      for (int t = 0; t < a.n_heads; ++t)
        if (a.heads.v[t] / a.group == g) add_head(t);
      if (n > start) a.group_start.v[a.n_groups++] = start;
    }
  } else {
    for (int t = 0; t < a.n_heads; ++t) add_head(t);
    a.group_start.v[a.n_groups++] = 0;
  }
  static_assert(kMaxHeads <= 256, "an entry of the work order holds two slots of eight bits");
  static_assert(sizeof(a.group_start.v) / sizeof(a.group_start.v[0]) == kMaxHeads + 1, "room for the end of the last group");
  a.group_start.v[a.n_groups] = n;
}

// Position `raw` of the work order -> the two tiles (slot and row-block of each); what the producer warp does on the
// device, here for host-side checks of the order.  False past the end.
bool attn_pair_item(const AttnArgs& a, int raw, int* slot_a, int* rb_a, int* slot_b, int* rb_b) {
  const int n_pairs = (a.Nb + 1) / 2;
  if (raw < 0 || raw >= a.n_heads * n_pairs) return false;
  WorkItemTiles w = resolve_item(a.order, a.group_start, a.n_groups, n_pairs, raw);
  *slot_a = w.slot_a; *rb_a = w.rb_a; *slot_b = w.slot_b; *rb_b = w.rb_b;
  return true;
}

cudaError_t launch_attn_pair(const AttnArgs& a_in, cudaStream_t s) {
  if (!attn_pair_supported(a_in) || !a_in.work_counter) return cudaErrorInvalidValue;
  AttnArgs a = a_in;
  attn_pair_work_order(a, sm_count());
  CUtensorMap tq, tk, tv;
  if (!make_map(&tq, a.q, a.q_sh, a.q_sn, a.n_q_heads, a.N, D, BLK) ||
      !make_map(&tk, a.k, a.k_sh, a.k_sn, a.n_kv_heads, a.N, D, BLK) ||
      !make_map(&tv, a.v, a.v_sh, a.v_sn, a.n_kv_heads, a.N, D, BLK))
    return cudaErrorInvalidValue;
  auto kernel = a.trace ? attn_pair_kernel<true> : attn_pair_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemTotal);
  if (e != cudaSuccess) return e;
  // Persistent CTAs, one per SM, take the items of the work order from a counter that starts at zero.
  e = cudaMemsetAsync(a.work_counter, 0, sizeof(int), s);
  if (e != cudaSuccess) return e;
  kernel<<<attn_pair_ctas(a.n_heads, a.Nb), kThreadsPair, kSmemTotal, s>>>(a, tq, tk, tv);
  return cudaGetLastError();
}

}  // namespace sp
