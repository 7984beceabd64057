// liblightkv kernels, part 2: tcgen05 tensor-core contractions fed by TMA (sm_100a).
#include <algorithm>

#include "launch.h"
#include "tc_common.cuh"

namespace lkv {

using namespace tc;

// ------------------------------------------------------------------------------------------------------
// Host: tensor maps.  cuTensorMapEncodeTiled is fetched through the runtime so that the library does not
// link against libcuda.
// ------------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [batch, heads, rows, width] with element strides (width contiguous); box = 64 x box_rows
// elements, 128-byte swizzle.
static bool make_map_bhnd(CUtensorMap* map, const void* base, int width, int rows, int heads, int batch,
                          int64_t row_stride, int64_t head_stride, int64_t batch_stride, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)width, (cuuint64_t)rows, (cuuint64_t)heads, (cuuint64_t)batch};
  const cuuint64_t strides[3] = {(cuuint64_t)row_stride * 2, (cuuint64_t)head_stride * 2,
                                 (cuuint64_t)(batch > 1 ? batch_stride : head_stride * heads) * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ======================================================================================================
// xi per head on tensor cores (Eq. "attention-factor" over the softmax rows of Eq. "attention-matrix").
//
// A work item is (tile of 128 vision queries, head, sample).  Persistent CTAs, two per SM, draw items from a
// ticket counter in global memory (the list interleaves groups of 64 (sample, head) pairs whose K stays in L2
// together, longest rows first inside a group).  Warp 0 is the scheduler and the TMA producer: it
// publishes the ticket to the other roles through a two-slot ring in shared memory, streams the item's Q tile
// once and its K tiles (128 keys) through a 2-stage ring; the next item's Q and first K tiles are requested as
// soon as the MMAs of the current item have drained, i.e. while its last tiles are still in the softmax warps.
// Warp 1 issues S = Q K^T (128 x 128 x dh, bf16 -> fp32) into one of two TMEM accumulators.  Warps 2-9 are
// the softmax warps, two threads per query row (= TMEM lane): a thread pulls 32 of the 64 logits of a half of the
// accumulator into registers (the warp that takes the last piece releases the accumulator) and adds
// exp(logit - reference) to two sums (all visible keys / prompt keys J); the two threads of a row combine their
// references and sums once per item through shared memory.
// Output per head: sum_J / sum_all.
//
// The kernel is bound by the exponentials (one per logit on the special-function unit, 16 per clock per SM,
// against one MMA per tile), so the softmax arithmetic is kept to three instructions per logit:
//   * the reference subtracted before the exponential is the thread's maximum over its FIRST 32 keys only
//     (softmax is invariant to the reference; fp32 holds exp of any later logit up to 88 above it), so the
//     other tiles need no maximum and no rescaling;
//   * on halves that need neither the causal mask nor the prompt mask, every eighth exponential is evaluated
//     on the FMA pipe instead (range reduction + cubic, relative error 7.5e-5).  With the softmax warps alone
//     on an SM a quarter is the best share; in the whole kernel, which runs into the power limit (SM clock
//     about 1.78 GHz instead of 1.965), the dozen instructions of the cubic cost more than the special-function
//     slot they free, and an eighth measured fastest (none: +1 %, a quarter: +4 %, three eighths: +10 %).
// A row whose sum left the fp32 range (a later logit more than 88 above the first keys' maximum) is found at
// the end of its item, which is then appended to a list in global memory; a second launch of the kernel
// (SAFE) walks that list with a running maximum and rescaling on every half, as an ordinary online softmax
// does, and overwrites the item's results.  With an empty list that launch returns at once.
// Halves that straddle the diagonal (or the end of the sample) are masked, and the columns no row of a warp
// can see are skipped.  With the caller's row log-sum-exp (LSE) only the prompt key tiles are visited.
// ======================================================================================================
__device__ __forceinline__ float ex2(float x) {          // one MUFU op, flush-to-zero
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x on the FMA and integer pipes: x is clamped to [-126, 128], split into the nearest integer j (magic-number
// add) and r in [-0.5, 0.5]; 2^r by a minimax cubic; j is added to the exponent field.  x = 128 gives the bit
// pattern of a non-finite value, which the overflow check at the end of the item sees.
__device__ __forceinline__ float ex2_fma(float x) {
  x = fminf(fmaxf(x, -126.f), 128.f);
  const float t = x + 12582912.f;                         // 1.5 * 2^23: the integer lands in the low mantissa bits
  const float r = x - (t - 12582912.f);
  float p = fmaf(r, 0.0551716685f, 0.2426111251f);
  p = fmaf(p, r, 0.6932609677f);
  p = fmaf(p, r, 0.9999280572f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// Scheduler words in the workspace (zeroed on the stream before the first launch of a call).
struct XiSched {
  unsigned int ticket;               // next item of the first launch
  unsigned int safe_ticket;          // next entry of the list, second launch
  unsigned int n_redo;               // items appended to the list
  unsigned int pad;
};

struct XiTcArgs {
  const int* n_vis;
  const int* seq_start;              // first row of each sample in q, k, lse, lse_out (packed batches) or nullptr
  float* xi_h;
  uint32_t* status;
  const float* lse;                  // [B, H, N] row log-sum-exp (natural log) from the caller, or nullptr
  int64_t lse_bs, lse_hs;
  float* lse_out;                    // [B, H, N] receives the row log-sum-exp of the vision rows, or nullptr
  int64_t lse_out_bs, lse_out_hs;
  TextSet text;                      // prompt-token set J
  int n_text_after, bidirectional;   // bidirectional: every query sees all keys of its sample
  int cap_in, vis_begin, n_q_heads, group;
  int batch, n_qt;                   // samples, query tiles of 128 rows per (sample, head)
  float scale2;                      // log2(e) / sqrt(dh)
  XiSched* sched;
  int* redo_list;                    // [n_qt * H * B] items whose sums left the fp32 range
};

constexpr int XT_STAGES = 2;         // K tiles in the shared-memory ring
constexpr int XT_SBUF = 2;           // S accumulators in tensor memory
constexpr int XT_CTAS = 2;           // CTAs per SM
constexpr int XT_KEY_TILE = 128;     // keys per K tile and per MMA (the softmax warps read it as two halves of 64)
constexpr int XT_SUB = 64;           // keys per half
constexpr int XT_THREADS = 320;      // TMA / scheduler warp, MMA warp, eight softmax warps
constexpr int XT_SAMPLE_CACHE = 256;  // samples whose token count and row offset are kept in shared memory
constexpr int XT_HEAD_GROUP = 64;    // (sample, head) pairs whose work items are interleaved (their K: 64 x ~1 MB)

// LSE: the caller supplied the row log-sum-exp (a.lse != nullptr).  SAFE: second launch, items from the list.
template <int DH, bool LSE, bool SAFE>
__global__ void __launch_bounds__(XT_THREADS, XT_CTAS)
xi_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map, XiTcArgs a) {
  grid_dependency_sync();
  constexpr int BK = XT_KEY_TILE;
  static_assert(BK == 2 * XT_SUB && XT_SUB == 64, "a K tile is two halves of 64 keys; the prompt mask of a half is one 64-bit word");
  static_assert(!(LSE && SAFE), "with the caller's normaliser no sum can leave the fp32 range");
  constexpr int HALVES = DH / 64;
  constexpr uint32_t TILE_BYTES = HALVES * 16384;          // Q tile: 128 rows x DH bf16
  constexpr uint32_t KHALF_BYTES = BK * 128;               // BK key rows x 64 columns
  constexpr uint32_t KT_BYTES = HALVES * KHALF_BYTES;      // K tile: BK rows x DH bf16
  // With the caller's normaliser an item is one or two key tiles and the kernel is bound by reading Q from HBM:
  // then the Q tile is double buffered (two items' Q in flight per CTA) and one K stage is enough.
  constexpr int QBUF = LSE ? 2 : 1, KSTAGES = LSE ? 1 : XT_STAGES;
  const unsigned int n_items = SAFE ? a.sched->n_redo : unsigned(a.n_qt) * a.n_q_heads * a.batch;
  if (n_items == 0) return;                                // nothing on the list: the usual case of the second launch

  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* q_s = base;                   // [QBUF] Q tiles
  unsigned char* k_s = base + QBUF * TILE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + QBUF * TILE_BYTES + KT_BYTES * KSTAGES);
  uint64_t* q_full = bars;                     // [2]
  uint64_t* q_empty = bars + 2;                // [2] every MMA that reads the Q tile has completed
  uint64_t* k_full = bars + 4;                 // [XT_STAGES]
  uint64_t* k_empty = k_full + XT_STAGES;      // [XT_STAGES]
  uint64_t* s_full = k_empty + XT_STAGES;      // [XT_SBUF]
  uint64_t* s_empty = s_full + XT_SBUF;        // [XT_SBUF]
  uint64_t* item_full = s_empty + XT_SBUF;     // [2] the scheduler published an item
  uint64_t* item_empty = item_full + 2;        // [2] the MMA thread and the eight softmax warps have read it
  uint64_t* pair_full = item_empty + 2;        // the upper column group has stored its partial sums of an item
  uint64_t* pair_empty = pair_full + 1;        // the lower column group has read them
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pair_empty + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* item_slot = abort_flag + 1;    // [2]
  int* redo_mark = const_cast<int*>(item_slot) + 2;      // last item this CTA put on the list
  float* pair_m = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(bars) + 256);   // [128] each
  float* pair_all = pair_m + 128;
  float* pair_txt = pair_all + 128;
  // per-sample token counts and row offsets, read once (every role decodes every item; a trip to global memory
  // per item would be a good part of a short item); samples beyond the cache are read from global memory
  int* s_nvis = reinterpret_cast<int*>(pair_txt + 128);    // [XT_SAMPLE_CACHE]
  int* s_row0 = s_nvis + XT_SAMPLE_CACHE;                   // [XT_SAMPLE_CACHE]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // key tiles to visit: all tiles up to the last query's own key, or, when the caller supplies the row
  // log-sum-exp, only the tiles that hold prompt keys (J lies before the vision block, so it is visible)
  const int kt_lo = LSE ? a.text.begin / BK : 0;
  const int nkt_lse = a.text.end > a.text.begin ? (a.text.end - 1) / BK + 1 - kt_lo : 0;
  struct Item { int h, b, t0, nq, s_first, nkt, n_seq, nsub, row0, bc; };   // nsub: halves of 64 keys the item visits;
                                                                           // row0, bc: row offset and batch coordinate of the TMA loads
  // item -> (query tile, head, sample).  The (sample, head) pairs are taken in groups of XT_HEAD_GROUP whose keys
  // stay in L2 together; inside a group the list runs over the query tiles from the longest rows to the shortest,
  // all pairs of the group for each, so that the work left for the last tickets is short.
  auto decode = [&](int item, Item& it) -> bool {
    const int n_hb = a.n_q_heads * a.batch, per_group = XT_HEAD_GROUP * a.n_qt;
    const int grp = item / per_group, within = item - grp * per_group;
    const int gsize = min(XT_HEAD_GROUP, n_hb - grp * XT_HEAD_GROUP);
    const int hb = grp * XT_HEAD_GROUP + within % gsize, qt = a.n_qt - 1 - within / gsize;
    it.h = hb % a.n_q_heads; it.b = hb / a.n_q_heads;
    const int n = it.b < XT_SAMPLE_CACHE ? s_nvis[it.b] : (a.n_vis ? min(a.n_vis[it.b], a.cap_in) : a.cap_in);
    it.t0 = qt * 128;
    if (it.t0 >= n) return false;
    it.nq = min(128, n - it.t0);
    it.s_first = a.vis_begin + it.t0;
    it.n_seq = a.vis_begin + n + a.n_text_after;
    it.nsub = LSE ? 2 * nkt_lse : ((a.bidirectional ? it.n_seq : it.s_first + it.nq) - 1) / XT_SUB + 1;
    it.nkt = (it.nsub + 1) / 2;
    it.row0 = it.b < XT_SAMPLE_CACHE ? s_row0[it.b] : (a.seq_start ? a.seq_start[it.b] : 0);   // packed batch: one long
                                                                                              // row axis, batch coordinate 0
    it.bc = a.seq_start ? 0 : it.b;
    return true;
  };

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) { mbar_init(&q_full[i], 1); mbar_init(&q_empty[i], 1); }
    for (int i = 0; i < XT_STAGES; ++i) { mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1); }
    for (int i = 0; i < XT_SBUF; ++i) { mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 8); }
    for (int i = 0; i < 2; ++i) { mbar_init(&item_full[i], 1); mbar_init(&item_empty[i], 9); }
    mbar_init(pair_full, 4);
    mbar_init(pair_empty, 4);
    *abort_flag = 0;
    *redo_mark = -1;
    fence_barrier_init();
  }
  if (warp == 1) { tmem_alloc(tmem_slot, XT_SBUF * BK); tmem_relinquish(); }
  for (int i = threadIdx.x; i < min(a.batch, XT_SAMPLE_CACHE); i += blockDim.x) {
    s_nvis[i] = a.n_vis ? min(a.n_vis[i], a.cap_in) : a.cap_in;
    s_row0[i] = a.seq_start ? a.seq_start[i] : 0;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ---- scheduler + TMA producer
      prefetch_tensormap(&q_map);
      prefetch_tensormap(&k_map);
      uint32_t kf = 0, n = 0, nq_loaded = 0;           // K tiles fetched / items published / Q tiles loaded
      for (;;) {
        const uint32_t slot = n & 1;
        if (!mbar_wait(&item_empty[slot], ((n >> 1) & 1) ^ 1, abort_flag)) break;
        // items of the LSE form are all alike: a fixed round-robin split balances them and saves the atomic's
        // round trip, which would otherwise be a good part of such a short item
        const unsigned int t = LSE ? blockIdx.x + n * gridDim.x
                                   : atomicAdd(SAFE ? &a.sched->safe_ticket : &a.sched->ticket, 1u);
        const int item = t < n_items ? (SAFE ? a.redo_list[t] : int(t)) : -1;
        item_slot[slot] = item;
        mbar_arrive(&item_full[slot]);                 // release: the slot is written before the arrival is seen
        ++n;
        if (item < 0) break;
        Item it;
        if (!decode(item, it) || it.nkt == 0) continue;
        // a Q buffer is free once every MMA of the item that used it last has completed
        const uint32_t qb = nq_loaded % QBUF, q_use = nq_loaded / QBUF;
        if (q_use > 0 && !mbar_wait(&q_empty[qb], (q_use - 1) & 1, abort_flag)) break;
        mbar_expect_tx(&q_full[qb], TILE_BYTES);
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf)
          tma_load_4d(q_s + qb * TILE_BYTES + hf * 16384, &q_map, &q_full[qb], hf * 64, it.row0 + it.s_first, it.h, it.bc);
        ++nq_loaded;
        const int hk = it.h / a.group;
        bool ok = true;
        for (int kt = 0; kt < it.nkt; ++kt, ++kf) {
          const uint32_t s = kf % KSTAGES;
          if (!mbar_wait(&k_empty[s], ((kf / KSTAGES) & 1) ^ 1, abort_flag)) { ok = false; break; }
          mbar_expect_tx(&k_full[s], KT_BYTES);
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_4d(k_s + s * KT_BYTES + hf * KHALF_BYTES, &k_map, &k_full[s], hf * 64, it.row0 + (kt_lo + kt) * BK, hk, it.bc);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issue
      constexpr uint32_t idesc_full = idesc_bf16(128, BK), idesc_half = idesc_bf16(128, XT_SUB);
      // the operand descriptors are built once (Q: one per 16-column step; K: those of ring stage 0, a stage
      // adds a constant to the address field)
      uint64_t q_desc[DH / 16], k_desc[DH / 16];
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        q_desc[kk] = smem_desc_sw128(smem_u32(q_s) + (kk >> 2) * 16384 + (kk & 3) * 32);
        k_desc[kk] = smem_desc_sw128(smem_u32(k_s) + (kk >> 2) * KHALF_BYTES + (kk & 3) * 32);
      }
      uint32_t kc = 0, n = 0, nq_used = 0;             // K tiles consumed / items read / Q tiles used
      for (;;) {
        const uint32_t slot = n & 1;
        if (!mbar_wait(&item_full[slot], (n >> 1) & 1, abort_flag)) break;
        const int item = item_slot[slot];
        mbar_arrive(&item_empty[slot]);
        ++n;
        if (item < 0) break;
        Item it;
        if (!decode(item, it) || it.nkt == 0) continue;
        const uint32_t qb = nq_used % QBUF;
        if (!mbar_wait(&q_full[qb], (nq_used / QBUF) & 1, abort_flag)) break;
        const uint64_t q_off = uint64_t(qb * (TILE_BYTES >> 4));
        bool ok = true;
        for (int kt = 0; kt < it.nkt; ++kt, ++kc) {
          const uint32_t s = kc % KSTAGES, buf = kc % XT_SBUF;
          if (!mbar_wait(&s_empty[buf], ((kc / XT_SBUF) & 1) ^ 1, abort_flag) ||
              !mbar_wait(&k_full[s], (kc / KSTAGES) & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t stage_off = uint64_t(s * (KT_BYTES >> 4));     // the address field counts 16-byte units
          const uint32_t d_addr = tmem_base + buf * BK;
          // the last tile of an odd number of halves needs its first 64 keys only
          const uint32_t idesc = (2 * kt + 2 > it.nsub) ? idesc_half : idesc_full;
#pragma unroll
          for (int kk = 0; kk < DH / 16; ++kk) umma_bf16(d_addr, q_desc[kk] + q_off, k_desc[kk] + stage_off, idesc, kk > 0);
          umma_commit(&k_empty[s]);
          umma_commit(&s_full[buf]);
        }
        if (!ok) break;
        umma_commit(&q_empty[qb]);
        ++nq_used;
      }
    }
  } else {
    // ---- softmax warps: two threads per query row.  Warps 2-5 take the lower 32 columns of every half of 64
    //      keys, warps 6-9 the upper 32; warp w may read the TMEM lanes of quadrant w % 4.  Each thread keeps
    //      its own reference and sums; the two partial results of a row are combined once per item.
    const int sw = warp - 2, quad = warp & 3, cg = sw >> 2;   // softmax warp 0..7, lane quadrant, column group
    const int r = quad * 32 + lane;                     // query row of this thread
    const uint32_t lane_addr = tmem_base + (uint32_t(quad * 32) << 16) + cg * 32;
    const float sc = a.scale2;
    uint32_t kc = 0, n = 0, np = 0;                     // key tiles consumed / items read / exchanges done by this CTA
    bool alive = true;
    while (alive) {
      const uint32_t slot = n & 1;
      const bool published = mbar_wait(&item_full[slot], (n >> 1) & 1, abort_flag);
      if (!__all_sync(0xffffffffu, published)) break;
      const int item = item_slot[slot];
      __syncwarp();                                     // every lane has read the slot
      if (lane == 0) mbar_arrive(&item_empty[slot]);
      ++n;
      if (item < 0) break;
      Item it;
      if (!decode(item, it)) continue;
      const int h = it.h, b = it.b, nq = it.nq, s_first = it.s_first;
      float m_run = -INFINITY, l_all = 0.f, l_txt = 0.f;
      // the caller's normaliser of this row, in log2 units (fetched before the first wait: its latency hides there)
      float l2 = 0.f;
      if (LSE && r < nq) l2 = a.lse[size_t(b) * a.lse_bs + size_t(h) * a.lse_hs + it.row0 + s_first + r] * 1.4426950408889634f;
      for (int kt = 0; kt < it.nkt; ++kt, ++kc) {
        const uint32_t buf = kc % XT_SBUF;
        const bool landed = mbar_wait(&s_full[buf], (kc / XT_SBUF) & 1, abort_flag);
        if (!__all_sync(0xffffffffu, landed)) { alive = false; break; }   // the TMEM loads below are warp-wide
        tc_fence_after();
        const int n_half = min(2, it.nsub - 2 * kt);     // halves of this tile the item needs
        for (int half = 0; half < n_half; ++half) {
          const int j0 = (kt_lo + kt) * BK + half * XT_SUB + cg * 32;      // first key of this thread's 32 columns
          float v[32];
          tmem_ld32(lane_addr + buf * BK + half * XT_SUB, v);
          tmem_ld_wait();
          if (half == n_half - 1) {                       // the accumulator is in registers: hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_empty[buf]);
          }

          if (LSE) {                                      // normaliser known: only the prompt columns count
            const unsigned int tm = (unsigned int)a.text.mask64(j0);
            l_all = 1.f;
            if (tm == 0xffffffffu) {                      // all 32 keys are prompt keys: no tests, four chains
              float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int i = 0; i < 32; ++i) part[i & 3] += ex2(fmaf(v[i], sc, -l2));
              l_txt += (part[0] + part[1]) + (part[2] + part[3]);
            } else if (tm != 0u) {
              float st = 0.f;
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if ((tm >> i) & 1u) st += ex2(fmaf(v[i], sc, -l2));
              l_txt += st;
            }
            continue;
          }
          const bool in_j = j0 < a.text.end && j0 + 32 > a.text.begin;     // the columns reach into the prompt set J
          // some row does not see all of these keys: the diagonal, or the end of the sample
          const bool edge = j0 + 31 > (a.bidirectional ? it.n_seq - 1 : s_first);
          int lim_max = 32;                                // columns at least one row of this warp sees
          if (edge) {
            const int lim = (a.bidirectional ? it.n_seq - 1 : s_first + r) - j0;   // last visible column of this row
            lim_max = __reduce_max_sync(0xffffffffu, lim);
            if (lim_max < 0) continue;                     // no row of this warp sees any of these keys
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i > lim) v[i] = -INFINITY;
          }
          if (SAFE || __any_sync(0xffffffffu, m_run == -INFINITY)) {
            // reference of the thread: maximum of the first 32 columns of its own in which it sees a key (the
            // first 64 keys of the row, unless the row is among the first 32 of a sequence), of every half when
            // SAFE.  While some row of the warp has no reference yet the others update theirs, which is exact.
            float mx[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              mx[j] = v[j * 8];
#pragma unroll
              for (int i = 1; i < 8; ++i) mx[j] = fmaxf(mx[j], v[j * 8 + i]);
            }
            const float m_new = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), m_run);
            if (m_new > -INFINITY) {                        // (a thread whose 32 columns are all masked keeps none)
              const float resc = ex2((m_run - m_new) * sc); // 0 on the first half
              l_all *= resc;
              l_txt *= resc;
              m_run = m_new;
            }
          }
          if (m_run == -INFINITY) continue;                // this thread has not seen a key yet
          const float ms = m_run * sc;
          if (!edge && !in_j) {
            // the bulk: every eighth exponential on the FMA pipe
            float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float x = fmaf(v[i], sc, -ms);
              part[i & 3] += (i & 7) == 7 ? ex2_fma(x) : ex2(x);
            }
            l_all += (part[0] + part[1]) + (part[2] + part[3]);
          } else {
            const unsigned int tm = in_j ? (unsigned int)a.text.mask64(j0) : 0u;
            float sa = 0.f, st = 0.f;
#pragma unroll
            for (int blk = 0; blk < 4; ++blk)
              if (blk * 8 <= lim_max) {                     // warp-uniform: masked blocks cost no exponentials
                float pa = 0.f, pt = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const float p = ex2(fmaf(v[blk * 8 + i], sc, -ms));   // exp2(-inf) = 0 on masked columns
                  pa += p;
                  if ((tm >> (blk * 8 + i)) & 1u) pt += p;
                }
                sa += pa;
                st += pt;
              }
            l_all += sa;
            l_txt += st;
          }
        }  // halves
      }  // key tiles
      // ---- the two threads of a row meet: the upper column group hands its reference and sums over.  Every warp
      //      that entered the item takes part, also after a failed wait (the flag is raised, nothing is stored).
      if (cg == 1) {
        const bool free_again = np == 0 || mbar_wait(pair_empty, (np - 1) & 1, abort_flag);
        if (!__all_sync(0xffffffffu, free_again)) alive = false;
        pair_m[r] = m_run; pair_all[r] = l_all; pair_txt[r] = l_txt;
        __syncwarp();
        if (lane == 0) mbar_arrive(pair_full);
        ++np;
        if (!alive) break;
        continue;
      }
      {
        const bool handed = mbar_wait(pair_full, np & 1, abort_flag);
        if (!__all_sync(0xffffffffu, handed)) alive = false;
        ++np;
        if (!alive) break;
        if (!LSE) {
          const float m_o = pair_m[r], m_new = fmaxf(m_run, m_o);
          const float f_own = ex2((m_run - m_new) * sc), f_o = m_o > -INFINITY ? ex2((m_o - m_new) * sc) : 0.f;
          l_all = fmaf(l_all, f_own, pair_all[r] * f_o);
          l_txt = fmaf(l_txt, f_own, pair_txt[r] * f_o);
          m_run = m_new;
        } else {
          l_txt += pair_txt[r];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(pair_empty);             // the exchange buffers are free for the next item
      }
      if (!LSE && !SAFE) {
        // a sum that is not a finite number means some logit lay more than 88 above the reference: the item
        // goes on the list of the second launch (once per CTA)
        const bool bad = r < nq && !(l_all <= 3.0e38f);
        if (__any_sync(0xffffffffu, bad) && lane == 0 && atomicExch(redo_mark, item) != item)
          a.redo_list[atomicAdd(&a.sched->n_redo, 1u)] = item;
      }
      if (r < nq && !*abort_flag) {
        a.xi_h[(size_t(b) * a.n_q_heads + h) * a.cap_in + it.t0 + r] = LSE ? l_txt : l_txt / l_all;
        if (!LSE && a.lse_out)
          a.lse_out[size_t(b) * a.lse_out_bs + size_t(h) * a.lse_out_hs + it.row0 + s_first + r] =
              fmaf(m_run, sc, log2f(l_all)) * 0.6931471805599453f;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, XT_SBUF * BK);
  }
  if (threadIdx.x == 0 && *abort_flag && a.status) atomicOr(a.status, LIGHTKV_STATUS_TIMEOUT);
}

bool tc_xi_supported(int head_dim) { return head_dim == 64 || head_dim == 128; }

static int sm_count();

cudaError_t launch_xi_tc(const LayerLaunch& L) {
  const lightkv_layer_args_t* a = L.a;
  const int rows = a->seq_rows > 0 ? a->seq_rows : a->vis_begin + L.ws.cap_in + a->n_text_after;
  CUtensorMap qm, km;
  const int map_batch = a->seq_start ? 1 : L.batch;       // packed batch: every sample lives on one row axis
  if (!make_map_bhnd(&qm, a->q, L.head_dim, rows, L.n_q_heads, map_batch, a->q_row_stride, a->q_head_stride,
                     a->q_batch_stride, 128) ||
      !make_map_bhnd(&km, a->k, L.head_dim, rows, L.n_kv_heads, map_batch, a->k_row_stride, a->k_head_stride,
                     a->k_batch_stride, XT_KEY_TILE))
    return cudaErrorInvalidValue;
  XiTcArgs x;
  x.n_vis = a->n_vis; x.seq_start = a->seq_start; x.xi_h = L.ws.xi_h; x.status = a->status; x.cap_in = L.ws.cap_in;
  x.lse = L.xi_mode == LIGHTKV_XI_ATTN_LSE ? a->lse : nullptr; x.lse_bs = a->lse_batch_stride; x.lse_hs = a->lse_head_stride;
  x.lse_out = L.xi_mode == LIGHTKV_XI_ATTN_FULL ? a->lse_out : nullptr;
  x.lse_out_bs = a->lse_out_batch_stride; x.lse_out_hs = a->lse_out_head_stride;
  x.text = L.text; x.n_text_after = a->n_text_after; x.bidirectional = a->bidirectional;
  x.vis_begin = a->vis_begin;
  x.n_q_heads = L.n_q_heads; x.group = L.n_q_heads / L.n_kv_heads;
  x.scale2 = 1.4426950408889634f / sqrtf((float)L.head_dim);
  x.batch = L.batch; x.n_qt = (L.ws.cap_in + 127) / 128;
  x.sched = reinterpret_cast<XiSched*>(L.ws.xi_sched); x.redo_list = L.ws.xi_redo;
  const long long n_items = (long long)x.n_qt * L.n_q_heads * L.batch;
  if (n_items > 0x7fffffffLL) return cudaErrorInvalidValue;
  // As many CTAs as stay resident (two per SM) draw work items from a ticket counter; with the caller's
  // log-sum-exp an item is one or two key tiles, otherwise up to the whole row.
  const dim3 grid((unsigned)std::min<long long>(n_items, XT_CTAS * sm_count()));
  // Q tiles + K ring (LSE: two Q tiles, one K stage; otherwise one Q tile, XT_STAGES K stages) + barriers + exchange
  const size_t smem = size_t(L.head_dim / 64) * (x.lse ? 2 * 16384 + XT_KEY_TILE * 128
                                                        : 16384 + size_t(XT_STAGES) * XT_KEY_TILE * 128) + 1024 + 256 + 1536 + 2 * XT_SAMPLE_CACHE * sizeof(int);
  cudaError_t e = cudaMemsetAsync(x.sched, 0, sizeof(XiSched), L.stream);      // tickets and list length start at 0
  if (e != cudaSuccess) return e;
  auto launch = [&](auto kernel, dim3 g) -> cudaError_t {
    const cudaError_t rc = ensure_dynamic_smem(kernel, (int)smem);
    if (rc != cudaSuccess) return rc;
    return launch_kernel(kernel, g, XT_THREADS, smem, L.stream, 1, qm, km, x);
  };
  if (x.lse) return L.head_dim == 128 ? launch(xi_tc_kernel<128, true, false>, grid) : launch(xi_tc_kernel<64, true, false>, grid);
  e = L.head_dim == 128 ? launch(xi_tc_kernel<128, false, false>, grid) : launch(xi_tc_kernel<64, false, false>, grid);
  if (e != cudaSuccess) return e;
  // second launch: the items whose sums left the fp32 range, with a running maximum (returns at once when the
  // list is empty; one CTA per SM is plenty for what is an exception)
  const dim3 grid2((unsigned)std::min<long long>(n_items, sm_count()));
  return L.head_dim == 128 ? launch(xi_tc_kernel<128, false, true>, grid2) : launch(xi_tc_kernel<64, false, true>, grid2);
}

// ======================================================================================================
// FD + best partner on tensor cores (Eq. "similarity", Step 2).
//
// Persistent CTAs, two per SM; a work item is a tile of up to 128 A entries x 128 B entries (see
// FdTiling): a group of whole windows, or one 128 x 128 block of a large window.  The rows of a tile are
// scattered over the sequence (they are listed by a_tok / b_tok), so eight warps gather them with 16-byte
// cp.async copies, eight threads per 128-byte row segment, straight into the 128-byte-swizzled K-major
// layout tcgen05 reads.  The copies go through a ring of six 16 KB stages; a stage is 128 row slots of
// 128 bytes (64 columns) and every loader thread fills four slots of it.  What the slots hold depends
// on the tile's size (passes = 1, 2, 4 <=> at most 32, 64, 128 entries per operand):
//   passes 4: even fills = the 128 A rows of a chunk, odd fills = its 128 B rows   (2 fills per chunk)
//   passes 2: [64 A rows | 64 B rows] of one chunk                                  (1 fill per chunk)
//   passes 1: [32 A rows, chunk c | 32 A rows, chunk c+1 | 32 B rows, c | 32 B rows, c+1]   (2 chunks per fill)
// Four fills are in flight while a fifth is being consumed and a sixth may still be held by the tensor
// core, so the loaders never wait for an MMA on their critical path.  Each thread re-reads the pieces
// it fetched to accumulate the rows' squared norms: X is read from HBM exactly once.  A ninth warp
// issues G += X_A X_B^T (128 x N x 64 per chunk, N = B entries rounded up to 16, bf16 -> fp32 in TMEM).
// The MMA always reads 128 A rows (16 KB) from the start of a chunk's A block: rows the tile does not
// have are never written, may overlap other blocks or the 4 KB pad behind the ring, and only feed
// accumulator rows nobody reads.  After the last chunk the loader warps turn into the epilogue: one
// thread per A row scans the FD of the columns that belong to the row's own window and keeps the
// minimum (ties: lowest B index).  Blocks of a large window combine through a 64-bit atomicMin on
// (orderable FD, B index), which is order independent.
// ======================================================================================================
struct FdTcArgs {
  const __nv_bfloat16* x;              // first vision row of sample 0
  const int* seq_start;                // first row of each sample (packed batches) or nullptr
  int64_t batch_stride, row_stride;    // elements
  int d, batch;
  int metric;                          // LIGHTKV_FD_*
  Workspace ws;
  uint32_t* status;
};

// pair score from the inner product g and the norms of the two rows: the norms themselves for FD = 1 - cosine,
// the squared norms for the Euclidean scores |a|^2 + |b|^2 - 2 g
__device__ __forceinline__ float pair_score(int metric, float g, float na, float nb) {
  if (metric == LIGHTKV_FD_COSINE) {
    const float den = na * nb;
    return 1.0f - (den > 0.f ? g / den : 0.f);
  }
  const float sq = fmaxf(fmaf(-2.0f, g, na + nb), 0.f);
  return metric == LIGHTKV_FD_L2 ? sqrtf(sq) : sq;
}

constexpr int FT_LOADERS = 256;
constexpr int FT_STAGES = 6;
constexpr int FT_AHEAD = 4;                               // fills in flight
constexpr int kFdPitch = kFdTile + 1;                     // row pitch (floats) of a partial G in shared memory
constexpr uint32_t FT_STAGE_BYTES = 16 * 1024;
constexpr uint32_t FT_RING_BYTES = FT_STAGES * FT_STAGE_BYTES + 4096;   // + pad for the 16 KB A read
constexpr size_t FT_SMEM = size_t(FT_RING_BYTES) + 1024 /* alignment */ + 128 /* barriers */ +
                           4 * kFdTile * sizeof(float);

// Second half of the cluster epilogue (kept out of line so that it does not weigh on the registers of the
// streaming loop): full norms = partial squared sums added in rank order; then CTA `rank` finishes rows
// [rank * 128 / ks, (rank + 1) * 128 / ks), a warp per row, lanes over the columns of the row's window.
__device__ __noinline__ void fd_cluster_finish(int metric, const int* a_win, unsigned long long* a_key, int ks, int rank, int a0, int a1,
                                               int b0, int b1,
                                               bool combine, const int* win_off, const int* a_off, uint32_t p0,
                                               const float* a_nrm, const float* b_nrm, float* nrm_a, float* nrm_b,
                                               volatile int* abort_flag) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  {
    const int i = tid & (kFdTile - 1);
    const uint32_t src = smem_u32(tid < kFdTile ? a_nrm + i : b_nrm + i);
    float ss = 0.f;
    for (int j = 0; j < ks; ++j) ss += ld_cluster_f32(map_to_cta(src, j));
    (tid < kFdTile ? nrm_a : nrm_b)[i] = metric == LIGHTKV_FD_COSINE ? sqrtf(ss) : ss;
  }
  named_barrier(1, FT_LOADERS);
  // CTA `rank` finishes rows [rank * 128 / ks, (rank + 1) * 128 / ks): a warp per row, lanes over the
  // columns of the row's window, partial sums added in rank order
  const int rows_mine = kFdTile / ks, r0 = rank * rows_mine;
  for (int rr = warp; rr < rows_mine; rr += 8) {
    const int row = r0 + rr, e = a0 + row;
    if (e >= a1) break;                               // warp-uniform; later rows are further out
    const int w = a_win[e];
    const int lo = max(win_off[w] - a_off[w], b0) - b0, hi = min(win_off[w + 1] - a_off[w + 1], b1) - b0;
    const float na = nrm_a[row];
    float best = 3.0e38f;
    int best_c = -1;
    for (int col = lo + lane; col < hi; col += 32) {
      const uint32_t src = p0 + uint32_t(row * kFdPitch + col) * 4;
      float gsum = 0.f;
      for (int j = 0; j < ks; ++j) gsum += ld_cluster_f32(map_to_cta(src, j));
      const float fd = pair_score(metric, gsum, na, nrm_b[col]);
      if (fd < best) { best = fd; best_c = col; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {                // minimum over the lanes, ties to the lower column
      const float of = __shfl_xor_sync(0xffffffffu, best, o);
      const int oc = __shfl_xor_sync(0xffffffffu, best_c, o);
      if (oc >= 0 && (best_c < 0 || of < best || (of == best && oc < best_c))) { best = of; best_c = oc; }
    }
    if (lane == 0 && best_c >= 0 && !*abort_flag) {
      const unsigned long long key = ((unsigned long long)orderable(best) << 32) | (unsigned)(b0 + best_c);
      unsigned long long* dst = a_key + e;
      if (combine) atomicMin(dst, key); else *dst = key;
    }
  }
}

// CLUSTER = false is the plain launch (ks = 1) with the cluster code compiled out.
template <bool CLUSTER>
__global__ void __launch_bounds__(FT_LOADERS + 32, 2) fd_tc_kernel(FdTcArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + FT_RING_BYTES);
  uint64_t* full = bars;                        // [FT_STAGES] fill landed (one arrival per loader warp)
  uint64_t* empty = full + FT_STAGES;           // [FT_STAGES] fill consumed (MMA commit)
  uint64_t* acc_full = empty + FT_STAGES;       // accumulator complete
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* a_nrm = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(bars) + 128);   // [128]
  float* b_nrm = a_nrm + kFdTile;                                                          // [128]
  float* red_f = b_nrm + kFdTile;                                                          // [128]
  int* red_c = reinterpret_cast<int*>(red_f + kFdTile);                                    // [128]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int i = 0; i < FT_STAGES; ++i) { mbar_init(&full[i], FT_LOADERS / 32); mbar_init(&empty[i], 1); }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 8) { tmem_alloc(tmem_slot, kFdTile); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // barriers and tensor memory are set up while the kernel before this one may still be running; from here on
  // global memory is read (and written), so that kernel must have completed
  grid_dependency_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t ring = smem_u32(base);
  const int nW = a.ws.n_windows;
  // A cluster of ks CTAs shares every tile: CTA `rank` contracts chunks [c_lo, c_lo + nk) of the hidden
  // dimension and the partial results are combined through distributed shared memory (ks = 1: no cluster).
  const int ks = CLUSTER ? (int)cluster_nctarank() : 1, rank = CLUSTER ? (int)cluster_ctarank() : 0;
  const int nk_all = (a.d + 63) >> 6;           // 64-column chunks of the whole hidden dimension
  const int c_lo = rank * nk_all / ks, nk = (rank + 1) * nk_all / ks - c_lo;

  // Work items are the (sample, tile) pairs of the whole batch in sample order; this CTA takes items
  // cluster id, cluster id + number of clusters, ...  Barrier phases run on across items: `done` counts the
  // fills this CTA has completed, `n_items` its finished tiles.
  uint32_t done = 0, n_items = 0;
  for (int item = blockIdx.x / ks;; item += gridDim.x / ks) {
  int b = 0, tile = item;
  while (b < a.batch) {
    const int nt = a.ws.fd_tiling[b].n_tiles;
    if (tile < nt) break;
    tile -= nt;
    ++b;
  }
  if (b >= a.batch) break;                      // same for every thread of the CTA
  const FdTiling tl = a.ws.fd_tiling[b];
  const int* win_off = a.ws.win_off + size_t(b) * (nW + 1);
  const int* a_off = a.ws.a_off + size_t(b) * (nW + 1);
  const int per_group = tl.blocks_a * tl.blocks_b;
  const int grp = tile / per_group, rem = tile - grp * per_group;
  const int ia = rem / tl.blocks_b, ib = rem - ia * tl.blocks_b;
  const int w0 = min(grp * tl.wpt, nW), w1 = min(nW, w0 + tl.wpt);
  const int passes = tl.passes;                                      // 1, 2 or 4
  const int cap_rows = 32 * passes;
  const int a0 = a_off[w0] + ia * kFdTile, a1 = min(a_off[w1], a0 + cap_rows);
  const int b0 = win_off[w0] - a_off[w0] + ib * kFdTile, b1 = min(win_off[w1] - a_off[w1], b0 + cap_rows);
  if (a0 >= a1 || b0 >= b1) continue;           // same for every thread of the CTA
  const int n_cols = (b1 - b0 + 15) & ~15;      // MMA N
  const int nf = passes == 4 ? 2 * nk : (passes == 2 ? nk : (nk + 1) >> 1);   // fills of this tile

  if (warp < 8) {
    // ---- gather: thread = 16-byte piece c of row slots g, g + 32, g + 64, g + 96 of every fill
    const int c = tid & 7, g = tid >> 3;
    const unsigned char* xb = reinterpret_cast<const unsigned char*>(
        a.x + size_t(b) * a.batch_stride + size_t(a.seq_start ? a.seq_start[b] : 0) * a.row_stride) + size_t(c_lo) * 128;
    const int* a_tok = a.ws.a_tok + size_t(b) * a.ws.cap_a;
    const int* b_tok = a.ws.b_tok + size_t(b) * a.ws.cap_b;
    // source row of slot t on even / odd fills (they differ only when passes = 4), validity bits, and the
    // chunk of slot t relative to the fill's first chunk (passes = 1 packs two chunks into a fill)
    const unsigned char* src_e[4];
    const unsigned char* src_o[4];
    uint32_t ok_e = 0, ok_o = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int i = passes == 4 ? t : (passes == 2 ? (t & 1) : 0);          // row g + 32 i of the operand
      const bool slot_b = passes == 4 ? false : (t >> 1) != 0;              // operand of slot t on even fills
      const int ea = a0 + g + 32 * i, eb = b0 + g + 32 * i;
      const int ta = ea < a1 ? a_tok[ea] : -1, tb = eb < b1 ? b_tok[eb] : -1;
      const unsigned char* pa = xb + (size_t(max(ta, 0)) * a.row_stride + c * 8) * 2;
      const unsigned char* pb = xb + (size_t(max(tb, 0)) * a.row_stride + c * 8) * 2;
      const size_t sub = passes == 1 ? size_t(t & 1) * 128 : 0;             // second chunk of the fill
      src_e[t] = (slot_b ? pb : pa) + sub;
      src_o[t] = (passes == 4 ? pb : (slot_b ? pb : pa)) + sub;
      ok_e |= ((slot_b ? tb : ta) >= 0 ? 1u : 0u) << t;
      ok_o |= ((passes == 4 ? tb : (slot_b ? tb : ta)) >= 0 ? 1u : 0u) << t;
    }
    const uint32_t slot0 = uint32_t(g) * 128 + (uint32_t(c ^ (g & 7)) << 4);   // swizzled offset of slot g; slot g+32t is 4096 t further
    const int chunk_shift = passes == 4 ? 1 : 0, chunk_mul = passes == 1 ? 2 : 1;
    float acc_e[4] = {0.f, 0.f, 0.f, 0.f}, acc_o[4] = {0.f, 0.f, 0.f, 0.f};
    // columns of this thread's A row in the epilogue (row = TMEM lane): the B entries of the row's own window.
    // Fetched here, two dependent loads deep, so that their latency hides behind the rows that stream below.
    const int q = warp & 3, half = warp >> 2, row = q * 32 + lane, e = a0 + row;
    int lo = 0x7fffffff, hi = 0;
    if (e < a1) {
      const int w = a.ws.a_win[size_t(b) * a.ws.cap_a + e];
      lo = max(win_off[w] - a_off[w], b0) - b0;
      hi = min(win_off[w + 1] - a_off[w + 1], b1) - b0;
    }

    // rows the tile does not have and chunks past the hidden size are not fetched at all; the pieces of
    // the last chunk that lie past the hidden size are zero-filled
    auto issue = [&](int f, uint32_t stage) {
      const uint32_t sb = ring + stage * FT_STAGE_BYTES + slot0;
      const bool odd = passes == 4 && (f & 1);
      const int kc0 = (f >> chunk_shift) * chunk_mul;
      const uint32_t okm = odd ? ok_o : ok_e;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int kc = kc0 + (passes == 1 ? (t & 1) : 0);
        if (kc >= nk || !((okm >> t) & 1)) continue;
        const uint32_t bytes = ((c_lo + kc) * 64 + c * 8 < a.d) ? 16u : 0u;   // d is a multiple of 8
        const unsigned char* p = odd ? src_o[t] : src_e[t];
        cp_async16(sb + t * 4096, p + (bytes ? size_t(kc0) * 128 : 0), bytes);
      }
    };
    // acc += lo^2 + hi^2 for the four bf16 pairs of v, each product exact in fp32 and added with one rounding
    // (the mixed-precision fma reads the bf16 halves directly: no unpacking instructions)
    auto sumsq = [](const uint4& v, float acc) {
      const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\t"
            "fma.rn.f32.bf16 %0, lo, lo, %0;\n\tfma.rn.f32.bf16 %0, hi, hi, %0;\n\t}" : "+f"(acc) : "r"(u[j]));
      return acc;
    };

    // fill F of this CTA (counted across tiles) uses stage F % 6; it may be written once the MMAs that read
    // fill F - 6 have completed, and is complete for the MMA warp on phase (F / 6) & 1 of full[]
    bool ok = true;
    for (int f = 0; f < FT_AHEAD; ++f) {
      if (f < nf && ok) {
        const uint32_t F = done + f;
        ok = mbar_wait(&empty[F % FT_STAGES], ((F / FT_STAGES) & 1) ^ 1, abort_flag);
        if (ok) issue(f, F % FT_STAGES);
      }
      cp_async_commit();
    }
    for (int f = 0; ok && f < nf; ++f) {
      const int fn = f + FT_AHEAD;
      if (fn < nf) {
        const uint32_t F = done + fn;
        if (!mbar_wait(&empty[F % FT_STAGES], ((F / FT_STAGES) & 1) ^ 1, abort_flag)) { ok = false; break; }
        issue(fn, F % FT_STAGES);
      }
      cp_async_commit();
      cp_async_wait<FT_AHEAD>();                          // this thread's pieces of fill f have landed
      const uint32_t s_cur = (done + f) % FT_STAGES;
      const uint32_t sb = ring + s_cur * FT_STAGE_BYTES + slot0;
      const bool odd = passes == 4 && (f & 1);
      const int kc0 = (f >> chunk_shift) * chunk_mul;
      const uint32_t okm = odd ? ok_o : ok_e;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        if (kc0 + (passes == 1 ? (t & 1) : 0) >= nk || !((okm >> t) & 1)) continue;
        const uint4 v = ld_shared16(sb + t * 4096);
        if (odd) acc_o[t] = sumsq(v, acc_o[t]); else acc_e[t] = sumsq(v, acc_e[t]);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&full[s_cur]);           // the MMA warp fences the proxies after its wait
    }
    cp_async_wait<0>();

    // ---- norms: squared sums of A row g + 32 i and B row g + 32 i, then across the eight threads of a row
    float ssa[4], ssb[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { ssa[i] = acc_e[i]; ssb[i] = acc_o[i]; }                 // passes 4
    if (passes == 2) { ssb[0] = acc_e[2]; ssb[1] = acc_e[3]; }
    if (passes == 1) { ssa[0] = acc_e[0] + acc_e[1]; ssb[0] = acc_e[2] + acc_e[3]; }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
        ssa[i] += __shfl_xor_sync(0xffffffffu, ssa[i], o);
        ssb[i] += __shfl_xor_sync(0xffffffffu, ssb[i], o);
      }
      if (c == 0 && i < passes) {                         // a cluster exchanges the squared partial sums
        const bool root = ks == 1 && a.metric == LIGHTKV_FD_COSINE;
        a_nrm[g + 32 * i] = root ? sqrtf(ssa[i]) : ssa[i];
        b_nrm[g + 32 * i] = root ? sqrtf(ssb[i]) : ssb[i];
      }
    }
    named_barrier(1, FT_LOADERS);

    // ---- epilogue: thread = A row (TMEM lane); warps 0-3 scan columns 0-63, warps 4-7 columns 64-127
    ok = ok && mbar_wait(acc_full, n_items & 1, abort_flag);
    ok = __all_sync(0xffffffffu, ok);                     // the TMEM loads below are warp-wide
    tc_fence_after();
    // columns some row of this warp needs: blocks of eight outside that range are skipped as a whole
    const int lo_w = __reduce_min_sync(0xffffffffu, lo), hi_w = __reduce_max_sync(0xffffffffu, hi);
    const float na = row < cap_rows ? a_nrm[row] : 0.f;
    float best = 3.0e38f;
    int best_c = -1;
    if (CLUSTER && ok && ks > 1) {
      // cluster: this CTA's partial G goes to shared memory as float [128][kFdPitch] over the drained ring
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int c0 = half * 64 + j * 32;
        if (c0 >= n_cols) break;                          // warp-uniform
        float v[32];
        tmem_ld32(tmem_base + (uint32_t(q * 32) << 16) + c0, v);
        tmem_ld_wait();
        float* prow = reinterpret_cast<float*>(base) + row * kFdPitch + c0;
#pragma unroll
        for (int i = 0; i < 32; ++i) prow[i] = v[i];
      }
    }
    if (ok && ks == 1) {
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int c0 = half * 64 + j * 32;
        if (c0 >= n_cols) break;                          // warp-uniform
        if (c0 + 32 <= lo_w || c0 >= hi_w) continue;      // warp-uniform
        float v[32];
        tmem_ld32(tmem_base + (uint32_t(q * 32) << 16) + c0, v);
        tmem_ld_wait();
#pragma unroll
        for (int blk = 0; blk < 4; ++blk) {
          if (c0 + blk * 8 + 8 <= lo_w || c0 + blk * 8 >= hi_w) continue;   // warp-uniform
#pragma unroll
          for (int i = blk * 8; i < blk * 8 + 8; ++i) {
            const int col = c0 + i;
            if (col >= lo && col < hi) {
              const float fd = pair_score(a.metric, v[i], na, b_nrm[col]);
              if (fd < best) { best = fd; best_c = col; }
            }
          }
        }
      }
    }
    if (ks == 1) {
    if (half == 1) { red_f[row] = best; red_c[row] = best_c; }
    named_barrier(1, FT_LOADERS);
    if (half == 0 && ok && e < a1) {
      if (red_f[row] < best) { best = red_f[row]; best_c = red_c[row]; }   // ties stay with the lower column
      if (best_c >= 0) {
        const unsigned long long key = ((unsigned long long)orderable(best) << 32) | (unsigned)(b0 + best_c);
        unsigned long long* dst = a.ws.a_key + size_t(b) * a.ws.cap_a + e;
        if (tl.blocks_b > 1) atomicMin(dst, key); else *dst = key;
      }
    }
    }
    tc_fence_before();                                    // TMEM reads done before the next tile's MMAs
  } else if (lane == 0) {
    // ---- MMA issue: one chunk = four K = 16 steps inside the 128-byte rows
    const uint32_t idesc = idesc_bf16(kFdTile, n_cols);
    auto chunk_mma = [&](uint32_t a_addr, uint32_t b_addr, bool first) {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
        umma_bf16(tmem_base, smem_desc_sw128(a_addr + kk * 32), smem_desc_sw128(b_addr + kk * 32), idesc,
                  !(first && kk == 0));
    };
    if (passes == 4) {
      for (int k = 0; k < nk; ++k) {
        const uint32_t FA = done + 2 * k, FB = FA + 1, sA = FA % FT_STAGES, sB = FB % FT_STAGES;
        if (!mbar_wait(&full[sA], (FA / FT_STAGES) & 1, abort_flag)) break;
        if (!mbar_wait(&full[sB], (FB / FT_STAGES) & 1, abort_flag)) break;
        fence_proxy_async();                              // the loaders' cp.async writes -> visible to the tensor core
        tc_fence_after();
        chunk_mma(ring + sA * FT_STAGE_BYTES, ring + sB * FT_STAGE_BYTES, k == 0);
        umma_commit(&empty[sA]);
        umma_commit(&empty[sB]);
      }
    } else {
      for (int f = 0; f < nf; ++f) {
        const uint32_t F = done + f, s = F % FT_STAGES;
        if (!mbar_wait(&full[s], (F / FT_STAGES) & 1, abort_flag)) break;
        fence_proxy_async();
        tc_fence_after();
        const uint32_t sa = ring + s * FT_STAGE_BYTES;
        if (passes == 2) {
          chunk_mma(sa, sa + 8192, f == 0);
        } else {
          chunk_mma(sa, sa + 8192, f == 0);
          if (2 * f + 1 < nk) chunk_mma(sa + 4096, sa + 12288, false);
        }
        umma_commit(&empty[s]);
      }
    }
    umma_commit(acc_full);
  }
  if (CLUSTER && ks > 1) {
    // ---- cluster epilogue.  Every thread of every CTA of the cluster passes both barriers for every tile,
    //      whatever happened before (an aborted CTA contributes garbage and the status bit, never a hang).
    __syncwarp();
    cluster_sync();                                       // all partial G and squared norms are in shared memory
    if (warp < 8)
      fd_cluster_finish(a.metric, a.ws.a_win + size_t(b) * a.ws.cap_a, a.ws.a_key + size_t(b) * a.ws.cap_a, ks, rank, a0, a1, b0, b1,
                        tl.blocks_b > 1, win_off, a_off, smem_u32(base), a_nrm, b_nrm, red_f,
                        reinterpret_cast<float*>(red_c), abort_flag);
    __syncwarp();
    cluster_sync();                                       // nobody reads this CTA's shared memory any more
  }
  done += nf;
  ++n_items;
  if (*abort_flag && ks == 1) break;
  }  // work items
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kFdTile);
  }
  if (tid == 0 && *abort_flag && a.status) atomicOr(a.status, LIGHTKV_STATUS_TIMEOUT);
}

bool tc_fd_supported(int hidden) { return hidden % 8 == 0; }

// SMs of the current device (cached per device ordinal).
static int sm_count() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (!cached[dev]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

cudaError_t launch_fd_tc(const LayerLaunch& L) {
  const lightkv_layer_args_t* a = L.a;
  FdTcArgs f;
  f.x = static_cast<const __nv_bfloat16*>(a->hidden) + size_t(a->vis_begin) * a->hidden_row_stride;
  f.seq_start = a->seq_start;
  f.batch_stride = a->hidden_batch_stride; f.row_stride = a->hidden_row_stride; f.d = L.hidden; f.batch = L.batch;
  f.metric = L.divergence; f.ws = L.ws; f.status = a->status;
  // Persistent CTAs, two per SM, no more than the plan expects tiles.  When that estimate leaves SMs idle,
  // clusters of 2, 4 or 8 CTAs split the hidden dimension of every tile.
  const long long bound = std::max<long long>(1, (long long)L.fd_tiles * L.batch);   // an estimate, see the plan
  const int slots = 2 * sm_count(), nk_all = (L.hidden + 63) / 64;
  int ks = 1;
  while (ks < 8 && bound * (2 * ks) <= slots && 2 * ks <= nk_all) ks *= 2;
  const int clusters = (int)std::min<long long>(bound, slots / ks);
  cudaError_t e;
  if (ks == 1) {
    if ((e = ensure_dynamic_smem(fd_tc_kernel<false>, (int)FT_SMEM)) != cudaSuccess) return e;
    return launch_kernel(fd_tc_kernel<false>, clusters, FT_LOADERS + 32, FT_SMEM, L.stream, 1, f);
  }
  if ((e = ensure_dynamic_smem(fd_tc_kernel<true>, (int)FT_SMEM)) != cudaSuccess) return e;
  return launch_kernel(fd_tc_kernel<true>, clusters * ks, FT_LOADERS + 32, FT_SMEM, L.stream, ks, f);
}

}  // namespace lkv
