// Tile bookkeeping of the tensor-core attention kernels, built once per call.
//
// Which 64-key tiles a 128-row query tile has to visit (the blocks its query blocks selected,
// Eq. 13, and the tiles its window reaches, Eq. 15), in which order, and which of its warps a tile
// concerns, depends only on the block indices and the sequence lengths.  Building that inside the
// attention kernels cost every CTA several thousand cycles before its first product; here one warp
// per attention CTA builds the image of the bookkeeping the attention kernel wants in shared
// memory, and the attention kernel fetches it with one bulk copy while its first tiles load.
//
// Query-major image (forward and dQ kernel), see meta_layout():
//   [8][nT] selection bytes   bit c of byte (g, jt): query block g of the CTA selected key block
//                             jt * (64 / Bk) + c
//   list[nT], flags[nT]       the tiles any row of the CTA needs, ascending; bit 0: some selected
//                             block lies in the tile, bit 1: the window of some row reaches it
//   items[2 nT], icls[2 nT][4] (forward) the long-term tiles, then the short-term tiles, and the
//                             class of every (item, softmax warp)
//   jcls[nT][2][8]            (dQ) class of every (listed tile, half tile, compute warp)
//   counts                    {tiles on the list, long-term items, short-term items}
// Head-packed variant (Shape::pack): the CTA's rows 0..63 and 64..127 are the same 64 positions of
// two query heads with a common key/value head, so both halves have the same selection bytes and
// every listed tile concerns both.
// With a selection per query position the key-major images would each have to scan the index rows
// of every later position; instead the query-major images, which read every index row once, set
// one bit per (key block, position) in a table in global memory (launch 1), and the key-major
// images copy the words of their key blocks from it (launch 2).
// Key-major image (dK/dV kernel): [8][nT] bytes: bit c of byte (g, qt): query block
// qt * (64 / Bk) + c selected key block g of the CTA; list / flags of the 64-query tiles that
// visit the CTA's keys; jcls[nT][2][8] class of every (listed tile, half tile, compute warp);
// counts {tiles on the list}.
#include "tc_common.cuh"

namespace blossom {
namespace tc {
namespace {

constexpr int kMetaWarps = 4;  // images per CTA, one warp each

// One warp builds one image: no block-wide barrier anywhere, so the (latency-bound) images of a
// whole launch are in flight at once.
__global__ void __launch_bounds__(kMetaWarps * 32) tc_meta_kernel(Shape s, const int32_t *__restrict__ seq_lens,
                                                                  const int32_t *__restrict__ idx,
                                                                  uint8_t *__restrict__ qmeta,
                                                                  uint8_t *__restrict__ kmeta, int nT,
                                                                  int n_query_ctas, int image0, int image_end,
                                                                  int branches, int with_fwd,
                                                                  uint32_t *__restrict__ inv_bits) {
  grid_chain_enter();
  extern __shared__ __align__(16) uint8_t meta_all[];
  const MetaLayout ml = meta_layout(nT, s.pq);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int image = image0 + (int)blockIdx.x * kMetaWarps + warp;  // this launch builds [image0, image_end)
  if (image >= image_end) return;
  const int Lw = (s.L + 31) >> 5;  // words per key block of the bit table
  const int slice = ml.bytes + ((3 * nT + 15) / 16) * 16;  // the image and a scratch list behind it
  uint8_t *meta = meta_all + (size_t)warp * slice;
  const int nST = (s.L + 127) >> 7;
  const bool key_major = image >= n_query_ctas;
  const int cta = key_major ? image - n_query_ctas : image;
  // query-major CTAs count (batch, query head) pairs, key-major CTAs (batch, key/value head) pairs;
  // uk = the (batch, key/value head) pair whose selection the image is built from
  // (head-packed query-major CTAs count (batch, pair of query heads) pairs, one CTA per 64 positions)
  const bool pack = !key_major && s.pack;
  const int u = pack ? cta / nT : cta / nST;
  const int n = key_major ? u / s.Hkv : (pack ? u / (s.H / 2) : u / s.H);
  const int uk = key_major ? u : n * s.Hkv + (pack ? 2 * (u % (s.H / 2)) : u % s.H) / s.G;
  int len = seq_lens ? seq_lens[n] : s.L;
  len = min(max(len, 0), s.L);
  const int pad0 = s.L - len;
  uint32_t *selw = reinterpret_cast<uint32_t *>(meta);
  uint8_t *selb = meta;
  uint16_t *list = reinterpret_cast<uint16_t *>(meta + ml.list);
  uint8_t *lflags = meta + ml.flags;
  uint16_t *items = reinterpret_cast<uint16_t *>(meta + ml.items);
  uint8_t *icls = meta + ml.icls;
  uint8_t *jcls = meta + ml.jcls;
  int *counts = reinterpret_cast<int *>(meta + ml.counts);
  const unsigned lt = (1u << lane) - 1u;
  const int G = 128 / s.Bk, nb = 64 / s.Bk;
  const int bk_shift = __ffs(s.Bk) - 1;  // Bk is a power of two

  for (int i = lane; i < ml.bytes / 4; i += 32) selw[i] = 0u;  // the whole image
  __syncwarp();

  if (!key_major) {
    const int st = pack ? nT - 1 - cta % nT : nST - 1 - cta % nST;  // the attention kernels take long rows first
    const int row0 = pack ? st * 64 : st * 128, row_last = min(s.L - 1, row0 + (pack ? 63 : 127));
    // first position of the 32 rows of TMEM lane quarter w, and of the 64-row half hf
    auto quarter_row0 = [&](int w) { return row0 + 32 * (pack ? (w & 1) : w); };
    auto half_row0 = [&](int hf) { return pack ? row0 : row0 + 64 * hf; };
    if (s.pq) {
      // a selection per query position: every row's own bytes, and their union per query block
      // (which is what the tile list and the item order below are built from)
      uint32_t *roww = reinterpret_cast<uint32_t *>(meta + ml.rows);
      // the bit table is per key/value head: the group's first query head (or pair of heads) fills it
      const bool fills = inv_bits && (pack ? (2 * (u % (s.H / 2))) % s.G == 0 : (u % s.H) % s.G == 0);
      for (int i = lane; i < 128 * s.topk; i += 32) {
        const int r = i / s.topk, slot = i % s.topk, t = pack ? row0 + (r & 63) : row0 + r;
        if (t < s.L) {
          const int blk = idx[((int64_t)uk * s.L + t) * s.topk + slot];
          if (blk >= 0 && blk <= (t >> bk_shift)) {
            const int a = (r >> bk_shift) * nT + blk / nb, b2 = r * nT + blk / nb;
            atomicOr(&selw[a >> 2], (1u << (blk % nb)) << ((a & 3) * 8));
            atomicOr(&roww[b2 >> 2], (1u << (blk % nb)) << ((b2 & 3) * 8));
            if (fills && (!pack || r < 64))
              atomicOr(&inv_bits[((int64_t)uk * s.M + blk) * Lw + (t >> 5)], 1u << (t & 31));
          }
        }
      }
    } else {
    for (int i = lane; i < G * s.topk; i += 32) {  // the selections of the CTA's query blocks
      const int g = i / s.topk, slot = i % s.topk, qb = pack ? st * nb + g % nb : st * G + g;
      if (qb < s.M) {
        const int blk = idx[((int64_t)uk * s.M + qb) * s.topk + slot];
        if (blk >= 0 && blk < s.M && (blk <= qb || !s.causal)) {
          const int a = g * nT + blk / nb;
          atomicOr(&selw[a >> 2], (1u << (blk % nb)) << ((a & 3) * 8));
        }
      }
    }
    }
    __syncwarp();
    int nv = 0;
    {  // the tiles any row of the CTA needs, ascending
      const int jt_max = (s.causal ? row_last : s.L - 1) >> 6;
      for (int base = 0; base <= jt_max; base += 32) {
        const int jt = base + lane;
        int f = 0;
        if (jt <= jt_max && row_last >= pad0 && jt * 64 + 63 >= pad0) {
          for (int g = 0; g < G; ++g) f |= selb[g * nT + jt] ? 1 : 0;
          if (st_ranges_touch(s, row0, row_last, jt * 64, jt * 64 + 63)) f |= 2;
          f &= branches;
        }
        const unsigned bal = __ballot_sync(0xffffffffu, f != 0);
        if (f) {
          const int pos = nv + __popc(bal & lt);
          list[pos] = (uint16_t)jt;
          lflags[pos] = (uint8_t)f;
        }
        nv += __popc(bal);
      }
    }
    __syncwarp();
    const int gh = G / 2;
    if (lane == 0) counts[0] = nv;
    if (with_fwd) {  // ---- the forward's items and their classes ----
    // Long-term items: the tiles both 64-row halves of the CTA need, then alternately a tile only
    // rows 0..63 need and a tile only rows 64..127 need.  A softmax warp may run ahead of the
    // slowest one, so with alternating items both pairs of warps have work at once.
    int nA = 0, nB = 0, nC = 0;
    for (int pass = 0; pass < 2; ++pass) {
      int cA = 0, cB = 0, cC = 0;
      for (int base = 0; base < nv; base += 32) {
        const int j = base + lane;
        int c = 0;
        if (j < nv && (lflags[j] & 1)) {
          const int jt = list[j];
          for (int g = 0; g < G; ++g)
            if (selb[g * nT + jt]) c |= g < gh ? 1 : 2;
        }
        const unsigned bA = __ballot_sync(0xffffffffu, c == 1), bB = __ballot_sync(0xffffffffu, c == 2),
                       bC = __ballot_sync(0xffffffffu, c == 3);
        if (pass == 1 && c) {
          int pos;
          if (c == 3) pos = cC + __popc(bC & lt);
          else if (c == 1) {
            const int k = cA + __popc(bA & lt);
            pos = nC + (k < nB ? 2 * k : nB + k);
          } else {
            const int k = cB + __popc(bB & lt);
            pos = nC + (k < nA ? 2 * k + 1 : nA + k);
          }
          items[pos] = list[j];
        }
        cA += __popc(bA);
        cB += __popc(bB);
        cC += __popc(bC);
      }
      nA = cA;
      nB = cB;
      nC = cC;
    }
    const int nl = nA + nB + nC;
    int count = nl;
    for (int base = 0; base < nv; base += 32) {  // short-term items in ascending order
      const int j = base + lane;
      const bool on = j < nv && (lflags[j] & 2);
      const unsigned bal = __ballot_sync(0xffffffffu, on);
      if (on) items[count + __popc(bal & lt)] = list[j];
      count += __popc(bal);
    }
    if (lane == 0) {
      counts[0] = nv;
      counts[1] = nl;
      counts[2] = count - nl;
    }
    __syncwarp();
    // Class of every (item, softmax warp): 0 = no row of the warp needs the tile, 1 = every row
    // sees all 64 keys, 2 = mixed (the warp builds per-lane column masks).
    const bool uni = s.Bk >= 32;  // a warp's 32 rows share one query block
    const uint32_t allbits = (1u << (64 / s.Bk)) - 1u;
    for (int e = lane; e < count * 4; e += 32) {
      const int it = e >> 2, w = e & 3;
      const int jt = items[it], p0 = jt * 64, t_lo = quarter_row0(w);
      const bool some = (p0 <= t_lo + 31 || !s.causal) && p0 + 63 >= pad0 && t_lo + 31 >= pad0 && t_lo < s.L;
      // every row of the warp may see every key of the tile as far as validity and causality go
      const bool inner = t_lo >= pad0 && t_lo + 31 < s.L && p0 >= pad0 && (s.causal ? p0 + 63 <= t_lo : p0 + 63 < s.L);
      int cls = 0;
      if (some) {
        if (it < nl) {
          if (!uni) cls = 2;
          else {
            const uint32_t bits = selb[((w * 32) / s.Bk) * nT + jt];
            cls = bits == 0u ? 0 : ((!s.pq && inner && bits == allbits) ? 1 : 2);  // (per position: the rows differ)
          }
        } else if (st_ranges_touch(s, t_lo, t_lo + 31, p0, p0 + 63)) {
          cls = (inner && p0 >= t_lo + 31 - s.window + 1 && (s.causal || p0 + 63 <= t_lo + s.window - 1)) ? 1 : 2;  // 1: inside every row's window
        }
      }
      icls[e] = (uint8_t)cls;
    }
    }  // the forward's part
    __syncwarp();
    // The dQ kernel walks `list` itself (a tile serves both branches there).  Same idea as above:
    // tiles both 64-row halves need first, then alternately a tile only rows 0..63 need and one
    // only rows 64..127 need, so that the two halves' warps work on neighbouring tiles at once.
    // (Backward call only; the forward reads `items`.)
    if (kmeta) {
      uint16_t *tlist = reinterpret_cast<uint16_t *>(meta + ml.bytes);
      uint8_t *tflags = meta + ml.bytes + 2 * nT;
      int nA = 0, nB = 0, nC = 0;
      for (int pass = 0; pass < 2; ++pass) {
        int cA = 0, cB = 0, cC = 0;
        for (int base = 0; base < nv; base += 32) {
          const int j = base + lane;
          int c = 0;
          if (j < nv) {
            const int jt = list[j], p0 = jt * 64;
            if (lflags[j] & 1)
              for (int g = 0; g < G; ++g)
                if (selb[g * nT + jt]) c |= g < gh ? 1 : 2;
            if (lflags[j] & 2)
              for (int hf = 0; hf < 2; ++hf)
                if ((p0 <= half_row0(hf) + 63 || !s.causal) &&
                    st_ranges_touch(s, half_row0(hf), half_row0(hf) + 63, p0, p0 + 63))
                  c |= 1 << hf;
            if (c == 0) c = 3;
          }
          const unsigned bA = __ballot_sync(0xffffffffu, c == 1), bB = __ballot_sync(0xffffffffu, c == 2),
                         bC = __ballot_sync(0xffffffffu, c == 3);
          if (pass == 1 && c) {
            int pos;
            if (c == 3) pos = cC + __popc(bC & lt);
            else if (c == 1) {
              const int k = cA + __popc(bA & lt);
              pos = nC + (k < nB ? 2 * k : nB + k);
            } else {
              const int k = cB + __popc(bB & lt);
              pos = nC + (k < nA ? 2 * k + 1 : nA + k);
            }
            tlist[pos] = list[j];
            tflags[pos] = lflags[j];
          }
          cA += __popc(bA);
          cB += __popc(bB);
          cC += __popc(bC);
        }
        nA = cA;
        nB = cB;
        nC = cC;
      }
      __syncwarp();
      for (int j = lane; j < nv; j += 32) {
        list[j] = tlist[j];
        lflags[j] = tflags[j];
      }
    }
    __syncwarp();
    // dQ kernel: class of every (listed tile, half tile of 32 keys, compute warp).  Warp w works
    // on rows 32 (w % 4) ... and keys 16 (w / 4) ... of the half tile.  Bit 0 / bit 1: every row of
    // the warp sees all 16 keys through the long-term / short-term branch and no row sees only a
    // part of them; 8: mixed, the warp builds per-lane column masks.  (A forward-only call has no
    // use for them.)
    for (int e = lane; e < (kmeta ? nv * 16 : 0); e += 32) {
      const int it = e >> 4, hh = (e >> 3) & 1, w = e & 7, qtr = w & 3, c = w >> 2;
      const int jt = list[it], f = lflags[it];
      const int k_lo = jt * 64 + 32 * hh + 16 * c, k_hi = k_lo + 15, t_lo = quarter_row0(qtr), t_hi = t_lo + 31;
      const bool rows_in = t_lo >= pad0 && t_hi < s.L, rows_none = t_hi < pad0 || t_lo >= s.L;
      const bool past = rows_in && k_lo >= pad0 && (s.causal ? k_hi <= t_lo : k_hi < s.L);  // every key visible to every row (validity, causality)
      const bool reach = !rows_none && (k_lo <= t_hi || !s.causal) && k_hi >= pad0 && k_lo < s.L;  // some key may be visible to some row
      int cL = 0, cS = 0;  // 0 none, 1 all, 2 mixed
      if ((f & 1) && reach) {
        const int kb = (32 * hh + 16 * c) >> bk_shift;  // key block within the tile
        bool any_sel = false, all_sel = true;
        for (int gq = (qtr * 32) >> bk_shift; gq <= (qtr * 32 + 31) >> bk_shift; ++gq) {
          const bool sel = (selb[gq * nT + jt] >> kb) & 1u;
          any_sel |= sel;
          all_sel &= sel;
        }
        if (any_sel) cL = (all_sel && past && !s.pq) ? 1 : 2;
      }
      if ((f & 2) && reach && st_ranges_touch(s, t_lo, t_hi, k_lo, k_hi))
        cS = (past && k_lo >= t_hi - s.window + 1 && (s.causal || k_hi <= t_lo + s.window - 1)) ? 1 : 2;  // 1: inside every row's window
      jcls[e] = (uint8_t)((cL == 2 || cS == 2) ? 8 : (cL | (cS << 1)));
    }
  } else {
    const int kt = cta % nST;  // the dK/dV kernel takes early keys first
    const int key0 = kt * 128, key_last = min(s.L - 1, key0 + 127);
    if (s.pq) {
      // a selection per query position: which positions selected each of this CTA's key blocks
      // (one bit per position), and per 64-query tile which query blocks hold such a position
      // (the words of this CTA's key blocks from the bit table the query-major images filled: word w
      // of a block holds positions 32 w ...; a position before the block never selected it)
      uint32_t *invw = reinterpret_cast<uint32_t *>(meta + ml.rows);
      const int qb0 = kt * G, w_lo = key0 >> 5;
      for (int i = lane; i < G * (Lw - w_lo); i += 32) {
        const int g = i / (Lw - w_lo), w = w_lo + i % (Lw - w_lo);
        if (qb0 + g >= s.M) continue;
        const uint32_t bits = inv_bits[((int64_t)uk * s.M + qb0 + g) * Lw + w];
        if (!bits) continue;
        const int a = g * nT + (w >> 1);
        invw[2 * a + (w & 1)] = bits;
        // the 32 positions lie in one query block (Bk >= 32) or in two (Bk = 16)
        uint32_t qbits;
        if (s.Bk >= 32) qbits = 1u << (((w & 1) * 32) >> bk_shift);
        else qbits = (((bits & 0xffffu) ? 1u : 0u) | ((bits >> 16) ? 2u : 0u)) << ((w & 1) * 2);
        atomicOr(&selw[a >> 2], qbits << ((a & 3) * 8));
      }
    } else {  // which query blocks selected each of this CTA's key blocks, per 64-query tile
      // (the index rows of query blocks qb0 .. M-1 are contiguous; eight loads in flight per lane)
      // (without the causal mask every query block may have selected them: the rows start at block 0)
      const int qb0 = kt * G, qb_first = s.causal ? qb0 : 0, total = (s.M - qb_first) * s.topk;
      const int32_t *rows = idx + ((int64_t)uk * s.M + qb_first) * s.topk;
      for (int base = 0; base < total; base += 256) {
        int blk[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int i = base + e * 32 + lane;
          blk[e] = i < total ? rows[i] : -1;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int i = base + e * 32 + lane, qb = qb_first + i / s.topk;
          if (blk[e] >= qb0 && blk[e] < qb0 + G && (blk[e] <= qb || !s.causal)) {
            const int a = (blk[e] - qb0) * nT + qb / nb;
            atomicOr(&selw[a >> 2], (1u << (qb % nb)) << ((a & 3) * 8));
          }
        }
      }
    }
    __syncwarp();
    const int qt_min = s.causal ? key0 >> 6 : 0, qt_max = (s.L - 1) >> 6;
    int count = 0;
    for (int base = qt_min; base <= qt_max; base += 32) {
      const int qt = base + lane;
      int f = 0;
      if (qt <= qt_max && key_last >= pad0) {
        for (int g = 0; g < G; ++g) f |= selb[g * nT + qt] ? 1 : 0;
        if (st_ranges_touch(s, qt * 64, min(qt * 64 + 63, s.L - 1), key0, key_last)) f |= 2;
        f &= branches;
      }
      const unsigned bal = __ballot_sync(0xffffffffu, f != 0);
      if (f) {
        const int pos = count + __popc(bal & lt);
        list[pos] = (uint16_t)qt;
        lflags[pos] = (uint8_t)f;
      }
      count += __popc(bal);
    }
    if (lane == 0) counts[0] = count;
    __syncwarp();
    // dK/dV kernel: class of every (listed tile, half tile of 32 queries, compute warp).  Warp w
    // works on key rows 32 (w % 4) ... of the CTA and on query columns 16 (w / 4) ... of the half
    // tile.  Same code as for the dQ kernel: bit 0 / bit 1 = every key row of the warp is seen in
    // full by all 16 queries through the long-term / short-term branch and none in part; 8 = mixed.
    for (int e = lane; e < count * 16; e += 32) {
      const int it = e >> 4, hh = (e >> 3) & 1, w = e & 7, qtr = w & 3, hf = w >> 2;
      const int qt = list[it], f = lflags[it], c_lo = 32 * hh + 16 * hf;
      const int p_lo = key0 + 32 * qtr, p_hi = p_lo + 31, t_lo = qt * 64 + c_lo, t_hi = t_lo + 15;
      const bool rows_in = p_lo >= pad0 && p_hi < s.L, rows_none = p_hi < pad0 || p_lo >= s.L;
      const bool past = rows_in && t_hi < s.L && (s.causal ? t_lo >= p_hi : t_lo >= pad0);  // every query sees every key (validity, causality)
      const bool reach = !rows_none && (t_hi >= p_lo || !s.causal) && t_hi >= pad0 && t_lo < s.L;  // some query may see some key
      int cL = 0, cS = 0;  // 0 none, 1 all, 2 mixed
      if ((f & 1) && reach) {
        bool any_sel = false, all_sel = true;
        for (int gk = (qtr * 32) >> bk_shift; gk <= (qtr * 32 + 31) >> bk_shift; ++gk) {
          const uint32_t bits = selb[gk * nT + qt];
          for (int c = c_lo >> bk_shift; c <= (c_lo + 15) >> bk_shift; ++c) {
            const bool sel = (bits >> c) & 1u;
            any_sel |= sel;
            all_sel &= sel;
          }
        }
        if (any_sel) cL = (all_sel && past && !s.pq) ? 1 : 2;
      }
      if ((f & 2) && reach && st_ranges_touch(s, t_lo, min(t_hi, s.L - 1), p_lo, min(p_hi, s.L - 1)))
        cS = (past && p_lo >= t_hi - s.window + 1 && (s.causal || p_hi <= t_lo + s.window - 1)) ? 1 : 2;  // 1: inside every query's window
      jcls[e] = (uint8_t)((cL == 2 || cS == 2) ? 8 : (cL | (cS << 1)));
    }
  }
  __syncwarp();
  uint4 *dst = reinterpret_cast<uint4 *>((key_major ? kmeta : qmeta) + (size_t)cta * ml.bytes);
  const uint4 *src = reinterpret_cast<const uint4 *>(meta);
  for (int i = lane; i < ml.bytes / 16; i += 32) dst[i] = src[i];
}

}  // namespace

int launch_tc_meta(const Shape &s, const int32_t *seq_lens, const int32_t *idx, uint8_t *qmeta,
                   uint8_t *kmeta, cudaStream_t st, int branches, int with_fwd) {
  if (with_fwd < 0) with_fwd = kmeta == nullptr;
  const int nT = (s.L + 63) / 64, nST = (s.L + 127) / 128;
  const int nq = s.pack ? nT * s.B * (s.H / 2) : nST * s.B * s.H, n_images = kmeta ? nq + nST * s.B * s.Hkv : nq;
  const size_t smem = (size_t)kMetaWarps * (meta_bytes(nT, s.pq) + ((3 * nT + 15) / 16) * 16);
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(tc_meta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return BLOSSOM_ERR_CUDA;
  auto launch = [&](int image0, int image_end, uint32_t *inv_bits) {
    LaunchScope ls(K_TC_META, st);
    launch_chained(tc_meta_kernel, dim3((unsigned)((image_end - image0 + kMetaWarps - 1) / kMetaWarps)),
                   dim3(kMetaWarps * 32), smem, st, s, seq_lens, idx, qmeta, kmeta, nT, nq, image0, image_end, branches,
                   with_fwd, inv_bits);
  };
  if (s.pq && kmeta) {
    // selection per position: the query-major images fill the bit table, then the key-major ones read it
    uint32_t *inv_bits = reinterpret_cast<uint32_t *>(kmeta + tc_meta_bytes(s));
    if (cudaMemsetAsync(inv_bits, 0, tc_inv_bits_bytes(s), st) != cudaSuccess) return BLOSSOM_ERR_CUDA;
    launch(0, nq, inv_bits);
    launch(nq, n_images, inv_bits);
  } else {
    launch(0, n_images, nullptr);
  }
  return cudaGetLastError() == cudaSuccess ? BLOSSOM_OK : BLOSSOM_ERR_CUDA;
}

}  // namespace tc
}  // namespace blossom
