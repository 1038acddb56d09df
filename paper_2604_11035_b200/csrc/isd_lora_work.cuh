// Work assignment of the LoRA GEMM kernels (isd_lora_tc.cu), shared by the device code, the host launchers and a
// host-only test entry, so that the item-to-CTA mapping can be checked without a GPU.
//
// A "unit" is what owns one output tile at a time: a CTA (tiles of 128 x bn) in the one-CTA kernel, a pair of
// CTAs (tiles of 256 x 256) in the pair kernel.  Units are numbered by the MIRRORED block index
// v = units - 1 - (block or pair index).  With the fused down-projection the units v >= units - tiles_m * t_chunks
// (the ones with the fewest output tiles) start with one block of t; then come the whole rounds of output tiles
// v, v + units, ...; the tiles of the last, partial round are cut into tail_split column strips, one per unit
// v < n_strips.  The mirror puts the blocks of t on the LOWEST block indices: the hardware hands out CTAs in index
// order, so the producers of t are resident before any reader of it and never wait before they publish, and a
// grid that is only partly resident still makes progress.
#pragma once

struct LoraWorkItem {
  int pre;   // 1: a block of t (rows m0 .., columns n0 .. of t); 0: a tile or strip of the output
  int m0, n0, cols;
};

struct LoraWork {
  int tiles_m, n_tiles, units, v, bm, bn, Rc, tail_split;
  int t_block, t_chunk, n_pre, rounds, tail0, n_strips, strip_cols, n_items;
#ifdef __CUDACC__
  __host__ __device__
#endif
  void init(int unit_index, int units_, int M, int N, int bm_, int bn_, int fuse, int t_chunks, int Rc_, int tail_split_) {
    units = units_; bm = bm_; bn = bn_; Rc = Rc_; tail_split = tail_split_;
    tiles_m = (M + bm - 1) / bm;
    n_tiles = tiles_m * ((N + bn - 1) / bn);
    v = units - 1 - unit_index;
    const int t_item = fuse ? v - (units - tiles_m * t_chunks) : -1;  // >= 0: this unit computes a block of t
    t_block = t_item >= 0 ? t_item % tiles_m : 0;
    t_chunk = t_item >= 0 ? t_item / tiles_m : 0;
    n_pre = t_item >= 0 ? 1 : 0;
    rounds = n_tiles / units;
    tail0 = rounds * units;
    n_strips = (n_tiles - tail0) * tail_split;
    strip_cols = bn / tail_split;
    n_items = n_pre + rounds + (v < n_strips ? 1 : 0);
  }
#ifdef __CUDACC__
  __host__ __device__
#endif
  LoraWorkItem item(int it) const {
    LoraWorkItem w;
    w.pre = it < n_pre ? 1 : 0;
    if (w.pre) {
      w.m0 = t_block * bm; w.n0 = t_chunk * Rc; w.cols = Rc;
    } else if (it - n_pre < rounds) {
      const int tile = v + (it - n_pre) * units;
      w.m0 = (tile % tiles_m) * bm; w.n0 = (tile / tiles_m) * bn; w.cols = bn;  // neighbouring units share a B panel
    } else {
      const int tile = tail0 + v / tail_split;
      w.m0 = (tile % tiles_m) * bm; w.n0 = (tile / tiles_m) * bn + (v % tail_split) * strip_cols; w.cols = strip_cols;
    }
    return w;
  }
};

// What isd_lora_linear launches for a shape: the kernel form and its grid.
struct LoraPlan {
  int form;      // 2: CTA pairs, fused; 1: one-CTA kernel, fused; 0: two launches of the one-CTA kernel (t first)
  int units;     // units of the launch that writes y (CTAs, or pairs)
  int bm, bn;    // tile of a unit
  int fuse, t_chunks, Rc, tail_split;
};

// Units and column strips of one launch: as many units as tiles (at least one per block of t), at most max_units;
// the last, partial round is cut into as many strips as the units without a block of t can take.
inline void lora_grid(int M, int N, int bm, int bn, int fuse, int t_chunks, int max_units, bool strips_need_32, int& units,
                      int& tail_split) {
  const int tiles_m = (M + bm - 1) / bm;
  const int n_tiles = tiles_m * ((N + bn - 1) / bn), n_t = fuse ? tiles_m * t_chunks : 0;
  int u = n_tiles < n_t ? n_t : n_tiles;
  if (u > max_units) u = max_units;
  const int tail = n_tiles % u;
  tail_split = 1;
  for (int sp = 4; sp > 1; sp >>= 1)
    if (tail > 0 && tail * sp <= u - n_t && (!strips_need_32 || (bn / sp) % 32 == 0)) { tail_split = sp; break; }
  units = u;
}

inline LoraPlan lora_plan(int m, int n, int rank, int num_sms, int max_flags) {
  LoraPlan p;
  const int kBM = 128, kWide = 256;
  const int chunks = rank <= kWide ? 1 : (rank % kWide == 0 ? rank / kWide : 0);
  const int tiles_m = (m + kBM - 1) / kBM, blocks2 = (m + 2 * kBM - 1) / (2 * kBM);
  p.fuse = 0; p.t_chunks = 1; p.Rc = rank;
  if (chunks > 0 && blocks2 * chunks <= num_sms / 2 && blocks2 <= max_flags) {
    p.form = 2; p.fuse = 1; p.t_chunks = chunks; p.Rc = rank / chunks; p.bm = 2 * kBM; p.bn = kWide;
    lora_grid(m, n, p.bm, p.bn, 1, chunks, num_sms / 2, false, p.units, p.tail_split);
  } else if (chunks > 0 && tiles_m * chunks <= num_sms && tiles_m <= max_flags) {
    p.form = 1; p.fuse = 1; p.t_chunks = chunks; p.Rc = rank / chunks; p.bm = kBM; p.bn = kWide;
    lora_grid(m, n, p.bm, p.bn, 1, chunks, num_sms, true, p.units, p.tail_split);
  } else {
    p.form = 0; p.bm = kBM; p.bn = kWide;
    lora_grid(m, n, p.bm, p.bn, 0, 1, num_sms, true, p.units, p.tail_split);
  }
  return p;
}
