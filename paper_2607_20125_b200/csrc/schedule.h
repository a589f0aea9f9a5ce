// Host-side tile scheduler of the attention kernel: turns (heads, labels, cache fill) into the per-CTA work lists, the
// shared queue of the dynamic tail and the merge lists.  Host code only; private to headcast_api.cu.
#pragma once
#include "context.h"

namespace {

// ---------------------------------------------------------------------------------- scheduling
struct Proto {  // one (head, query-tile pair, key range) before it is cut into parts
  WorkItem w;
  int n_tiles;
  int tile_off = 0;  // first tile of this proto inside the key sweep (key chunks of a long stream; else 0)
  int group = -1;    // pieces with the same group id are partial results of one query-tile pair (assigned in finalize_schedule)
  int phase = -1;    // phase this proto is placed in (-1: the last line)
  bool always_partial = false;  // one of several key chunks of its pair: never a final result on its own
  int cls_group = -1;  // classification: every piece writes a partial result that belongs to this group ...
  int cls_tag = 0;     // ... with this tag (0 first block, 1 middle blocks, 2 newest block)
};

// Query-tile pairs of rows [q_lo, q_hi) (q_lo a multiple of 256; by default all rows) of one head and key range.
void add_query_pairs(std::vector<Proto>& out, WorkItem base, int n_queries, int n_tiles, int q_lo = 0, int q_hi = -1) {
  const int q_end = (q_hi < 0) ? n_queries : std::min(q_hi, n_queries);
  for (int q0 = q_lo; q0 < q_end; q0 += 256) {
    Proto p;
    p.w = base;
    p.w.q_start[0] = q0;
    p.w.q_start[1] = q0 + 128;
    p.w.q_count[0] = std::min(128, n_queries - q0);
    p.w.q_count[1] = std::max(0, std::min(128, n_queries - q0 - 128));
    p.w.tile_begin = 0;
    p.w.tile_end = n_tiles;
    p.n_tiles = n_tiles;
    out.push_back(p);
  }
}

WorkItem range_item(int head, int map, int x0, long long row0, int n_keys) {
  WorkItem w;
  std::memset(&w, 0, sizeof(w));
  w.head = head;
  w.cell = -1;
  w.kv_map = map;
  w.kv_x0 = x0;
  w.kv_row0 = static_cast<int32_t>(row0);
  w.seg_stride = 0;
  w.seg_len = n_keys;
  w.tiles_per_seg = (n_keys + 127) / 128;
  w.out_mode = OUT_BF16;
  return w;
}

// Cost model of the scheduler, in units of the time one key tile takes with both query tiles in flight (about 2.0 us),
// fitted by least squares to the per-item timings of headcast_read_trace on B200 (480P, 720P and 1080P work lists,
// residual 1-3 % of an item): a lone query tile still needs 0.86 of that because the chain S -> softmax -> P -> next S
// is latency bound; every item pays for its query load, pipeline fill and epilogue; a partial result costs an extra
// round trip through global memory; the tiles of Spatial items measure 2 % slower.
#ifndef HC_COST_ITEM
#define HC_COST_ITEM 2.4
#endif
#ifndef HC_COST_ITEM_SINGLE
#define HC_COST_ITEM_SINGLE 1.0
#endif
#ifndef HC_COST_PARTIAL
#define HC_COST_PARTIAL 0.75
#endif
#ifndef HC_COST_SPATIAL
#define HC_COST_SPATIAL 1.02
#endif
#ifndef HC_COST_SINGLE
#define HC_COST_SINGLE 0.86
#endif
constexpr double TILE_COST_PAIR = 1.0, TILE_COST_SINGLE = HC_COST_SINGLE;
constexpr double ITEM_OVERHEAD = HC_COST_ITEM, ITEM_OVERHEAD_SINGLE = HC_COST_ITEM_SINGLE;
constexpr double PARTIAL_EXTRA = HC_COST_PARTIAL;
constexpr double SPATIAL_FACTOR = HC_COST_SPATIAL;  // tiles of Spatial items (queries gathered by cell, short cell-major key runs)
constexpr int MIN_PART_TILES = 4;  // never cut a key range into pieces shorter than this

double tile_cost(const WorkItem& w) {
  return (w.q_count[1] > 0 ? TILE_COST_PAIR : TILE_COST_SINGLE) * (w.cell >= 0 ? SPATIAL_FACTOR : 1.0);
}

double item_overhead(const WorkItem& w) { return w.q_count[1] > 0 ? ITEM_OVERHEAD : ITEM_OVERHEAD_SINGLE; }

double item_cost(const WorkItem& w) {
  return tile_cost(w) * (w.tile_end - w.tile_begin) + item_overhead(w) + (w.out_mode == OUT_PARTIAL ? PARTIAL_EXTRA : 0.0);
}

// Assigns work to the persistent CTAs (one per SM).
//  - allow_split: the items, longest first, are laid end to end and the line is cut into one equal share per
//    CTA; an item that straddles a cut is divided along its key range, its pieces write unnormalised partial
//    results and combine_kernel merges them.  Every CTA then carries the same number of tile-times.
//  - otherwise (outputs that cannot be merged afterwards): whole items, longest first, onto the least loaded CTA.
void finalize_schedule(headcast_ctx* c, Schedule& s, std::vector<Proto>& protos, bool allow_split) {
  s.items.clear();
  s.combine.clear();
  s.combine_long.clear();
  s.n_slots = 0;
  const int n_cta = c->n_sm;
  std::vector<std::vector<WorkItem>> bins(n_cta + 1);  // bins[n_cta]: the shared queue (dynamic tail)
  bool tail_mode = false;
  int tail_piece_tiles = 8;
  std::stable_sort(protos.begin(), protos.end(),
                   [](const Proto& a, const Proto& b) { return item_cost(a.w) > item_cost(b.w); });
  if (allow_split) {
    // Lay the items end to end and give every CTA the same share Q of the line, cutting the item that straddles a
    // boundary.  Cuts add cost of their own (a second query load and epilogue, partial results), so the share that
    // makes everything fit on n_cta CTAs is found by bisection: lay_out(Q) reports the load of the last CTA.
    struct RawPart { int group, slot, tag; };
    std::vector<RawPart> cls_raw;
    // what earlier phases (see below) have already placed; lay_out() starts over from here on every trial
    std::vector<size_t> bin_base(n_cta, 0);
    size_t combine_base = 0, cls_base = 0, first_proto = 0, last_proto = protos.size();
    int slot_base = 0;
    auto lay_out = [&](double quota) -> double {
      for (int b = 0; b < n_cta; ++b) bins[b].resize(bin_base[b]);
      bins[n_cta].clear();
      s.combine.resize(combine_base);
      cls_raw.resize(cls_base);
      s.n_slots = slot_base;
      int cta = 0;
      double room = quota, last_load = 0.0;
      const int last_bin = tail_mode ? n_cta : n_cta - 1;
      auto next_cta = [&]() {
        if (cta < last_bin) {
          ++cta;
          room = quota;
        }
      };
      for (size_t pi = first_proto; pi < last_proto; ++pi) {
        const Proto& p = protos[pi];
        const double per_tile = tile_cost(p.w), overhead = item_overhead(p.w);
        std::vector<std::pair<int, WorkItem>> parts;  // (cta, piece)
        int begin = 0;
        while (begin < p.n_tiles) {
          const int left = p.n_tiles - begin;
          const double need = per_tile * left + overhead + (begin > 0 ? PARTIAL_EXTRA : 0.0);
          int take = left;
          if (tail_mode && cta == n_cta) {
            // the shared queue: pieces of a fixed size, drawn by whichever CTA is free
            take = std::min(left, tail_piece_tiles);
            if (left - take < MIN_PART_TILES) take = left;
          } else if (need > room && cta < last_bin) {
            // as many tiles as fit, but both pieces must be worth having
            const int can = std::min(static_cast<int>(std::floor((room - overhead - PARTIAL_EXTRA) / per_tile)),
                                     left - MIN_PART_TILES);
            if (can >= MIN_PART_TILES) {
              take = can;
            } else if (room < quota) {  // nothing worth cutting fits into what is left of this CTA
              next_cta();
              continue;
            }  // else: an empty CTA cannot take a proper piece either (a remainder of fewer than 2 * MIN_PART_TILES
               // tiles, or a share smaller than one piece): it takes the rest whole
          }
          WorkItem w = p.w;
          w.tile_begin = p.tile_off + begin;
          w.tile_end = p.tile_off + begin + take;
          parts.push_back(std::make_pair(cta, w));
          const bool cut = (take < left) || begin > 0 || (p.cls_group >= 0) || p.always_partial;
          const double cost = per_tile * take + overhead + (cut ? PARTIAL_EXTRA : 0.0);
          room -= cost;
          if (cta == n_cta - 1) last_load += cost;
          begin += take;
        }
        if (p.cls_group >= 0) {
          for (auto& pr : parts) {
            pr.second.out_mode = OUT_PARTIAL;
            pr.second.out_slot = s.n_slots++;
            bins[pr.first].push_back(pr.second);
            cls_raw.push_back({p.cls_group, pr.second.out_slot, p.cls_tag});
          }
          continue;
        }
        // pieces of ordinary items: whether a piece is a final or a partial result, and its slot, is settled once every
        // phase is placed (the pieces of one query-tile pair may come from several key chunks); until then out_slot
        // carries the pair's group id
        for (auto& pr : parts) {
          pr.second.out_mode = OUT_PARTIAL;
          pr.second.out_slot = p.group;
          bins[pr.first].push_back(pr.second);
        }
      }
      return last_load;
    };
    // The share is found by bisection between the ideal share and one that surely fits.  "Fits" is not quite monotone
    // in the share (room an item could not be cut into is lost, and how much depends on where the cuts fall), so the
    // bisection can settle on a share far too large and leave many CTAs idle; when that happens the shares are
    // scanned upwards from the ideal one instead, coarsely and then finely, and the first that fits is taken.
    auto fits = [&](double share) { return lay_out(share) <= share; };
    auto idle_ctas = [&]() {
      int n = 0;
      for (int b = 0; b < n_cta; ++b) n += bins[b].size() == bin_base[b];
      return n;
    };
    double tail_budget = 0.0;
    auto place = [&](size_t first, size_t last) {  // spreads protos [first, last) over all CTAs, after what is there
      first_proto = first;
      last_proto = last;
      double total = 0.0, biggest = 0.0;
      for (size_t pi = first; pi < last; ++pi) {
        total += item_cost(protos[pi].w);
        biggest = std::max(biggest, item_cost(protos[pi].w));
      }
      const double ideal = total / n_cta;
      if (tail_budget > 0.0 && last == protos.size() && total > 20.0 * n_cta) {
        // last phase: every CTA gets an equal share of all but the tail budget; the rest goes to the shared queue
        const double budget = std::min(tail_budget, 0.5 * total);
        tail_mode = true;
        tail_piece_tiles = std::max(8, static_cast<int>(budget / (4.0 * n_cta)));
        lay_out((total - budget) / n_cta);
        tail_mode = false;
        for (int b = 0; b < n_cta; ++b) bin_base[b] = bins[b].size();
        return;
      }
      double lo = ideal, hi = ideal + biggest + ITEM_OVERHEAD + PARTIAL_EXTRA;
      while (!fits(hi)) hi *= 1.25;
      for (int iter = 0; iter < 24 && hi - lo > 0.25; ++iter) {
        const double mid = 0.5 * (lo + hi);
        if (fits(mid)) hi = mid; else lo = mid;
      }
      lay_out(hi);
      if (idle_ctas() > std::max(2, n_cta / 20)) {
        double share = ideal;
        int step = 0;
        while (!fits(share) && step < 400) share = ideal * (1.0 + 0.02 * ++step);
        if (step > 0) {
          const double below = ideal * (1.0 + 0.02 * (step - 1));
          for (int k = 1; k < 8; ++k) {
            const double fine = below + (share - below) * k / 8.0;
            if (fits(fine)) {
              share = fine;
              break;
            }
          }
        }
        lay_out(share);
      }
      for (int b = 0; b < n_cta; ++b) bin_base[b] = bins[b].size();
      combine_base = s.combine.size();
      cls_base = cls_raw.size();
      slot_base = s.n_slots;
    };
    // Phases.  In one line over everything, the CTAs work on all long key streams at once (at 720P three Global
    // heads: 116 MB of K/V against 126 MB of L2) and the streams evict each other.  So the long streams (plain row
    // ranges of one head: Global heads, every head of the dense sweep) are packed, largest first, into phases of at
    // most HC_PHASE_BYTES of K/V, and every phase that is worth at least 60 tile-steps per CTA is spread over ALL
    // CTAs on its own, one phase after the other: the CTAs then read the same tens of MB at the same time.
    // Everything else (short streams, Spatial cells) follows in one last line.  Measured: 9-13 % off the 720P and
    // 1080P attention and dense sweeps, 6 % off the 480P dense sweep; at 480P the three Global heads (50 MB) are
    // left in one line, where phases only add partial results to merge.
    // A stream too long for that on its own (1080P: 88 MB of K/V per Global head) is ALSO cut along its keys into
    // chunks of at most HC_CHUNK_BYTES, every chunk a phase of its own: all CTAs sweep the same ~30 MB of keys at the
    // same time, each query-tile pair leaves one partial result per chunk, and combine_kernel merges them.  Without the
    // chunks the CTAs sit at 148 different places of the sweep, the whole stream is the working set, and 8.4x the
    // algorithmic bytes came from DRAM at 1080P (ncu: 6.97 GB per launch).
    {
#ifndef HC_PHASE_MB
#define HC_PHASE_MB 60
#endif
#ifndef HC_CHUNK_MB
#define HC_CHUNK_MB 30
#endif
      constexpr long long HC_PHASE_BYTES = static_cast<long long>(HC_PHASE_MB) << 20, HC_CHUNK_BYTES = static_cast<long long>(HC_CHUNK_MB) << 20;
      for (size_t pi = 0; pi < protos.size(); ++pi)
        if (protos[pi].group < 0) protos[pi].group = static_cast<int>(pi);
      struct Stream { int map, head, phase, n_chunks; double cost; long long bytes; };
      std::vector<Stream> streams;
      double all_cost = 0.0;
      auto stream_of = [&](const Proto& p) {
        return std::find_if(streams.begin(), streams.end(), [&](const Stream& st) { return st.map == p.w.kv_map && st.head == p.w.head; });
      };
      for (const Proto& p : protos) {
        all_cost += item_cost(p.w);
        if (p.w.cell >= 0) continue;
        auto it = stream_of(p);
        if (it == streams.end()) {
          const long long segs = (p.n_tiles + p.w.tiles_per_seg - 1) / p.w.tiles_per_seg;
          streams.push_back({p.w.kv_map, p.w.head, -1, 1, 0.0, segs * p.w.seg_len * c->D * 4ll});
          it = streams.end() - 1;
        }
        it->cost += item_cost(p.w);
      }
      // Dynamic tail.  Identical work takes +-3 % longer or shorter from SM to SM, which no static list can absorb: the
      // last HC_TAIL_FRAC of the launch's work is held back from the equal shares and cut into small pieces that the
      // CTAs draw from a shared queue when their own lists are done (measured: 0.02 is the best of 0.02 / 0.04 / 0.06;
      // -3.5 % at 480P, -0.7 % at 720P, -0.5 % at 1080P).  Not for classification sweeps (their pieces are merged by group).
#ifndef HC_TAIL_FRAC
#define HC_TAIL_FRAC 0.02
#endif
      if (s.cls_groups.empty() && all_cost > 40.0 * n_cta) tail_budget = HC_TAIL_FRAC * all_cost;
      std::stable_sort(streams.begin(), streams.end(), [](const Stream& a, const Stream& b) { return a.cost > b.cost; });
      // first-fit of the streams into phases; a phase too light to be cut 148 ways is dissolved again
      std::vector<double> phase_cost;
      std::vector<long long> phase_bytes;
      long long long_bytes = 0;
      for (Stream& st : streams) {
        if (st.cost < 20.0 * n_cta) continue;
        long_bytes += st.bytes;
        // key chunks only for plain row ranges (one segment) that are not part of a classification sweep
        const int chunks = static_cast<int>((st.bytes + HC_CHUNK_BYTES - 1) / HC_CHUNK_BYTES);
        if (st.bytes > HC_PHASE_BYTES && s.cls_groups.empty() && st.cost / chunks >= 60.0 * n_cta) {
          st.n_chunks = chunks;
          st.phase = static_cast<int>(phase_bytes.size());
          for (int k = 0; k < chunks; ++k) {
            phase_bytes.push_back(HC_PHASE_BYTES);  // closed to other streams
            phase_cost.push_back(st.cost / chunks);
          }
          continue;
        }
        size_t ph = 0;
        while (ph < phase_bytes.size() && phase_bytes[ph] + st.bytes > HC_PHASE_BYTES) ++ph;
        if (ph == phase_bytes.size()) {
          phase_bytes.push_back(0);
          phase_cost.push_back(0.0);
        }
        phase_bytes[ph] += st.bytes;
        phase_cost[ph] += st.cost;
        st.phase = static_cast<int>(ph);
      }
      size_t done = 0;
      if (long_bytes > (64ll << 20) && all_cost >= 120.0 * n_cta) {  // below that the streams share L2 anyway (480P: 50 MB)
        // every proto learns its phase; protos of a chunked stream are replaced by one proto per key chunk
        std::vector<Proto> expanded;
        expanded.reserve(protos.size());
        for (const Proto& p : protos) {
          auto it = (p.w.cell >= 0) ? streams.end() : stream_of(p);
          if (it == streams.end() || it->phase < 0) {
            expanded.push_back(p);
            continue;
          }
          if (it->n_chunks == 1 || p.w.seg_stride != 0 || p.n_tiles < 2 * it->n_chunks * MIN_PART_TILES) {
            Proto q = p;
            q.phase = it->phase;
            expanded.push_back(q);
            continue;
          }
          for (int k = 0; k < it->n_chunks; ++k) {
            Proto q = p;
            const int lo = static_cast<int>(static_cast<long long>(p.n_tiles) * k / it->n_chunks);
            const int hi = static_cast<int>(static_cast<long long>(p.n_tiles) * (k + 1) / it->n_chunks);
            q.tile_off = p.tile_off + lo;
            q.n_tiles = hi - lo;
            q.w.tile_begin = q.tile_off;
            q.w.tile_end = q.tile_off + q.n_tiles;
            q.phase = it->phase + k;
            q.always_partial = true;
            expanded.push_back(q);
          }
        }
        protos.swap(expanded);
        // what belongs to no phase (short streams, Spatial cells, phases too light to be cut 148 ways) goes FIRST, the
        // phases follow: the launch then ends inside a long stream, whose last stretch feeds the shared queue
        auto heavy = [&](const Proto& p) { return p.phase >= 0 && phase_cost[p.phase] >= 60.0 * n_cta; };
        bool any_heavy = false;
        for (const Proto& p : protos) any_heavy = any_heavy || heavy(p);
        if (any_heavy) {
          auto mid0 = std::stable_partition(protos.begin(), protos.end(), [&](const Proto& p) { return !heavy(p); });
          const size_t n_left = static_cast<size_t>(mid0 - protos.begin());
          if (n_left > 0) place(0, n_left);
          done = n_left;
        }
        for (size_t ph = 0; ph < phase_cost.size(); ++ph) {
          if (phase_cost[ph] < 60.0 * n_cta) continue;
          auto in_phase = [&](const Proto& p) { return p.phase == static_cast<int>(ph); };
          auto mid = std::stable_partition(protos.begin() + done, protos.end(), in_phase);
          const size_t next = static_cast<size_t>(mid - protos.begin());
          if (next > done) place(done, next);
          done = next;
        }
      }
      if (done < protos.size() || protos.empty()) place(done, protos.size());
    }
    // ordinary items: the pieces of one query-tile pair (same group id, parked in out_slot) become a final result if
    // there is only one, else partial results in consecutive slots, in key order, plus one merge entry per query tile
    if (s.cls_groups.empty()) {
      struct Piece { int bin, pos, tile_begin; };
      std::vector<std::vector<Piece>> by_group;
      for (int b = 0; b <= n_cta; ++b)
        for (size_t i = 0; i < bins[b].size(); ++i) {
          const WorkItem& w = bins[b][i];
          if (static_cast<size_t>(w.out_slot) >= by_group.size()) by_group.resize(w.out_slot + 1);
          by_group[w.out_slot].push_back({b, static_cast<int>(i), w.tile_begin});
        }
      s.combine.clear();
      s.combine_long.clear();
      s.n_slots = 0;
      for (auto& pieces : by_group) {
        if (pieces.empty()) continue;
        if (pieces.size() == 1) {
          WorkItem& w = bins[pieces[0].bin][pieces[0].pos];
          w.out_mode = OUT_BF16;
          w.out_slot = 0;
          continue;
        }
        std::sort(pieces.begin(), pieces.end(), [](const Piece& a, const Piece& b) { return a.tile_begin < b.tile_begin; });
        const int first_slot = s.n_slots;
        for (const Piece& pc : pieces) bins[pc.bin][pc.pos].out_slot = s.n_slots++;
        const WorkItem& w0 = bins[pieces[0].bin][pieces[0].pos];
        for (int t = 0; t < (w0.q_count[1] > 0 ? 2 : 1); ++t) {
          CombineEntry e;
          e.head = w0.head;
          e.cell = w0.cell;
          e.q_start = w0.q_start[t];
          e.q_count = w0.q_count[t];
          e.first_slot = first_slot;
          e.n_parts = static_cast<int32_t>(pieces.size());
          e.sub = t;
          e.pad = 0;
          (e.n_parts > COMBINE_LONG_PARTS ? s.combine_long : s.combine).push_back(e);
        }
      }
    }
    // classification: the pieces of every group, in group order
    std::stable_sort(cls_raw.begin(), cls_raw.end(), [](const RawPart& a, const RawPart& b) { return a.group < b.group; });
    s.cls_parts.clear();
    for (ClsGroup& g : s.cls_groups) g.n_parts = 0;
    for (const RawPart& rp : cls_raw) {
      ClsGroup& g = s.cls_groups[rp.group];
      if (g.n_parts == 0) g.first_part = static_cast<int32_t>(s.cls_parts.size());
      ++g.n_parts;
      s.cls_parts.push_back(ClsPart{rp.slot, rp.tag});
    }
  } else {
    typedef std::pair<double, int> Load;
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> pq;
    for (int b = 0; b < n_cta; ++b) pq.push(Load(0.0, b));
    for (const Proto& p : protos) {
      Load l = pq.top();
      pq.pop();
      bins[l.second].push_back(p.w);
      pq.push(Load(l.first + item_cost(p.w), l.second));
    }
  }
  s.cta_first.assign(n_cta + 1, 0);
  for (int b = 0; b < n_cta; ++b) {
    s.cta_first[b] = static_cast<int32_t>(s.items.size());
    s.items.insert(s.items.end(), bins[b].begin(), bins[b].end());
  }
  s.cta_first[n_cta] = static_cast<int32_t>(s.items.size());
  s.dyn_first = static_cast<int32_t>(s.items.size());
  s.items.insert(s.items.end(), bins[n_cta].begin(), bins[n_cta].end());
  s.dyn_end = static_cast<int32_t>(s.items.size());
  s.uploaded = false;
}

int n_filled(const headcast_ctx* c) { return static_cast<int>(c->slots.size()); }

void build_dense_schedule(headcast_ctx* c, Schedule& s, int out_mode, bool allow_split) {
  std::vector<Proto> protos;
  const int n_keys = n_filled(c) * c->L;
  for (int h = 0; h < c->H; ++h) {
    WorkItem w = range_item(h, MAP_MONO, h * c->D, 0, n_keys);
    w.out_mode = out_mode;
    add_query_pairs(protos, w, c->L, w.tiles_per_seg);
  }
  s.flops = 4.0 * c->H * static_cast<double>(c->L) * n_keys * c->D;
  finalize_schedule(c, s, protos, allow_split);
  s.key_filled = n_filled(c);
}

// group < 0: every head; 0: Global heads only; 1: Spatial; 2: Sink and Dummy
// group < 0: every head; else only the heads of one archetype group (0 Global, 1 Spatial, 2 Sink + Dummy), and for
// groups 0 and 2 only the query rows [q_lo, q_hi) (q_lo a multiple of 256; q_hi < 0: to the end).
void build_headcast_schedule(headcast_ctx* c, Schedule& s, int group = -1, int q_lo = 0, int q_hi = -1) {
  std::vector<Proto> protos;
  const int nf = n_filled(c);
  const long long win = static_cast<long long>(c->n_blk) * c->L;
  double flops = 0.0;
  for (int h = 0; h < c->H; ++h) {
    const int cl = c->cls[h], ix = c->idx[h];
    if (group >= 0 && group != (cl == CLS_GLOBAL ? 0 : cl == CLS_SPATIAL ? 1 : 2)) continue;
    if (cl == CLS_SINK || cl == CLS_DUMMY) {
      const int j = (cl == CLS_SINK) ? ix : c->n_cls[CLS_SINK] + ix;
      // the head's blocks are adjacent; with two of them the order does not matter to attention
      long long row0 = static_cast<long long>(j) * c->sd_slots * c->L;
      if (cl == CLS_DUMMY && c->sd_valid == 1) row0 += static_cast<long long>(c->dummy_cur) * c->L;
      WorkItem w = range_item(h, MAP_SD, 0, row0, c->sd_valid * c->L);
      add_query_pairs(protos, w, c->L, w.tiles_per_seg, q_lo, q_hi);
      flops += 4.0 * c->L * static_cast<double>(c->sd_valid) * c->L * c->D;
    } else if (cl == CLS_GLOBAL) {
      WorkItem w = range_item(h, MAP_GLOBAL, 0, ix * win, nf * c->L);
      add_query_pairs(protos, w, c->L, w.tiles_per_seg, q_lo, q_hi);
      flops += 4.0 * c->L * static_cast<double>(nf) * c->L * c->D;
    } else {
      for (size_t ci = 0; ci < c->cells.size(); ++ci) {
        const int nc = c->cells[ci].ch * c->cells[ci].cw;
        const long long row0 = ix * win + static_cast<long long>(c->n_blk) * c->F_b * c->cell_tok_off[ci];
        WorkItem w = range_item(h, MAP_SPATIAL, 0, row0, nf * c->F_b * nc);
        w.cell = static_cast<int32_t>(ci);
        add_query_pairs(protos, w, c->F_b * nc, w.tiles_per_seg);
        flops += 4.0 * (c->F_b * nc) * static_cast<double>(nf * c->F_b * nc) * c->D;
      }
    }
  }
  s.flops = flops;
  finalize_schedule(c, s, protos, true);
  s.key_filled = nf * 4 + c->sd_valid;
}

}  // namespace
