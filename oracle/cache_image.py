"""Byte-level image of the mixed-rank paged cache, built on the CPU.

TEST INFRASTRUCTURE ONLY (same rules as the rest of `oracle/`).

The paper fixes WHAT is persisted (Eq. 2 and the sentence after it: only the
retained components x^[I] of every token); the container format is the
library's own and is restated here, independently of the CUDA code, so the
packed bytes and tables the GPU writes can be compared bit for bit.

Format
------
* Rank class of a token side (K or V): c = ceil(r / 64), row width w = 64 c
  16-bit elements.  Elements r .. w-1 of a stored row are +0 (0x0000).
* A tile holds up to 128 tokens of one (layer, side, sequence, class).  It owns
  c consecutive 16 KiB blocks; block j of the tile is the panel
  [128 rows x 64 elements] of elements 64 j .. 64 j + 63, row-major
  (row s at byte 128 s).  Rows past the last valid token are zero.
* Tokens of one (side, sequence, class) fill tiles in arrival order
  (order of the compress calls, then index within a call).
* A compress call is cut into pieces of PIECE_TOKENS tokens, handled in order.
  Within a piece, new tiles are created in ascending key order
  key = (side * max_seqs + seq) * n_classes + (c - 1)   (side: K = 0, V = 1),
  and, within a key, in ascending tile ordinal.  Tile ids count up per
  (layer, side); blocks come from one bump pointer shared by all layers.
* Per tile and slot: K side stores the token position, V side stores the
  score link ktile_id * 128 + kslot of the same token's K row; both sides store
  the rank r.
* K tiles are also listed per class (creation order); V tiles per sequence
  (creation order).
* Eviction (the paper combines the method with token eviction, Sec. 5.2
  "Implementation Details": one token set for all heads) keeps, of one
  sequence in one layer, the tokens at the listed positions.  Per (side,
  class) of the sequence the survivors move to the front of the key's tiles in
  their stored order; the rows behind the last survivor in the last tile still
  in use become zero; emptied tiles leave the lists (n_valid 0, blocks left as
  they are and not reused); V slots are relinked to the K rows' new slots.
"""
import numpy as np

TILE = 128
PANEL = 64
BLOCK_ELEMS = TILE * PANEL
PIECE_TOKENS = 131072


class CacheImage:
    def __init__(self, n_layers, d_kv, max_seqs, max_tokens_per_seq, n_blocks):
        self.L = n_layers
        self.d = d_kv
        self.NC = d_kv // PANEL
        self.S = max_seqs
        self.tmax = max_tokens_per_seq
        self.n_blocks = n_blocks
        self.tiles_per_seq = -(-max_tokens_per_seq // TILE) + self.NC
        self.NT = max_seqs * self.tiles_per_seq
        self.blocks = np.zeros((n_blocks, BLOCK_ELEMS), dtype=np.uint16)
        self.next_block = 0
        nk = 2 * self.S * self.NC
        self.fill = np.zeros((self.L, nk), dtype=np.int64)
        self.key_tiles = [[[] for _ in range(nk)] for _ in range(self.L)]
        # per (layer, side): tile tables
        self.n_tiles = np.zeros((self.L, 2), dtype=np.int64)
        self.tile_desc = np.zeros((self.L, 2, self.NT, 4), dtype=np.int32)  # seq, cls, n_valid, base
        self.tile_aux = np.zeros((self.L, 2, self.NT, TILE), dtype=np.int32)
        self.tile_rank = np.zeros((self.L, 2, self.NT, TILE), dtype=np.uint16)
        self.kclass_tiles = [[[] for _ in range(self.NC)] for _ in range(self.L)]
        self.seq_vtiles = [[[] for _ in range(self.S)] for _ in range(self.L)]
        self.seq_tokens = np.zeros((self.L, self.S), dtype=np.int64)

    def key(self, side, seq, cls):
        return (side * self.S + seq) * self.NC + (cls - 1)

    def append(self, layer, xk, xv, seq_ids, positions, ranks):
        """xk, xv: [n, d] uint16 bit patterns of x~; ranks [n, 2] (r_K, r_V).
        Returns False (image unchanged) if a piece does not fit."""
        n = len(seq_ids)
        for lo in range(0, n, PIECE_TOKENS):
            hi = min(n, lo + PIECE_TOKENS)
            if not self._piece(layer, xk[lo:hi], xv[lo:hi], seq_ids[lo:hi], positions[lo:hi], ranks[lo:hi]):
                return False
        return True

    def _piece(self, layer, xk, xv, seq_ids, positions, ranks):
        n = len(seq_ids)
        ranks = np.asarray(ranks, dtype=np.int64)
        cls = (ranks + PANEL - 1) // PANEL
        keys = np.empty((n, 2), dtype=np.int64)
        for side in range(2):
            keys[:, side] = (side * self.S + np.asarray(seq_ids)) * self.NC + (cls[:, side] - 1)
        # stable rank inside the piece
        within = np.zeros((n, 2), dtype=np.int64)
        counts = {}
        for side in range(2):
            for i in range(n):
                k = int(keys[i, side])
                within[i, side] = counts.get(k, 0)
                counts[k] = within[i, side] + 1
        # capacity: tokens per sequence, tiles, blocks
        add_tok = np.bincount(np.asarray(seq_ids), minlength=self.S)
        if np.any(self.seq_tokens[layer] + add_tok > self.tmax):
            return False
        need_blocks = 0
        need_tiles = [0, 0]
        for k in sorted(counts):
            c = k % self.NC + 1
            side = k // (self.S * self.NC)
            old = -(-int(self.fill[layer, k]) // TILE)
            new = -(-int(self.fill[layer, k] + counts[k]) // TILE)
            need_blocks += (new - old) * c
            need_tiles[side] += new - old
        if self.next_block + need_blocks > self.n_blocks:
            return False
        for side in range(2):
            if self.n_tiles[layer, side] + need_tiles[side] > self.NT:
                return False
        # allocate new tiles in ascending key order
        for k in sorted(counts):
            c = k % self.NC + 1
            side = k // (self.S * self.NC)
            seq = (k // self.NC) % self.S
            old = -(-int(self.fill[layer, k]) // TILE)
            new = -(-int(self.fill[layer, k] + counts[k]) // TILE)
            for _ in range(old, new):
                tid = int(self.n_tiles[layer, side])
                self.n_tiles[layer, side] += 1
                self.tile_desc[layer, side, tid] = (seq, c, 0, self.next_block)
                self.next_block += c
                self.key_tiles[layer][k].append(tid)
                if side == 0:
                    self.kclass_tiles[layer][c - 1].append(tid)
                else:
                    self.seq_vtiles[layer][seq].append(tid)
        # write rows
        kslot_of = np.zeros(n, dtype=np.int64)
        for side, x in ((0, xk), (1, xv)):
            for i in range(n):
                k = int(keys[i, side])
                g = int(self.fill[layer, k]) + int(within[i, side])
                tid = self.key_tiles[layer][k][g // TILE]
                slot = g % TILE
                c = k % self.NC + 1
                r = int(ranks[i, side])
                base = int(self.tile_desc[layer, side, tid, 3])
                row = np.zeros(c * PANEL, dtype=np.uint16)
                row[:r] = x[i, :r]
                for j in range(c):
                    self.blocks[base + j, slot * PANEL:(slot + 1) * PANEL] = row[j * PANEL:(j + 1) * PANEL]
                self.tile_rank[layer, side, tid, slot] = r
                if side == 0:
                    self.tile_aux[layer, 0, tid, slot] = positions[i]
                    kslot_of[i] = tid * TILE + slot
                else:
                    self.tile_aux[layer, 1, tid, slot] = kslot_of[i]
                self.tile_desc[layer, side, tid, 2] = max(int(self.tile_desc[layer, side, tid, 2]), slot + 1)
        for k, cnt in counts.items():
            self.fill[layer, k] += cnt
        self.seq_tokens[layer] += add_tok
        return True

    def evict(self, layer, seq, keep_positions):
        """Keeps the tokens of `seq` whose position is listed; returns, per side, {old global slot: new global slot}."""
        keep = set(int(p) for p in keep_positions)
        moved = [{}, {}]
        kept_tokens = 0
        # who survives is decided on the tables as they are (a V slot finds its position through its K row)
        survivors_of = {}
        for side in range(2):
            for c in range(1, self.NC + 1):
                found = []
                for tid in self.key_tiles[layer][self.key(side, seq, c)]:
                    for slot in range(int(self.tile_desc[layer, side, tid, 2])):
                        a = int(self.tile_aux[layer, side, tid, slot])
                        pos = a if side == 0 else int(self.tile_aux[layer, 0, a // TILE, a % TILE])
                        if pos in keep:
                            found.append((tid, slot))
                survivors_of[side, c] = found
        for side in range(2):
            for c in range(1, self.NC + 1):
                k = self.key(side, seq, c)
                tiles = self.key_tiles[layer][k]
                survivors = survivors_of[side, c]
                rows = []
                for tid, slot in survivors:                      # everything is read before anything is written
                    base = int(self.tile_desc[layer, side, tid, 3])
                    rows.append(([self.blocks[base + j, slot * PANEL:(slot + 1) * PANEL].copy() for j in range(c)],
                                 int(self.tile_aux[layer, side, tid, slot]), int(self.tile_rank[layer, side, tid, slot])))
                for g, ((tid, slot), (row, a, r)) in enumerate(zip(survivors, rows)):
                    dt, ds = tiles[g // TILE], g % TILE
                    moved[side][tid * TILE + slot] = dt * TILE + ds
                    base = int(self.tile_desc[layer, side, dt, 3])
                    for j in range(c):
                        self.blocks[base + j, ds * PANEL:(ds + 1) * PANEL] = row[j]
                    self.tile_aux[layer, side, dt, ds] = a
                    self.tile_rank[layer, side, dt, ds] = r
                n = len(survivors)
                n_kept = -(-n // TILE)
                if n % TILE:
                    base = int(self.tile_desc[layer, side, tiles[n_kept - 1], 3])
                    for j in range(c):
                        self.blocks[base + j, (n % TILE) * PANEL:] = 0
                for ordinal, tid in enumerate(tiles):
                    self.tile_desc[layer, side, tid, 2] = min(TILE, n - ordinal * TILE) if ordinal < n_kept else 0
                gone = set(tiles[n_kept:])
                self.key_tiles[layer][k] = tiles[:n_kept]
                if side == 0:
                    self.kclass_tiles[layer][c - 1] = [t for t in self.kclass_tiles[layer][c - 1] if t not in gone]
                    kept_tokens += n
                else:
                    self.seq_vtiles[layer][seq] = [t for t in self.seq_vtiles[layer][seq] if t not in gone]
                self.fill[layer, k] = n
        # V slots follow their tokens' K rows
        for c in range(1, self.NC + 1):
            for tid in self.key_tiles[layer][self.key(1, seq, c)]:
                for slot in range(int(self.tile_desc[layer, 1, tid, 2])):
                    self.tile_aux[layer, 1, tid, slot] = moved[0][int(self.tile_aux[layer, 1, tid, slot])]
        self.seq_tokens[layer, seq] = kept_tokens
        return moved

    # ---- logical views used by the decode oracle ---------------------------------
    def stored_bytes(self, layer=None):
        """Bytes physically held by tiles' valid rows (padding to the class width included)."""
        total = 0
        for l in range(self.L) if layer is None else [layer]:
            for side in range(2):
                for tid in range(int(self.n_tiles[l, side])):
                    _, c, nv, _ = self.tile_desc[l, side, tid]
                    total += int(nv) * int(c) * PANEL * 2
        return total
