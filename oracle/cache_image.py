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
