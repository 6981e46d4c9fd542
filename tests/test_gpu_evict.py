"""GPU parity of global token eviction with compaction (twkv_evict) against the CPU oracle.

The cache image after eviction (tables and every block, bit for bit) is compared with the oracle's image after the
same operation; decode attention afterwards must equal the oracle's attention over the surviving tokens; appends after
an eviction continue behind the survivors.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle.cache_image import CacheImage
from paper_2603_04411_b200 import workloads
from tests.helpers import GpuCache, attn_errors, bits16, compare_cache_with_image, oracle_decode

pytestmark = pytest.mark.gpu

MAX_ABS, REL_L2 = 2e-3, 1e-3


def _setup(B, li, ranks, n_first):
    n_seq = int(li.seq_ids.max()) + 1
    tmax = int(np.bincount(li.seq_ids.numpy(), minlength=n_seq).max())
    gc = GpuCache(B, n_layers=1, n_q_heads=li.n_q_heads, n_kv_heads=li.n_kv_heads, dtype=li.dtype, out_dtype=torch.float32,
                  max_seqs=n_seq, max_tokens_per_seq=tmax, payload_bytes=int((-(-ranks // 64) * 128).sum()))
    img = CacheImage(1, li.d_kv, n_seq, tmax, int(gc.lay.n_blocks))
    dev = {n: getattr(li, n).cuda().contiguous() for n in ["Uinv_k", "Uinv_v", "xt_k", "xt_v", "seq_ids", "positions"]}
    B.twkv_cache_set_layer_params(gc.h, 0, dev["Uinv_k"], dev["Uinv_v"])
    lv = torch.from_numpy(ranks.astype(np.int16)).cuda().contiguous()

    def append(lo, hi):
        B.twkv_compress(gc.h, 0, dev["xt_k"][lo:hi], dev["xt_v"][lo:hi], dev["seq_ids"][lo:hi], dev["positions"][lo:hi], None,
                        lv[lo:hi], B.TWKV_GATE_FORCED)
        assert img.append(0, bits16(li.xt_k[lo:hi]), bits16(li.xt_v[lo:hi]), li.seq_ids[lo:hi].numpy(), li.positions[lo:hi].numpy(),
                          ranks[lo:hi])
    append(0, n_first)
    return gc, img, append


def _decode_check(B, gc, li, ranks, alive, seqs):
    out = torch.full((len(seqs), li.n_q_heads, 128), float("nan"), device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q[seqs].cuda().contiguous(), torch.tensor(seqs, dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    sub = torch.from_numpy(np.nonzero(alive)[0])
    li2 = workloads.LayerInputs(**{**li.__dict__})
    for n in ["xt_k", "xt_v", "seq_ids", "positions"]:
        setattr(li2, n, getattr(li, n)[sub].contiguous())
    li2.q = li.q[seqs]
    want = oracle_decode(li2, ranks[alive], seqs)
    return attn_errors(out.cpu().numpy(), want)


def test_evict_compacts_and_decode_sees_survivors_only():
    from paper_2603_04411_b200 import build
    build.build()
    from paper_2603_04411_b200 import binding as B
    # three sequences x 700 tokens, every rank, K and V ranks independent, shuffled positions
    li = workloads.build_layer(801, n_seq=3, ctx=700, n_q_heads=32, mode="forced", rank_recipe="any", outlier="pct:1",
                               shuffle_positions=True)
    ranks = li.ranks.numpy().astype(np.int64)
    n = ranks.shape[0]
    gc, img, append = _setup(B, li, ranks, 1800)                        # sequences 0 and 1 whole, 400 tokens of sequence 2
    compare_cache_with_image(gc, img)
    rng = np.random.default_rng(5)
    seq_np, pos_np = li.seq_ids.numpy(), li.positions.numpy()
    alive = np.zeros(n, bool); alive[:1800] = True
    # sequence 1 keeps about a quarter of its tokens (plus positions nothing is cached at, which are ignored)
    keep1 = np.concatenate([rng.permutation(700)[:180], [5000, 123456]]).astype(np.int32)
    B.twkv_evict(gc.h, 0, 1, torch.from_numpy(keep1).cuda())
    img.evict(0, 1, keep1)
    alive &= ~((seq_np == 1) & ~np.isin(pos_np, keep1))
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    compare_cache_with_image(gc, img)
    st = B.twkv_cache_stats(gc.h, 0)
    assert st.tokens == int(alive.sum()) and st.bytes_algorithmic == int(2 * ranks[alive].sum())
    assert st.bytes_stored == img.stored_bytes(0)
    max_abs, rel_l2 = _decode_check(B, gc, li, ranks, alive, [0, 1, 2])
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    # sequence 2 gets the rest of its tokens, then sequence 0 is cut to 3 tokens and sequence 2 evicted twice in a row
    append(1800, n)
    alive[1800:] = True
    keep0 = pos_np[seq_np == 0][[0, 350, 699]].astype(np.int32)
    B.twkv_evict(gc.h, 0, 0, torch.from_numpy(keep0).cuda())
    img.evict(0, 0, keep0)
    alive &= ~((seq_np == 0) & ~np.isin(pos_np, keep0))
    for frac in (0.5, 0.3):
        cur = pos_np[(seq_np == 2) & alive]
        keep2 = rng.permutation(cur)[:int(frac * len(cur))].astype(np.int32)
        B.twkv_evict(gc.h, 0, 2, torch.from_numpy(keep2).cuda())
        img.evict(0, 2, keep2)
        alive &= ~((seq_np == 2) & ~np.isin(pos_np, keep2))
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    compare_cache_with_image(gc, img)
    max_abs, rel_l2 = _decode_check(B, gc, li, ranks, alive, [2, 0, 1])
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    # appends after an eviction continue behind the survivors: sequence 1's dropped tokens come back as new tokens
    back = np.nonzero((seq_np == 1) & ~alive)[0][:150]
    sel = torch.from_numpy(back)
    B.twkv_compress(gc.h, 0, li.xt_k[sel].cuda().contiguous(), li.xt_v[sel].cuda().contiguous(), li.seq_ids[sel].cuda().contiguous(),
                    li.positions[sel].cuda().contiguous(), None, torch.from_numpy(ranks[back].astype(np.int16)).cuda().contiguous(),
                    B.TWKV_GATE_FORCED)
    assert img.append(0, bits16(li.xt_k[sel]), bits16(li.xt_v[sel]), seq_np[back], pos_np[back], ranks[back])
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK
    compare_cache_with_image(gc, img)
    alive[back] = True
    max_abs, rel_l2 = _decode_check(B, gc, li, ranks, alive, [1])
    assert max_abs < MAX_ABS and rel_l2 < REL_L2, (max_abs, rel_l2)
    # dropping everything leaves an empty sequence (zeros), the others untouched
    B.twkv_evict(gc.h, 0, 1, torch.zeros(0, dtype=torch.int32, device="cuda"))
    img.evict(0, 1, [])
    compare_cache_with_image(gc, img)
    out = torch.full((1, 32, 128), 3.0, device="cuda")
    B.twkv_decode_attn(gc.h, 0, li.q[1:2].cuda().contiguous(), torch.tensor([1], dtype=torch.int32, device="cuda"), out)
    assert B.twkv_cache_status(gc.h) == B.TWKV_OK and torch.count_nonzero(out).item() == 0
    gc.close()
