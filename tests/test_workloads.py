"""The synthetic inputs have the shapes, value distributions and structure the benchmark's configs name."""
import numpy as np

from paper_2507_01438_b200 import workloads as wl


def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 (even mantissa) and 1 + 2^-7: goes to 1.0;
    # 1 + 3*2^-8 is a tie between 1+2^-7 (odd) and 1+2^-6 (even): goes up.
    a = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -16, -2.5, 0.0],
                 dtype=np.float32)
    b = wl.f32_to_bf16_bits(a)
    assert b.tolist() == [0x3F80, 0x3F80, 0x3F82, 0x3F81, 0xC020, 0x0000]
    back = wl.bf16_bits_to_f32(b)
    assert np.all(np.abs(back - a) <= np.abs(a) * 2.0 ** -8)


def test_tiny_and_decode_shapes():
    w = wl.tiny()
    assert (w.h_in, w.h_out, w.n_slots, w.max_rank, w.T) == (256, 256, 4, 8, 16)
    assert all(ad.rank == 8 and ad.scale == 2.0 for ad in w.adapters.values())
    std = wl.bf16_bits_to_f32(w.W).std()
    assert 0.018 < std < 0.022
    d = wl.q_proj_decode(h=512, n=32)
    assert sorted(d.ids.tolist()) == list(range(32))          # every token its own adapter
    assert abs(wl.bf16_bits_to_f32(d.x).std() - 1.0) < 0.05


def test_prefill_segments_are_contiguous():
    p = wl.gate_up_prefill(h_in=64, h_out=96, seg_len=32)
    assert p.T == 256
    runs = p.ids.reshape(8, 32)
    assert np.all(runs == runs[:, :1]) and sorted(runs[:, 0].tolist()) == list(range(8))


def test_many_tenant_ids_follow_the_bounded_power_law():
    m = wl.down_proj_many_tenant(h_in=64, h_out=32, n_tokens=256, only_used=True)
    assert m.n_slots == 1000 and m.T == 256
    assert int((m.ids == -1).sum()) == 26                      # 10 % of 256, rounded
    used = m.distinct_adapters()
    assert 60 <= len(used) <= 140 and set(used) == set(m.adapters)
    # heavy head: the most popular adapter holds roughly P(1) = 0.18 of the adapter tokens
    _, counts = np.unique(m.ids[m.ids >= 0], return_counts=True)
    assert 0.08 < counts.max() / counts.sum() < 0.30
    full = wl.down_proj_many_tenant(h_in=64, h_out=32, n_tokens=256, n_adapters=50, only_used=False)
    assert len(full.adapters) == 50


def test_full_set_batch_layout():
    b = wl.full_set_batch()
    assert b.ids.shape == (2112,) and set(np.unique(b.ranks)) <= {8, 16, 32}
    tail = b.ids[64:].reshape(2, 1024)
    assert np.all(tail == tail[:, :1]) and tail[0, 0] != tail[1, 0]
    assert not (set(tail[:, 0].tolist()) & set(b.ids[:64].tolist()))
    assert sum(hi * ho for _, hi, ho in wl.LLAMA8B_SITES) == 218103808
