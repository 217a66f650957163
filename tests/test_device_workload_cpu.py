"""The torch generator the benchmark uses, run on the CPU device: deterministic per seed, same
layout as the numpy generator, and it plants a structure the oracle recovers."""
import numpy as np

from helpers import OracleLayer, delta_gap_ok
from paper_2604_12056_b200 import workloads as wl


def test_device_workload_recipe_on_cpu():
    cfg = wl.config("c5", kv_lens=(300, 170), n_blocks=2, steps=3, topk=4)
    a = wl.DeviceWorkload(cfg, replica=1, layer=2, device="cpu")
    b = wl.DeviceWorkload(cfg, replica=1, layer=2, device="cpu")
    c = wl.DeviceWorkload(cfg, replica=1, layer=3, device="cpu")
    ha, hb, hc = a.host_copy(), b.host_copy(), c.host_copy()
    assert (ha.k_pages == hb.k_pages).all() and (ha.page_table == hb.page_table).all()
    assert not (ha.k_pages == hc.k_pages).all()
    assert ha.k_pages.dtype == np.uint16 and ha.k_pages.shape == (2 * cfg.max_pages_per_seq, 8, 32, 128)
    assert sorted(ha.page_table.ravel().tolist()) == list(range(2 * cfg.max_pages_per_seq))
    # the partial last page's tail is NaN-filled, as in the numpy generator
    tail = wl.bf16_bits_to_f32(ha.k_pages[ha.page_table[0, 300 // 32], 0, 300 % 32:, :])
    assert np.isnan(tail).all()
    # all layers share the per-step active counts
    steps_a = [a.start_block(), a.next_step(), a.next_step()]
    steps_c = [c.start_block(), c.next_step(), c.next_step()]
    for x, y in zip(steps_a, steps_c):
        assert (x.host_copy().m_per_seq == y.host_copy().m_per_seq).all()
    # the oracle finds the planted tokens
    o = OracleLayer(ha)
    for t, inp in enumerate(steps_a):
        h = inp.host_copy()
        r = o.run_step(h)
        if t:
            m = int(h.m_per_seq[0])
            for s in range(2):
                assert r["act"][s, :m].tolist() == sorted(h.planted[s].tolist())
                assert delta_gap_ok(r["delta"][s], m)
