"""Input generators: determinism, structure and the save / load round trip (no method arithmetic here)."""
import numpy as np

from paper_2310_09443_b200 import traces


def test_generators_are_seeded_and_valid():
    for idx in (0, 1, 2):
        a = traces.make_config(idx)
        b = traces.make_config(idx)
        a.validate()
        assert a.sha256() == b.sha256()
    assert traces.config0_mlp_chain(seed=0).sha256() != traces.config0_mlp_chain(seed=5).sha256()


def test_structure_of_dnn_shaped_traces():
    tr = traces.make_config(1)
    deg = np.diff(tr.kernel_ptr)
    assert deg.min() >= 1 and deg.max() <= 16            # a kernel touches a handful of tensors
    used = np.zeros(tr.N, dtype=bool)
    used[tr.kernel_tensors] = True
    assert used.all()                                    # every tensor is used by some kernel
    assert tr.tensor_global.sum() > 0                    # parameters / optimizer state are global


def test_save_load_round_trip(tmp_path):
    tr = traces.make_config(0)
    digest = tr.save(str(tmp_path / "t.npz"))
    back = traces.Trace.load(str(tmp_path / "t.npz"))
    assert back.sha256() == digest == tr.sha256()
    assert back.name == tr.name
    assert back.capacity_bytes == tr.capacity_bytes and back.capacity_frac == tr.capacity_frac
    assert (back.host_bw, back.ssd_bw, back.host_capacity_bytes) == (tr.host_bw, tr.ssd_bw, tr.host_capacity_bytes)
    for f in ("kernel_ptr", "kernel_tensors", "tensor_bytes", "kernel_ns", "tensor_global"):
        assert getattr(back, f).dtype == getattr(tr, f).dtype
        assert np.array_equal(getattr(back, f), getattr(tr, f))
