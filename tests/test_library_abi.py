"""The C library builds for sm_100a, loads, and exports every symbol include/bsr.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

from conftest import ROOT


def _declared():
    text = open(os.path.join(ROOT, "include", "bsr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bsr_[a-z_]+)\s*\(", text)))


def test_header_declares_the_four_protocol_calls():
    names = _declared()
    for n in ("bsr_probe", "bsr_restore", "bsr_commit", "bsr_invalidate"):
        assert n in names
    assert len(names) >= 15


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2608_17826_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    for n in _declared():
        assert hasattr(lib, n), f"{n} declared in bsr.h but not exported"


def test_binding_covers_the_header_and_struct_sizes_match():
    from paper_2608_17826_b200 import binding as B
    assert sorted(B.EXPORTS) == _declared()
    for n in B.EXPORTS:
        assert callable(getattr(B, n))
    assert ctypes.sizeof(B.bsr_config) == 64  # as gcc lays out include/bsr.h
    assert ctypes.sizeof(B.bsr_tensor_desc) == 16
    assert ctypes.sizeof(B.bsr_stats) == 8 * 8 * 5 + 8 * 7 + 8 * 4 + 8 * 2 + 8 * 3


def test_context_creation_fails_loudly_without_a_gpu_or_with_bad_arguments():
    import torch
    from paper_2608_17826_b200 import binding as B
    assert B.bsr_ctx_create(0, 1)[0] == B.BSR_ERR_INVALID
    if not torch.cuda.is_available():
        rc, ctx = B.bsr_ctx_create(4, 1)
        assert rc == B.BSR_ERR_CUDA and ctx is None


def _fake_sysfs(tmp_path, nodes, dev_node, bus="0000:1b:00.0"):
    d = tmp_path / "bus" / "pci" / "devices" / bus
    d.mkdir(parents=True)
    (d / "numa_node").write_text(f"{dev_node}\n")
    for k, cpus in enumerate(nodes):
        n = tmp_path / "devices" / "system" / "node" / f"node{k}"
        n.mkdir(parents=True)
        (n / "cpulist").write_text(cpus + "\n")
    return str(tmp_path)


def test_numa_placement_helper_reads_a_sysfs_tree(tmp_path):
    """The host-topology helper behind the automatic placement of fill threads and pinned pool,
    against a fake sysfs tree: two sockets, the GPU on the second; upper-case bus id as CUDA prints it."""
    from paper_2608_17826_b200 import binding as B
    root = _fake_sysfs(tmp_path, ["0-15,32-47", "16-31,48-63"], 1)
    assert B.bsr_numa_of_pci(root, "0000:1B:00.0") == (B.BSR_OK, 1, "16-31,48-63", 2)
    assert B.bsr_numa_of_pci(root, "0000:ff:00.0")[0] == B.BSR_ERR_MISSING


def test_numa_placement_helper_unknown_node_and_bad_list(tmp_path):
    from paper_2608_17826_b200 import binding as B
    root = _fake_sysfs(tmp_path / "a", ["0-7"], -1)
    assert B.bsr_numa_of_pci(root, "0000:1b:00.0") == (B.BSR_OK, -1, "", 1)   # the platform does not say
    root = _fake_sysfs(tmp_path / "b", ["0-7", "9-x"], 1)
    assert B.bsr_numa_of_pci(root, "0000:1b:00.0")[0] == B.BSR_ERR_INVALID
