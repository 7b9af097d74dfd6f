"""The C-ABI library builds, loads, exports what include/qlora.h declares, and validates arguments on the host
before anything is launched (so these run without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2306_08162_b200 import build as qbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ql():
    qbuild.build_library()
    import paper_2306_08162_b200 as mod
    mod.library()
    return mod


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(qlora_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(ql):
    lib = ctypes.CDLL(ql.library_path())
    names = declared_symbols()
    assert {"qlora_fwd", "qlora_bwd_input", "qlora_bwd_lora", "qlora_pack", "qlora_unpack", "qlora_dequant",
            "qlora_workspace_bytes", "qlora_status_string"} <= names
    for name in names:
        assert hasattr(lib, name), name


def test_binding_has_the_same_names(ql):
    for name in declared_symbols():
        assert hasattr(ql, name), name


def test_status_strings(ql):
    assert ql.qlora_status_string(0) == "ok"
    seen = {ql.qlora_status_string(c) for c in range(-6, 1)}
    assert len(seen) == 7
    assert ql.qlora_status_string(-99) == "unknown status"


def test_workspace_query_and_desc_validation(ql):
    d = ql.desc(4, 128, 4096, 4096, 8, 16.0)
    assert ql.qlora_workspace_bytes(d, 2048) >= 2 * 2048 * 8 * 4
    assert ql.qlora_workspace_bytes(d, 0) > 0
    for bad in (ql.desc(5, 128, 4096, 4096, 8, 16.0),     # bits
                ql.desc(4, 100, 4096, 4096, 8, 16.0),     # group not a multiple of 32
                ql.desc(4, 96, 4096, 4096, 8, 16.0),      # group does not divide K
                ql.desc(4, 128, 4100, 4096, 8, 16.0),     # K % 32
                ql.desc(4, 128, 4096, 4100, 8, 16.0),     # N % 8
                ql.desc(4, 128, 4096, 4096, 12, 16.0),    # rank % 8
                ql.desc(4, 128, 4096, 4096, 72, 16.0)):   # rank > 64
        with pytest.raises(ql.QloraError) as e:
            ql.qlora_workspace_bytes(bad, 16)
        assert e.value.status == -2
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_workspace_bytes(d, -1)
    assert e.value.status == -1


def test_calls_reject_bad_arguments_before_launch(ql):
    """NULL, misaligned and undersized arguments are refused on the host; nothing reaches a device."""
    d = ql.desc(4, 128, 256, 256, 8, 16.0)
    ok = 0x1000  # an aligned non-NULL value; never dereferenced because a later argument is refused first
    need = ql.qlora_workspace_bytes(d, 4)
    # NULL tensor
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_fwd(d, 4, None, ok, ok, ok, ok, ok, ok, None, ok, stream=0, workspace_bytes=need)
    assert e.value.status == -1
    # misaligned
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_fwd(d, 4, ok + 2, ok, ok, ok, ok, ok, ok, None, ok, stream=0, workspace_bytes=need)
    assert e.value.status == -3
    # workspace too small / missing
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_fwd(d, 4, ok, ok, ok, ok, ok, ok, ok, None, ok, stream=0, workspace_bytes=need - 1)
    assert e.value.status == -4
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_bwd_input(d, 4, ok, ok, ok, ok, ok, ok, ok, None, None, stream=0, workspace_bytes=0)
    assert e.value.status == -4
    # LoRA operands required when r > 0
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_bwd_input(d, 4, ok, ok, ok, ok, None, ok, ok, None, ok, stream=0, workspace_bytes=need)
    assert e.value.status == -1
    # accumulate flag
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_bwd_lora(d, 4, ok, ok, ok, ok, None, None, ok, ok, 2, ok, stream=0, workspace_bytes=need)
    assert e.value.status == -1
    # negative M
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_fwd(d, -4, ok, ok, ok, ok, ok, ok, ok, None, ok, stream=0, workspace_bytes=need)
    assert e.value.status == -1
    # format utilities
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_pack(5, 32, 8, ok, ok, stream=0)
    assert e.value.status == -2
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_unpack(4, 33, 8, ok, ok, stream=0)
    assert e.value.status == -2
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_dequant(ql.desc(4, 128, 256, 256, 0, 0.0), ok, ok, None, ok, stream=0)
    assert e.value.status == -1
    # dropout variants: the mask is required, the keep scale is 1 / (1 - p) >= 1
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_fwd_dropout(d, 4, ok, None, 1.25, ok, ok, ok, ok, ok, ok, None, ok, stream=0, workspace_bytes=need)
    assert e.value.status == -1
    with pytest.raises(ql.QloraError) as e:
        ql.qlora_bwd_input_dropout(d, 4, ok, ok, 0.5, ok, ok, ok, ok, ok, ok, None, ok, stream=0, workspace_bytes=need)
    assert e.value.status == -1
    # column gather: element size, NULL, in-place
    lib = ql.library()
    assert lib.qlora_gather_columns(3, 4, 8, ok, ok, ok + 64, 0) == -2
    assert lib.qlora_gather_columns(2, 4, 8, ok, None, ok + 64, 0) == -1
    assert lib.qlora_gather_columns(2, 4, 8, ok, ok, ok, 0) == -1


def test_missing_library_fails_loudly(ql, monkeypatch, tmp_path):
    from paper_2306_08162_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.library()


def test_host_state_is_per_device_and_nothing_is_keyed_by_caller_pointers():
    """What the library remembers between calls is kept per device ordinal (arrays of kMaxDevices in device_state.h and
    beside the occupancy queries); there is no process-wide 'configured' flag and no table keyed by a workspace address."""
    import glob
    import re
    csrc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2306_08162_b200", "csrc")
    text = {os.path.basename(p): open(p).read() for p in glob.glob(os.path.join(csrc, "*"))}
    for name, src in text.items():
        assert "unordered_map" not in src and "static bool configured" not in src, name
        assert not re.search(r"static\s+int\s+n\s*=\s*\[\]", src), name          # a process-wide cached SM count
    ds = text["device_state.h"]
    assert "size_t done[kMaxDevices]" in ds and "int cached[kMaxDevices]" in ds and "cudaGetDevice" in ds
    assert "max_clusters_dev[kMaxDevices]" in text["umma_kernel.cu"]
    assert "DeviceFacts facts[ST_MAX_DEVICES]" in text["stream_kernel.cu"]


def test_which_way_db_goes_is_a_host_side_plan(ql):
    """qlora_bwd_input_db_on_producers launches nothing: it replays the backward call's plan (tiles against SM pairs,
    idle pairs against row blocks).  Without a GPU the library plans for 148 SMs, so the LLaMA-7B answers are fixed."""
    yes = [(4096, 4096, 8, 2048), (4096, 4096, 8, 8192), (4096, 4096, 8, 4096), (1024, 1024, 16, 1536)]
    no = [(4096, 4096, 8, 128),        # single-CTA tensor-core kernel: no producer pairs
          (4096, 4096, 8, 16),         # few-token kernels
          (4096, 4096, 24, 2048),      # three rank tiles
          (4096, 11008, 16, 2048),     # 64 tiles leave ten idle pairs: too few for 128 row blocks at three per CTA
          (11008, 4096, 16, 2048)]     # split last wave: the producers are only half a tile ahead
    for K, N, r, M in yes:
        assert ql.qlora_bwd_input_db_on_producers(ql.desc(2, 64, K, N, r, 16.0), M) is True, (K, N, r, M)
    for K, N, r, M in no:
        assert ql.qlora_bwd_input_db_on_producers(ql.desc(2, 64, K, N, r, 16.0), M) is False, (K, N, r, M)
    # the optional workspace areas exist exactly where they can be used
    d = ql.desc(4, 128, 4096, 4096, 8, 16.0)
    assert ql.qlora_workspace_bytes(d, 2048) >= 2 * 10 * 4096 * 8 * 4 + 8 * 8192 * 8 * 4       # the parts of dB of 20 producer CTAs + gradient partial sums of 8 row slices
    assert ql.qlora_workspace_bytes(d, 128) < 2**20                                            # nothing optional with few tokens
    gate = ql.desc(2, 64, 4096, 11008, 16, 32.0)
    assert ql.qlora_workspace_bytes(gate, 2048) >= 24 * 512 * 1024      # 24 split tiles of the forward
    with pytest.raises(ql.QloraError):
        ql.qlora_bwd_input_db_on_producers(ql.desc(5, 64, 4096, 4096, 8, 16.0), 2048)
