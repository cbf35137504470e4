"""The C-ABI library loads without a GPU and exports every function the header declares."""
import ctypes
import os
import re

from paper_2609_35140_b200 import build as tik_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "tik.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tik_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = _declared_functions()
    for required in ("tik_attn_train_fwd", "tik_attn_prefill", "tik_attn_decode", "tik_token_logprob",
                     "tik_kv_cache_write", "tik_create", "tik_destroy", "tik_workspace_bytes"):
        assert required in names


def test_library_exports_every_declared_symbol():
    path = tik_build.build()
    lib = ctypes.CDLL(path)
    for name in _declared_functions():
        assert hasattr(lib, name), name


def test_host_only_calls_work_without_a_gpu():
    from paper_2609_35140_b200 import binding
    assert binding.contract_id().startswith("tik")
    lib = binding.load()
    assert lib.tik_status_str(0) == b"ok"
    assert lib.tik_status_str(-3) == b"workspace too small"
    # decode scratch: B * Hq * chunks * (d + 4) floats; log-prob: T * (2 * super-chunks + 1) floats
    assert binding.workspace_bytes(binding.OP_ATTN_DECODE, 16, 32, 8, 128, 16384) == 16 * 32 * 8 * 132 * 4
    assert binding.workspace_bytes(binding.OP_ATTN_DECODE, 16, 32, 8, 128, 2049) == 16 * 32 * 2 * 132 * 4
    assert binding.workspace_bytes(binding.OP_TOKEN_LOGPROB, 5000, H=4096, V=151936) == 5000 * (2 * 149 + 1) * 4
    # calls of at most 2048 rows keep one partial per 128-column tile: ceil(151936 / 128) = 1187
    assert binding.workspace_bytes(binding.OP_TOKEN_LOGPROB, 64, H=4096, V=151936) == 64 * (2 * 1187 + 1) * 4
    assert binding.workspace_bytes(binding.OP_TOKEN_LOGPROB, 2048, H=4096, V=151936) == 2048 * (2 * 1187 + 1) * 4
    assert binding.workspace_bytes(binding.OP_TOKEN_LOGPROB, 2049, H=4096, V=151936) == 2049 * (2 * 149 + 1) * 4
    # full-sequence kernels: a plan of 16 bytes per (sequence, candidate item) + header; 4096 positions
    # = 32 tiles = 8 pairs + 16 single tiles
    assert binding.workspace_bytes(binding.OP_ATTN_TRAIN_FWD, 1000, 8, 2, 128, 4096) == 16 + 16 * 1000 * 24
    assert binding.workspace_bytes(binding.OP_ATTN_PREFILL, 3, 8, 2, 128, 1000) == 16 + 16 * 3 * 4
    assert binding.workspace_bytes(binding.OP_ATTN_TRAIN_FWD, 0, 8, 2, 128, 4096) == 0


def test_per_device_launch_setup_bookkeeping():
    """The shared-memory opt-in is kept per device: a second GPU of the process is not skipped."""
    from paper_2609_35140_b200 import binding
    lib = binding.load()
    lib.tik_selftest_host.restype = ctypes.c_int
    assert lib.tik_selftest_host() == 0
