"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2603_17803_b200 import build
    return build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "swarm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(swarm_[a-z_]+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = declared_functions()
    for required in ("swarm_select", "swarm_resolve_clusters", "swarm_gather", "swarm_sparse_attn", "swarm_step"):
        assert required in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in swarm.h but not exported"
    lib.swarm_version.restype = ctypes.c_int32
    assert lib.swarm_version() >= 100


def test_binding_covers_every_declared_symbol(lib_path):
    from paper_2603_17803_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()
    for name in declared_functions():
        assert callable(getattr(binding, name))


def test_shape_validation_runs_without_a_gpu(lib_path):
    from paper_2603_17803_b200 import binding as B
    ok = dict(batch=1, n_q_heads=32, n_kv_heads=8, page_size=16, top_k=256, n_queues=8, max_pages_per_req=8192,
              max_clusters_total=1024, n_pool_pages=8192)
    n = B.swarm_workspace_bytes(B.make_shape(**ok))
    assert n > 32 * 8192 * 4 and n % 256 == 0
    with pytest.raises(B.SwarmError) as e:
        B.swarm_workspace_bytes(B.make_shape(**{**ok, "head_dim": 96}))
    assert e.value.code == B.ERR_UNSUPPORTED
    with pytest.raises(B.SwarmError) as e:
        B.swarm_workspace_bytes(B.make_shape(**{**ok, "n_queues": 0}))
    assert e.value.code == B.ERR_INVALID_ARG


def test_switches_reject_a_null_ctx_without_a_gpu(lib_path):
    """The ctx switches validate their arguments on the host (no CUDA call is made for a null ctx)."""
    lib = ctypes.CDLL(lib_path)
    for name in ("swarm_set_index_prefetch", "swarm_set_scorer", "swarm_set_select_sms", "swarm_set_attn_splits"):
        fn = getattr(lib, name)
        fn.restype = ctypes.c_int32
        assert fn(None, ctypes.c_int32(1)) == 1, name      # SWARM_ERR_INVALID_ARG


def test_struct_layouts_match_the_header():
    from paper_2603_17803_b200 import binding as B
    assert ctypes.sizeof(B.swarm_shape) == 56          # 9 x int32 + uint32 + int64 + 2 x int32
    assert ctypes.sizeof(B.swarm_inputs) == 9 * 8
    assert ctypes.sizeof(B.swarm_outputs) == 12 * 8
