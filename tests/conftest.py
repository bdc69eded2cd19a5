import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


# The GPU parity modules run once per merge mode: the barrier merge with the combine kernel, the chained merge
# with the final merge of cut units inside the decode kernel (the default), the chained merge with the
# combine kernel, and the short-piece instantiation of the latter (forced on for every batch it can run) must
# each pass every case, whatever the library would pick by itself.  Values: (merge mode, short-piece path).
MERGE_MODE_MODULES = ("test_gpu_parity", "test_gpu_grouped", "test_gpu_decode_loop", "test_gpu_multi_token")
MERGE_MODES = {"barrier": (0, -1), "chain": (1, -1), "chain_combine": (2, -1), "chain_short": (2, 1)}


# ... and the grouped-decode module once per kernel for the shared prompt tiles.
PREFIX_ENGINE_MODULES = ("test_gpu_grouped",)
PREFIX_ENGINES = {"tcgen05": 1, "warp_mma": 0}


def pytest_generate_tests(metafunc):
    name = metafunc.module.__name__.split(".")[-1]
    if name in MERGE_MODE_MODULES:
        metafunc.parametrize("merge_mode", list(MERGE_MODES), indirect=True)
    if name in PREFIX_ENGINE_MODULES:
        metafunc.parametrize("prefix_engine", list(PREFIX_ENGINES), indirect=True)


@pytest.fixture(autouse=True)
def prefix_engine(request):
    name = getattr(request, "param", None)
    if name is None:
        yield None
        return
    from paper_2607_09207_b200 import pdattn
    pdattn.set_prefix_engine(PREFIX_ENGINES[name])
    try:
        yield name
    finally:
        pdattn.set_prefix_engine(-1)


@pytest.fixture(autouse=True)
def merge_mode(request):
    name = getattr(request, "param", None)
    if name is None:
        yield None
        return
    from paper_2607_09207_b200 import pdattn
    pdattn.set_merge_mode(MERGE_MODES[name][0])
    pdattn.set_short_piece_path(MERGE_MODES[name][1])
    try:
        yield name
    finally:
        pdattn.set_merge_mode(-1)
        pdattn.set_short_piece_path(-1)


# The fp64 oracle's output for a benchmark configuration at full size, every (sequence, head) row.  The
# configurations are seeded, so the reference is a function of the configuration number alone and is computed
# once per session (a few seconds of all host cores each); several GPU test modules compare against it.
_FULL_REFERENCE = {}


@pytest.fixture(scope="session")
def full_reference():
    def get(cfg, w_gpu):
        if cfg not in _FULL_REFERENCE:
            from oracle import pdattn_oracle
            _FULL_REFERENCE[cfg] = pdattn_oracle.decode_workload(w_gpu.to("cpu"))
        return _FULL_REFERENCE[cfg]
    return get
