"""The C-ABI library: it loads without a GPU, exports every symbol include/pods.h declares, and the
binding's signature table covers the same set.  Host-visible argument errors come back as status
codes before any launch (no compute call is made here)."""
import ctypes as C
import re

from paper_2504_13818_b200 import binding
from paper_2504_13818_b200.csrc import build as cuda_build


def _declared(rootpath):
    text = (rootpath / "include" / "pods.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b((?:pods|grpo)_[a-z0-9_]+)\s*\(", text))


def test_library_builds_loads_and_exports_every_declared_symbol(request):
    cuda_build.build()
    lib = binding.load()
    names = _declared(request.config.rootpath)
    assert {"pods_select", "pods_compact", "grpo_loss_fwd_bwd", "grpo_loss_chunk"} <= names
    for name in names:
        assert hasattr(lib, name), name
    assert names == set(binding.SIGNATURES), names ^ set(binding.SIGNATURES)
    assert b"sm_100a" in lib.pods_version()


def test_host_side_argument_checks_return_codes_without_launching():
    lib = binding.load()
    bad = lib.pods_select(None, 4, 16, 17, 0, 0, 0, None, None, None, None, None)      # m > n
    assert bad == 1 and lib.pods_status_string(bad) == b"invalid argument"
    assert lib.pods_select(None, 4, 2048, 4, 0, 0, 0, None, None, None, None, None) == 2   # n > PODS_MAX_N
    assert lib.pods_select(None, 4, 16, 4, 9, 0, 0, None, None, None, None, None) == 2     # unknown rule
    assert lib.pods_select(None, 4, 16, 4, 0, 0, 0, None, None, None, None, None) == 1     # null pointers
    assert lib.pods_select(None, 0, 16, 4, 0, 0, 0, None, None, None, None, None) == 0     # empty batch
    assert lib.pods_compact(None, 1, 4, 2, None, None, 8, None, 0, None, None, None, 16, None, None) == 1
    assert lib.grpo_loss_chunk_workspace_bytes(1000) >= 8000
    assert lib.grpo_loss_workspace_bytes(1000, 16, 0) >= 8000 + 128
    fake = C.c_void_p(256)      # non-null, never dereferenced: the size checks come first
    rc = lib.grpo_loss_chunk(fake, 8, fake, fake, fake, fake, fake, fake, 1, 0, None, 4, 16, 0.2, 0.0, 1.0,
                             fake, fake, fake, 16, None, 0, None, None)
    assert rc == 1              # ldl < V
    rc = lib.grpo_loss_chunk(fake, 16, fake, fake, fake, fake, fake, fake, 1, 0, None, 4, 16, 0.2, 0.0, 1.0,
                             fake, fake, fake, 16, None, 0, None, None)
    assert rc == 3              # no workspace
    rc = lib.grpo_loss_chunk(fake, 16, fake, fake, None, fake, fake, fake, 1, 0, None, 4, 16, 0.2, 0.04, 1.0,
                             fake, fake, fake, 16, fake, 4096, None, None)
    assert rc == 1              # beta != 0 needs ref_logp


def test_binding_refuses_host_tensors():
    import pytest
    import torch
    with pytest.raises(binding.PodsError):
        binding.pods_select(torch.zeros(2, 4), 2)


def test_cluster_vocabulary_limit_is_a_process_wide_setting_with_a_floor():
    lib = binding.load()
    default = lib.pods_set_loss_cluster_min_vocab(100000)
    assert default == 8192
    assert lib.pods_set_loss_cluster_min_vocab(5) == 100000       # values below 2048 are raised to 2048
    assert lib.pods_set_loss_cluster_min_vocab(default) == 2048
    assert lib.pods_set_loss_cluster_min_vocab(default) == default
