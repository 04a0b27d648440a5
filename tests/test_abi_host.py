"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_1906_11024_b200 import binding as B
from paper_1906_11024_b200 import build as san_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    san_build.build()
    return B.lib()


def _cfg(**kw):
    base = dict(n_layers=6, n_heads=8, d_head=64, max_sent=2, beam=4, max_tgt_len=32, max_src_len=16,
                dtype=B.SAN_BF16, self_is_aan=0, encdec_shared_context=0)
    base.update(kw)
    return B.san_config(**base)


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "san.h")).read()
    declared = set(re.findall(r"\b(san_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert B.san_status_string(B.SAN_OK) == "ok"
    seen = {B.san_status_string(i) for i in range(11)}
    assert len(seen) == 11 and "unknown status" not in seen
    assert B.san_status_string(99) == "unknown status"


def test_query_bytes_counts_key_planes_only_for_block_first_layers(lib):
    """Section 3.2: layers that take their weights from another layer keep no keys, so
    the self-attention key cache holds one plane per block."""
    cfg = _cfg()
    e, seqs = 2, 2 * 4
    self_plane = seqs * 8 * 32 * 64 * e
    mem_plane = 2 * 8 * 16 * 64 * e
    for ns, ne in ((6, 6), (3, 1), (1, 2), (2, 6)):
        rc, cb, wb = B.san_query_bytes(cfg, ns, ne)
        assert rc == B.SAN_OK
        assert cb == (ns + 6) * self_plane + (ne + 6) * mem_plane
        assert wb > 0 and wb % 4 == 0
    rc, cb_ctx, _ = B.san_query_bytes(_cfg(encdec_shared_context=1), 3, 2)
    assert cb_ctx == (3 + 6) * self_plane + (2 + 2) * mem_plane          # Eq. 5: one V plane per block
    rc, cb_aan, _ = B.san_query_bytes(_cfg(self_is_aan=1), 6, 3)
    assert cb_aan == (3 + 6) * mem_plane + 6 * seqs * 512 * 4            # float32 running sums


@pytest.mark.parametrize("kw,status", [
    (dict(d_head=32), B.SAN_ERR_UNSUPPORTED),
    (dict(n_layers=0), B.SAN_ERR_SHAPE),
    (dict(n_layers=65), B.SAN_ERR_SHAPE),
    (dict(beam=B.SAN_MAX_BEAM + 1), B.SAN_ERR_SHAPE),
    (dict(beam=0), B.SAN_ERR_SHAPE),
    (dict(max_tgt_len=0), B.SAN_ERR_SHAPE),
    (dict(dtype=7), B.SAN_ERR_DTYPE),
])
def test_query_bytes_rejects_bad_configs(lib, kw, status):
    rc, _, _ = B.san_query_bytes(_cfg(**kw), 1, 1)
    assert rc == status


def test_query_bytes_rejects_bad_block_counts(lib):
    assert B.san_query_bytes(_cfg(), 0, 1)[0] == B.SAN_ERR_POLICY
    assert B.san_query_bytes(_cfg(), 7, 1)[0] == B.SAN_ERR_POLICY
    assert lib.san_query_bytes(None, 1, 1, None, None) == B.SAN_ERR_NULL


def test_create_rejects_before_touching_the_device(lib):
    cfg = _cfg()
    fake = 0x10000        # never dereferenced: every call below fails its host checks first
    big = 1 << 40
    assert B.san_create(cfg, [2, 2, 3], [6], fake, big, fake, big)[0] == B.SAN_ERR_POLICY   # sums to 7
    assert B.san_create(cfg, [2, 0, 4], [6], fake, big, fake, big)[0] == B.SAN_ERR_POLICY   # empty block
    assert B.san_create(cfg, [2, 2, 2], [3, 2], fake, big, fake, big)[0] == B.SAN_ERR_POLICY
    assert B.san_create(cfg, [2, 2, 2], [6], None, big, fake, big)[0] == B.SAN_ERR_NULL
    assert B.san_create(cfg, [2, 2, 2], [6], fake, big, None, big)[0] == B.SAN_ERR_NULL
    assert B.san_create(cfg, [2, 2, 2], [6], fake + 8, big, fake, big)[0] == B.SAN_ERR_SHAPE   # misaligned
    assert B.san_create(cfg, [2, 2, 2], [6], fake, 16, fake, big)[0] == B.SAN_ERR_CAPACITY
    assert B.san_create(cfg, [2, 2, 2], [6], fake, big, fake, 16)[0] == B.SAN_ERR_CAPACITY


def test_null_context_is_an_error_everywhere(lib):
    assert B.san_destroy(None) == B.SAN_ERR_NULL
    assert B.san_policy_set_sizes(None, B.SAN_SELF, [6]) == B.SAN_ERR_NULL
    assert B.san_policy_get_map(None, B.SAN_SELF)[0] == B.SAN_ERR_NULL
    assert B.san_cache_append(None, 0, 0, 1, 0, 0, 0, 0, 0, 1, 1, stream=0) == B.SAN_ERR_NULL
    assert B.san_attn_weights(None, 0, 0, 0, 0, 0, 1, 0, 0, 8, stream=0) == B.SAN_ERR_NULL
    assert B.san_attn_apply(None, 0, 0, 0, 1, 0, 8, 0, 0, 0, 1, 0, 0, 0, stream=0) == B.SAN_ERR_NULL
    assert B.san_aan_step(None, 0, 1, 0, 0, 0, 1, 0, stream=0) == B.SAN_ERR_NULL
    assert lib.san_device_status(None, None, None, None) == B.SAN_ERR_NULL
