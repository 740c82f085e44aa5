"""A library that does not match its sources is never loaded silently: staleness is decided by content, and a
failed rebuild is an error even when an older libatts.so is lying around."""
import pytest

from paper_2509_15148_b200 import binding
from paper_2509_15148_b200 import build as b


def test_stamp_decides_staleness(tmp_path, monkeypatch):
    binding.load()                                   # whatever state the tree is in, this leaves a matching pair
    assert not b.is_stale()
    stamp = tmp_path / "stamp"
    monkeypatch.setattr(b, "STAMP_PATH", str(stamp))
    assert b.is_stale()                              # no stamp: unknown provenance counts as stale
    stamp.write_text("0" * 64 + "\n")
    assert b.is_stale()                              # built from other sources
    stamp.write_text(b.source_digest() + "\n")
    assert not b.is_stale()


def test_failed_rebuild_of_a_stale_library_raises(tmp_path, monkeypatch):
    binding.load()
    stamp = tmp_path / "stamp"
    stamp.write_text("0" * 64 + "\n")
    monkeypatch.setattr(b, "STAMP_PATH", str(stamp))
    monkeypatch.setattr(binding, "_lib", None)

    def broken(*a, **k):
        raise RuntimeError("nvcc failed building libatts.so")

    monkeypatch.setattr(b, "build_library", broken)
    with pytest.raises(RuntimeError, match="nvcc failed"):
        binding.load()                               # the old .so exists, and is still refused
    assert binding._lib is None
