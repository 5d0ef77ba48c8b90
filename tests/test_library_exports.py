"""The C-ABI library loads without a GPU and exports every symbol include/egtp.h declares."""
import os
import re

from paper_2602_11812_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "egtp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"EGTP_API\s+[\w\s\*]+?\b(\w+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    build.build()
    lib = binding.load()
    declared = _declared_symbols()
    assert len(declared) >= 17
    assert sorted(binding.EXPORTED_SYMBOLS) == declared
    for name in declared:
        assert hasattr(lib, name), name
    assert binding.status_string(0) == "ok"
    assert "offsets" in binding.status_string(binding.EGTP_ERR_BAD_OFFSETS)
    assert binding.egtp_kernel_name(binding.EGTP_K_LMHEAD_ENTROPY) == "lmhead_entropy"
    assert [binding.egtp_kernel_name(k) for k in range(binding.EGTP_NUM_KERNELS)] == binding.KERNEL_IDS
