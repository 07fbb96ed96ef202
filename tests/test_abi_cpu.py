"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, validates arguments before touching CUDA, and refuses to compute without a device."""
import ctypes
import os
import re

import pytest

import paper_2411_19870_b200 as demo
from paper_2411_19870_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return demo.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "demo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(demo_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert "demo_init" in names and "demo_compress" in names and "demo_decode_apply" in names and "demo_free" in names
    for n in names:
        assert hasattr(lib, n), "missing export " + n
    assert set(names) == set(binding.EXPORTS)


def test_status_strings(lib):
    seen = {demo.demo_status_string(i) for i in range(9)}
    assert len(seen) == 9 and "ok" in seen


def _init(shapes, **kw):
    args = dict(chunk=64, topk=32, beta=0.999, lr=1e-3, weight_decay=0.1, num_workers=2)
    args.update(kw)
    return demo.DemoTransform(shapes, **args)


@pytest.mark.parametrize("shapes,kw,status", [
    ([(64, 60)], {}, 2),            # dim not a multiple of s
    ([(32, 64)], {}, 2),            # dim smaller than s
    ([(64, 64, 64)], {}, 2),        # 3-D tensor
    ([(64, 64)], {"topk": 0}, 3),
    ([(64, 64)], {"topk": 4097}, 3),
    ([(64, 64)], {"chunk": 48}, 4),
    ([(64, 64)], {"grad_dtype": 7}, 4),
    ([(64, 64)], {"num_workers": 0}, 1),
    ([(64, 64)], {"beta": float("nan")}, 1),
])
def test_init_argument_errors_come_before_cuda(lib, shapes, kw, status):
    with pytest.raises(demo.DemoError) as e:
        _init(shapes, **kw)
    assert e.value.status == status


def test_null_arguments(lib):
    assert lib.demo_init(None, None, None, 0, 0) == 1
    assert lib.demo_payload_bytes(None) == 0
    assert lib.demo_payload_layout(None, 0, None, None, None) == 1
    assert lib.demo_compress(None, 0, None, None, None, None) == 1
    assert lib.demo_decode_apply(None, None, 0, None, None) == 1
    assert lib.demo_step_host(None, None, None, None, None, None, None, None) == 1
    assert lib.demo_set_lr(None, 1.0) == 1
    assert lib.demo_set_path(None, 0) == 1
    assert lib.demo_set_alpha(None, 0.5) == 1
    assert lib.demo_set_decode_mode(None, 0, 0) == 1
    assert lib.demo_selftest_bounded_wait(None, 1000, None) == 1
    assert lib.demo_device_status(None, None) == 1
    assert lib.demo_launch_count(None) == 0
    lib.demo_free(None)  # NULL-safe


def test_no_cpu_fallback_without_device(lib):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(demo.DemoError) as e:
        _init([(64, 64)])
    assert e.value.status == 6  # DEMO_ERR_CUDA: the product path fails loudly without a GPU


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError):
        demo.load_library(str(tmp_path / "libnot_there.so"))


def test_binding_checks_the_layout_the_abi_assumes():
    """The C ABI takes bare pointers; the binding refuses tensors whose layout differs from the shapes
    the context was built for (checked without a GPU: the device test is skipped with None)."""
    import torch

    from paper_2411_19870_b200.binding import validate_tensors

    shapes = [(4, 6), (8,)]
    good = [torch.zeros(4, 6), torch.zeros(8)]
    validate_tensors(good, shapes, torch.float32, None, "m")
    with pytest.raises(ValueError, match="expected 2 tensors"):
        validate_tensors(good[:1], shapes, torch.float32, None, "m")
    with pytest.raises(ValueError, match="shape"):
        validate_tensors([torch.zeros(6, 4), good[1]], shapes, torch.float32, None, "m")
    with pytest.raises(ValueError, match="dtype"):
        validate_tensors([good[0].double(), good[1]], shapes, torch.float32, None, "m")
    with pytest.raises(ValueError, match="not contiguous"):
        validate_tensors([torch.zeros(6, 4).t(), good[1]], shapes, torch.float32, None, "m")
    with pytest.raises(ValueError, match="expected cuda:0"):
        validate_tensors(good, shapes, torch.float32, 0, "m")


def test_divisor_chunk_shapes():
    """Chunk extents for dimensions that are not multiples of the target: always divisors, never above the
    target or the library's limits, and the target itself wherever it divides."""
    import math

    from paper_2411_19870_b200 import chunking

    assert chunking.largest_divisor_at_most(50304, 64) == 64
    assert chunking.largest_divisor_at_most(50257, 64) == 29      # 50257 = 29 * 1733
    assert chunking.largest_divisor_at_most(97, 64) == 1          # prime
    assert chunking.divisor_chunk_shape((2048, 8192), 64) == (64, 64)
    assert chunking.divisor_chunk_shape((50257, 768), 64) == (29, 64)
    assert chunking.divisor_chunk_shape((512, 512, 3, 3), 64) == (32, 32, 3, 3)   # 64*64*9 elements is too many
    assert chunking.divisor_chunk_shape((1000,), 64) == (50,)
    for shape in ((768, 3072), (50257, 1600), (6, 10, 14), (256, 256, 7, 7), (129,), (16, 16, 16, 16)):
        for target in (8, 32, 64, 128, 500):
            ch = chunking.divisor_chunk_shape(shape, target)
            assert len(ch) == len(shape)
            assert all(n % s == 0 and 1 <= s <= min(target, chunking.MAX_EXTENT) for n, s in zip(shape, ch))
            assert math.prod(ch) <= chunking.MAX_CHUNK_ELEMS
