"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and classifies expressions (Sec. 2.2) without a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2404_04541_b200 import build, binding
    build.build()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spws.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spws_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(binding):
    names = declared_functions()
    assert len(names) >= 12
    L = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(L, n), f"{n} declared in spws.h but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_status_strings(binding):
    seen = {binding.status_string(s) for s in range(0, 11)}
    assert len(seen) == 11 and "ok" in seen
    assert binding.status_string(99) == "unknown status"


@pytest.mark.parametrize("expr,fmts,ok", [
    ("C(i,j)=A(i,k)*B(k,j)", (0, 0, 0), True),
    ("  Out( r , c ) = X(r, t) * Y( t ,c)", (0, 0, 0), True),
    ("C(i,j) += A(i,k) * B(k,j)", (0, 0, 0), True),
    ("C(i,j,l)=A(i,j,k)*B(k,l)", (1, 1, 0), True),
    ("Z(a,b,c) = T(a,b,x) * M(x,c)", (1, 1, 0), True),
    ("C(i,j)=A(i,k)*B(k,j)", (0, 1, 0), False),        # formats do not fit the order
    ("C(i,j,l)=A(i,j,k)*B(k,l)", (0, 0, 0), False),
    ("C(i,j)=A(k,i)*B(k,j)", (0, 0, 0), True),         # outer-product order: second-order scatter
    ("R(u,v) = P(w,u) * Q(w,v)", (0, 0, 0), True),
    ("C(i,j)=A(k,i)*B(k,j)", (0, 1, 0), False),
    ("C(i,j)=A(k,j)*B(k,i)", (0, 0, 0), False),        # outer-product order with the output transposed
    ("C(j,i)=A(i,k)*B(k,j)", (0, 0, 0), False),        # transposed output
    ("C(i,j)=A(i,k)*B(j,k)", (0, 0, 0), False),        # B accessed against its storage order
    ("C(i,j)=A(i,j)*B(i,j)", (0, 0, 0), False),        # element-wise: no reduction variable
    ("C(i,j,l)=A(k,i,j)*B(k,l)", (1, 1, 0), False),    # contraction of the outermost mode needs a COO result
    ("C(i,j,l)=A(k,i,j)*B(k,l)", (2, 1, 0), True),     # SpTTM, third-order scatter
    ("C(k,j,l)=A(k,i,j)*B(i,l)", (2, 1, 0), True),     # SpTTM-I
    ("C(i,j,l)=A(i,j,k)*B(k,l)", (2, 1, 0), False),    # the first-order form has a CSF result
    ("C(k,j,l)=A(k,i,j)*B(i,l)", (2, 0, 0), False),
    ("C(i,j)=A(i,k)+B(k,j)", (0, 0, 0), False),
    ("C(i,j)=A(i,k)*B(k,j)*D(j,j)", (0, 0, 0), False),
    ("C(i,i)=A(i,k)*B(k,i)", (0, 0, 0), False),
    ("C(i,j)=C(i,k)*B(k,j)", (0, 0, 0), False),
    ("C(i,j)=A(i,k)*B(k,j", (0, 0, 0), False),
    ("", (0, 0, 0), False),
])
def test_expression_classification(binding, expr, fmts, ok):
    st = binding.check_expression(expr, fmts)
    assert st == (binding.SPWS_OK if ok else binding.SPWS_UNSUPPORTED_EXPRESSION)


def test_no_device_is_reported_not_faked(binding):
    """Without a CUDA device the library reports an error; it never computes on the CPU."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(binding.SpwsError) as e:
        binding.Handle()
    assert e.value.status == binding.SPWS_CUDA_ERROR
    from paper_2404_04541_b200 import api
    with pytest.raises(RuntimeError):
        api.Context()
