"""The binding's host-side argument check, without a GPU: stand-in tensors (only the attributes
the check reads) go through `check_args`, which must refuse everything that would make a kernel
read or write out of bounds, before any pointer is taken."""
import pytest

from paper_2601_21238_b200 import binding as B


class FakeDevice:
    def __init__(self, index):
        self.index = index


class FakeTensor:
    def __init__(self, shape, dtype="torch.float32", cuda=True, device=0, contiguous=True):
        self.shape = tuple(shape)
        self.dtype = dtype
        self.is_cuda = cuda
        self.device = FakeDevice(device if cuda else None)
        self._contiguous = contiguous

    def is_contiguous(self):
        return self._contiguous

    def numel(self):
        n = 1
        for d in self.shape:
            n *= d
        return n

    def data_ptr(self):
        raise AssertionError("the check must not take addresses")


def layer(M=8, K=32, N=16, P=4, **over):
    t = dict(X=FakeTensor((M, K)), pos_ids=FakeTensor((M,), "torch.int32"), Wq=FakeTensor((N, K), "torch.int8"),
             s_w=FakeTensor((N,)), s_tok=FakeTensor((P,)), s_ch=FakeTensor((K,)), bias=FakeTensor((N,)),
             Y=FakeTensor((M, N), "torch.bfloat16"))
    t.update(over)
    return t


def run(t, out=B.OUT_BF16, x_dtype="torch.float32", device=0):
    M, K, N, P, specs = B._layer_specs("qlinear", t["X"], x_dtype, t["pos_ids"], t["Wq"], t["s_w"], t["s_tok"],
                                       t["s_ch"], t["bias"], out, t["Y"])
    B.check_args("qlinear", device, *specs)
    return M, K, N, P


def code_of(fn):
    with pytest.raises(B.StwqError) as ei:
        fn()
    return ei.value.code


def test_a_consistent_layer_passes_and_sizes_are_derived_from_the_tensors():
    assert run(layer()) == (8, 32, 16, 4)
    assert run(layer(s_ch=None, bias=None)) == (8, 32, 16, 4)            # the optional ones


def test_wrong_dtype_is_refused():
    assert code_of(lambda: run(layer(Y=FakeTensor((8, 16), "torch.float32")))) == B.ERR_BITS   # bf16 asked, fp32 given
    assert code_of(lambda: run(layer(), out=B.OUT_F32)) == B.ERR_BITS
    assert code_of(lambda: run(layer(Wq=FakeTensor((16, 32), "torch.float32")))) == B.ERR_BITS
    assert code_of(lambda: run(layer(pos_ids=FakeTensor((8,), "torch.int64")))) == B.ERR_BITS
    assert code_of(lambda: run(layer(), out=7)) == B.ERR_BITS


def test_wrong_shapes_are_refused():
    assert code_of(lambda: run(layer(Wq=FakeTensor((16, 48), "torch.int8")))) == B.ERR_DIM     # Wq.shape[1] != K
    assert code_of(lambda: run(layer(pos_ids=FakeTensor((7,), "torch.int32")))) == B.ERR_DIM   # short pos_ids
    assert code_of(lambda: run(layer(s_w=FakeTensor((15,))))) == B.ERR_DIM
    assert code_of(lambda: run(layer(bias=FakeTensor((17,))))) == B.ERR_DIM
    assert code_of(lambda: run(layer(s_ch=FakeTensor((16,))))) == B.ERR_DIM
    assert code_of(lambda: run(layer(Y=FakeTensor((16, 8), "torch.bfloat16")))) == B.ERR_DIM   # transposed output
    assert code_of(lambda: run(layer(X=FakeTensor((8, 4, 8))))) == B.ERR_DIM


def test_views_devices_and_missing_tensors_are_refused():
    assert code_of(lambda: run(layer(X=FakeTensor((8, 32), contiguous=False)))) == B.ERR_ALIGN   # a transposed view
    assert code_of(lambda: run(layer(Wq=FakeTensor((16, 32), "torch.int8", cuda=False)))) == B.ERR_CUDA
    assert code_of(lambda: run(layer(bias=FakeTensor((16,), device=1)))) == B.ERR_CUDA
    assert code_of(lambda: run(layer(s_tok=None))) == B.ERR_NULL
    assert code_of(lambda: run(layer(Y=None))) == B.ERR_NULL


def test_raw_accumulator_calls_need_no_scales():
    t = layer(pos_ids=None, s_w=None, s_tok=None, s_ch=None, bias=None, X=FakeTensor((8, 32), "torch.int8"),
              Y=FakeTensor((8, 16), "torch.int32"))
    M, K, N, P, specs = B._layer_specs("qlinear_q", t["X"], "torch.int8", None, t["Wq"], None, None, None, None,
                                       B.OUT_INT32, t["Y"], need_scales=False)
    B.check_args("qlinear_q", 0, *specs)
    assert (M, K, N, P) == (8, 32, 16, 1)
