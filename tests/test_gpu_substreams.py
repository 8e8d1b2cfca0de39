"""The optional two-sub-stream softmax of the tcgen05 path (ORTHRUS_TC_NSUB=2) is chosen
when the library is first used in a process, so its parity run happens in a child
process: the shape, split and mask tests of test_gpu_attend.py with the variable set."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_parity_with_two_substreams():
    env = dict(os.environ, ORTHRUS_TC_NSUB="2")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(HERE, "test_gpu_attend.py"), "-x", "-q",
                        "-k", "tcgen05 and (shapes or forced or peaked or planted)"],
                       env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
