"""CPU oracle for the Anakin hot path.  TEST INFRASTRUCTURE, NOT THE PRODUCT (see anakin_oracle.cpp)."""
